// Medusa heads (Section 3.1): residual SiLU block, vocabulary projection as a
// weight-streaming matrix-vector product, per-head top-k fused into the projection,
// and the expansion of the candidates into the T tree tokens (Section 3.2).
//
// HBM-bound by construction: every weight is read once and used for B <= 16
// multiply-adds, so the kernels are organised around 16-byte coalesced weight loads
// with many loads in flight; activations stay in shared memory in fp32 so that no
// intermediate is rounded.
#include "common.cuh"

namespace mtv {

constexpr int HEADS_THREADS = 256;
constexpr int HEADS_WARPS = HEADS_THREADS / 32;
constexpr int NB_MAX = 4;  // batch rows handled by one pass over the weights

HeadsWs heads_ws_layout(const mtv_tree *t, int B, int H, int V) {
    HeadsWs w;
    // CTAs per head for the vocabulary projection: fill the GPU about twice over all heads
    int per_head = (2 * sm_count() + t->K - 1) / t->K;
    int max_useful = (V + HEADS_WARPS - 1) / HEADS_WARPS;  // at least one row per warp
    if (per_head > max_useful) per_head = max_useful;
    if (per_head < 1) per_head = 1;
    w.ctas_per_head = per_head;
    size_t off = 0;
    w.hprime_off = off;   off = align_up(off + (size_t)t->K * B * H * sizeof(float), 256);
    w.part_val_off = off; off = align_up(off + (size_t)t->K * B * per_head * MTV_MAX_TOPK * sizeof(float), 256);
    w.part_idx_off = off; off = align_up(off + (size_t)t->K * B * per_head * MTV_MAX_TOPK * sizeof(int32_t), 256);
    w.total = off;
    return w;
}

__device__ __forceinline__ void bf16x8_to_float(const uint4 &u, float *f) {
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

__device__ __forceinline__ uint4 ld_stream(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// (value, id) ordering of the candidate lists: larger value first, equal values by smaller id.
__device__ __forceinline__ bool cand_before(float va, int ia, float vb, int ib) {
    return va > vb || (va == vb && ia < ib);
}

// ---------------------------------------------------------------------------
// Residual block:  hprime[k][b][o] = h[b][o] + SiLU(W1[k][o][:] . h[b][:] + b1[k][o])
// One warp per output row, NB batch rows per pass; h staged in shared memory as fp32.
template <int NB>
__global__ void __launch_bounds__(HEADS_THREADS)
heads_resblock_kernel(int B, int H, int K, const __nv_bfloat16 *__restrict__ hidden,
                      const __nv_bfloat16 *__restrict__ W1, const __nv_bfloat16 *__restrict__ b1,
                      float *__restrict__ hprime) {
    extern __shared__ float sh[];  // [NB][H]
    const int b0 = blockIdx.y * NB;
    for (int i = threadIdx.x; i < NB * H; i += HEADS_THREADS) {
        int b = b0 + i / H;
        sh[i] = b < B ? __bfloat162float(hidden[(size_t)b * H + i % H]) : 0.f;
    }
    __syncthreads();
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int rows = K * H;
    for (int row = blockIdx.x * HEADS_WARPS + warp; row < rows; row += gridDim.x * HEADS_WARPS) {
        const __nv_bfloat16 *w = W1 + (size_t)row * H;
        float acc[NB];
#pragma unroll
        for (int b = 0; b < NB; ++b) acc[b] = 0.f;
        for (int h0 = lane * 8; h0 < H; h0 += 256) {
            float wf[8];
            bf16x8_to_float(ld_stream(w + h0), wf);
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                const float4 x0 = *reinterpret_cast<const float4 *>(sh + b * H + h0);
                const float4 x1 = *reinterpret_cast<const float4 *>(sh + b * H + h0 + 4);
                acc[b] = fmaf(wf[0], x0.x, acc[b]); acc[b] = fmaf(wf[1], x0.y, acc[b]);
                acc[b] = fmaf(wf[2], x0.z, acc[b]); acc[b] = fmaf(wf[3], x0.w, acc[b]);
                acc[b] = fmaf(wf[4], x1.x, acc[b]); acc[b] = fmaf(wf[5], x1.y, acc[b]);
                acc[b] = fmaf(wf[6], x1.z, acc[b]); acc[b] = fmaf(wf[7], x1.w, acc[b]);
            }
        }
        const int k = row / H, o = row % H;
        const float bias = b1 ? __bfloat162float(b1[row]) : 0.f;
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            float y = warp_sum(acc[b]) + bias;
            if (lane == 0 && b0 + b < B) {
                float silu = y / (1.f + expf(-y));
                hprime[((size_t)k * B + b0 + b) * H + o] = sh[b * H + o] + silu;
            }
        }
    }
}

// ---------------------------------------------------------------------------
// Vocabulary projection with fused partial top-k.
// grid = (ctas_per_head, K, ceil(B/NB)).  A CTA owns a contiguous slab of vocabulary
// rows of one head; each warp walks its rows two at a time, keeps the dot products of
// NB batch rows in registers and inserts a logit into its private sorted list only
// when it beats the list's last entry.  At the end the warps' lists are merged and
// the CTA's best kd entries per batch row go to the workspace.
template <int NB>
__global__ void __launch_bounds__(HEADS_THREADS)
heads_vocab_topk_kernel(int B, int H, int V, const __nv_bfloat16 *__restrict__ W2,
                        const float *__restrict__ hprime, const int32_t *__restrict__ kd_arr,
                        float *__restrict__ part_val, int32_t *__restrict__ part_idx) {
    extern __shared__ float sh[];                   // [NB][H] then the lists
    float *xs = sh;
    float *lval = sh + (size_t)NB * H;              // [WARPS][NB][16]
    int32_t *lidx = reinterpret_cast<int32_t *>(lval + HEADS_WARPS * NB * MTV_MAX_TOPK);
    const int k = blockIdx.y, b0 = blockIdx.z * NB;
    const int kd = kd_arr[k];
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int per = gridDim.x;
    if (kd == 0) return;

    for (int i = threadIdx.x; i < NB * H; i += HEADS_THREADS) {
        int b = b0 + i / H;
        xs[i] = b < B ? hprime[((size_t)k * B + b) * H + i % H] : 0.f;
    }
    for (int i = threadIdx.x; i < HEADS_WARPS * NB * MTV_MAX_TOPK; i += HEADS_THREADS) {
        lval[i] = -INFINITY;
        lidx[i] = 0x7fffffff;
    }
    __syncthreads();

    // slab of this CTA
    const int rows_per = (V + per - 1) / per;
    const int v_begin = blockIdx.x * rows_per;
    const int v_end = min(V, v_begin + rows_per);
    float *my_val = lval + (warp * NB) * MTV_MAX_TOPK;
    int32_t *my_idx = lidx + (warp * NB) * MTV_MAX_TOPK;
    float thr_v[NB];
    int thr_i[NB];
#pragma unroll
    for (int b = 0; b < NB; ++b) { thr_v[b] = -INFINITY; thr_i[b] = 0x7fffffff; }

    const __nv_bfloat16 *Wk = W2 + (size_t)k * V * H;
    constexpr int R = 2;  // rows per warp iteration
    for (int v0 = v_begin + warp * R; v0 < v_end; v0 += HEADS_WARPS * R) {
        float acc[R][NB];
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int b = 0; b < NB; ++b) acc[r][b] = 0.f;
        const bool has1 = v0 + 1 < v_end;
        const __nv_bfloat16 *w0 = Wk + (size_t)v0 * H;
        const __nv_bfloat16 *w1 = has1 ? w0 + H : w0;
#pragma unroll 2
        for (int h0 = lane * 8; h0 < H; h0 += 256) {
            float wf[R][8];
            const uint4 u0 = ld_stream(w0 + h0);
            const uint4 u1 = ld_stream(w1 + h0);
            bf16x8_to_float(u0, wf[0]);
            bf16x8_to_float(u1, wf[1]);
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                const float4 x0 = *reinterpret_cast<const float4 *>(xs + b * H + h0);
                const float4 x1 = *reinterpret_cast<const float4 *>(xs + b * H + h0 + 4);
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    float a = acc[r][b];
                    a = fmaf(wf[r][0], x0.x, a); a = fmaf(wf[r][1], x0.y, a);
                    a = fmaf(wf[r][2], x0.z, a); a = fmaf(wf[r][3], x0.w, a);
                    a = fmaf(wf[r][4], x1.x, a); a = fmaf(wf[r][5], x1.y, a);
                    a = fmaf(wf[r][6], x1.z, a); a = fmaf(wf[r][7], x1.w, a);
                    acc[r][b] = a;
                }
            }
        }
#pragma unroll
        for (int r = 0; r < R; ++r) {
            if (r == 1 && !has1) break;
            const int v = v0 + r;
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                const float z = warp_sum(acc[r][b]);  // identical in every lane
                if (cand_before(z, v, thr_v[b], thr_i[b])) {
                    if (lane == 0) {
                        // insertion into the sorted list of kd entries
                        int pos = kd - 1;
                        while (pos > 0 && cand_before(z, v, my_val[b * MTV_MAX_TOPK + pos - 1],
                                                      my_idx[b * MTV_MAX_TOPK + pos - 1])) {
                            my_val[b * MTV_MAX_TOPK + pos] = my_val[b * MTV_MAX_TOPK + pos - 1];
                            my_idx[b * MTV_MAX_TOPK + pos] = my_idx[b * MTV_MAX_TOPK + pos - 1];
                            --pos;
                        }
                        my_val[b * MTV_MAX_TOPK + pos] = z;
                        my_idx[b * MTV_MAX_TOPK + pos] = v;
                    }
                    __syncwarp();
                    thr_v[b] = my_val[b * MTV_MAX_TOPK + kd - 1];
                    thr_i[b] = my_idx[b * MTV_MAX_TOPK + kd - 1];
                }
            }
        }
    }
    __syncthreads();
    // merge the warps' lists: rank each entry among all HEADS_WARPS*kd entries of its batch row
    for (int e = threadIdx.x; e < NB * HEADS_WARPS * MTV_MAX_TOPK; e += HEADS_THREADS) {
        const int b = e / (HEADS_WARPS * MTV_MAX_TOPK);
        const int w = (e / MTV_MAX_TOPK) % HEADS_WARPS, s = e % MTV_MAX_TOPK;
        if (s >= kd || b0 + b >= B) continue;
        const float z = lval[(w * NB + b) * MTV_MAX_TOPK + s];
        const int id = lidx[(w * NB + b) * MTV_MAX_TOPK + s];
        int rank = 0;
        for (int w2 = 0; w2 < HEADS_WARPS; ++w2)
            for (int s2 = 0; s2 < kd; ++s2) {
                const float z2 = lval[(w2 * NB + b) * MTV_MAX_TOPK + s2];
                const int id2 = lidx[(w2 * NB + b) * MTV_MAX_TOPK + s2];
                // entries with the sentinel id are all "equal"; order them by position
                if (cand_before(z2, id2, z, id) || (z2 == z && id2 == id && (w2 * MTV_MAX_TOPK + s2) < (w * MTV_MAX_TOPK + s)))
                    ++rank;
            }
        if (rank < kd) {
            const size_t o = (((size_t)k * B + b0 + b) * per + blockIdx.x) * MTV_MAX_TOPK + rank;
            part_val[o] = z;
            part_idx[o] = id;
        }
    }
}

// ---------------------------------------------------------------------------
// Final merge + expansion.  grid = B, block = K * 128 threads: thread group d merges
// head d's per-CTA lists into cand[b][offset_d ..], then the block gathers
// tree_tok[b][i] = cand[b][tree_indices[i]].
constexpr int MERGE_GROUP = 128;
__global__ void heads_merge_expand_kernel(int B, int K, int T, int C, int per,
                                          const float *__restrict__ part_val,
                                          const int32_t *__restrict__ part_idx,
                                          const int32_t *__restrict__ kd_arr,
                                          const int32_t *__restrict__ off_arr,
                                          const int32_t *__restrict__ tree_indices,
                                          const int32_t *__restrict__ root_tok,
                                          int32_t *__restrict__ cand, float *__restrict__ cand_logit,
                                          int32_t *__restrict__ tree_tok) {
    extern __shared__ float sh[];  // per group: per*16 values, per*16 ids
    const int b = blockIdx.x;
    const int d = threadIdx.x / MERGE_GROUP, t = threadIdx.x % MERGE_GROUP;
    const int kd = kd_arr[d], off = off_arr[d];
    const int n = per * kd;
    float *val = sh + (size_t)d * per * MTV_MAX_TOPK * 2;
    int32_t *idx = reinterpret_cast<int32_t *>(val + per * MTV_MAX_TOPK);
    for (int e = t; e < n; e += MERGE_GROUP) {
        const size_t o = (((size_t)d * B + b) * per + e / kd) * MTV_MAX_TOPK + e % kd;
        val[e] = part_val[o];
        idx[e] = part_idx[o];
    }
    __syncthreads();
    for (int e = t; e < n; e += MERGE_GROUP) {
        const float z = val[e];
        const int id = idx[e];
        int rank = 0;
        for (int e2 = 0; e2 < n && rank < kd; ++e2)
            if (cand_before(val[e2], idx[e2], z, id) || (val[e2] == z && idx[e2] == id && e2 < e)) ++rank;
        if (rank < kd) {
            cand[(size_t)b * C + off + rank] = id;
            if (cand_logit) cand_logit[(size_t)b * (C - 1) + off - 1 + rank] = z;
        }
    }
    if (threadIdx.x == 0) cand[(size_t)b * C] = root_tok[b];
    __threadfence_block();
    __syncthreads();
    for (int i = threadIdx.x; i < T; i += blockDim.x)
        tree_tok[(size_t)b * T + i] = cand[(size_t)b * C + tree_indices[i]];
}

template <int NB>
static int launch_heads(const mtv_tree *t, int B, int H, int V, const __nv_bfloat16 *hidden,
                        const __nv_bfloat16 *W1, const __nv_bfloat16 *b1, const __nv_bfloat16 *W2,
                        const HeadsWs &L, char *ws, cudaStream_t st) {
    float *hprime = reinterpret_cast<float *>(ws + L.hprime_off);
    float *pv = reinterpret_cast<float *>(ws + L.part_val_off);
    int32_t *pi = reinterpret_cast<int32_t *>(ws + L.part_idx_off);
    const int btiles = (B + NB - 1) / NB;
    const size_t sm1 = (size_t)NB * H * sizeof(float);
    const size_t sm2 = sm1 + (size_t)HEADS_WARPS * NB * MTV_MAX_TOPK * 8;
    if (sm2 > 227 * 1024) return MTV_ERR_UNSUPPORTED_SHAPE;
    static bool attr_done = false;
    if (!attr_done) {
        MTV_CUDA_CHECK(cudaFuncSetAttribute(heads_resblock_kernel<NB>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        MTV_CUDA_CHECK(cudaFuncSetAttribute(heads_vocab_topk_kernel<NB>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        attr_done = true;
    }
    int g1 = (t->K * H + HEADS_WARPS - 1) / HEADS_WARPS;
    const int cap = 4 * sm_count();
    if (g1 > cap) g1 = cap;
    {
        TapScope tap(MTV_KERNEL_HEADS_RESBLOCK, st);
        heads_resblock_kernel<NB><<<dim3(g1, btiles), HEADS_THREADS, sm1, st>>>(B, H, t->K, hidden, W1, b1, hprime);
    }
    {
        TapScope tap(MTV_KERNEL_HEADS_VOCAB_TOPK, st);
        heads_vocab_topk_kernel<NB><<<dim3(L.ctas_per_head, t->K, btiles), HEADS_THREADS, sm2, st>>>(
            B, H, V, W2, hprime, t->d_kd, pv, pi);
    }
    return MTV_OK;
}

}  // namespace mtv

extern "C" int medusa_heads_topk(const mtv_tree_t *tree, int B, int H, int V,
                                 const mtv_bf16 *hidden, const mtv_bf16 *W1, const mtv_bf16 *b1,
                                 const mtv_bf16 *W2, const int32_t *root_tok,
                                 int32_t *cand, float *cand_logit, int32_t *tree_tok,
                                 void *ws, size_t ws_bytes, void *stream) {
    using namespace mtv;
    if (!tree || !tree->on_device || !hidden || !W1 || !W2 || !root_tok || !cand || !tree_tok || !ws)
        return MTV_ERR_INVALID_ARG;
    if (B < 1 || H < 8 || V < 1) return MTV_ERR_INVALID_ARG;
    if (B > 16 || H % 8 != 0) return MTV_ERR_UNSUPPORTED_SHAPE;
    for (int d = 0; d < tree->K; ++d)
        if (tree->k_d[d] > V) return MTV_ERR_INVALID_ARG;
    const HeadsWs L = heads_ws_layout(tree, B, H, V);
    if (ws_bytes < L.total) return MTV_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    auto *h = reinterpret_cast<const __nv_bfloat16 *>(hidden);
    auto *w1 = reinterpret_cast<const __nv_bfloat16 *>(W1);
    auto *bb = reinterpret_cast<const __nv_bfloat16 *>(b1);
    auto *w2 = reinterpret_cast<const __nv_bfloat16 *>(W2);
    int rc;
    if (B == 1) rc = launch_heads<1>(tree, B, H, V, h, w1, bb, w2, L, (char *)ws, st);
    else if (B == 2) rc = launch_heads<2>(tree, B, H, V, h, w1, bb, w2, L, (char *)ws, st);
    else rc = launch_heads<NB_MAX>(tree, B, H, V, h, w1, bb, w2, L, (char *)ws, st);
    if (rc != MTV_OK) return rc;
    const size_t smm = (size_t)tree->K * L.ctas_per_head * MTV_MAX_TOPK * 8;
    if (smm > 200 * 1024) return MTV_ERR_UNSUPPORTED_SHAPE;
    static bool attr_done = false;
    if (!attr_done) {
        MTV_CUDA_CHECK(cudaFuncSetAttribute(heads_merge_expand_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
        attr_done = true;
    }
    TapScope tap(MTV_KERNEL_HEADS_MERGE, st);
    heads_merge_expand_kernel<<<B, tree->K * MERGE_GROUP, smm, st>>>(
        B, tree->K, tree->T, tree->C, L.ctas_per_head,
        reinterpret_cast<const float *>((char *)ws + L.part_val_off),
        reinterpret_cast<const int32_t *>((char *)ws + L.part_idx_off), tree->d_kd, tree->d_cand_offset,
        tree->d_tree_indices, root_tok, cand, cand_logit, tree_tok);
    MTV_CUDA_CHECK(cudaGetLastError());
    return MTV_OK;
}
