// Tree attention (Section 3.2 / Fig. 2(b)): all T tree nodes attend to the prefix and to
// their ancestors-or-self among the tree rows of the KV cache.
//
// GQA-grouped: the G = Hq/Hkv query heads that share a KV head and the T nodes form one
// (T*G) x D query block, so every K/V row fetched from HBM serves T*G queries.  Split
// over the key range (flash-decoding): each CTA produces an unnormalised partial
// (running max m, sum l, O) for its key range; a second kernel merges the partials.
// The visibility matrix is applied as a per-node ancestor bitmask, and only on the key
// tiles that overlap the tree rows.
#include "common.cuh"

namespace mtv {

constexpr int BM = 128;          // query rows per CTA (8 warps x 16 rows)
constexpr int BN = 64;           // keys per tile
constexpr int ATT_THREADS = 256;
constexpr float LOG2E = 1.4426950408889634f;

bool attn_tc_eligible(int D, int G);
int attn_tc_plan(int T, int G, int B, int Hkv, int Lcap, int *n_rt_out);
int launch_tree_attn_tc(const mtv_tree *tree, int B, int Hq, int Hkv, const __nv_bfloat16 *q, const __nv_bfloat16 *k,
                        const __nv_bfloat16 *v, int64_t sb, int64_t sh, int64_t st, int Lcap, const int32_t *seq_lens,
                        float scale_log2, __nv_bfloat16 *out, int32_t *status, void *ws_o, float *ws_ml, int32_t *ws_order,
                        cudaStream_t stream);

AttnWs attn_ws_layout(const mtv_tree *t, int B, int Hq, int Hkv, int D, int Lcap) {
    AttnWs w;
    const int G = Hq / Hkv;
    const int M = t->T * G;
    w.use_tc = attn_tc_eligible(D, G);
    if (w.use_tc) {   // one launch; partials of the key splits pass through the workspace
        int n_rt = 1;
        w.nsplit = attn_tc_plan(t->T, G, B, Hkv, Lcap, &n_rt);
        w.m_rows = 256;
        const size_t slabs = w.nsplit > 1 ? (size_t)B * Hkv * n_rt * w.nsplit : 0;
        w.o_off = 0;
        w.ml_off = align_up(slabs * 256 * D * sizeof(__nv_bfloat16), 256);
        w.order_off = align_up(w.ml_off + slabs * 256 * 2 * sizeof(float), 256);   // sequences by descending length
        w.total = align_up(w.order_off + (size_t)B * sizeof(int32_t), 256) + 256;
        return w;
    }
    const int mblocks = (M + BM - 1) / BM;
    w.m_rows = mblocks * BM;
    long ctas = (long)B * Hkv * mblocks;
    int ns = (int)(sm_count() / ctas);
    const int tiles = (Lcap + BN - 1) / BN;
    if (ns > tiles) ns = tiles;
    if (ns < 1 || tiles <= 4) ns = 1;   // a few tiles: one CTA per block writes the output itself (one launch instead of two)
    w.nsplit = ns;
    size_t off = 0;
    w.o_off = off;  off = align_up(off + (size_t)B * Hkv * ns * w.m_rows * D * sizeof(float), 256);
    w.ml_off = off; off = align_up(off + (size_t)B * Hkv * ns * w.m_rows * 2 * sizeof(float), 256);
    w.total = off;
    return w;
}

struct AttnParams {
    const __nv_bfloat16 *q, *k, *v;
    __nv_bfloat16 *out;
    int64_t sb, sh, st;
    const int32_t *seq_lens;
    const uint64_t *anc;  // [T][2]
    int32_t *status;
    float *ws_o, *ws_ml;
    float scale_log2;
    int B, T, Hq, Hkv, G, Lcap, nsplit, m_rows;
};

__device__ __forceinline__ void cp_async16(uint32_t smem, const void *gmem, bool valid) {
    const int sz = valid ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem), "l"(gmem), "r"(sz));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N)); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&h);
}

// Range of key tiles handled by split s of a sequence with n_keys visible-candidate rows.
__device__ __forceinline__ void split_range(int n_keys, int nsplit, int s, int &t_begin, int &t_end) {
    const int tiles = (n_keys + BN - 1) / BN;
    const int per = (tiles + nsplit - 1) / nsplit;
    t_begin = min(tiles, s * per);
    t_end = min(tiles, t_begin + per);
}

template <int D>
__global__ void __launch_bounds__(ATT_THREADS, 1)
tree_attn_partial_kernel(const AttnParams p) {
    constexpr int ROWB = D * 2;       // bytes per K/V row
    constexpr int CH = D / 8;         // 16-byte chunks per row
    constexpr int TILE_B = BN * ROWB; // bytes per tile
    extern __shared__ __align__(128) unsigned char smem[];
    const uint32_t s_k = (uint32_t)__cvta_generic_to_shared(smem);  // 2 stages of K then 2 of V
    const uint32_t s_v = s_k + 2 * TILE_B;

    const int split = blockIdx.x;
    const int mblocks = p.m_rows / BM;
    const int g = blockIdx.y / mblocks, mb = blockIdx.y % mblocks;
    const int b = blockIdx.z;
    const int L = p.seq_lens[b];
    if (p.nsplit == 1 && p.status && blockIdx.y == 0 && threadIdx.x == 0)   // no combine kernel follows: report here
        p.status[b] = L + p.T > p.Lcap ? MTV_ERR_CAPACITY : MTV_OK;
    if (L + p.T > p.Lcap) return;     // (with splits: reported by the combine kernel)
    const int n_keys = L + p.T;
    int t_begin, t_end;
    split_range(n_keys, p.nsplit, split, t_begin, t_end);

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int gq = lane / 4, tq = lane % 4;
    const int M = p.T * p.G;
    const int r0 = mb * BM + warp * 16 + gq, r1 = r0 + 8;

    // Q fragments straight from global memory (row r = node*G + head-in-group)
    uint32_t qf[D / 16][4];
    {
        const int i0 = r0 / p.G, j0 = r0 % p.G, i1 = r1 / p.G, j1 = r1 % p.G;
        const uint32_t *q0 = reinterpret_cast<const uint32_t *>(p.q + (((size_t)b * p.T + i0) * p.Hq + g * p.G + j0) * D);
        const uint32_t *q1 = reinterpret_cast<const uint32_t *>(p.q + (((size_t)b * p.T + i1) * p.Hq + g * p.G + j1) * D);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
            qf[kk][0] = r0 < M ? q0[kk * 8 + tq] : 0u;
            qf[kk][1] = r1 < M ? q1[kk * 8 + tq] : 0u;
            qf[kk][2] = r0 < M ? q0[kk * 8 + 4 + tq] : 0u;
            qf[kk][3] = r1 < M ? q1[kk * 8 + 4 + tq] : 0u;
        }
    }
    // ancestor bitmasks of the two rows' nodes (rows past M see everything: they are never stored)
    uint64_t a0lo = ~0ull, a0hi = ~0ull, a1lo = ~0ull, a1hi = ~0ull;
    if (r0 < M) { a0lo = p.anc[(r0 / p.G) * 2]; a0hi = p.anc[(r0 / p.G) * 2 + 1]; }
    if (r1 < M) { a1lo = p.anc[(r1 / p.G) * 2]; a1hi = p.anc[(r1 / p.G) * 2 + 1]; }

    const __nv_bfloat16 *kbase = p.k + b * p.sb + g * p.sh;
    const __nv_bfloat16 *vbase = p.v + b * p.sb + g * p.sh;

    auto load_tile = [&](int tile, int stage) {
        const int key0 = tile * BN;
#pragma unroll
        for (int it = 0; it < BN * CH / ATT_THREADS; ++it) {
            const int e = it * ATT_THREADS + threadIdx.x;
            const int row = e / CH, c = e % CH;
            const int key = key0 + row;
            const bool ok = key < n_keys;
            const int64_t goff = (int64_t)(ok ? key : 0) * p.st + c * 8;
            const uint32_t soff = stage * TILE_B + row * ROWB + ((c ^ (row & 7)) * 16);
            cp_async16(s_k + soff, kbase + goff, ok);
            cp_async16(s_v + soff, vbase + goff, ok);
        }
    };

    float o[D / 8][4];
#pragma unroll
    for (int j = 0; j < D / 8; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

    if (t_begin < t_end) load_tile(t_begin, 0);
    cp_async_commit();

    for (int tile = t_begin; tile < t_end; ++tile) {
        const int stage = (tile - t_begin) & 1;
        if (tile + 1 < t_end) load_tile(tile + 1, stage ^ 1);
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();

        // S = Q K^T  (16 x BN per warp)
        float s[BN / 8][4];
#pragma unroll
        for (int j = 0; j < BN / 8; ++j) s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
        const uint32_t kst = s_k + stage * TILE_B;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
#pragma unroll
            for (int j = 0; j < BN / 8; j += 2) {
                const int mi = lane / 8;
                const int row = (j + mi / 2) * 8 + lane % 8;
                const int c = kk * 2 + (mi & 1);
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4(kst + row * ROWB + ((c ^ (row & 7)) * 16), b0, b1, b2, b3);
                mma_bf16(s[j], qf[kk], b0, b1);
                mma_bf16(s[j + 1], qf[kk], b2, b3);
            }
        }
        // scale, mask
        const int key0 = tile * BN;
        const bool need_mask = key0 + BN > L;
#pragma unroll
        for (int j = 0; j < BN / 8; ++j) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float x = s[j][e] * p.scale_log2;
                if (need_mask) {
                    const int key = key0 + j * 8 + tq * 2 + (e & 1);
                    bool vis = key < L;
                    if (!vis && key < n_keys) {
                        const int a = key - L;
                        const uint64_t lo = (e & 2) ? a1lo : a0lo, hi = (e & 2) ? a1hi : a0hi;
                        vis = ((a < 64 ? lo >> a : hi >> (a - 64)) & 1ull) != 0;
                    }
                    if (!vis) x = -INFINITY;
                }
                s[j][e] = x;
            }
        }
        // online softmax (base 2)
        float mx0 = m0, mx1 = m1;
#pragma unroll
        for (int j = 0; j < BN / 8; ++j) {
            mx0 = fmaxf(mx0, fmaxf(s[j][0], s[j][1]));
            mx1 = fmaxf(mx1, fmaxf(s[j][2], s[j][3]));
        }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        const float use0 = mx0 == -INFINITY ? 0.f : mx0, use1 = mx1 == -INFINITY ? 0.f : mx1;
        const float al0 = exp2f(m0 - use0), al1 = exp2f(m1 - use1);  // m = -inf -> 0
        m0 = mx0; m1 = mx1;
        l0 *= al0; l1 *= al1;
#pragma unroll
        for (int j = 0; j < D / 8; ++j) { o[j][0] *= al0; o[j][1] *= al0; o[j][2] *= al1; o[j][3] *= al1; }
        uint32_t pa[BN / 16][4];
#pragma unroll
        for (int j = 0; j < BN / 8; ++j) {
            const float p0 = exp2f(s[j][0] - use0), p1 = exp2f(s[j][1] - use0);
            const float p2 = exp2f(s[j][2] - use1), p3 = exp2f(s[j][3] - use1);
            l0 += p0 + p1; l1 += p2 + p3;
            pa[j / 2][(j & 1) * 2] = pack_bf16(p0, p1);
            pa[j / 2][(j & 1) * 2 + 1] = pack_bf16(p2, p3);
        }
        // O += P V
        const uint32_t vst = s_v + stage * TILE_B;
#pragma unroll
        for (int kk = 0; kk < BN / 16; ++kk) {
#pragma unroll
            for (int j = 0; j < D / 8; j += 2) {
                const int mi = lane / 8;
                const int row = kk * 16 + (mi & 1) * 8 + lane % 8;
                const int c = j + mi / 2;
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4_trans(vst + row * ROWB + ((c ^ (row & 7)) * 16), b0, b1, b2, b3);
                mma_bf16(o[j], pa[kk], b0, b1);
                mma_bf16(o[j + 1], pa[kk], b2, b3);
            }
        }
        __syncthreads();  // the stage is free for the load issued next iteration
    }
    cp_async_wait<0>();

    l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);

    if (p.nsplit == 1) {
        // the only split of its block: normalise and write the output rows (row r = node * G + head-in-group)
        const float inv0 = l0 > 0.f ? 1.f / l0 : 0.f, inv1 = l1 > 0.f ? 1.f / l1 : 0.f;
        __nv_bfloat16 *o0 = p.out + (((size_t)b * p.T + r0 / p.G) * p.Hq + g * p.G + r0 % p.G) * D;
        __nv_bfloat16 *o1 = p.out + (((size_t)b * p.T + r1 / p.G) * p.Hq + g * p.G + r1 % p.G) * D;
#pragma unroll
        for (int j = 0; j < D / 8; ++j) {
            if (r0 < M) *reinterpret_cast<uint32_t *>(o0 + j * 8 + tq * 2) = pack_bf16(o[j][0] * inv0, o[j][1] * inv0);
            if (r1 < M) *reinterpret_cast<uint32_t *>(o1 + j * 8 + tq * 2) = pack_bf16(o[j][2] * inv1, o[j][3] * inv1);
        }
        return;
    }
    const size_t slab = (((size_t)b * p.Hkv + g) * p.nsplit + split) * p.m_rows;
    float *wo0 = p.ws_o + (slab + r0) * D, *wo1 = p.ws_o + (slab + r1) * D;
#pragma unroll
    for (int j = 0; j < D / 8; ++j) {
        *reinterpret_cast<float2 *>(wo0 + j * 8 + tq * 2) = make_float2(o[j][0], o[j][1]);
        *reinterpret_cast<float2 *>(wo1 + j * 8 + tq * 2) = make_float2(o[j][2], o[j][3]);
    }
    if (tq == 0) {
        *reinterpret_cast<float2 *>(p.ws_ml + (slab + r0) * 2) = make_float2(m0, l0);
        *reinterpret_cast<float2 *>(p.ws_ml + (slab + r1) * 2) = make_float2(m1, l1);
    }
}

// grid = B*T*Hq, block = D threads: merge the splits of one output row.
template <int D>
__global__ void __launch_bounds__(D)
tree_attn_combine_kernel(const AttnParams p) {
    const int row = blockIdx.x;
    const int h = row % p.Hq, i = (row / p.Hq) % p.T, b = row / (p.Hq * p.T);
    const int L = p.seq_lens[b];
    if (L + p.T > p.Lcap) {
        if (p.status && h == 0 && i == 0 && threadIdx.x == 0) p.status[b] = MTV_ERR_CAPACITY;
        return;
    }
    if (p.status && h == 0 && i == 0 && threadIdx.x == 0) p.status[b] = MTV_OK;
    const int g = h / p.G, r = i * p.G + h % p.G;
    const size_t base = ((size_t)b * p.Hkv + g) * p.nsplit * p.m_rows + r;
    float m = -INFINITY;
    for (int s = 0; s < p.nsplit; ++s) m = fmaxf(m, p.ws_ml[(base + (size_t)s * p.m_rows) * 2]);
    float l = 0.f, acc = 0.f;
    for (int s = 0; s < p.nsplit; ++s) {
        const size_t e = base + (size_t)s * p.m_rows;
        const float ms = p.ws_ml[e * 2];
        if (ms == -INFINITY) continue;
        const float w = exp2f(ms - m);
        l += w * p.ws_ml[e * 2 + 1];
        acc += w * p.ws_o[e * D + threadIdx.x];
    }
    p.out[(size_t)row * D + threadIdx.x] = __float2bfloat16_rn(acc / l);
}

}  // namespace mtv

extern "C" int tree_verify_attention(const mtv_tree_t *tree, int B, int Hq, int Hkv, int D,
                                     const mtv_bf16 *q, const mtv_bf16 *k_cache, const mtv_bf16 *v_cache,
                                     int64_t stride_b, int64_t stride_h, int64_t stride_t, int Lcap,
                                     const int32_t *seq_lens, float scale,
                                     mtv_bf16 *out, int32_t *status,
                                     void *ws, size_t ws_bytes, void *stream) {
    using namespace mtv;
    MTV_RANGE("tree_verify_attention");
    if (!tree || !tree->on_device || !q || !k_cache || !v_cache || !seq_lens || !out || !ws) return MTV_ERR_INVALID_ARG;
    if (B < 1 || Hq < 1 || Hkv < 1 || Lcap < tree->T) return MTV_ERR_INVALID_ARG;
    if ((D != 64 && D != 128) || Hq % Hkv != 0 || Hq / Hkv > 8 || B > 65535) return MTV_ERR_UNSUPPORTED_SHAPE;
    if (stride_t % 8 || stride_h % 8 || stride_b % 8 || stride_t < D) return MTV_ERR_INVALID_ARG;
    if (((uintptr_t)k_cache | (uintptr_t)v_cache | (uintptr_t)q | (uintptr_t)out) & 15) return MTV_ERR_INVALID_ARG;
    const AttnWs Lw = attn_ws_layout(tree, B, Hq, Hkv, D, Lcap);
    if (ws_bytes < Lw.total) return MTV_ERR_WORKSPACE;
    AttnParams p;
    p.q = reinterpret_cast<const __nv_bfloat16 *>(q);
    p.k = reinterpret_cast<const __nv_bfloat16 *>(k_cache);
    p.v = reinterpret_cast<const __nv_bfloat16 *>(v_cache);
    p.out = reinterpret_cast<__nv_bfloat16 *>(out);
    p.sb = stride_b; p.sh = stride_h; p.st = stride_t;
    p.seq_lens = seq_lens;
    p.anc = tree->d_anc;
    p.status = status;
    p.ws_o = reinterpret_cast<float *>((char *)ws + Lw.o_off);
    p.ws_ml = reinterpret_cast<float *>((char *)ws + Lw.ml_off);
    p.scale_log2 = (scale == 0.f ? 1.f / sqrtf((float)D) : scale) * LOG2E;
    p.B = B; p.T = tree->T; p.Hq = Hq; p.Hkv = Hkv; p.G = Hq / Hkv; p.Lcap = Lcap;
    p.nsplit = Lw.nsplit; p.m_rows = Lw.m_rows;
    cudaStream_t st = (cudaStream_t)stream;
    if (Lw.use_tc && scale >= 0.f) {
        // tcgen05 path: head_dim 128, query groups of up to 8 heads; one launch
        TapScope tap(MTV_KERNEL_ATTN_PARTIAL, st);
        const int rc = launch_tree_attn_tc(tree, B, Hq, Hkv, p.q, p.k, p.v, stride_b, stride_h, stride_t, Lcap, seq_lens,
                                           p.scale_log2, p.out, status, p.ws_o, p.ws_ml,
                                           reinterpret_cast<int32_t *>((char *)ws + Lw.order_off), st);
        if (rc != MTV_OK) return rc;
        MTV_CUDA_CHECK(cudaGetLastError());
        return MTV_OK;
    } else {
        if (Lw.use_tc) return MTV_ERR_INVALID_ARG;   // a negative scale
        const dim3 grid(Lw.nsplit, Hkv * (Lw.m_rows / BM), B);
        const size_t smem = (size_t)4 * BN * D * 2;
        static PerDeviceOnce attr_once;
        bool *attr_done = attr_once.flag();
        if (!attr_done || !*attr_done) {
            MTV_CUDA_CHECK(cudaFuncSetAttribute(tree_attn_partial_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, 4 * BN * 64 * 2));
            MTV_CUDA_CHECK(cudaFuncSetAttribute(tree_attn_partial_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, 4 * BN * 128 * 2));
            if (attr_done) *attr_done = true;
        }
        TapScope tap(MTV_KERNEL_ATTN_PARTIAL, st);
        if (D == 64) tree_attn_partial_kernel<64><<<grid, ATT_THREADS, smem, st>>>(p);
        else tree_attn_partial_kernel<128><<<grid, ATT_THREADS, smem, st>>>(p);
    }
    if (Lw.nsplit > 1) {
        TapScope tap(MTV_KERNEL_ATTN_COMBINE, st);
        if (D == 64) tree_attn_combine_kernel<64><<<B * tree->T * Hq, 64, 0, st>>>(p);
        else tree_attn_combine_kernel<128><<<B * tree->T * Hq, 128, 0, st>>>(p);
    }
    MTV_CUDA_CHECK(cudaGetLastError());
    return MTV_OK;
}
