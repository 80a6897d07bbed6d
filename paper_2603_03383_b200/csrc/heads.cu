// Medusa heads (Section 3.1): residual SiLU block, vocabulary projection as a
// weight-streaming matrix-vector product, per-head top-k fused into the projection,
// and the expansion of the candidates into the T tree tokens (Section 3.2).
//
// HBM-bound by construction: every weight is read once and used for B <= 16
// multiply-adds, so the kernels are organised around 16-byte coalesced weight loads
// with many loads in flight; activations stay in shared memory in fp32 so that no
// intermediate is rounded.
#include "common.cuh"
#include "heads_common.cuh"
#include "sm100_ptx.cuh"

namespace mtv {

constexpr int HEADS_THREADS = 256;
constexpr int HEADS_WARPS = HEADS_THREADS / 32;
// one pass over the weights serves 1, 2, 4 or 8 batch rows:
// batch rows per pass for a batch of B rows
static inline int nb_for(int B) { return B == 1 ? 1 : B == 2 ? 2 : B <= 4 ? 4 : 8; }

// vocabulary projection: 2 groups of 8 consumer warps + 1 producer warp
constexpr int VT_GROUP_WARPS = 8;
constexpr int VT_GROUPS = 2;
constexpr int VT_CONS_WARPS = VT_GROUP_WARPS * VT_GROUPS;
constexpr int VT_THREADS = (VT_CONS_WARPS + 1) * 32;
constexpr int VT_MAX_STAGES = 6;
constexpr uint32_t VT_SMEM_MAX = 226 * 1024;  // the opt-in limit minus room for static shared memory

// Shared-memory plan of the vocabulary projection for one (NB, H): rows per stage, number
// of stages, and the byte offsets of every region.
struct VocabSmem {
    int rows_per_stage, n_stages, n_it;
    uint32_t stage_bytes, ring_bytes, xs_off, lists_off, zbuf_off, bars_off, total;
};
static VocabSmem vocab_smem_plan(int NB, int H, int ctas_per_head) {
    VocabSmem s;
    s.n_it = (H / 8 + 31) / 32;                       // 16-byte chunks per lane and row
    const uint32_t row_bytes = (uint32_t)H * 2;
    const uint32_t xs_bytes = (uint32_t)NB * s.n_it * 64 * 16;
    const uint32_t lists_bytes = (uint32_t)VT_CONS_WARPS * NB * MTV_MAX_TOPK * 8;
    const uint32_t merge_bytes = (uint32_t)ctas_per_head * MTV_MAX_TOPK * 8;   // final merge reuses the ring
    const uint32_t zbuf_bytes = NB > 1 ? VT_GROUPS * 2 * VT_GROUP_WARPS * 32 * 4 : 0;   // partial logits of the column parts
    const uint32_t fixed = xs_bytes + lists_bytes + zbuf_bytes + 256;
    s.rows_per_stage = 0;
    for (int rs = VT_GROUP_WARPS; rs >= 1; rs /= 2) {
        const uint32_t sb = rs * row_bytes;
        if (fixed + 2 * sb > VT_SMEM_MAX) continue;
        int n = (int)((VT_SMEM_MAX - fixed) / sb);
        if (n > VT_MAX_STAGES) n = VT_MAX_STAGES;
        // keep at least ~96 KB in flight when the rows are long enough
        s.rows_per_stage = rs; s.n_stages = n; s.stage_bytes = sb;
        break;
    }
    if (s.rows_per_stage == 0) { s.total = 0; return s; }
    s.ring_bytes = s.n_stages * s.stage_bytes;
    if (s.ring_bytes < merge_bytes) s.ring_bytes = (merge_bytes + 127) / 128 * 128;
    s.xs_off = (s.ring_bytes + 127) / 128 * 128;
    s.lists_off = s.xs_off + xs_bytes;
    s.zbuf_off = s.lists_off + lists_bytes;
    s.bars_off = s.zbuf_off + zbuf_bytes;
    s.total = s.bars_off + 256;
    if (s.total > VT_SMEM_MAX) s.total = 0;
    return s;
}

HeadsWs heads_ws_layout(const mtv_tree *t, int B, int H, int V) {
    HeadsWs w;
    // one persistent CTA per SM, the SMs divided evenly among the heads
    int per_head = sm_count() / t->K;
    const int max_useful = (V + VT_GROUP_WARPS - 1) / VT_GROUP_WARPS;
    if (per_head > max_useful) per_head = max_useful;
    if (per_head < 1) per_head = 1;
    w.ctas_per_head = per_head;
    const int btiles = (B + nb_for(B) - 1) / nb_for(B);
    size_t off = 0;
    w.hprime_off = off;   off = align_up(off + (size_t)t->K * B * H * sizeof(float), 256);
    w.part_val_off = off; off = align_up(off + (size_t)t->K * B * per_head * MTV_MAX_TOPK * sizeof(float), 256);
    w.part_idx_off = off; off = align_up(off + (size_t)t->K * B * per_head * MTV_MAX_TOPK * sizeof(int32_t), 256);
    w.counters_off = off; off = align_up(off + (size_t)(t->K + 1) * btiles * sizeof(int32_t), 256);
    w.n_counters = (t->K + 1) * btiles;
    w.use_tc = heads_tc_eligible(B, H);
    w.xsplit_off = off;
    if (w.use_tc) off = align_up(off + heads_tc_xsplit_bytes(t->K, H), 256);
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

// Sum over the 32 lanes of N per-lane values at once (N a power of two <= 32): afterwards lane l holds
// in v[0] the sum of value number l / (32 / N).  N - 1 + log2(32 / N) shuffles instead of 5 N.
template <int N>
__device__ __forceinline__ void warp_sum_scatter(float (&v)[N], int lane) {
    int n = N;
#pragma unroll
    for (int bit = 16; bit >= 1; bit >>= 1) {
        if (n > 1) {
            n >>= 1;
            const bool up = (lane & bit) != 0;
#pragma unroll
            for (int i = 0; i < N / 2; ++i) {
                if (i < n) {
                    const float send = up ? v[i] : v[i + n];
                    const float keep = up ? v[i + n] : v[i];
                    v[i] = keep + __shfl_xor_sync(0xffffffffu, send, bit);
                }
            }
        } else {
            v[0] += __shfl_xor_sync(0xffffffffu, v[0], bit);
        }
    }
}

// ---------------------------------------------------------------------------
// Residual block:  hprime[k][b][o] = h[b][o] + SiLU(W1[k][o][:] . h[b][:] + b1[k][o])
// One warp per output row, NB batch rows per pass; h staged in shared memory as fp32.
template <int NB>
__global__ void __launch_bounds__(HEADS_THREADS)
heads_resblock_kernel(int B, int H, int K, const __nv_bfloat16 *__restrict__ hidden,
                      const __nv_bfloat16 *__restrict__ W1, const __nv_bfloat16 *__restrict__ b1,
                      float *__restrict__ hprime, int32_t *__restrict__ counters, int n_counters) {
    extern __shared__ float sh[];  // [NB][H]
    const int b0 = blockIdx.y * NB;
    // tickets of the vocabulary kernel (the next launch on the stream) start at zero
    if (blockIdx.x == 0 && blockIdx.y == 0)
        for (int i = threadIdx.x; i < n_counters; i += HEADS_THREADS) counters[i] = 0;
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
#pragma unroll 4
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
// Vocabulary projection with fused top-k, merge and tree expansion.
//
// grid = (ctas_per_head, K, ceil(B/NB)): one persistent CTA per SM, each owning a
// contiguous slab of one head's vocabulary rows.  A producer warp streams the slab
// through a ring of shared-memory stages with bulk (TMA) copies, one copy per weight
// row, completion counted on an mbarrier per stage, so that the bytes in flight per SM
// do not depend on how many registers the consumers have.  Two groups of eight consumer
// warps take alternate stages; a warp computes the dot products of one weight row with
// NB activation rows (fp32 activations in shared memory, laid out so that a warp's
// 16-byte reads are conflict-free) and inserts a logit into its private sorted list only
// when it beats the list's last entry.  Afterwards the warps' lists are merged per CTA;
// the last CTA of a head (atomic ticket, no waiting) merges the CTAs' lists into the
// candidate buffer, and the last head to finish expands the candidates into tree tokens.
template <int NB>
__global__ void __launch_bounds__(VT_THREADS, 1)
heads_vocab_topk_kernel(const VocabParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    float4 *xs4 = reinterpret_cast<float4 *>(smem + p.xs_off);            // [NB][n_it][2][32]
    float *lval = reinterpret_cast<float *>(smem + p.lists_off);          // [CONS_WARPS][NB][16]
    int32_t *lidx = reinterpret_cast<int32_t *>(lval + VT_CONS_WARPS * NB * MTV_MAX_TOPK);
    const uint32_t bars = ptx::smem_u32(smem + p.bars_off);               // full[n_stages], empty[n_stages]
    __shared__ int s_abort;

    const int k = blockIdx.y, bz = blockIdx.z, b0 = bz * NB;
    const int per = gridDim.x;
    const int kd = p.kd_arr[k];
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int H = p.H, RS = p.rows_per_stage, NST = p.n_stages;
    const uint32_t row_bytes = (uint32_t)H * 2;
    const int n_chunk16 = H / 8;

    // activations: chunk c = it*32 + lane of row b lives at xs4[((b*n_it + it)*2 + half)*32 + lane]
    for (int i = threadIdx.x; i < NB * p.n_it * 64; i += VT_THREADS) {
        const int ln = i % 32, half = (i / 32) % 2, it = (i / 64) % p.n_it, b = i / (64 * p.n_it);
        const int c = it * 32 + ln;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c < n_chunk16 && b0 + b < p.B)
            v = *reinterpret_cast<const float4 *>(p.hprime + ((size_t)k * p.B + b0 + b) * H + c * 8 + half * 4);
        xs4[i] = v;
    }
    for (int i = threadIdx.x; i < VT_CONS_WARPS * NB * MTV_MAX_TOPK; i += VT_THREADS) {
        lval[i] = -INFINITY;
        lidx[i] = 0x7fffffff;
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < NST; ++s) {
            ptx::mbar_init(bars + s * 8, 1);                               // full: the producer's expect_tx arrival
            ptx::mbar_init(bars + (NST + s) * 8, VT_GROUP_WARPS);          // empty: one arrival per consumer warp
        }
        ptx::fence_mbar_init();
        s_abort = 0;
    }
    __syncthreads();

    // slab of this CTA
    const int rows_per = (p.V + per - 1) / per;
    const int v_begin = min(p.V, (int)blockIdx.x * rows_per);
    const int v_end = kd > 0 ? min(p.V, v_begin + rows_per) : v_begin;
    const int n_chunks = (v_end - v_begin + RS - 1) / RS;
    const __nv_bfloat16 *Wk = p.W2 + (size_t)k * p.V * H;
    const uint32_t ring = ptx::smem_u32(smem);
    volatile int *abort_flag = &s_abort;

    if (warp == VT_CONS_WARPS) {
        // ---- producer
        for (int t = 0; t < n_chunks && !*abort_flag; ++t) {
            const int s = t % NST, use = t / NST;
            if (use > 0 && !ptx::mbar_wait(bars + (NST + s) * 8, (use - 1) & 1)) { *abort_flag = 1; break; }
            const int v0 = v_begin + t * RS;
            const int rows = min(RS, v_end - v0);
            if (lane == 0) ptx::mbar_arrive_expect_tx(bars + s * 8, rows * row_bytes);
            __syncwarp();
            if (lane < rows)
                ptx::bulk_g2s(ring + s * p.stage_bytes + lane * row_bytes, Wk + (size_t)(v0 + lane) * H, row_bytes,
                              bars + s * 8);
        }
    } else {
        // ---- consumers
        if constexpr (NB == 1) {
        const int group = warp / VT_GROUP_WARPS, wr = warp % VT_GROUP_WARPS;
        float *my_val = lval + (warp * NB) * MTV_MAX_TOPK;
        int32_t *my_idx = lidx + (warp * NB) * MTV_MAX_TOPK;
        float thr_v[NB];
        int thr_i[NB];
#pragma unroll
        for (int b = 0; b < NB; ++b) { thr_v[b] = -INFINITY; thr_i[b] = 0x7fffffff; }
        for (int t = group; t < n_chunks; t += VT_GROUPS) {
            const int s = t % NST, use = t / NST;
            if (*abort_flag) break;
            // The two groups take turns on a stage when n_stages is odd.  A parity wait cannot
            // tell phase `use` from phase `use - 2`, so first make sure that the stage's previous
            // use was released (by whichever group had it): after that its full barrier is in
            // phase `use` and the wait below cannot be satisfied by an older phase.
            if (use > 0 && !ptx::mbar_wait(bars + (NST + s) * 8, (use - 1) & 1)) { *abort_flag = 1; break; }
            if (!ptx::mbar_wait(bars + s * 8, use & 1)) { *abort_flag = 1; break; }
            const int v0 = v_begin + t * RS;
            const int rows = min(RS, v_end - v0);
            float acc[NB];
#pragma unroll
            for (int b = 0; b < NB; ++b) acc[b] = 0.f;
            if (wr < rows) {
                const uint4 *wrow = reinterpret_cast<const uint4 *>(smem + s * p.stage_bytes + wr * row_bytes);
                float acc2[NB];
#pragma unroll
                for (int b = 0; b < NB; ++b) acc2[b] = 0.f;
#pragma unroll 4
                for (int it = 0; it < p.n_it; ++it) {
                    const int c = it * 32 + lane;
                    if (c < n_chunk16) {
                        float wf[8];
                        bf16x8_to_float(wrow[c], wf);
#pragma unroll
                        for (int b = 0; b < NB; ++b) {
                            const float4 x0 = xs4[((b * p.n_it + it) * 2) * 32 + lane];
                            const float4 x1 = xs4[((b * p.n_it + it) * 2 + 1) * 32 + lane];
                            float a = acc[b], a2 = acc2[b];
                            a = fmaf(wf[0], x0.x, a); a2 = fmaf(wf[1], x0.y, a2);
                            a = fmaf(wf[2], x0.z, a); a2 = fmaf(wf[3], x0.w, a2);
                            a = fmaf(wf[4], x1.x, a); a2 = fmaf(wf[5], x1.y, a2);
                            a = fmaf(wf[6], x1.z, a); a2 = fmaf(wf[7], x1.w, a2);
                            acc[b] = a; acc2[b] = a2;
                        }
                    }
                }
#pragma unroll
                for (int b = 0; b < NB; ++b) acc[b] += acc2[b];
            }
            float z[NB];
#pragma unroll
            for (int b = 0; b < NB; ++b) z[b] = warp_sum(acc[b]);     // identical in every lane
            // every lane's reads of the stage are complete (their values fed the sums): release it
            if (lane == 0) ptx::mbar_arrive(bars + (NST + s) * 8);
            if (wr < rows) {
                const int v = v0 + wr;
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    if (cand_before(z[b], v, thr_v[b], thr_i[b])) {
                        if (lane == 0) {
                            // insertion into the sorted list of kd entries
                            int pos = kd - 1;
                            while (pos > 0 && cand_before(z[b], v, my_val[b * MTV_MAX_TOPK + pos - 1],
                                                          my_idx[b * MTV_MAX_TOPK + pos - 1])) {
                                my_val[b * MTV_MAX_TOPK + pos] = my_val[b * MTV_MAX_TOPK + pos - 1];
                                my_idx[b * MTV_MAX_TOPK + pos] = my_idx[b * MTV_MAX_TOPK + pos - 1];
                                --pos;
                            }
                            my_val[b * MTV_MAX_TOPK + pos] = z[b];
                            my_idx[b * MTV_MAX_TOPK + pos] = v;
                        }
                        __syncwarp();
                        thr_v[b] = my_val[b * MTV_MAX_TOPK + kd - 1];
                        thr_i[b] = my_idx[b * MTV_MAX_TOPK + kd - 1];
                    }
                }
            }
        }
            } else {
        // Several batch rows: every activation chunk read from shared memory must serve several weight
        // rows, or shared-memory bandwidth, not HBM, sets the pace.  A group's eight warps split a stage
        // into row blocks of R rows and column parts: warp (rb, cp) multiplies rows [R rb, R rb + R) by
        // the batch rows over the iterations it = cp, cp + ncp, ...; the column parts' partial logits
        // meet in shared memory and the warp with cp = 0 of each row block keeps the candidate lists.
        constexpr int R = NB >= 4 ? 4 : 2;
        constexpr int NV = R * NB;                       // logits per warp and stage
        const int group = warp / VT_GROUP_WARPS, wr = warp % VT_GROUP_WARPS;
        const int nrb = RS / R, ncp = VT_GROUP_WARPS / nrb;   // the host guarantees RS >= R
        const int rb = wr % nrb, cp = wr / nrb;
        float *zbuf = reinterpret_cast<float *>(smem + p.zbuf_off) + group * 2 * VT_GROUP_WARPS * 32;   // [2][8 warps][32]
        float *my_val = lval + (warp * NB) * MTV_MAX_TOPK;
        int32_t *my_idx = lidx + (warp * NB) * MTV_MAX_TOPK;
        bool ok = true;   // a warp whose wait ran out keeps the group barrier matched without waiting again
        for (int t = group; t < n_chunks; t += VT_GROUPS) {
            const int s = t % NST, use = t / NST;
            if (*abort_flag) ok = false;
            if (ok && use > 0) ok = ptx::mbar_wait(bars + (NST + s) * 8, (use - 1) & 1);   // see the single-row path
            if (ok) ok = ptx::mbar_wait(bars + s * 8, use & 1);
            if (!ok) *abort_flag = 1;
            const int v0 = v_begin + t * RS;
            const int rows = min(RS, v_end - v0);
            float acc[NV];
#pragma unroll
            for (int i = 0; i < NV; ++i) acc[i] = 0.f;
            const unsigned char *wblock = smem + s * p.stage_bytes + (size_t)(rb * R) * row_bytes;
            for (int it = cp; it < p.n_it; it += ncp) {
                const int c = it * 32 + lane;
                if (c < n_chunk16) {
                    float wf[R][8];
#pragma unroll
                    for (int r = 0; r < R; ++r)
                        bf16x8_to_float(reinterpret_cast<const uint4 *>(wblock + (size_t)r * row_bytes)[c], wf[r]);
#pragma unroll
                    for (int b = 0; b < NB; ++b) {
                        const float4 x0 = xs4[((b * p.n_it + it) * 2) * 32 + lane];
                        const float4 x1 = xs4[((b * p.n_it + it) * 2 + 1) * 32 + lane];
#pragma unroll
                        for (int r = 0; r < R; ++r) {
                            float a = acc[r * NB + b];
                            a = fmaf(wf[r][0], x0.x, a); a = fmaf(wf[r][1], x0.y, a);
                            a = fmaf(wf[r][2], x0.z, a); a = fmaf(wf[r][3], x0.w, a);
                            a = fmaf(wf[r][4], x1.x, a); a = fmaf(wf[r][5], x1.y, a);
                            a = fmaf(wf[r][6], x1.z, a); a = fmaf(wf[r][7], x1.w, a);
                            acc[r * NB + b] = a;
                        }
                    }
                }
            }
            warp_sum_scatter<NV>(acc, lane);   // lane l: partial logit number l / (32 / NV) of this column part
            // every lane's reads of the stage are complete (their values fed the sums): release it
            if (ok && lane == 0) ptx::mbar_arrive(bars + (NST + s) * 8);
            float *zb = zbuf + ((t / VT_GROUPS) & 1) * VT_GROUP_WARPS * 32;
            if (lane % (32 / NV) == 0) zb[wr * 32 + lane / (32 / NV)] = acc[0];
            asm volatile("bar.sync %0, 256;" ::"r"(2 + group) : "memory");
            if (cp == 0) {
                // lane l < NV: row r = l / NB of the block, batch row b = l % NB
                const int r = lane / NB, b = lane % NB;
                float z = 0.f;
                if (lane < NV)
                    for (int q = 0; q < ncp; ++q) z += zb[(q * nrb + rb) * 32 + lane];
                const int v = v0 + rb * R + r;
                const bool live = lane < NV && rb * R + r < rows && b0 + b < p.B;
#pragma unroll 1
                for (int rr = 0; rr < R; ++rr) {
                    if (live && r == rr &&
                        cand_before(z, v, my_val[b * MTV_MAX_TOPK + kd - 1], my_idx[b * MTV_MAX_TOPK + kd - 1])) {
                        // this lane is the only one that touches list b now: insertion into the sorted list
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
                }
            }
        }
        }
    }
    __syncthreads();
    if (s_abort) {
        // A wait ran out.  Raise the sticky error; the producer gives its copies in flight one
        // more bounded chance to land before the CTA (and its shared memory) goes away.
        if (threadIdx.x == 0) atomicExch(p.dev_error, MTV_ERR_TIMEOUT);
        if (warp == VT_CONS_WARPS && lane == 0)
            for (int s = 0; s < NST; ++s) { ptx::mbar_wait(bars + s * 8, 0); ptx::mbar_wait(bars + s * 8, 1); }
        return;
    }

    vocab_tail(p, NB, VT_CONS_WARPS, lval, lidx, smem, k, bz, b0, per, kd, p.xs_off);
}

template <int NB>
static int launch_heads(const mtv_tree *t, int B, int H, int V, const __nv_bfloat16 *hidden,
                        const __nv_bfloat16 *W1, const __nv_bfloat16 *b1, const __nv_bfloat16 *W2,
                        const int32_t *root_tok, int32_t *cand, float *cand_logit, int32_t *tree_tok,
                        const HeadsWs &L, char *ws, cudaStream_t st) {
    float *hprime = reinterpret_cast<float *>(ws + L.hprime_off);
    const int btiles = (B + NB - 1) / NB;
    const size_t sm1 = (size_t)NB * H * sizeof(float);
    const VocabSmem S = vocab_smem_plan(NB, H, L.ctas_per_head);
    if (sm1 > VT_SMEM_MAX || S.total == 0) return MTV_ERR_UNSUPPORTED_SHAPE;
    if (NB > 1 && S.rows_per_stage < (NB >= 4 ? 4 : 2)) return MTV_ERR_UNSUPPORTED_SHAPE;   // rows too long for a block of rows per stage
    static PerDeviceOnce attr_once;
    bool *attr_done = attr_once.flag();
    if (!attr_done || !*attr_done) {
        MTV_CUDA_CHECK(cudaFuncSetAttribute(heads_resblock_kernel<NB>, cudaFuncAttributeMaxDynamicSharedMemorySize, VT_SMEM_MAX));
        MTV_CUDA_CHECK(cudaFuncSetAttribute(heads_vocab_topk_kernel<NB>, cudaFuncAttributeMaxDynamicSharedMemorySize, VT_SMEM_MAX));
        if (attr_done) *attr_done = true;
    }
    int g1 = (t->K * H + HEADS_WARPS - 1) / HEADS_WARPS;
    const int cap = 4 * sm_count();
    if (g1 > cap) g1 = cap;
    int32_t *counters = reinterpret_cast<int32_t *>(ws + L.counters_off);
    {
        TapScope tap(MTV_KERNEL_HEADS_RESBLOCK, st);
        heads_resblock_kernel<NB><<<dim3(g1, btiles), HEADS_THREADS, sm1, st>>>(B, H, t->K, hidden, W1, b1, hprime,
                                                                               counters, L.n_counters);
    }
    VocabParams p;
    p.B = B; p.H = H; p.V = V; p.K = t->K; p.T = t->T; p.C = t->C;
    p.W2 = W2; p.hprime = hprime;
    p.kd_arr = t->d_kd; p.off_arr = t->d_cand_offset; p.tree_indices = t->d_tree_indices; p.root_tok = root_tok;
    p.part_val = reinterpret_cast<float *>(ws + L.part_val_off);
    p.part_idx = reinterpret_cast<int32_t *>(ws + L.part_idx_off);
    p.counters = counters;
    p.cand = cand; p.cand_logit = cand_logit; p.tree_tok = tree_tok;
    p.dev_error = t->d_error;
    p.rows_per_stage = S.rows_per_stage; p.n_stages = S.n_stages; p.n_it = S.n_it;
    p.stage_bytes = S.stage_bytes; p.xs_off = S.xs_off; p.lists_off = S.lists_off; p.zbuf_off = S.zbuf_off; p.bars_off = S.bars_off;
    {
        TapScope tap(MTV_KERNEL_HEADS_VOCAB_TOPK, st);
        heads_vocab_topk_kernel<NB><<<dim3(L.ctas_per_head, t->K, btiles), VT_THREADS, S.total, st>>>(p);
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
    MTV_RANGE("medusa_heads_topk");
    if (!tree || !tree->on_device || !hidden || !W1 || !W2 || !root_tok || !cand || !tree_tok || !ws)
        return MTV_ERR_INVALID_ARG;
    if (B < 1 || H < 8 || V < 1) return MTV_ERR_INVALID_ARG;
    if (B > 16 || H % 8 != 0) return MTV_ERR_UNSUPPORTED_SHAPE;
    if (((uintptr_t)W2 | (uintptr_t)W1 | (uintptr_t)hidden | (uintptr_t)ws) & 15) return MTV_ERR_INVALID_ARG;
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
    if (L.use_tc) rc = launch_heads_tc(tree, B, H, V, h, w1, bb, w2, root_tok, cand, cand_logit, tree_tok, L, (char *)ws, st);
    else if (B == 1) rc = launch_heads<1>(tree, B, H, V, h, w1, bb, w2, root_tok, cand, cand_logit, tree_tok, L, (char *)ws, st);
    else if (B == 2) rc = launch_heads<2>(tree, B, H, V, h, w1, bb, w2, root_tok, cand, cand_logit, tree_tok, L, (char *)ws, st);
    else if (B <= 4) rc = launch_heads<4>(tree, B, H, V, h, w1, bb, w2, root_tok, cand, cand_logit, tree_tok, L, (char *)ws, st);
    else rc = launch_heads<8>(tree, B, H, V, h, w1, bb, w2, root_tok, cand, cand_logit, tree_tok, L, (char *)ws, st);
    if (rc != MTV_OK) return rc;
    MTV_CUDA_CHECK(cudaGetLastError());
    return MTV_OK;
}
