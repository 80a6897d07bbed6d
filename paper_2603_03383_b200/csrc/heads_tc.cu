// Vocabulary projection of the Medusa heads (Section 3.1) for several batch rows, on the tcgen05
// tensor cores.  With B > 1 the fp32 FMA pipe cannot keep up with the weight stream (B multiply-adds
// per weight element), the tensor cores can; what has to be kept is the precision of the single-row
// path, where activations stay fp32 and the candidate ids must match a double-precision checker:
//   * the fp32 activations h' are split into three bf16 terms hi + mid + lo (24 bits of mantissa, exact
//     to 2^-25); the three terms of up to 16 batch rows are the 48 rows of the MMA's N operand, and their
//     products with the bf16 weights are exact;
//   * the tensor core's fp32 accumulator truncates: over H = 4096 the sums drift by ~3e-6 of the largest
//     logit.  The K chunks therefore take turns over four accumulators that are added in the epilogue
//     with ordinary fp32 additions, which divides the drift by four.
// Layout of the work as in the fused LM head: persistent CTAs (a contiguous slab of one head's vocabulary
// rows each), TMA producer warp -> ring of stages (64 columns of 128 weight rows + the 48 activation
// rows) -> MMA issuer, accumulators double-buffered in tensor memory -> four epilogue warps, one thread
// per vocabulary row, that keep per-warp sorted candidate lists (a logit is inserted only if it beats
// the list's last entry).  What follows the projection is shared with the single-row kernel.
#include <cuda.h>

#include "common.cuh"
#include "heads_common.cuh"
#include "sm100_ptx.cuh"
#include "tma_host.cuh"

namespace mtv {

constexpr int HT_THREADS = 192;            // warps 0-3 epilogue, warp 4 MMA issuer, warp 5 TMA producer
constexpr int HT_EPI_WARPS = 4;
constexpr int HT_N = 3 * HT_NB;            // hi | mid | lo rows of the activation operand
constexpr int HT_NACC = 4;                 // accumulators that take turns over the K chunks
constexpr int HT_ACC_COLS = 64;            // tensor-memory columns reserved per accumulator (48 used)
constexpr uint32_t HT_W_BYTES = 128 * 128; // 128 weight rows x 64 columns
constexpr uint32_t HT_X_BYTES = HT_N * 128;
constexpr uint32_t HT_STAGE_BYTES = HT_W_BYTES + HT_X_BYTES;   // 22 KB, a multiple of 1024
constexpr int HT_STAGES = 8;
constexpr uint32_t HT_LIST_BYTES = HT_EPI_WARPS * HT_NB * MTV_MAX_TOPK * 8;
constexpr uint32_t HT_SMEM_BYTES = 1024 + HT_STAGES * HT_STAGE_BYTES + HT_LIST_BYTES;
static_assert(HT_STAGE_BYTES % 1024 == 0, "stages must keep the 1024-byte alignment of the swizzled tiles");
static_assert(2 * HT_NACC * HT_ACC_COLS <= 512, "tensor memory");
static_assert(HT_SMEM_BYTES <= 220 * 1024, "shared memory");

constexpr uint32_t HT_IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(HT_N >> 3) << 17) | ((128u >> 4) << 24);

__device__ __forceinline__ uint64_t ht_desc(uint32_t saddr) {   // K-major, 128-byte swizzle
    uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(16u >> 4) << 16;
    d |= (uint64_t)(1024u >> 4) << 32;
    d |= 1ull << 46;
    d |= 2ull << 61;
    return d;
}
__device__ __forceinline__ void ht_tma_2d(uint32_t dst, const void *map, uint32_t bar, int c0, int c1) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}

// ---------------------------------------------------------------------------
// Residual block for several batch rows:  h'[k][b][o] = h[b][o] + SiLU(W1[k][o][:] . h[b][:] + b1[k][o]).
// The same pipeline with the K H rows of W1 as the MMA's M side (tiles of 128 rows, persistent CTAs) and the
// bf16 hidden states of up to 16 batch rows as its N side (exact: they are bf16 to begin with).  The epilogue
// (thread = output row) adds the four accumulators, the bias and the residual in fp32 and writes h' as the
// three bf16 terms the vocabulary projection multiplies: xsplit[k][part][b][o], part = 0 (hi), 1 (mid),
// 2 (lo), h' = hi + mid + lo up to 2^-25.  Batch rows b >= B hold finite values nobody reads.
constexpr int RT_STAGES = 8;
constexpr uint32_t RT_X_BYTES = HT_NB * 128;
constexpr uint32_t RT_STAGE_BYTES = HT_W_BYTES + RT_X_BYTES;   // 18 KB
constexpr uint32_t RT_SMEM_BYTES = 1024 + RT_STAGES * RT_STAGE_BYTES;
constexpr uint32_t RT_IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(HT_NB >> 3) << 17) | ((128u >> 4) << 24);
static_assert(RT_STAGE_BYTES % 1024 == 0, "stages must keep the 1024-byte alignment of the swizzled tiles");

struct ResblockTcParams {
    int B, H, K;
    const __nv_bfloat16 *hidden, *b1;
    __nv_bfloat16 *xsplit;
    int32_t *counters;
    int n_counters;
    int32_t *dev_error;
};

// w_map: [K H][H] rows of W1, box 64 x 128; h_map: [B][H] hidden states, box 64 x 16 (rows >= B read as zero).
__global__ void __launch_bounds__(HT_THREADS, 1)
heads_resblock_tc_kernel(const __grid_constant__ CUtensorMap w_map, const __grid_constant__ CUtensorMap h_map,
                         const ResblockTcParams p) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag_s;
    __shared__ int issued_s;
    __shared__ __align__(8) unsigned long long bar_mem[2 * RT_STAGES + 5];
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t ring = raw + ((1024u - (raw & 1023u)) & 1023u);
    const uint32_t bars = ptx::smem_u32(bar_mem);
    auto full = [&](int s) { return bars + (uint32_t)s * 8u; };
    auto empty = [&](int s) { return bars + (uint32_t)(RT_STAGES + s) * 8u; };
    auto acc_full = [&](int u) { return bars + (uint32_t)(2 * RT_STAGES + u) * 8u; };
    auto acc_empty = [&](int u) { return bars + (uint32_t)(2 * RT_STAGES + 2 + u) * 8u; };
    const uint32_t drain_bar = bars + (uint32_t)(2 * RT_STAGES + 4) * 8u;
    volatile int *abort_flag = &abort_flag_s;
    constexpr uint32_t TMEM_COLS = 2 * HT_NACC * HT_NB;   // 128

    // tickets of the vocabulary kernel (the next launch on the stream) start at zero
    if (blockIdx.x == 0)
        for (int i = threadIdx.x; i < p.n_counters; i += HT_THREADS) p.counters[i] = 0;
    if (threadIdx.x == 0) {
        for (int s = 0; s < RT_STAGES; ++s) { ptx::mbar_init(full(s), 1); ptx::mbar_init(empty(s), 1); }
        for (int u = 0; u < 2; ++u) { ptx::mbar_init(acc_full(u), 1); ptx::mbar_init(acc_empty(u), 128); }
        ptx::mbar_init(drain_bar, 1);
        ptx::fence_mbar_init();
        abort_flag_s = 0;
        issued_s = 0;
        ptx::prefetch_tensormap(&w_map);
        ptx::prefetch_tensormap(&h_map);
    }
    if (warp == 4) {
        ptx::tmem_alloc(ptx::smem_u32(&tmem_slot), TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = tmem_slot;

    const int rows = p.K * p.H;
    const int n_tiles_all = (rows + 127) / 128;
    const int my_tiles = (int)blockIdx.x < n_tiles_all ? (n_tiles_all - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
    const int n_kc = p.H / 64;

    if (warp == 5) {
        // ---------------------------------------------------------------- TMA producer
        int it = 0;
        for (int q = 0; q < my_tiles && !*abort_flag; ++q) {
            const int row0 = ((int)blockIdx.x + q * (int)gridDim.x) * 128;
            for (int kc = 0; kc < n_kc; ++kc, ++it) {
                const int s = it % RT_STAGES, use = it / RT_STAGES;
                if (use > 0 && !ptx::mbar_wait(empty(s), (use - 1) & 1)) { *abort_flag = 1; break; }
                if (lane == 0) {
                    const uint32_t base = ring + s * RT_STAGE_BYTES;
                    ptx::mbar_arrive_expect_tx(full(s), RT_STAGE_BYTES);
                    ht_tma_2d(base, &w_map, full(s), kc * 64, row0);
                    ht_tma_2d(base + HT_W_BYTES, &h_map, full(s), kc * 64, 0);
                }
                __syncwarp();
            }
        }
        if (lane == 0) issued_s = it;
    } else if (warp == 4) {
        // ---------------------------------------------------------------- MMA issuer
        int it = 0;
        bool ok = true;
        for (int q = 0; ok && q < my_tiles && !*abort_flag; ++q) {
            const int u = q & 1;
            if (q >= 2) ok = ptx::mbar_wait(acc_empty(u), ((q >> 1) - 1) & 1);
            if (!ok) break;
            ptx::tc_fence_after();
            for (int kc = 0; kc < n_kc; ++kc, ++it) {
                const int s = it % RT_STAGES;
                ok = ptx::mbar_wait(full(s), (it / RT_STAGES) & 1);
                if (!ok) break;
                ptx::tc_fence_after();
                if (lane == 0) {
                    const uint32_t base = ring + s * RT_STAGE_BYTES;
                    const uint32_t d = tmem + (u * HT_NACC + kc % HT_NACC) * HT_NB;
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        ptx::mma_ss(d, ht_desc(base + kk * 32), ht_desc(base + HT_W_BYTES + kk * 32), RT_IDESC,
                                    kc >= HT_NACC || kk > 0);
                    ptx::tc_commit(empty(s));
                    if (kc == n_kc - 1) ptx::tc_commit(acc_full(u));
                }
                __syncwarp();
            }
        }
        if (!ok) *abort_flag = 1;
    } else {
        // ---------------------------------------------------------------- epilogue: thread = output row
        const int n_acc = min(HT_NACC, n_kc);
        bool ok = true;
        for (int q = 0; q < my_tiles; ++q) {
            const int u = q & 1;
            if (*abort_flag) ok = false;
            if (ok) ok = ptx::mbar_wait(acc_full(u), (q >> 1) & 1);
            __syncwarp();
            ptx::tc_fence_after();
            float y[HT_NB];
#pragma unroll
            for (int b = 0; b < HT_NB; ++b) y[b] = 0.f;
            for (int a = 0; a < n_acc; ++a) {
                uint32_t acc[16];
                ptx::tmem_ld16(tmem + ((uint32_t)(warp * 32) << 16) + (u * HT_NACC + a) * HT_NB, acc);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int b = 0; b < HT_NB; ++b) y[b] += __uint_as_float(acc[b]);
            }
            ptx::tc_fence_before();
            ptx::mbar_arrive(acc_empty(u));
            const int r = ((int)blockIdx.x + q * (int)gridDim.x) * 128 + warp * 32 + lane;
            if (ok && r < rows) {
                const int k = r / p.H, o = r % p.H;
                const float bias = p.b1 ? __bfloat162float(p.b1[(size_t)k * p.H + o]) : 0.f;
#pragma unroll
                for (int b = 0; b < HT_NB; ++b) {
                    const float yy = y[b] + bias;
                    const float h = b < p.B ? __bfloat162float(p.hidden[(size_t)b * p.H + o]) : 0.f;
                    float x = h + yy / (1.f + expf(-yy));
                    const __nv_bfloat16 hi = __float2bfloat16_rn(x);
                    x -= __bfloat162float(hi);                         // exact
                    const __nv_bfloat16 mid = __float2bfloat16_rn(x);
                    x -= __bfloat162float(mid);                        // exact
                    __nv_bfloat16 *dst = p.xsplit + ((size_t)k * HT_N + b) * p.H + o;
                    dst[0] = hi;
                    dst[(size_t)HT_NB * p.H] = mid;
                    dst[(size_t)2 * HT_NB * p.H] = __float2bfloat16_rn(x);
                }
            }
        }
        if (!ok) *abort_flag = 1;
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 4) {
        if (*abort_flag) {
            if (lane == 0) ptx::tc_commit(drain_bar);
            __syncwarp();
            ptx::mbar_wait(drain_bar, 0);
        }
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem, TMEM_COLS);
    }
    if (*abort_flag) {
        if (threadIdx.x == 0) atomicExch(p.dev_error, MTV_ERR_TIMEOUT);
        if (warp == 5 && lane == 0)
            for (int s = 0; s < RT_STAGES; ++s) {
                const int uses = (issued_s - s + RT_STAGES - 1) / RT_STAGES;
                if (issued_s > s) ptx::mbar_wait(full(s), (uses - 1) & 1);
            }
    }
}

// grid = (ctas_per_head, K).  w_map: [K V][H] weights, box 64 x 128; x_map: [K 48][H] split activations, box 64 x 48.
__global__ void __launch_bounds__(HT_THREADS, 1)
heads_vocab_topk_tc_kernel(const __grid_constant__ CUtensorMap w_map, const __grid_constant__ CUtensorMap x_map,
                           const VocabParams p) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag_s;
    __shared__ int issued_s;
    __shared__ __align__(8) unsigned long long bar_mem[2 * HT_STAGES + 5];
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
    const uint32_t ring = raw + pad;
    unsigned char *ring_gen = smem_raw + pad;
    float *lval = reinterpret_cast<float *>(ring_gen + HT_STAGES * HT_STAGE_BYTES);   // [4 warps][16 rows][16]
    int32_t *lidx = reinterpret_cast<int32_t *>(lval + HT_EPI_WARPS * HT_NB * MTV_MAX_TOPK);
    const uint32_t bars = ptx::smem_u32(bar_mem);
    auto full = [&](int s) { return bars + (uint32_t)s * 8u; };
    auto empty = [&](int s) { return bars + (uint32_t)(HT_STAGES + s) * 8u; };
    auto acc_full = [&](int u) { return bars + (uint32_t)(2 * HT_STAGES + u) * 8u; };
    auto acc_empty = [&](int u) { return bars + (uint32_t)(2 * HT_STAGES + 2 + u) * 8u; };
    const uint32_t drain_bar = bars + (uint32_t)(2 * HT_STAGES + 4) * 8u;
    volatile int *abort_flag = &abort_flag_s;

    const int k = blockIdx.y, per = gridDim.x;
    const int kd = p.kd_arr[k];
    for (int i = threadIdx.x; i < HT_EPI_WARPS * HT_NB * MTV_MAX_TOPK; i += HT_THREADS) {
        lval[i] = -INFINITY;
        lidx[i] = 0x7fffffff;
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < HT_STAGES; ++s) { ptx::mbar_init(full(s), 1); ptx::mbar_init(empty(s), 1); }
        for (int u = 0; u < 2; ++u) { ptx::mbar_init(acc_full(u), 1); ptx::mbar_init(acc_empty(u), 128); }
        ptx::mbar_init(drain_bar, 1);
        ptx::fence_mbar_init();
        abort_flag_s = 0;
        issued_s = 0;
        ptx::prefetch_tensormap(&w_map);
        ptx::prefetch_tensormap(&x_map);
    }
    if (warp == 4) {
        ptx::tmem_alloc(ptx::smem_u32(&tmem_slot), 512);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = tmem_slot;

    // slab of this CTA: vocabulary rows [v_begin, v_end) of head k, in tiles of 128 rows
    const int rows_per = (p.V + per - 1) / per;
    const int v_begin = min(p.V, (int)blockIdx.x * rows_per);
    const int v_end = kd > 0 ? min(p.V, v_begin + rows_per) : v_begin;
    const int n_tiles = (v_end - v_begin + 127) / 128;
    const int n_kc = p.H / 64;

    if (warp == 5) {
        // ---------------------------------------------------------------- TMA producer
        int it = 0;
        for (int q = 0; q < n_tiles && !*abort_flag; ++q) {
            const int row0 = k * p.V + v_begin + q * 128;     // rows past the slab are loaded and ignored
            for (int kc = 0; kc < n_kc; ++kc, ++it) {
                const int s = it % HT_STAGES, use = it / HT_STAGES;
                if (use > 0 && !ptx::mbar_wait(empty(s), (use - 1) & 1)) { *abort_flag = 1; break; }
                if (lane == 0) {
                    const uint32_t base = ring + s * HT_STAGE_BYTES;
                    ptx::mbar_arrive_expect_tx(full(s), HT_STAGE_BYTES);
                    ht_tma_2d(base, &w_map, full(s), kc * 64, row0);
                    ht_tma_2d(base + HT_W_BYTES, &x_map, full(s), kc * 64, k * HT_N);
                }
                __syncwarp();
            }
        }
        if (lane == 0) issued_s = it;
    } else if (warp == 4) {
        // ---------------------------------------------------------------- MMA issuer
        int it = 0;
        bool ok = true;
        for (int q = 0; ok && q < n_tiles && !*abort_flag; ++q) {
            const int u = q & 1;
            if (q >= 2) ok = ptx::mbar_wait(acc_empty(u), ((q >> 1) - 1) & 1);   // the epilogue has read this buffer
            if (!ok) break;
            ptx::tc_fence_after();
            for (int kc = 0; kc < n_kc; ++kc, ++it) {
                const int s = it % HT_STAGES;
                ok = ptx::mbar_wait(full(s), (it / HT_STAGES) & 1);
                if (!ok) break;
                ptx::tc_fence_after();
                if (lane == 0) {
                    const uint32_t base = ring + s * HT_STAGE_BYTES;
                    const uint32_t d = tmem + (u * HT_NACC + kc % HT_NACC) * HT_ACC_COLS;
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        ptx::mma_ss(d, ht_desc(base + kk * 32), ht_desc(base + HT_W_BYTES + kk * 32), HT_IDESC,
                                    kc >= HT_NACC || kk > 0);
                    ptx::tc_commit(empty(s));
                    if (kc == n_kc - 1) ptx::tc_commit(acc_full(u));
                }
                __syncwarp();
            }
        }
        if (!ok) *abort_flag = 1;
    } else {
        // ---------------------------------------------------------------- epilogue: thread = vocabulary row
        float *my_val = lval + warp * HT_NB * MTV_MAX_TOPK;
        int32_t *my_idx = lidx + warp * HT_NB * MTV_MAX_TOPK;
        const int n_acc = min(HT_NACC, n_kc);
        bool ok = true;
        for (int q = 0; q < n_tiles; ++q) {
            const int u = q & 1;
            if (*abort_flag) ok = false;
            if (ok) ok = ptx::mbar_wait(acc_full(u), (q >> 1) & 1);
            __syncwarp();
            ptx::tc_fence_after();
            float z[HT_NB];
#pragma unroll
            for (int b = 0; b < HT_NB; ++b) z[b] = 0.f;
            for (int a = 0; a < n_acc; ++a) {
                uint32_t hi[16], mid[16], lo[16];
                const uint32_t col = tmem + ((uint32_t)(warp * 32) << 16) + (u * HT_NACC + a) * HT_ACC_COLS;
                ptx::tmem_ld16(col, hi);
                ptx::tmem_ld16(col + 16, mid);
                ptx::tmem_ld16(col + 32, lo);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int b = 0; b < HT_NB; ++b)
                    z[b] += (__uint_as_float(hi[b]) + __uint_as_float(mid[b])) + __uint_as_float(lo[b]);
            }
            ptx::tc_fence_before();
            ptx::mbar_arrive(acc_empty(u));
            const int v = v_begin + q * 128 + warp * 32 + lane;
            const bool valid = ok && v < v_end;
#pragma unroll
            for (int b = 0; b < HT_NB; ++b) {
                if (b >= p.B) break;
                float *bv = my_val + b * MTV_MAX_TOPK;
                int32_t *bi = my_idx + b * MTV_MAX_TOPK;
                unsigned m = __ballot_sync(0xffffffffu, valid && cand_before(z[b], v, bv[kd - 1], bi[kd - 1]));
                while (m) {
                    // the whole warp inserts the candidate of lane src: lane s holds entry s, the entries ahead
                    // of the candidate stay, the others move down by one
                    const int src = __ffs(m) - 1;
                    m &= m - 1;
                    const float zc = __shfl_sync(0xffffffffu, z[b], src);
                    const int vc = __shfl_sync(0xffffffffu, v, src);
                    const float ev = lane < kd ? bv[lane] : 0.f;
                    const int ei = lane < kd ? bi[lane] : 0;
                    const int pos = __popc(__ballot_sync(0xffffffffu, lane < kd && cand_before(ev, ei, zc, vc)));
                    __syncwarp();
                    if (pos < kd) {          // else the list has moved on since the ballot
                        if (lane >= pos && lane < kd - 1) { bv[lane + 1] = ev; bi[lane + 1] = ei; }
                        if (lane == pos) { bv[pos] = zc; bi[pos] = vc; }
                    }
                    __syncwarp();
                }
            }
        }
        if (!ok) *abort_flag = 1;
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 4) {
        if (*abort_flag) {           // issued tensor-core work gets one more bounded wait
            if (lane == 0) ptx::tc_commit(drain_bar);
            __syncwarp();
            ptx::mbar_wait(drain_bar, 0);
        }
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem, 512);
    }
    if (*abort_flag) {
        if (threadIdx.x == 0) atomicExch(p.dev_error, MTV_ERR_TIMEOUT);
        if (warp == 5 && lane == 0)  // ... and so do the copies in flight, before the shared memory is given back
            for (int s = 0; s < HT_STAGES; ++s) {
                const int uses = (issued_s - s + HT_STAGES - 1) / HT_STAGES;
                if (issued_s > s) ptx::mbar_wait(full(s), (uses - 1) & 1);
            }
        return;
    }
    vocab_tail(p, HT_NB, HT_EPI_WARPS, lval, lidx, ring_gen, k, 0, 0, per, kd, HT_STAGES * HT_STAGE_BYTES);
}

bool heads_tc_eligible(int B, int H) { return B >= 2 && B <= HT_NB && H >= 64 && H % 64 == 0; }

size_t heads_tc_xsplit_bytes(int K, int H) { return (size_t)K * HT_N * H * sizeof(__nv_bfloat16); }

// Residual block, then projection, top-k, merges and tree expansion: the whole medusa_heads_topk for 2..16 rows.
int launch_heads_tc(const mtv_tree *t, int B, int H, int V, const __nv_bfloat16 *hidden, const __nv_bfloat16 *W1,
                    const __nv_bfloat16 *b1, const __nv_bfloat16 *W2, const int32_t *root_tok, int32_t *cand,
                    float *cand_logit, int32_t *tree_tok, const HeadsWs &L, char *ws, cudaStream_t st) {
    static PerDeviceOnce attr_once;
    bool *attr_done = attr_once.flag();
    if (!attr_done || !*attr_done) {
        MTV_CUDA_CHECK(cudaFuncSetAttribute(heads_vocab_topk_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, HT_SMEM_BYTES));
        MTV_CUDA_CHECK(cudaFuncSetAttribute(heads_resblock_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, RT_SMEM_BYTES));
        if (attr_done) *attr_done = true;
    }
    __nv_bfloat16 *xsplit = reinterpret_cast<__nv_bfloat16 *>(ws + L.xsplit_off);
    CUtensorMap w1_map, h_map, w2_map, x_map;
    if (!tma_map_2d_bf16(&w1_map, W1, t->K * H, H, 128) || !tma_map_2d_bf16(&h_map, hidden, B, H, HT_NB) ||
        !tma_map_2d_bf16(&w2_map, W2, t->K * V, H, 128) || !tma_map_2d_bf16(&x_map, xsplit, t->K * HT_N, H, HT_N))
        return MTV_ERR_CUDA;
    {
        ResblockTcParams r;
        r.B = B; r.H = H; r.K = t->K; r.hidden = hidden; r.b1 = b1; r.xsplit = xsplit;
        r.counters = reinterpret_cast<int32_t *>(ws + L.counters_off); r.n_counters = L.n_counters;
        r.dev_error = t->d_error;
        int ctas = (t->K * H + 127) / 128;
        if (ctas > sm_count()) ctas = sm_count();
        TapScope tap(MTV_KERNEL_HEADS_RESBLOCK, st);
        heads_resblock_tc_kernel<<<ctas, HT_THREADS, RT_SMEM_BYTES, st>>>(w1_map, h_map, r);
    }
    VocabParams p;
    p.B = B; p.H = H; p.V = V; p.K = t->K; p.T = t->T; p.C = t->C;
    p.W2 = W2; p.hprime = nullptr;
    p.kd_arr = t->d_kd; p.off_arr = t->d_cand_offset; p.tree_indices = t->d_tree_indices; p.root_tok = root_tok;
    p.part_val = reinterpret_cast<float *>(ws + L.part_val_off);
    p.part_idx = reinterpret_cast<int32_t *>(ws + L.part_idx_off);
    p.counters = reinterpret_cast<int32_t *>(ws + L.counters_off);
    p.cand = cand; p.cand_logit = cand_logit; p.tree_tok = tree_tok;
    p.dev_error = t->d_error;
    p.rows_per_stage = 0; p.n_stages = 0; p.n_it = 0;
    p.stage_bytes = 0; p.xs_off = 0; p.lists_off = 0; p.zbuf_off = 0; p.bars_off = 0;
    TapScope tap(MTV_KERNEL_HEADS_VOCAB_TOPK, st);
    heads_vocab_topk_tc_kernel<<<dim3(L.ctas_per_head, t->K), HT_THREADS, HT_SMEM_BYTES, st>>>(w2_map, x_map, p);
    return MTV_OK;
}

}  // namespace mtv
