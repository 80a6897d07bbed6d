// LM-head projection with the per-node argmax fused into its epilogue — the step between the
// tree attention and the acceptance (Section 3.2: acceptance needs, at every tree node, the base
// model's most likely next token).  logits[m][v] = <x[m], W[v]> for the M = B T tree nodes never go to
// memory: only argmax_v survives.
//
// A weight-streaming GEMM on the tcgen05 tensor cores.  With few nodes (M <= 128 per pass) the
// arithmetic intensity is M flop per weight byte, so HBM bounds it; the vocabulary rows are the
// MMA's M dimension, the nodes its N dimension:
//   D[128 vocabulary rows][N nodes] += W_tile[128][64 k] . X[N][64 k]^T      (both operands K-major)
// One persistent CTA per SM walks pairs of vocabulary tiles, so that a chunk of X fetched from L2
// serves two weight tiles.  A tile holds R <= 128 rows, R chosen by the host so that every CTA gets
// the same number of pairs (V = 32000 on 148 SMs: 112 rows); the MMA spans 128 rows all the same and
// the rows past R, whatever the shared memory held, are left out of the maximum.  From 129 nodes up a
// pass takes 256 nodes and one weight tile per stage: 128 x 256 x 16 is the MMA shape that runs at the
// full tensor rate (128 x 128 x 16 reaches about 60 % of it), and the large batches are tensor-bound.
// Warp roles: TMA producer (ring of stages, one stage = 64
// columns of the weight tiles and of the N node rows), MMA issuer (accumulators in tensor memory,
// double-buffered: the epilogue of one pair overlaps the MMAs of the next), four epilogue warps
// (one thread per vocabulary row: order-preserving (value, ~index) keys, butterfly max over the
// warp's 32 rows, shared-memory max across warps and pairs, one 64-bit atomic max per node at the end).
#include <cuda.h>

#include "common.cuh"
#include "sm100_ptx.cuh"
#include "tma_host.cuh"

namespace mtv {

constexpr int LM_THREADS = 192;            // warps 0-3 epilogue, warp 4 MMA issuer, warp 5 TMA producer
constexpr int LM_KC = 64;                  // columns per stage: one 128-byte swizzle span
constexpr uint32_t LM_TILE_BYTES = 128 * 128; // one weight tile of a stage: 128 rows x 64 columns
constexpr uint32_t LM_SMEM_MAX = 220 * 1024;   // dynamic part; the static part (keys, barriers) is about 1.2 KB
constexpr int LM_MAX_STAGES = 6;

constexpr uint32_t LM_IDESC_BASE = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 4) << 24);   // bf16 x bf16 -> fp32, M = 128

struct LmParams {
    unsigned long long *keys;   // [M] best (value, ~index) per node, zero before the launch
    int32_t *dev_error;
    int M, H, V, N;             // N = nodes per pass (64, 128 or 256)
    int R;                      // vocabulary rows per tile (<= 128, a multiple of 8), chosen so that the tiles
                                // divide evenly among the CTAs; the MMA still spans 128 rows, the rest is ignored
    int n_pairs;                // units (of two weight tiles, or of one when N = 256) over the vocabulary
    int n_stages;
    uint32_t stage_bytes;
};

__device__ __forceinline__ uint64_t lm_desc(uint32_t saddr) {   // K-major, 128-byte swizzle
    uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(16u >> 4) << 16;
    d |= (uint64_t)(1024u >> 4) << 32;
    d |= 1ull << 46;
    d |= 2ull << 61;
    return d;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const void *map, uint32_t bar, int c0, int c1) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
// larger fp32 first, equal values by lower index: one unsigned 64-bit max does both
__device__ __forceinline__ unsigned long long lm_key(uint32_t fbits, uint32_t idx) {
    uint32_t ord = (fbits & 0x80000000u) ? ~fbits : (fbits | 0x80000000u);
    if ((fbits << 1) == 0) ord = 0x80000000u;   // -0.0 and +0.0 compare equal
    return ((unsigned long long)ord << 32) | (0xffffffffu - idx);
}
__device__ __forceinline__ unsigned long long umax(unsigned long long a, unsigned long long b) { return a > b ? a : b; }

// Max over the 32 lanes of 32 per-lane keys at once: afterwards lane l holds the max of key number l.
__device__ __forceinline__ unsigned long long warp_max_scatter32(unsigned long long (&v)[32], int lane) {
    int n = 32;
#pragma unroll
    for (int bit = 16; bit >= 1; bit >>= 1) {
        n >>= 1;
        const bool up = (lane & bit) != 0;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            if (i < n) {
                const unsigned long long send = up ? v[i] : v[i + n];
                const unsigned long long keep = up ? v[i + n] : v[i];
                v[i] = umax(keep, __shfl_xor_sync(0xffffffffu, send, bit));
            }
        }
    }
    return v[0];
}

// N nodes per pass; TILES weight tiles per stage (2 for N <= 128, so that an X chunk serves two tiles; 1 for N = 256,
// the MMA shape that runs at the full tensor rate, where two tiles' accumulators would not fit tensor memory twice)
template <int N>
__global__ void __launch_bounds__(LM_THREADS, 1)
lm_head_argmax_kernel(const __grid_constant__ CUtensorMap w_map, const __grid_constant__ CUtensorMap x_map,
                      const LmParams p) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ unsigned long long best[N];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag_s;
    __shared__ int issued_s;                                    // stages the producer has issued (read when giving up)
    __shared__ __align__(8) unsigned long long bar_mem[2 * LM_MAX_STAGES + 5];
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t ring = raw + ((1024u - (raw & 1023u)) & 1023u);
    const uint32_t bars = ptx::smem_u32(bar_mem);
    const int NST = p.n_stages;
    auto full = [&](int s) { return bars + (uint32_t)s * 8u; };
    auto empty = [&](int s) { return bars + (uint32_t)(LM_MAX_STAGES + s) * 8u; };
    auto acc_full = [&](int u) { return bars + (uint32_t)(2 * LM_MAX_STAGES + u) * 8u; };
    auto acc_empty = [&](int u) { return bars + (uint32_t)(2 * LM_MAX_STAGES + 2 + u) * 8u; };
    const uint32_t drain_bar = bars + (uint32_t)(2 * LM_MAX_STAGES + 4) * 8u;
    volatile int *abort_flag = &abort_flag_s;
    constexpr int TILES = N <= 128 ? 2 : 1;
    constexpr uint32_t W_BYTES = TILES * LM_TILE_BYTES;
    constexpr uint32_t TMEM_COLS = 2 * TILES * N;   // 2 buffers x TILES x N columns (256 or 512)

    for (int i = threadIdx.x; i < N; i += LM_THREADS) best[i] = 0ull;
    if (threadIdx.x == 0) {
        for (int s = 0; s < NST; ++s) { ptx::mbar_init(full(s), 1); ptx::mbar_init(empty(s), 1); }
        for (int u = 0; u < 2; ++u) { ptx::mbar_init(acc_full(u), 1); ptx::mbar_init(acc_empty(u), 128); }
        ptx::mbar_init(drain_bar, 1);
        ptx::fence_mbar_init();
        abort_flag_s = 0;
        issued_s = 0;
        ptx::prefetch_tensormap(&w_map);
        ptx::prefetch_tensormap(&x_map);
    }
    if (warp == 4) {
        ptx::tmem_alloc(ptx::smem_u32(&tmem_slot), TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = tmem_slot;

    // grid = (passes, CTAs per pass): the CTAs that walk the same weight rows for different node
    // passes are neighbours in launch order, so all but the first find those rows in L2
    const int pass = blockIdx.x;                         // nodes [pass N, pass N + N)
    const int cta = blockIdx.y, n_cta = gridDim.y;
    const int n_pairs = p.n_pairs, R = p.R;
    const int my_pairs = cta < n_pairs ? (n_pairs - cta + n_cta - 1) / n_cta : 0;
    const int n_kc = p.H / LM_KC;
    const uint32_t x_off = W_BYTES;                      // X chunk sits after the weight chunk in a stage

    if (warp == 5) {
        // ---------------------------------------------------------------- TMA producer
        int it = 0;
        for (int q = 0; q < my_pairs && !*abort_flag; ++q) {
            const int row0 = (cta + q * n_cta) * TILES * R;
            for (int kc = 0; kc < n_kc; ++kc, ++it) {
                const int s = it % NST, use = it / NST;
                if (use > 0 && !ptx::mbar_wait(empty(s), (use - 1) & 1)) { *abort_flag = 1; break; }
                if (lane == 0) {
                    const uint32_t base = ring + s * p.stage_bytes;
                    ptx::mbar_arrive_expect_tx(full(s), (uint32_t)(TILES * R + N) * 128u);
                    tma_load_2d(base, &w_map, full(s), kc * LM_KC, row0);                 // rows past V arrive as zeros
                    if (TILES == 2) tma_load_2d(base + LM_TILE_BYTES, &w_map, full(s), kc * LM_KC, row0 + R);
                    tma_load_2d(base + x_off, &x_map, full(s), kc * LM_KC, pass * N);      // rows past M arrive as zeros
                }
                __syncwarp();
            }
        }
        if (lane == 0) issued_s = it;
    } else if (warp == 4) {
        // ---------------------------------------------------------------- MMA issuer
        constexpr uint32_t IDESC = LM_IDESC_BASE | ((uint32_t)(N >> 3) << 17);
        int it = 0;
        bool ok = true;
        for (int q = 0; ok && q < my_pairs && !*abort_flag; ++q) {
            const int u = q & 1;
            if (q >= 2) ok = ptx::mbar_wait(acc_empty(u), ((q >> 1) - 1) & 1);   // the epilogue has read this buffer
            if (!ok) break;
            ptx::tc_fence_after();
            for (int kc = 0; kc < n_kc; ++kc, ++it) {
                const int s = it % NST;
                ok = ptx::mbar_wait(full(s), (it / NST) & 1);
                if (!ok) break;
                ptx::tc_fence_after();
                if (lane == 0) {
                    const uint32_t base = ring + s * p.stage_bytes;
#pragma unroll
                    for (int t = 0; t < TILES; ++t)
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            ptx::mma_ss(tmem + (u * TILES + t) * N, lm_desc(base + t * LM_TILE_BYTES + kk * 32),
                                        lm_desc(base + x_off + kk * 32), IDESC, kc > 0 || kk > 0);
                    ptx::tc_commit(empty(s));                         // the stage is free once these MMAs are done
                    if (kc == n_kc - 1) ptx::tc_commit(acc_full(u));  // and so is the pair's accumulator
                }
                __syncwarp();
            }
        }
        if (!ok) *abort_flag = 1;
    } else {
        // ---------------------------------------------------------------- epilogue: thread = vocabulary row
        bool ok = true;
        for (int q = 0; q < my_pairs; ++q) {
            const int u = q & 1;
            if (*abort_flag) ok = false;
            if (ok) ok = ptx::mbar_wait(acc_full(u), (q >> 1) & 1);
            __syncwarp();
            ptx::tc_fence_after();
            const int row0 = (cta + q * n_cta) * TILES * R;
#pragma unroll 1
            for (int t = 0; t < TILES; ++t) {
                const int r = warp * 32 + lane;
                const int v = r < R ? row0 + t * R + r : p.V;          // this thread's vocabulary row (none past R)
#pragma unroll 1
                for (int c = 0; c < N / 32; ++c) {
                    uint32_t acc[32];
                    ptx::tmem_ld32(tmem + ((uint32_t)(warp * 32) << 16) + (u * TILES + t) * N + c * 32, acc);
                    ptx::tmem_ld_wait();
                    unsigned long long key[32];
#pragma unroll
                    for (int e = 0; e < 32; ++e) key[e] = v < p.V ? lm_key(acc[e], (uint32_t)v) : 0ull;
                    const unsigned long long k = warp_max_scatter32(key, lane);   // node c * 32 + lane, this warp's 32 rows
                    atomicMax(&best[c * 32 + lane], k);
                }
            }
            ptx::tc_fence_before();
            ptx::mbar_arrive(acc_empty(u));
        }
        if (!ok) *abort_flag = 1;
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0) atomicExch(p.dev_error, MTV_ERR_TIMEOUT);
        // copies in flight and issued tensor-core work get one more bounded wait before the shared
        // and tensor memory are given back
        if (warp == 5 && lane == 0)
            for (int s = 0; s < NST; ++s) {
                const int uses = (issued_s - s + NST - 1) / NST;   // how often stage s was filled
                if (issued_s > s) ptx::mbar_wait(full(s), (uses - 1) & 1);
            }
        if (warp == 4) {
            if (lane == 0) ptx::tc_commit(drain_bar);
            __syncwarp();
            ptx::mbar_wait(drain_bar, 0);
        }
        __syncthreads();
    }
    for (int n = threadIdx.x; n < N; n += LM_THREADS) {
        const int m = pass * N + n;
        if (m < p.M && best[n] != 0ull) atomicMax(p.keys + m, best[n]);
    }
    if (warp == 4) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem, TMEM_COLS);
    }
}

// keys -> (argmax, value)
__global__ void lm_head_finish_kernel(int M, const unsigned long long *__restrict__ keys, int32_t *__restrict__ am,
                                      float *__restrict__ am_val) {
    const int m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m >= M) return;
    const unsigned long long k = keys[m];
    am[m] = (int32_t)(0xffffffffu - (uint32_t)(k & 0xffffffffu));
    if (am_val) {
        const uint32_t ord = (uint32_t)(k >> 32);
        am_val[m] = __uint_as_float((ord & 0x80000000u) ? (ord & 0x7fffffffu) : ~ord);
    }
}

}  // namespace mtv

extern "C" int lm_head_argmax(const mtv_tree_t *tree, int B, int H, int V, const mtv_bf16 *x, const mtv_bf16 *W,
                              int32_t *am, float *am_val, unsigned long long *keys, void *stream) {
    using namespace mtv;
    MTV_RANGE("lm_head_argmax");
    if (!tree || !tree->on_device || !x || !W || !keys || B < 1 || V < 1 || (am_val && !am)) return MTV_ERR_INVALID_ARG;
    if (H < 64 || H % 64 != 0) return MTV_ERR_UNSUPPORTED_SHAPE;
    if (((uintptr_t)x | (uintptr_t)W) & 15) return MTV_ERR_INVALID_ARG;
    const int M = B * tree->T;
    const int N = M <= 64 ? 64 : M <= 128 ? 128 : 256;
    const int tiles = N <= 128 ? 2 : 1;                  // weight tiles per stage (see the kernel)
    const int passes = (M + N - 1) / N;
    cudaStream_t st = (cudaStream_t)stream;
    CUtensorMap w_map, x_map;
    LmParams p;
    p.keys = keys; p.dev_error = tree->d_error; p.M = M; p.H = H; p.V = V; p.N = N;
    p.stage_bytes = tiles * LM_TILE_BYTES + N * 128;
    p.n_stages = (int)((LM_SMEM_MAX - 1024) / p.stage_bytes);
    if (p.n_stages > LM_MAX_STAGES) p.n_stages = LM_MAX_STAGES;
    const size_t smem = 1024 + (size_t)p.n_stages * p.stage_bytes;
    static PerDeviceOnce attr_once;
    bool *attr_done = attr_once.flag();
    if (!attr_done || !*attr_done) {
        MTV_CUDA_CHECK(cudaFuncSetAttribute(lm_head_argmax_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, LM_SMEM_MAX));
        MTV_CUDA_CHECK(cudaFuncSetAttribute(lm_head_argmax_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, LM_SMEM_MAX));
        MTV_CUDA_CHECK(cudaFuncSetAttribute(lm_head_argmax_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, LM_SMEM_MAX));
        if (attr_done) *attr_done = true;
    }
    MTV_CUDA_CHECK(cudaMemsetAsync(keys, 0, (size_t)M * 8, st));
    int ctas = sm_count() / passes;                      // per pass; one CTA per SM in all
    const int min_pairs = (V + tiles * 128 - 1) / (tiles * 128);   // units of `tiles` weight tiles
    if (ctas > (V + 63) / 64) ctas = (V + 63) / 64;      // no tile below 32 rows
    if (ctas < 1) ctas = 1;
    // every CTA walks the same number of tile pairs; the tile height shrinks until they just cover V
    const int rounds = (min_pairs + ctas - 1) / ctas;
    p.n_pairs = ctas * rounds;
    p.R = ((V + tiles * p.n_pairs - 1) / (tiles * p.n_pairs) + 7) / 8 * 8;
    if (!tma_map_2d_bf16(&w_map, W, V, H, p.R) || !tma_map_2d_bf16(&x_map, x, M, H, N)) return MTV_ERR_CUDA;
    const dim3 grid(passes, ctas);
    if (N == 64) lm_head_argmax_kernel<64><<<grid, LM_THREADS, smem, st>>>(w_map, x_map, p);
    else if (N == 128) lm_head_argmax_kernel<128><<<grid, LM_THREADS, smem, st>>>(w_map, x_map, p);
    else lm_head_argmax_kernel<256><<<grid, LM_THREADS, smem, st>>>(w_map, x_map, p);
    if (am) lm_head_finish_kernel<<<(M + 127) / 128, 128, 0, st>>>(M, keys, am, am_val);
    MTV_CUDA_CHECK(cudaGetLastError());
    return MTV_OK;
}
