// Tree attention on the 5th-generation tensor cores (Section 3.2 / Fig. 2(b)), head_dim 128.
//
// One CTA owns up to 256 query rows (two 128-row tiles of the (node, head-in-group) block
// that shares one KV head) and a contiguous range of 128-key tiles.  Warp roles:
//   warps 0-7 / 8-15 softmax warps of row tile 0 / 1: two threads per query row, each with one
//                    half (64 keys) of the row of S from tensor memory in registers — two such warps
//                    per scheduler, so that one can use the special-function unit while the other
//                    issues the rest; they apply the ancestor bitmask on the tiles that overlap the
//                    tree rows, agree on the running max through shared memory, keep partial row
//                    sums and write P (bf16) back to tensor memory over S;
//   warp 16          issues tcgen05.mma: S_t = Q_t K^T (operands in shared memory) and
//                    O_t += P_t V (P from tensor memory, V from shared memory, N-major);
//   warp 17          TMA producer: Q once, then K and V tiles through a ring of 32 KB slots;
//   warps 18-19      only help with the copies of the merge.
// Tensor memory: S0 | S1 | O0 | O1, 128 fp32 columns each; P_t overlays the first 64 columns
// of S_t.  The softmax warpgroups take registers from the fifth warpgroup (setmaxnreg).
//
// The key splits of one query block are merged inside the same launch.  After its last key tile
// a CTA parks its partial in shared memory — its own normalised result O / l in bf16 plus the
// fp32 pair (m, l); the exchange of partials is bound by L2 bandwidth, so they travel in the
// output's precision — sends it to the workspace with bulk copies (it stays in L2), and arrives
// on a counter of its query block.  When all splits of
// the block have arrived, every CTA fetches a slice of the rows of all partials with bulk copies
// (plain loads would be throttled by the little L1 this kernel leaves), combines them in fp32 with
// the weights exp2(m_s - m) l_s / sum and writes bf16 output rows.  The grid never exceeds one CTA per SM, so all CTAs are resident together and
// the wait on the counter always ends; it is bounded all the same.  The counters live in the
// tree object, start at zero and are put back to zero by the last CTA that has seen them full.
//
// The running max is only raised when the new row max exceeds it by more than 8 (in log2
// units), so O in tensor memory is rescaled rarely; P stays below 2^8.
#include <cuda.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace mtv {

constexpr int TC_BN = 128;
constexpr int TC_SLOTS = 5;
constexpr int TC_THREADS = 640;   // 5 warpgroups: 4 of softmax warps, {MMA warp, TMA warp, 2 helper warps}
constexpr int TC_MMA_WARP = 16, TC_TMA_WARP = 17;
constexpr uint32_t TC_TILE_BYTES = 128 * 128 * 2;   // one 128 x 128 bf16 tile: two 64-column halves
constexpr uint32_t TC_HALF_BYTES = TC_TILE_BYTES / 2;
constexpr uint32_t TC_Q_BYTES = 2 * TC_TILE_BYTES;
constexpr uint32_t TC_RING_BYTES = TC_SLOTS * TC_TILE_BYTES;
constexpr uint32_t TC_BAR_BYTES = 256;
constexpr uint32_t TC_XMAX_BYTES = 2 * 2 * 128 * 2;   // running-max exchange of the two half-row threads, bf16
constexpr uint32_t TC_SMEM_BYTES = 1024 + TC_Q_BYTES + TC_RING_BYTES + TC_BAR_BYTES + TC_XMAX_BYTES;
static_assert(TC_SMEM_BYTES <= 227 * 1024, "shared memory budget");
constexpr float TC_RESCALE_THRESHOLD = 8.f;
constexpr int TC_MAX_SPLITS = 32;
constexpr int TC_MAX_GROUPS = 256;   // merge counters available in the tree object

// Register rebalancing.  The CTA's pool is what the launch allocates: TC_THREADS threads at the
// per-thread count the compiler derives from the launch bounds (65536 / 640 rounded down to a
// multiple of 8 = 96).  setmaxnreg.inc blocks until the pool has the registers, so the five
// warpgroups' targets must not add up to more than the pool: 4 x 104 + 64 = 5 x 96.
constexpr int TC_REGS_LAUNCH = 96, TC_REGS_SOFTMAX = 104, TC_REGS_OTHER = 64;
static_assert(4 * TC_REGS_SOFTMAX + TC_REGS_OTHER <= 5 * TC_REGS_LAUNCH, "setmaxnreg targets exceed the CTA's register pool");
static_assert(TC_REGS_LAUNCH * TC_THREADS <= 65536, "launch register count does not fit the register file");

// After the last key tile the Q / K / V buffers are reused:
//   [0, 64 KB)       the parked partial: 256 rows of 128 bf16 values O / l (the split's own normalised
//                    result; fp32 (m, l) travel beside it).  16-byte chunk j of row r sits at chunk
//                    position j ^ (r & 15): the one-row-per-thread stores are conflict-free while rows
//                    stay contiguous for one bulk copy.  The workspace holds partials in the same
//                    form; whoever reads a row undoes the permutation.  After the partial has left
//                    for the workspace the same space receives the rows this CTA merges.
//   the last 8 KB    parked (m, l) per row; (m, l) then the merge weights of every split
constexpr uint32_t TC_ROW_BYTES = 256;
constexpr uint32_t TC_TILES_BYTES = TC_Q_BYTES + TC_RING_BYTES;
constexpr uint32_t TC_PARK_ML_OFF = TC_TILES_BYTES - 8192;
constexpr uint32_t TC_WBUF_OFF = TC_PARK_ML_OFF + 256 * 8;
constexpr uint32_t TC_WBUF_ENTRIES = 256 + TC_MAX_SPLITS;
static_assert(TC_WBUF_OFF + TC_WBUF_ENTRIES * 8 <= TC_TILES_BYTES, "merge buffers must fit the tile buffers");
static_assert((256 + TC_MAX_SPLITS) * TC_ROW_BYTES <= TC_PARK_ML_OFF, "rows to merge must fit below the small buffers");

// barrier slots (8 bytes each) inside the barrier region
enum { BAR_Q = 0 /* one per row tile */, BAR_KV_FULL = 2, BAR_KV_EMPTY = BAR_KV_FULL + TC_SLOTS, BAR_S = BAR_KV_EMPTY + TC_SLOTS,
       BAR_P = BAR_S + 2, BAR_O = BAR_P + 2, BAR_FINAL = BAR_O + 2, BAR_MERGE = BAR_FINAL + 1, BAR_COUNT = BAR_MERGE + 1 };
static_assert(BAR_COUNT * 8 + 8 <= TC_BAR_BYTES, "barrier region too small");

// instruction descriptors: bf16 x bf16 -> fp32, M = 128, N = 128
constexpr uint32_t IDESC_BASE = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t IDESC_QK = IDESC_BASE;               // A, B both K-major
constexpr uint32_t IDESC_PV = IDESC_BASE | (1u << 16);  // B (= V) N-major

struct TcParams {
    const int32_t *seq_lens;
    const uint64_t *anc;   // [T][2]
    __nv_bfloat16 *out;    // [B][T][Hq][128]
    __nv_bfloat16 *ws_o;   // [groups][nsplit][256 rows][128] partial O / l, chunks permuted (only when nsplit > 1)
    float2 *ws_ml;         // [groups][nsplit][256] partial (m, l)
    int32_t *arrive, *depart;   // [groups] merge counters, zero between calls
    int32_t *status;       // [B] or null
    int32_t *dev_error;
    float scale_log2;
    int T, G, Hq, Hkv, Lcap, nsplit, n_rt, M_rows;
};

// 128-byte-swizzled shared-memory operand descriptor.
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(lbo_bytes >> 4) << 16;
    d |= (uint64_t)(sbo_bytes >> 4) << 32;
    d |= 1ull << 46;   // descriptor version of this architecture
    d |= 2ull << 61;   // 128-byte swizzle
    return d;
}
// K-major operand (rows 128 bytes apart inside an 8-row group, groups 1024 bytes apart)
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t saddr) { return smem_desc(saddr, 16, 1024); }
// N-major operand: 64-column halves TC_HALF_BYTES apart, 8-key groups 1024 bytes apart
__device__ __forceinline__ uint64_t desc_nmajor(uint32_t saddr) { return smem_desc(saddr, TC_HALF_BYTES, 1024); }

// Register rebalancing between warpgroups (all four warps of a warpgroup execute it).
template <int N> __device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }

// CTA-wide barrier usable from the diverged warp roles (every thread of the CTA arrives on it,
// from whichever copy of the epilogue it runs).
__device__ __forceinline__ void cta_sync() { asm volatile("bar.sync 1, %0;" ::"n"(TC_THREADS) : "memory"); }

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ int ld_acquire(const int32_t *p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Developer timeline (compiled out unless MTV_TRACE is defined): lane 0 of the calling warp
// stores the SM cycle counter of event `id` for this CTA.
#ifdef MTV_TRACE
__device__ long long *g_trace = nullptr;   // [ctas][64]
#define TRACE_CTA ((size_t)(blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x)
#define TRACE(id)                                                                      \
    do {                                                                               \
        if (g_trace && (threadIdx.x % 32) == 0) g_trace[TRACE_CTA * 64 + (id)] = clock64(); \
    } while (0)
#else
#define TRACE(id)
#endif

// What the epilogue needs from the main body.
struct TcCtx {
    unsigned char *tiles;   // 1024-byte aligned base of the tile buffers (generic address)
    uint32_t bars;          // shared address of the barrier region
    volatile int *abort_flag;
    uint32_t tmem;
    int nt, split, rows0, g, b, cnt;
    bool final_committed;
};

// Everything after the last key tile; instantiated once for the softmax warpgroups (which have
// the registers to keep many loads in flight) and once for the third warpgroup.
template <bool SOFTMAX>
__device__ __forceinline__ void tc_epilogue(const TcParams &p, const TcCtx &c) {
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    float2 *wbuf = reinterpret_cast<float2 *>(c.tiles + TC_WBUF_OFF);
    auto bar = [&](int i) { return c.bars + (uint32_t)i * 8u; };

    ptx::tc_fence_before();
    cta_sync();   // every role is done; partials are parked
    if (*c.abort_flag) {
        // A bounded wait ran out: raise the sticky error, give outstanding copies and tensor-core
        // work one more bounded chance to finish.  The CTA still takes part in the merge so that
        // the other splits never wait for it; the error word tells the host the output is invalid.
        if (threadIdx.x == 0) atomicExch(p.dev_error, MTV_ERR_TIMEOUT);
        if (!SOFTMAX) {
            if (warp == TC_TMA_WARP && lane == 0) {
                ptx::mbar_wait(bar(BAR_Q), 0);
                if (c.nt == 2) ptx::mbar_wait(bar(BAR_Q + 1), 0);
                for (int s = 0; s < TC_SLOTS; ++s) { ptx::mbar_wait(bar(BAR_KV_FULL + s), 0); ptx::mbar_wait(bar(BAR_KV_FULL + s), 1); }
            }
            if (warp == TC_MMA_WARP) {
                if (!c.final_committed && lane == 0) ptx::tc_commit(bar(BAR_FINAL));
                __syncwarp();
                ptx::mbar_wait(bar(BAR_FINAL), 0);
            }
        }
        cta_sync();
    }
    if (warp == 0) TRACE(44);   // partial parked

    const int act_rows = c.nt * 128;
    const int nsplit = p.nsplit;
    const int grp = blockIdx.z * gridDim.y + blockIdx.y;
    const unsigned char *rows_smem = c.tiles;   // parked rows, later the rows to merge
    // chunk j (8 bf16 values) of a 256-byte row whose index inside its 256-row slab is r
    auto chunk = [&](const unsigned char *row_ptr, int r, int j) {
        return *reinterpret_cast<const uint4 *>(row_ptr + ((j ^ (r & 15)) << 4));
    };
    auto out_ptr = [&](int r, int j) {   // 8 output values of query-block row r
        const int node = r / p.G, hq = c.g * p.G + r % p.G;
        return reinterpret_cast<uint4 *>(p.out + (((size_t)c.b * p.T + node) * p.Hq + hq) * 128 + j * 8);
    };
    if (nsplit == 1) {
        // the parked partial is the result
        for (int item = threadIdx.x; item < act_rows * 16; item += TC_THREADS) {
            const int row = item / 16, j = item % 16, r = c.rows0 + row;
            if (r < p.M_rows) *out_ptr(r, j) = chunk(rows_smem + row * TC_ROW_BYTES, row, j);
        }
    } else {
        const size_t slab0 = (size_t)grp * nsplit;   // first slab of this query block
        const int rows_per = (act_rows + nsplit - 1) / nsplit;
        const int row_begin = c.split * rows_per;
        const int n_my = max(0, min(act_rows, row_begin + rows_per) - row_begin);
        if (threadIdx.x == 0) {
            // ---- publish: two bulk copies out of shared memory, then arrive and wait for the others
            const size_t slab = slab0 + c.split;
            ptx::bulk_s2g(p.ws_o + slab * 256 * 128, ptx::smem_u32(c.tiles), act_rows * TC_ROW_BYTES);
            ptx::bulk_s2g(p.ws_ml + slab * 256, ptx::smem_u32(c.tiles + TC_PARK_ML_OFF), act_rows * 8);
            ptx::bulk_commit();
            ptx::bulk_wait_all();
            TRACE(51);   // partial left shared memory and is written
            ptx::fence_proxy_async_global();
            // release-arrive without waiting for the counter's old value
            asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(p.arrive + grp) : "memory");
            TRACE(52);   // arrived
            const long long t0 = clock64();
            while (ld_acquire(p.arrive + grp) < nsplit)
                if (clock64() - t0 > ptx::WAIT_CYCLE_LIMIT) { atomicExch(p.dev_error, MTV_ERR_TIMEOUT); break; }
            TRACE(53);   // everybody arrived
        }
        cta_sync();
        // ---- fetch rows [row_begin, row_begin + n_my) of every split: one bulk copy per split, each issued by a
        //      different warp (the copies of one warp's lanes are issued one after the other)
        if (n_my > 0 && lane == 0) {
            if (warp == 0) ptx::mbar_arrive_expect_tx(bar(BAR_MERGE), (uint32_t)(nsplit * n_my) * TC_ROW_BYTES);
            ptx::fence_proxy_async_global();   // the other CTAs' partials, acquired above, before the async-proxy reads
            for (int sp = warp; sp < nsplit; sp += TC_THREADS / 32)
                ptx::bulk_g2s(ptx::smem_u32(c.tiles) + (uint32_t)(sp * n_my) * TC_ROW_BYTES,
                              p.ws_o + ((slab0 + sp) * 256 + row_begin) * 128, (uint32_t)n_my * TC_ROW_BYTES, bar(BAR_MERGE));
        }
        if (warp == 0) TRACE(45);   // all splits arrived, rows on their way
        // Nobody polls the arrival counter once all have seen it full: the last one to get here puts both counters
        // back to zero (the next call cannot start before this kernel has ended).  Done here, behind the copies,
        // so that the round trip of the atomic is not on the way of anything.
        if (threadIdx.x == 0 && atomicAdd(p.depart + grp, 1) == nsplit - 1) {
            p.arrive[grp] = 0;
            p.depart[grp] = 0;
            __threadfence();
        }
        // ---- merge weights, one warp per row, lane s = split s: exp2(m_s - m) l_s / sum over the splits
        //      (split s contributes its own normalised result O_s / l_s)
        for (int rl = warp; rl < n_my; rl += TC_THREADS / 32) {
            float2 ml = make_float2(-INFINITY, 0.f);
            if (lane < nsplit) ml = __ldcg(p.ws_ml + (slab0 + lane) * 256 + row_begin + rl);
            float m = ml.x;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
            const float w = ml.x == -INFINITY ? 0.f : ex2(ml.x - m) * ml.y;
            float lsum = w;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, o);
            if (lane < nsplit) wbuf[rl * nsplit + lane].x = w / lsum;
        }
        cta_sync();
        if (warp == 0) TRACE(49);   // weights ready
        if (n_my > 0 && !ptx::mbar_wait(bar(BAR_MERGE), 0) && threadIdx.x == 0) atomicExch(p.dev_error, MTV_ERR_TIMEOUT);
        if (warp == 0) TRACE(50);   // rows landed
        for (int item = threadIdx.x; item < n_my * 16; item += TC_THREADS) {
            const int rl = item / 16, j = item % 16;
            const int r = c.rows0 + row_begin + rl;
            if (r >= p.M_rows) continue;
            float acc[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = 0.f;
            const unsigned char *row_ptr = rows_smem + rl * TC_ROW_BYTES;
#pragma unroll 6
            for (int sp = 0; sp < nsplit; ++sp) {
                const float w = wbuf[rl * nsplit + sp].x;
                const uint4 v = chunk(row_ptr + (size_t)(sp * n_my) * TC_ROW_BYTES, row_begin + rl, j);
                const uint32_t vw[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    acc[2 * e] = fmaf(w, __uint_as_float(vw[e] << 16), acc[2 * e]);
                    acc[2 * e + 1] = fmaf(w, __uint_as_float(vw[e] & 0xffff0000u), acc[2 * e + 1]);
                }
            }
            *out_ptr(r, j) = make_uint4(pack2_bf16(acc[0], acc[1]), pack2_bf16(acc[2], acc[3]),
                                        pack2_bf16(acc[4], acc[5]), pack2_bf16(acc[6], acc[7]));
        }
        if (warp == 0) TRACE(46);   // merge done
    }
    if (!SOFTMAX && warp == TC_MMA_WARP) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(c.tmem, 512);
    }
    if (warp == 0) TRACE(47);
}

__global__ void __launch_bounds__(TC_THREADS, 1)
tree_attn_tc_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                    const __grid_constant__ CUtensorMap v_map, const TcParams p) {
    extern __shared__ unsigned char smem_raw[];
    // Programmatic dependent launch: let the next kernel of the stream be set up while this one runs.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int split = blockIdx.x;
    const int g = blockIdx.y / p.n_rt, rt = blockIdx.y % p.n_rt;
    const int b = blockIdx.z;
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    if (warp == 0) TRACE(0);

    // carve shared memory (tiles need 1024-byte alignment for the 128-byte swizzle)
    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
    const uint32_t q_smem = raw + pad;
    const uint32_t ring = q_smem + TC_Q_BYTES;
    const uint32_t bars = ring + TC_RING_BYTES;
    unsigned char *tiles_gen = smem_raw + pad;
    unsigned char *bar_region = tiles_gen + TC_Q_BYTES + TC_RING_BYTES;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(bar_region + BAR_COUNT * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bar_region + BAR_COUNT * 8 + 4);
    auto bar = [&](int i) { return bars + (uint32_t)i * 8u; };
    float2 *park_ml = reinterpret_cast<float2 *>(tiles_gen + TC_PARK_ML_OFF);

    if (warp == TC_TMA_WARP && lane == 0) {
        ptx::mbar_init(bar(BAR_Q), 1);
        ptx::mbar_init(bar(BAR_Q + 1), 1);
        // the copy engine fetches the three descriptors while the CTA sets itself up (they are kernel parameters:
        // nothing the previous kernel of the stream could still be writing)
        ptx::prefetch_tensormap(&k_map);
        ptx::prefetch_tensormap(&q_map);
        ptx::prefetch_tensormap(&v_map);
        for (int s = 0; s < TC_SLOTS; ++s) { ptx::mbar_init(bar(BAR_KV_FULL + s), 1); ptx::mbar_init(bar(BAR_KV_EMPTY + s), 1); }
        for (int t = 0; t < 2; ++t) {
            ptx::mbar_init(bar(BAR_S + t), 1);
            ptx::mbar_init(bar(BAR_P + t), 256);
            ptx::mbar_init(bar(BAR_O + t), 1);
        }
        ptx::mbar_init(bar(BAR_FINAL), 1);
        ptx::mbar_init(bar(BAR_MERGE), 1);
        ptx::fence_mbar_init();
        *abort_flag = 0;
    }
    if (warp == TC_MMA_WARP) {
        ptx::tmem_alloc(ptx::smem_u32(const_cast<uint32_t *>(tmem_slot)), 512);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    if (warp == 0) TRACE(1);

    // Nothing above touched global memory.  From here on the previous kernel of the stream must be
    // complete (its outputs may be this kernel's inputs, and it may share the workspace and counters).
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int L = p.seq_lens[b];
    const bool reporter = blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0;
    if (L + p.T > p.Lcap) {         // the same for every CTA of the query block: nobody waits for anybody
        if (reporter && p.status) p.status[b] = MTV_ERR_CAPACITY;
        if (warp == TC_MMA_WARP) ptx::tmem_dealloc(*tmem_slot, 512);
        return;
    }
    if (reporter && p.status) p.status[b] = MTV_OK;
    const int n_keys = L + p.T;
    const int tiles = (n_keys + TC_BN - 1) / TC_BN;
    const int base_cnt = tiles / p.nsplit, rem = tiles % p.nsplit;
    const int t_begin = split * base_cnt + min(split, rem);
    const int cnt = base_cnt + (split < rem ? 1 : 0);
    const int rows0 = rt * 256;
    const int nt = p.M_rows - rows0 > 128 ? 2 : 1;

    // One K or V tile into ring slot (i mod TC_SLOTS): i = 2j is K of key tile j, i = 2j + 1 is V.
    auto issue_kv = [&](int i) {
        const int slot = i % TC_SLOTS;
        const CUtensorMap *map = (i & 1) ? &v_map : &k_map;
        ptx::mbar_arrive_expect_tx(bar(BAR_KV_FULL + slot), TC_TILE_BYTES);
        for (int half = 0; half < 2; ++half)
            ptx::tma_load_4d(ring + slot * TC_TILE_BYTES + half * TC_HALF_BYTES, map, bar(BAR_KV_FULL + slot), half * 64,
                             (t_begin + i / 2) * TC_BN, g, b);
    };
    const int n_loads = 2 * cnt;
    // Only the first K and V tiles are requested before the CTA syncs; the others wait until the first query tile
    // has landed, so that what the first MMAs need is not queued behind 160 KB of tiles that are needed later.
    const int n_early = min(n_loads, 2);

    if (warp == TC_TMA_WARP && lane == 0) {
        if (cnt > 0) {
            // first K tile, then Q (a barrier per row tile: the first MMA needs K_0 and the first tile only), then the rest
            issue_kv(0);
            for (int t = 0; t < nt; ++t) {
                ptx::mbar_arrive_expect_tx(bar(BAR_Q + t), TC_TILE_BYTES);
                for (int half = 0; half < 2; ++half)
                    ptx::tma_load_4d(q_smem + t * TC_TILE_BYTES + half * TC_HALF_BYTES, &q_map, bar(BAR_Q + t), half * 64,
                                     g * p.G, (rows0 + t * 128) / p.G, b);
            }
            for (int i = 1; i < n_early; ++i) issue_kv(i);
        }
    }
    __syncwarp();

    TcCtx ctx;
    ctx.tiles = tiles_gen; ctx.bars = bars; ctx.abort_flag = abort_flag; ctx.tmem = *tmem_slot;
    ctx.nt = nt; ctx.split = split; ctx.rows0 = rows0; ctx.g = g; ctx.b = b; ctx.cnt = cnt;
    ctx.final_committed = false;
    const uint32_t tmem = ctx.tmem;

    if (warp >= 16) {
        reg_dec<TC_REGS_OTHER>();   // the whole fifth warpgroup gives registers to the softmax warpgroups
        if (warp == TC_TMA_WARP) {
            // ------------------------------------------------------------ TMA producer (the rest of the tiles)
            if (cnt > 0 && !ptx::mbar_wait(bar(BAR_Q), 0)) *abort_flag = 1;
            for (int i = n_early; i < n_loads && !*abort_flag; ++i) {
                const int slot = i % TC_SLOTS, use = i / TC_SLOTS;
                if (use > 0 && !ptx::mbar_wait(bar(BAR_KV_EMPTY + slot), (use - 1) & 1)) { *abort_flag = 1; break; }
                if (lane == 0) issue_kv(i);
                __syncwarp();
            }
        } else if (warp == TC_MMA_WARP) {
            // ------------------------------------------------------------ MMA issuer
            auto issue_S = [&](int t, int j) {
                const uint32_t kbase = ring + ((2 * j) % TC_SLOTS) * TC_TILE_BYTES;
                const uint32_t qbase = q_smem + t * TC_TILE_BYTES;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint32_t off = (kk / 4) * TC_HALF_BYTES + (kk % 4) * 32;
                    ptx::mma_ss(tmem + t * 128, desc_kmajor(qbase + off), desc_kmajor(kbase + off), IDESC_QK, kk > 0);
                }
            };
            auto issue_PV = [&](int t, int j) {
                const uint32_t vbase = ring + ((2 * j + 1) % TC_SLOTS) * TC_TILE_BYTES;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    ptx::mma_ts(tmem + 256 + t * 128, tmem + t * 128 + kk * 8, desc_nmajor(vbase + kk * 2048), IDESC_PV,
                                j > 0 || kk > 0);
            };
            auto wait_kv = [&](int i) { return ptx::mbar_wait(bar(BAR_KV_FULL + i % TC_SLOTS), (i / TC_SLOTS) & 1); };
            bool ok = cnt == 0 || (wait_kv(0) && ptx::mbar_wait(bar(BAR_Q), 0));
            if (ok && cnt > 0) {
                TRACE(2);   // Q and K_0 landed
                ptx::tc_fence_after();
                if (lane == 0) {
                    issue_S(0, 0);
                    ptx::tc_commit(bar(BAR_S + 0));
                }
                __syncwarp();
                if (nt == 2) ok = ptx::mbar_wait(bar(BAR_Q + 1), 0);
                ptx::tc_fence_after();
                if (ok && lane == 0) {
                    if (nt == 2) { issue_S(1, 0); ptx::tc_commit(bar(BAR_S + 1)); }
                    ptx::tc_commit(bar(BAR_KV_EMPTY + 0));
                }
                __syncwarp();
            }
            for (int j = 0; ok && j < cnt && !*abort_flag; ++j) {
                const bool more = j + 1 < cnt;
                ok = wait_kv(2 * j + 1);
                if (!ok) break;
                {
                    // Rows of the V tile past the last valid key hold whatever the cache holds there; their
                    // P is zero, but 0 * NaN would still poison O: clear them before the tensor core reads.
                    const int valid = n_keys - (t_begin + j) * TC_BN;
                    if (valid < TC_BN) {
                        unsigned char *vt = tiles_gen + TC_Q_BYTES + ((2 * j + 1) % TC_SLOTS) * TC_TILE_BYTES;
                        for (int e = lane; e < (TC_BN - valid) * 16; e += 32) {
                            const int row = valid + e / 16, c16 = e % 16;     // 16 x 16 bytes per row: 8 per half
                            *reinterpret_cast<uint4 *>(vt + (c16 / 8) * TC_HALF_BYTES + row * 128 + (c16 % 8) * 16) =
                                make_uint4(0u, 0u, 0u, 0u);
                        }
                        ptx::fence_proxy_async();
                        __syncwarp();
                    }
                }
                ok = ptx::mbar_wait(bar(BAR_P + 0), j & 1);
                if (!ok) break;
                ptx::tc_fence_after();
                if (lane == 0) { issue_PV(0, j); ptx::tc_commit(bar(BAR_O + 0)); }
                __syncwarp();
                if (more) {
                    ok = wait_kv(2 * j + 2);
                    if (!ok) break;
                    ptx::tc_fence_after();
                    if (lane == 0) { issue_S(0, j + 1); ptx::tc_commit(bar(BAR_S + 0)); }
                    __syncwarp();
                }
                if (nt == 2) {
                    ok = ptx::mbar_wait(bar(BAR_P + 1), j & 1);
                    if (!ok) break;
                    ptx::tc_fence_after();
                    if (lane == 0) { issue_PV(1, j); ptx::tc_commit(bar(BAR_O + 1)); }
                    __syncwarp();
                }
                if (lane == 0) {
                    ptx::tc_commit(bar(BAR_KV_EMPTY + (2 * j + 1) % TC_SLOTS));   // V_j is free once its MMAs are done
                    if (more) {
                        if (nt == 2) { issue_S(1, j + 1); ptx::tc_commit(bar(BAR_S + 1)); }
                        ptx::tc_commit(bar(BAR_KV_EMPTY + (2 * j + 2) % TC_SLOTS));
                    }
                }
                __syncwarp();
            }
            if (ok && cnt > 0 && !*abort_flag) {
                if (lane == 0) ptx::tc_commit(bar(BAR_FINAL));   // follows every tensor-core operation issued
                __syncwarp();
                ctx.final_committed = true;
            }
            if (!ok) *abort_flag = 1;
        }
        tc_epilogue<false>(p, ctx);
    } else {
        reg_inc<TC_REGS_SOFTMAX>();
        if (warp / 8 < nt) {
            // ------------------------------------------------------------ softmax warps of row tile t
            // Thread (row, hf) owns keys [64 hf, 64 hf + 64) of its query row in every key tile.
            const int t = warp / 8, hf = (warp / 4) & 1;
            const int row = (warp % 4) * 32 + lane;
            const int r = rows0 + t * 128 + row;
            uint64_t alo = 0, ahi = 0;
            if (r < p.M_rows) { alo = p.anc[(r / p.G) * 2]; ahi = p.anc[(r / p.G) * 2 + 1]; }
            const uint32_t lane_base = (uint32_t)((warp % 4) * 32) << 16;
            const uint32_t t_s = tmem + lane_base + t * 128 + hf * 64;          // this thread's 64 columns of S_t
            const uint32_t t_p = tmem + lane_base + t * 128 + hf * 32;          // its 32 columns of P_t
            const uint32_t t_o = tmem + lane_base + 256 + t * 128 + hf * 64;    // its 64 columns of O_t
            __nv_bfloat16 *xmax = reinterpret_cast<__nv_bfloat16 *>(bar_region + TC_BAR_BYTES);   // [t][hf][row]
            auto pair_sync = [&]() { asm volatile("bar.sync %0, 256;" ::"r"(2 + t) : "memory"); };  // the 256 threads of row tile t
            float m_used = -INFINITY, l = 0.f;
            bool ok = true;
            // visibility of the tree rows as 32-bit words: word q covers tree rows 32q .. 32q+31
            auto anc_word = [&](int q) -> uint32_t {
                if (q < 0) return 0xffffffffu;     // prefix rows are visible to every node
                if (q == 0) return (uint32_t)alo;
                if (q == 1) return (uint32_t)(alo >> 32);
                if (q == 2) return (uint32_t)ahi;
                if (q == 3) return (uint32_t)(ahi >> 32);
                return 0u;                         // past the tree rows: nothing
            };
            // A thread whose wait ran out keeps going through the motions without waiting, so that
            // the barriers it shares with the other half-row threads stay matched.
            for (int j = 0; j < cnt; ++j) {
                if (*abort_flag) ok = false;
                if (ok) ok = ptx::mbar_wait(bar(BAR_S + t), j & 1);
                if (warp % 8 == 0 && j < 6) TRACE(8 + t * 16 + j * 2);       // S_t(j) ready
                ptx::tc_fence_after();
                // ---- this thread's half row of S in registers (raw scores; the scale is positive)
                uint32_t sr[2][32];
                ptx::tmem_ld32(t_s, sr[0]);
                ptx::tmem_ld32(t_s + 32, sr[1]);
                ptx::tmem_ld_wait();
                const int key0 = (t_begin + j) * TC_BN + hf * 64;
                if (key0 + 64 > L) {
                    // the half tile overlaps the tree rows or the end of the cache: bit e of vis is column 32c + e
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        const int a0 = key0 + c * 32 - L;        // tree row of the chunk's first column
                        const int q = a0 >> 5, sh = a0 & 31;     // floor division
                        const uint32_t vis = __funnelshift_r(anc_word(q), anc_word(q + 1), sh);
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if (!((vis >> e) & 1u)) sr[c][e] = 0xff800000u;   // -inf
                    }
                }
                float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
                for (int c = 0; c < 2; ++c)
#pragma unroll
                    for (int e = 0; e < 32; e += 4) {
                        mx0 = fmaxf(mx0, __uint_as_float(sr[c][e]));
                        mx1 = fmaxf(mx1, __uint_as_float(sr[c][e + 1]));
                        mx2 = fmaxf(mx2, __uint_as_float(sr[c][e + 2]));
                        mx3 = fmaxf(mx3, __uint_as_float(sr[c][e + 3]));
                    }
                // The two halves need the same reference, not the exact maximum (P may reach 2^8):
                // they exchange their maxima rounded to bf16 and both take the larger rounded value.
                const __nv_bfloat16 own = __float2bfloat16_rn(fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * p.scale_log2);
                xmax[(t * 2 + hf) * 128 + row] = own;
                pair_sync();   // also: both halves hold their S before anyone overwrites it with P
                const float mxs = fmaxf(__bfloat162float(own), __bfloat162float(xmax[(t * 2 + (hf ^ 1)) * 128 + row]));
                const float m_new = (j == 0 || mxs > m_used + TC_RESCALE_THRESHOLD) ? mxs : m_used;
                // O holds sums relative to m_used: rescale it when the reference moves (rare)
                const bool need = j > 0 && m_new != m_used && m_used != -INFINITY;
                if (__any_sync(0xffffffffu, need)) {
                    if (ok) ok = ptx::mbar_wait(bar(BAR_O + t), (j - 1) & 1);
                    ptx::tc_fence_after();
                    const float alpha = need ? ex2(m_used - m_new) : 1.f;
#pragma unroll 1
                    for (int c = 0; c < 4; ++c) {
                        uint32_t o[16];
                        ptx::tmem_ld16(t_o + c * 16, o);
                        ptx::tmem_ld_wait();
#pragma unroll
                        for (int e = 0; e < 16; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                        ptx::tmem_st16(t_o + c * 16, o);
                    }
                    ptx::tmem_st_wait();
                    l *= alpha;
                }
                m_used = m_new;
                const float m_eff = m_used == -INFINITY ? 0.f : m_used;
                // ---- P = exp2(scale * S - m), partial row sum, bf16 P over the first 64 columns of S_t
                float l0 = 0.f, l1 = 0.f, l2 = 0.f, l3 = 0.f;
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t pk[16];
#pragma unroll
                    for (int e = 0; e < 16; e += 2) {
                        const float p0 = ex2(fmaf(__uint_as_float(sr[c][2 * e]), p.scale_log2, -m_eff));
                        const float p1 = ex2(fmaf(__uint_as_float(sr[c][2 * e + 1]), p.scale_log2, -m_eff));
                        const float p2 = ex2(fmaf(__uint_as_float(sr[c][2 * e + 2]), p.scale_log2, -m_eff));
                        const float p3 = ex2(fmaf(__uint_as_float(sr[c][2 * e + 3]), p.scale_log2, -m_eff));
                        l0 += p0; l1 += p1; l2 += p2; l3 += p3;
                        pk[e] = pack2_bf16(p0, p1);
                        pk[e + 1] = pack2_bf16(p2, p3);
                    }
                    ptx::tmem_st16(t_p + c * 16, pk);
                }
                l += (l0 + l1) + (l2 + l3);
                ptx::tmem_st_wait();
                ptx::tc_fence_before();
                ptx::mbar_arrive(bar(BAR_P + t));
                if (warp % 8 == 0 && j < 6) TRACE(9 + t * 16 + j * 2);       // P_t(j) written
            }
            // ---- hand over the partial of this row
            if (cnt > 0) {
                // every tensor-core read of the tile buffers must be over before they are reused
                if (*abort_flag) ok = false;
                if (ok) ok = ptx::mbar_wait(bar(BAR_FINAL), 0);
                if (warp % 8 == 0) TRACE(40 + t);                            // all tensor-core work done
                ptx::tc_fence_after();
            }
            // the row sum is the sum of the two halves' sums
            float *lx = reinterpret_cast<float *>(tiles_gen + TC_WBUF_OFF);   // [t][hf][row], free once the tiles are
            lx[(t * 2 + hf) * 128 + row] = l;
            pair_sync();
            l += lx[(t * 2 + (hf ^ 1)) * 128 + row];
            const bool have_o = cnt > 0 && ok;
            {
                // park this thread's 64 columns of O / l as bf16: chunk j at position j ^ (row & 15); an empty
                // split parks zeros
                unsigned char *dst = tiles_gen + (t * 128 + row) * TC_ROW_BYTES;
                const int sw = (t * 128 + row) & 15;
                const float inv_l = have_o && l > 0.f ? 1.f / l : 0.f;
#pragma unroll 1
                for (int c = 0; c < 2; ++c) {
                    uint32_t o[32];
                    if (have_o) {
                        ptx::tmem_ld32(t_o + c * 32, o);
                        ptx::tmem_ld_wait();
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e) o[e] = 0u;
                    }
#pragma unroll
                    for (int e = 0; e < 32; e += 8) {
                        uint4 pk;
                        pk.x = pack2_bf16(__uint_as_float(o[e]) * inv_l, __uint_as_float(o[e + 1]) * inv_l);
                        pk.y = pack2_bf16(__uint_as_float(o[e + 2]) * inv_l, __uint_as_float(o[e + 3]) * inv_l);
                        pk.z = pack2_bf16(__uint_as_float(o[e + 4]) * inv_l, __uint_as_float(o[e + 5]) * inv_l);
                        pk.w = pack2_bf16(__uint_as_float(o[e + 6]) * inv_l, __uint_as_float(o[e + 7]) * inv_l);
                        *reinterpret_cast<uint4 *>(dst + (((hf * 8 + c * 4 + e / 8) ^ sw) << 4)) = pk;
                    }
                }
                if (hf == 0) park_ml[t * 128 + row] = make_float2(m_used, l);   // (-inf, 0) for an empty split
                ptx::fence_proxy_async();   // the bulk copy out of shared memory must see these stores
            }
            if (!ok) *abort_flag = 1;
        }
        tc_epilogue<true>(p, ctx);
    }
}

// ---------------------------------------------------------------------------------------- host
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// 4-D bf16 tensor map with a 128-byte-swizzled box whose innermost extent is 64 elements.
static bool encode_map(CUtensorMap *map, const void *base, const cuuint64_t dims[4], const cuuint64_t strides_bytes[3],
                       const cuuint32_t box[4]) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint32_t ones[4] = {1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides_bytes, box, ones,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool attn_tc_eligible(int D, int G) { return D == 128 && (G == 1 || G == 2 || G == 4 || G == 8); }

static int tc_prepare() {
    static bool done = false;
    if (!done) {
        MTV_CUDA_CHECK(cudaFuncSetAttribute(tree_attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_BYTES));
        // the register rebalancing inside the kernel assumes the pool of a 168-register launch
        cudaFuncAttributes fa;
        MTV_CUDA_CHECK(cudaFuncGetAttributes(&fa, tree_attn_tc_kernel));
        if (fa.numRegs < TC_REGS_LAUNCH) {
            set_last_error("tree_attn_tc_kernel was built with too few registers for its setmaxnreg targets", cudaErrorInvalidValue);
            return MTV_ERR_CUDA;
        }
        done = true;
    }
    return MTV_OK;
}

// Number of key splits of a problem: as many as keep the whole grid within one wave of SMs
// (one CTA per SM), at most one per key tile, at most TC_MAX_SPLITS.  More than one split needs
// a merge counter per query block.
int attn_tc_plan(int T, int G, int B, int Hkv, int Lcap, int *n_rt_out) {
    const int n_rt = (T * G + 255) / 256;
    const long base = (long)B * Hkv * n_rt;
    const int tiles = (Lcap + TC_BN - 1) / TC_BN;
    long ns = sm_count() / base;
    if (ns > tiles) ns = tiles;
    if (ns > TC_MAX_SPLITS) ns = TC_MAX_SPLITS;
#ifdef TC_FORCE_NSPLIT
    ns = TC_FORCE_NSPLIT;
#endif
    if (ns < 1 || base > TC_MAX_GROUPS) ns = 1;
    if (n_rt_out) *n_rt_out = n_rt;
    return (int)ns;
}

int launch_tree_attn_tc(const mtv_tree *tree, int B, int Hq, int Hkv, const __nv_bfloat16 *q, const __nv_bfloat16 *k,
                        const __nv_bfloat16 *v, int64_t sb, int64_t sh, int64_t st, int Lcap, const int32_t *seq_lens,
                        float scale_log2, __nv_bfloat16 *out, int32_t *status, void *ws_o, float *ws_ml,
                        cudaStream_t stream) {
    const int G = Hq / Hkv, T = tree->T, D = 128;
    CUtensorMap q_map, k_map, v_map;
    {
        const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)Hq, (cuuint64_t)T, (cuuint64_t)B};
        const cuuint64_t str[3] = {(cuuint64_t)D * 2, (cuuint64_t)Hq * D * 2, (cuuint64_t)T * Hq * D * 2};
        const cuuint32_t box[4] = {64, (cuuint32_t)G, (cuuint32_t)(128 / G), 1};
        if (!encode_map(&q_map, q, dims, str, box)) return MTV_ERR_CUDA;
    }
    {
        const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)Lcap, (cuuint64_t)Hkv, (cuuint64_t)B};
        const cuuint64_t str[3] = {(cuuint64_t)st * 2, (cuuint64_t)sh * 2, (cuuint64_t)sb * 2};
        const cuuint32_t box[4] = {64, 128, 1, 1};
        if (!encode_map(&k_map, k, dims, str, box) || !encode_map(&v_map, v, dims, str, box)) return MTV_ERR_CUDA;
    }
    if (tc_prepare() != MTV_OK) return MTV_ERR_CUDA;
    TcParams p;
    p.seq_lens = seq_lens; p.anc = tree->d_anc; p.out = out; p.status = status; p.dev_error = tree->d_error;
    p.ws_o = reinterpret_cast<__nv_bfloat16 *>(ws_o); p.ws_ml = reinterpret_cast<float2 *>(ws_ml);
    p.arrive = tree->d_counters; p.depart = tree->d_counters + TC_MAX_GROUPS;
    p.scale_log2 = scale_log2;
    p.T = T; p.G = G; p.Hq = Hq; p.Hkv = Hkv; p.Lcap = Lcap;
    p.nsplit = attn_tc_plan(T, G, B, Hkv, Lcap, &p.n_rt);
    p.M_rows = T * G;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.nsplit, Hkv * p.n_rt, B);
    cfg.blockDim = dim3(TC_THREADS, 1, 1);
    cfg.dynamicSmemBytes = TC_SMEM_BYTES;
    cfg.stream = stream;
    // Launched as a programmatic dependent of the previous kernel in the stream (the kernel itself
    // waits for that kernel before it reads anything), which hides most of the launch latency when
    // attention calls follow each other.  Not a cooperative launch: that costs about 2 us per
    // launch; the grid never exceeds one CTA per SM, so its CTAs are resident together whenever the
    // device is not shared with another long-running kernel, and the wait for the other splits is
    // bounded in any case.
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    MTV_CUDA_CHECK(cudaLaunchKernelEx(&cfg, tree_attn_tc_kernel, q_map, k_map, v_map, p));
    return MTV_OK;
}

}  // namespace mtv

#ifdef MTV_TRACE
extern "C" int mtv_trace_set(long long *buf) {
    return cudaMemcpyToSymbol(mtv::g_trace, &buf, sizeof buf) == cudaSuccess ? 0 : -1;
}
#endif
