// Tree attention on the 5th-generation tensor cores (Section 3.2 / Fig. 2(b)), head_dim 128.
//
// A pair of CTAs (a cluster of two) owns up to 256 query rows — the (node, head-in-group) rows that
// share one KV head: 128 / G whole tree nodes per CTA for a group of G <= 8 query heads (when G does not
// divide 128 the last rows of a CTA's tile stay unused) — and every nsplit-th 128-key group of the sequence.  The two CTAs form one
// tcgen05 CTA pair: each keeps 128 of the query rows, its own S / P / O in tensor memory and its own
// softmax warps, and each loads HALF of every K and V group from global memory (K: 64 of the 128 keys;
// V: 64 of the 128 columns), so a K/V byte crosses from L2 to the SMs once per 256 query rows.  The
// MMAs (M = 256 over the pair, N = 128) are issued by two threads of the even-ranked CTA and read both halves.
//
// The two 64-key halves of a group belong to two STREAMS, each with its own accumulator O and its own
// running (max, sum) per row; the streams are merged in registers at the end.  One softmax thread owns one
// query row of one stream: it reads the 64 scores of its half from tensor memory, needs nobody else for the
// row maximum, and writes P (bf16) back over them.  Every scheduler therefore runs two independent softmax
// warps (one per stream): while one uses the special-function unit for its exponentials, the other waits
// for tensor memory, barriers or the tensor core — the latencies that dominate a tile when all warps of a
// scheduler move in lockstep.
// Warp roles in each CTA:
//   warps 0-3 / 4-7  softmax warps of stream 0 / 1 (warp w: tensor-memory lanes 32 (w % 4) ..);
//   warp 8           (even CTA only) issues S = Q K^T of a whole group (operands in shared memory);
//   warp 9           TMA producer of this CTA's halves: Q once, K and V through rings of 16 KB slots;
//   warp 10          relay: tells the issuing CTA when this CTA's half of a group has landed (after clearing
//                    V rows past the last key);
//   warp 11          (even CTA only) issues O += P V per stream (P from tensor memory, V N-major from
//                    shared memory).
// Tensor memory per CTA: two S buffers of 128 columns (64 per stream; P overlays the first 32 columns of a
// stream's 64), then O of stream 0 and O of stream 1 (128 columns each).  S of group i + 2 is issued as soon as
// both O += P V of group i have completed, two groups ahead of the softmax.  Ring slots are handed back to the
// producer by the softmax warps, which see S of group i complete (its K slot is free) and with it O += P V
// of group i - 2 (its V slot is free): no tensor-core commit is spent on it.
//
// The key splits of a query block are merged inside the launch.  After its last group a CTA writes its own
// normalised result O / l (bf16) and (m, l) to the workspace, one thread release-arrives on a counter of the
// (query block, CTA rank), and when all splits have arrived each CTA combines a slice of the rows:
// out = sum_s w_s (O_s / l_s) with w_s = exp2(m_s - m) l_s / sum.  This wait needs all CTAs of a query
// block resident together: splits are only planned when the whole grid fits the device in one wave (one CTA
// per SM); the wait is bounded all the same.  Without splits CTAs never wait for CTAs outside their pair
// and the grid may be of any size.
//
// The running max of a stream moves only when a tile's max exceeds it by more than 8 (log2 units), so O is
// rescaled rarely and P stays below 2^8.
//
// Build option -DMTV_TRACE: per-CTA cycle stamps of the phases through mtv_trace_set (development aid).
#include <cuda.h>

#include <cstring>
#include <mutex>
#include <type_traits>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace mtv {

constexpr int TC_BN = 128;        // keys per group of a CTA pair (one S MMA set); a stream takes 64 of them
constexpr int TC_HALF = TC_BN / 2;
constexpr int TC_STAGES = 5;      // K and V ring slots per CTA
constexpr int TC_THREADS = 384;
constexpr int TC_SOFTMAX_WARPS = 8;
constexpr int TC_MMA_WARP = 8, TC_TMA_WARP = 9, TC_RELAY_WARP = 10, TC_PV_WARP = 11;
constexpr uint32_t TC_Q_BYTES = 128 * 128 * 2;   // this CTA's 128 query rows: two 64-column halves
constexpr uint32_t TC_Q_HALF = TC_Q_BYTES / 2;
constexpr uint32_t TC_K_BYTES = 64 * 128 * 2;    // this CTA's 64 keys of a group: two 64-column halves
constexpr uint32_t TC_K_HALF = TC_K_BYTES / 2;
constexpr uint32_t TC_V_BYTES = 128 * 64 * 2;    // 128 keys x this CTA's 64 columns
constexpr uint32_t TC_BAR_BYTES = 1024;
constexpr uint32_t TC_ML_BYTES = 2 * 128 * 8;    // (m, l) per stream and row, for the merge of the two streams
constexpr uint32_t TC_OFF_K = TC_Q_BYTES;
constexpr uint32_t TC_OFF_V = TC_OFF_K + TC_STAGES * TC_K_BYTES;
constexpr uint32_t TC_OFF_BAR = TC_OFF_V + TC_STAGES * TC_V_BYTES;
constexpr uint32_t TC_OFF_ML = TC_OFF_BAR + TC_BAR_BYTES;
constexpr uint32_t TC_SMEM_BYTES = 1024 + TC_OFF_ML + TC_ML_BYTES;
static_assert(TC_SMEM_BYTES <= 227 * 1024, "shared memory budget");
constexpr float TC_RESCALE_THRESHOLD = 8.f;
constexpr int TC_MAX_SPLITS = 32;
constexpr int TC_MAX_COUNTERS = 256;   // merge counters in the tree object: one per (query block, CTA rank)

// tensor-memory columns: S buffer b of stream t at 128 b + 64 t (P over its first 32 columns), O of stream t at 256 + 128 t
constexpr uint32_t TM_S = 0, TM_O = 256;

// mbarrier slots (8 bytes each).  "ready", "sfree" and "pready" are only used in the issuing CTA.
enum {
    BAR_QFULL = 0,
    BAR_KFULL = 1,
    BAR_VFULL = BAR_KFULL + TC_STAGES,
    BAR_KFREE = BAR_VFULL + TC_STAGES,
    BAR_VFREE = BAR_KFREE + TC_STAGES,
    BAR_QREADY = BAR_VFREE + TC_STAGES,
    BAR_KREADY = BAR_QREADY + 1,
    BAR_VREADY = BAR_KREADY + TC_STAGES,
    BAR_SREADY = BAR_VREADY + TC_STAGES,   // [2 buffers] S of a group is complete (tensor core -> softmax warps of both CTAs)
    // Barriers whose phases follow the groups come in pairs (even and odd groups): a waiter may then lag at most one
    // phase behind, which is all a parity wait can tell apart.
    BAR_PREADY = BAR_SREADY + 2,           // [2] both streams' P are in tensor memory (softmax warps of both CTAs -> issuer)
    BAR_ODONE = BAR_PREADY + 2,            // [2] both streams' O += P V of a group are complete (tensor core -> both CTAs)
    BAR_FINAL = BAR_ODONE + 2,
    BAR_COUNT = BAR_FINAL + 1
};
static_assert(BAR_COUNT * 8 + 16 <= TC_BAR_BYTES, "barrier region too small");

// instruction descriptors: bf16 x bf16 -> fp32, M = 256 over the CTA pair
constexpr uint32_t IDESC_BASE = (1u << 4) | (1u << 7) | (1u << 10) | ((256u >> 4) << 24);
constexpr uint32_t IDESC_QK = IDESC_BASE | ((128u >> 3) << 17);                // N = 128 keys; A, B both K-major
constexpr uint32_t IDESC_PV = IDESC_BASE | ((128u >> 3) << 17) | (1u << 16);   // N = 128 columns; B (= V) N-major

struct TcParams {
    const int32_t *seq_lens;
    const uint64_t *anc;   // [T][2]
    __nv_bfloat16 *out;    // [B][T][Hq][128]
    __nv_bfloat16 *ws_o;   // [query blocks][nsplit][256 rows][128] partial O / l (only when nsplit > 1)
    float2 *ws_ml;         // [query blocks][nsplit][256] partial (m, l)
    int32_t *arrive, *depart;   // [query blocks][2] merge counters, zero between calls
    int32_t *status;       // [B] or null
    const int32_t *order;  // [B] sequences by descending length, or null: grid index z -> sequence
    int32_t *dev_error;
    float scale_log2;
    int T, G, Hq, Hkv, Lcap, nsplit, n_blk;
    int npc, R;   // tree nodes per CTA (128 / G) and the query rows they fill (npc * G <= 128: the other rows of the tile idle)
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
// N-major operand one 64-column swizzle atom wide: 8-key groups 1024 bytes apart
__device__ __forceinline__ uint64_t desc_nmajor(uint32_t saddr) { return smem_desc(saddr, TC_V_BYTES, 1024); }

__device__ __forceinline__ void cta_sync() { asm volatile("bar.sync 1, %0;" ::"n"(TC_THREADS) : "memory"); }
__device__ __forceinline__ void softmax_sync() { asm volatile("bar.sync 6, %0;" ::"n"(TC_SOFTMAX_WARPS * 32) : "memory"); }

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// 2^x for two values on the FMA pipes: x = j + f with j the nearest integer (read off the low mantissa bits of
// x + 1.5 * 2^23) and f in [-0.5, 0.5]; 2^f by a cubic (relative error 7.5e-5, far below the bf16 rounding of P);
// 2^j by an add to the exponent field.  x is clamped at -126 (the result then underflows towards zero like ex2's).
__device__ __forceinline__ float2 exp2_poly2(float2 x) {
    const float magic = 12582912.f;
    x.x = fmaxf(x.x, -126.f);
    x.y = fmaxf(x.y, -126.f);
    const float2 t = __fadd2_rn(x, make_float2(magic, magic));
    const float2 jf = __fadd2_rn(t, make_float2(-magic, -magic));
    const float2 f = __fadd2_rn(x, make_float2(-jf.x, -jf.y));
    float2 q = __ffma2_rn(make_float2(0.055171650f, 0.055171650f), f, make_float2(0.24261113f, 0.24261113f));
    q = __ffma2_rn(q, f, make_float2(0.69326097f, 0.69326097f));
    q = __ffma2_rn(q, f, make_float2(0.99992806f, 0.99992806f));
    return make_float2(__int_as_float(__float_as_int(q.x) + (__float_as_int(t.x) << 23)),
                       __int_as_float(__float_as_int(q.y) + (__float_as_int(t.y) << 23)));
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

#ifdef MTV_TRACE
__device__ long long *g_trace = nullptr;   // [ctas][64]
// the buffer's address is read once per thread (TRACE_INIT); a stamp is then one clock read and one store
#define TRACE_INIT                                                                                                  \
    long long *trace_row = g_trace;                                                                                 \
    if (trace_row) trace_row += ((size_t)(blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x) * 64
#define TRACE(id)                                                            \
    do {                                                                     \
        if (trace_row && (threadIdx.x % 32) == 0) trace_row[(id)] = clock64(); \
    } while (0)
#else
#define TRACE_INIT
#define TRACE(id)
#endif

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(TC_THREADS, 1)
tree_attn_tc_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                    const __grid_constant__ CUtensorMap v_map, const TcParams p) {
    extern __shared__ unsigned char smem_raw[];
    // Programmatic dependent launch: let the next kernel of the stream be set up while this one runs.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const uint32_t rank = ptx::cluster_ctarank();     // 0: issues the MMAs, rows 0-127 of the block; 1: rows 128-255
    const int split = blockIdx.x >> 1;
    const int g = blockIdx.y / p.n_blk, blk = blockIdx.y % p.n_blk;
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    TRACE_INIT;
    if (warp == 0) TRACE(0);

    // carve shared memory (tiles need 1024-byte alignment for the 128-byte swizzle); both CTAs of the pair
    // get the same offsets, which the pair MMAs and the remote barrier addresses rely on
    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
    const uint32_t sbase = raw + pad;
    unsigned char *gbase = smem_raw + pad;
    const uint32_t q_smem = sbase, k_ring = sbase + TC_OFF_K, v_ring = sbase + TC_OFF_V, bars = sbase + TC_OFF_BAR;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(gbase + TC_OFF_BAR + BAR_COUNT * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(gbase + TC_OFF_BAR + BAR_COUNT * 8 + 4);
    float2 *ml_x = reinterpret_cast<float2 *>(gbase + TC_OFF_ML);
    auto bar = [&](int i) { return bars + (uint32_t)i * 8u; };
    auto lead = [&](int i) { return ptx::mapa(bar(i), 0); };        // the same barrier in the issuing CTA
    auto peer = [&](int i) { return ptx::mapa(bar(i), rank ^ 1); }; // the same barrier in the other CTA

    if (warp == TC_TMA_WARP && lane == 0) {
        ptx::prefetch_tensormap(&k_map);
        ptx::prefetch_tensormap(&q_map);
        ptx::prefetch_tensormap(&v_map);
        ptx::mbar_init(bar(BAR_QFULL), 1);
        ptx::mbar_init(bar(BAR_QREADY), 2);
        for (int s = 0; s < TC_STAGES; ++s) {
            ptx::mbar_init(bar(BAR_KFULL + s), 1);
            ptx::mbar_init(bar(BAR_VFULL + s), 1);
            ptx::mbar_init(bar(BAR_KFREE + s), TC_SOFTMAX_WARPS);   // the softmax warps of this CTA
            ptx::mbar_init(bar(BAR_VFREE + s), TC_SOFTMAX_WARPS);
            ptx::mbar_init(bar(BAR_KREADY + s), 2);    // the relay warp of each CTA
            ptx::mbar_init(bar(BAR_VREADY + s), 2);
        }
        for (int t = 0; t < 2; ++t) {
            ptx::mbar_init(bar(BAR_SREADY + t), 1);
            ptx::mbar_init(bar(BAR_PREADY + t), 2 * TC_SOFTMAX_WARPS);    // the softmax warps of both CTAs
            ptx::mbar_init(bar(BAR_ODONE + t), 1);
        }
        ptx::mbar_init(bar(BAR_FINAL), 1);
        ptx::fence_mbar_init();
        *abort_flag = 0;
    }
    if (warp == TC_MMA_WARP) {
        ptx::tmem_alloc_pair(ptx::smem_u32(const_cast<uint32_t *>(tmem_slot)), 512);
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before();
    __syncthreads();
    // The peer's barriers and tensor memory must exist before anything is sent its way: a cluster barrier,
    // whose wait comes after the sequence length has been read (both latencies overlap).
    ptx::cluster_arrive();
    ptx::tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    if (warp == 0) TRACE(1);

    // Nothing above touched global memory.  From here on the previous kernel of the stream must be
    // complete (its outputs may be this kernel's inputs, and it may share the workspace and counters).
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // With more query blocks than CTA pairs fit the device, blocks start in grid order as pairs retire: the longest
    // sequences go first (the order comes from a small kernel in front of this one), so that the last pairs to start
    // are the shortest.
    int b = p.order ? p.order[blockIdx.z] : blockIdx.z;
    if (!MTV_INDEX_OK(b, gridDim.z, p.dev_error)) b = blockIdx.z;   // (both CTAs of a pair read the same entry)
    const int L = p.seq_lens[b];
    // This CTA's query rows: row = (node - node0) * G + head-in-group for its npc nodes; with a group size that does not
    // divide 128 the last 128 - R rows of the tile belong to nobody (zeroed, computed, never written out).
    const int node0 = (blk * 2 + (int)rank) * p.npc;
    auto valid_row = [&](int lrow) { return lrow < p.R && node0 + lrow / p.G < p.T; };
    auto tile_of = [&](int j) { return split + j * p.nsplit; };
    auto issue_k = [&](int j) {
        const int s = j % TC_STAGES;
        ptx::mbar_arrive_expect_tx(bar(BAR_KFULL + s), TC_K_BYTES);
        for (int half = 0; half < 2; ++half)
            ptx::tma_load_4d(k_ring + s * TC_K_BYTES + half * TC_K_HALF, &k_map, bar(BAR_KFULL + s), half * 64,
                             tile_of(j) * TC_BN + (int)rank * TC_HALF, g, b);
    };
    auto issue_v = [&](int j) {
        const int s = j % TC_STAGES;
        ptx::mbar_arrive_expect_tx(bar(BAR_VFULL + s), TC_V_BYTES);
        ptx::tma_load_4d(v_ring + s * TC_V_BYTES, &v_map, bar(BAR_VFULL + s), (int)rank * 64, tile_of(j) * TC_BN, g, b);
    };
    constexpr int TC_EARLY = 2;   // tiles requested before the length is known
    if (warp == TC_TMA_WARP && lane == 0) {
        // The first tiles of this split and the query tile do not depend on the sequence length (the tiles of a split
        // are split, split + nsplit, ...; past the end of the cache a copy delivers zeros), so they are requested while
        // the length is still on its way; they only touch this CTA's own shared memory and barriers.
        issue_k(0);
        ptx::mbar_arrive_expect_tx(bar(BAR_QFULL), (uint32_t)p.R * 256u);
        for (int half = 0; half < 2; ++half)
            ptx::tma_load_4d(q_smem + half * TC_Q_HALF, &q_map, bar(BAR_QFULL), half * 64, g * p.G, node0, b);
        issue_k(1);
        issue_v(0);
        issue_v(1);
    }
    const bool reporter = blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0;
    const bool over = L + p.T > p.Lcap;   // the same for every CTA of the sequence: nobody waits for anybody
    if (reporter && p.status) p.status[b] = over ? MTV_ERR_CAPACITY : MTV_OK;
    const int n_keys = L + p.T;
    const int tiles = (n_keys + TC_BN - 1) / TC_BN;
    // key tiles split, split + nsplit, ... : the splits of a query block read neighbouring tiles at the same time
    const int cnt = over || split >= tiles ? 0 : (tiles - split + p.nsplit - 1) / p.nsplit;
    const bool have_rows = node0 < p.T;
    if (warp != TC_TMA_WARP) ptx::cluster_wait();   // the producer first requests this CTA's own tiles

    // A wait that ran out: flag both CTAs of the pair and raise the sticky error.
    auto give_up = [&]() {
        *abort_flag = 1;
        ptx::st_cluster_u32(ptx::mapa(ptx::smem_u32(const_cast<int *>(abort_flag)), rank ^ 1), 1u);
        atomicExch(p.dev_error, MTV_ERR_TIMEOUT);
    };

    if (warp == TC_TMA_WARP) {
        // ------------------------------------------------------------ TMA producer: this CTA's halves
        __syncwarp();
        ptx::cluster_wait();
        if (lane == 0) {
            // tiles requested before the length was known and not needed after all: let them land before the CTA can exit
            for (int j = cnt; j < TC_EARLY; ++j) {
                ptx::mbar_wait(bar(BAR_KFULL + j), 0);
                ptx::mbar_wait(bar(BAR_VFULL + j), 0);
            }
            if (cnt == 0) ptx::mbar_wait(bar(BAR_QFULL), 0);
        }
        if (lane == 0 && cnt > TC_EARLY) {
            // the other tiles are requested once the query tile has landed, so that what the first MMAs need is
            // not queued behind tiles that are needed later
            if (!ptx::mbar_wait(bar(BAR_QFULL), 0)) give_up();
            int issued = TC_EARLY;
            for (int j = TC_EARLY; j < cnt && !*abort_flag; ++j) {
                if (j >= TC_STAGES) {   // the slot's previous tile has been consumed by the tensor core
                    const uint32_t par = ((j / TC_STAGES) - 1) & 1;
                    if (!ptx::mbar_wait(bar(BAR_KFREE + j % TC_STAGES), par)) { give_up(); break; }
                    issue_k(j);
                    if (!ptx::mbar_wait(bar(BAR_VFREE + j % TC_STAGES), par)) { give_up(); break; }
                    issue_v(j);
                } else {
                    issue_k(j);
                    issue_v(j);
                }
                issued = j + 1;
            }
            if (*abort_flag) {
                // give every copy still in flight a bounded chance to land before the CTA can exit
                ptx::mbar_wait(bar(BAR_QFULL), 0);
                for (int j = max(0, issued - TC_STAGES); j < issued; ++j) {
                    ptx::mbar_wait(bar(BAR_KFULL + j % TC_STAGES), (j / TC_STAGES) & 1);
                    ptx::mbar_wait(bar(BAR_VFULL + j % TC_STAGES), (j / TC_STAGES) & 1);
                }
            }
        }
        __syncwarp();
        ptx::cluster_arrive();
    } else if (warp == TC_RELAY_WARP) {
        // ------------------------------------------------------------ relay: this CTA's half has landed
        bool ok = true;
        for (int j = 0; j < cnt && ok && !*abort_flag; ++j) {
            const int s = j % TC_STAGES;
            const uint32_t par = (j / TC_STAGES) & 1;
            ok = ptx::mbar_wait(bar(BAR_KFULL + s), par);
            if (!ok) break;
            if (j >= 2 && j < 7) TRACE(1 + j);   // K(j) landed
            if (lane == 0) ptx::mbar_arrive_remote(lead(BAR_KREADY + s));
            if (j == 0) {
                ok = ptx::mbar_wait(bar(BAR_QFULL), 0);
                if (!ok) break;
                if (p.R < 128) {
                    // the tile's unused rows hold whatever shared memory held: clear them (a row stays in its own 128
                    // bytes of each half under the swizzle), so that the scores of those rows are plain zeros
                    for (int e = p.R * 8 + lane; e < 128 * 8; e += 32) {
                        reinterpret_cast<uint4 *>(gbase)[e] = make_uint4(0u, 0u, 0u, 0u);
                        reinterpret_cast<uint4 *>(gbase + TC_Q_HALF)[e] = make_uint4(0u, 0u, 0u, 0u);
                    }
                    ptx::fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive_remote_release(lead(BAR_QREADY));
                } else if (lane == 0) {
                    ptx::mbar_arrive_remote(lead(BAR_QREADY));
                }
            }
            ok = ptx::mbar_wait(bar(BAR_VFULL + s), par);
            if (!ok) break;
            // Rows of the V tile past the last valid key hold whatever the cache holds there; their P is
            // zero, but 0 * NaN would still poison O: clear them before the tensor core reads.
            const int valid = n_keys - tile_of(j) * TC_BN;
            if (valid < TC_BN) {
                unsigned char *vt = gbase + TC_OFF_V + s * TC_V_BYTES;   // [128 keys][128 bytes]
                for (int e = valid * 8 + lane; e < TC_BN * 8; e += 32)
                    reinterpret_cast<uint4 *>(vt)[e] = make_uint4(0u, 0u, 0u, 0u);
                ptx::fence_proxy_async();
            }
            __syncwarp();
            if (lane == 0) {
                if (valid < TC_BN) ptx::mbar_arrive_remote_release(lead(BAR_VREADY + s));   // hands over the cleared rows
                else ptx::mbar_arrive_remote(lead(BAR_VREADY + s));
            }
        }
        if (!ok && lane == 0) give_up();
        __syncwarp();
        ptx::cluster_arrive();
    } else if (warp == TC_MMA_WARP) {
        // ------------------------------------------------------------ issuer of S = Q K^T (even CTA, one thread)
        // Two threads issue the MMAs, one per kind, so that the scores of the next groups never wait behind a P that
        // is still being written: this one follows the K groups and the completed O += P V, the other one (below)
        // the V groups and the finished P tiles.
        if (rank == 0 && lane == 0 && cnt > 0) {
            // Operand descriptors are built once; an instruction then costs its issuing thread one 64-bit add
            // per operand (the start-address field counts 16-byte units and never carries: shared-memory
            // addresses stay below 256 KB).
            const uint64_t dq0 = desc_kmajor(q_smem), dk0 = desc_kmajor(k_ring);
            bool ok = ptx::mbar_wait(bar(BAR_QREADY), 0);
            for (int j = 0; ok && j < cnt && !*abort_flag; ++j) {
                // the K group of both CTAs has landed; the S buffer (with P over it) has been consumed by both
                // streams' O += P V of group j - 2
                ok = ptx::mbar_wait(bar(BAR_KREADY + j % TC_STAGES), (j / TC_STAGES) & 1) &&
                     (j < 2 || ptx::mbar_wait(bar(BAR_ODONE + (j & 1)), ((j >> 1) - 1) & 1));
                if (!ok) break;
                if (j == 0) TRACE(2);   // Q and K_0 of both CTAs landed
                if (j >= 1 && j < 9) TRACE(55 + j);   // S(j) issued
                ptx::tc_fence_after();
                const uint64_t dk = dk0 + (uint64_t)(((j % TC_STAGES) * TC_K_BYTES) >> 4);
                const uint32_t d = tmem + TM_S + (uint32_t)(j & 1) * 128;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint64_t offq = (uint64_t)(((kk / 4) * TC_Q_HALF + (kk % 4) * 32) >> 4);
                    const uint64_t offk = (uint64_t)(((kk / 4) * TC_K_HALF + (kk % 4) * 32) >> 4);
                    ptx::mma_pair_ss(d, dq0 + offq, dk + offk, IDESC_QK, kk > 0);
                }
                ptx::tc_commit_pair(bar(BAR_SREADY + (j & 1)));
                ptx::tc_commit_pair(peer(BAR_SREADY + (j & 1)));
            }
            if (!ok) give_up();
        }
        __syncwarp();
        ptx::cluster_arrive();
    } else if (warp == TC_PV_WARP) {
        // ------------------------------------------------------------ issuer of O += P V (even CTA, one thread)
        if (rank == 0 && lane == 0 && cnt > 0) {
            const uint64_t dv0 = desc_nmajor(v_ring);
            bool ok = true;
            for (int j = 0; ok && j < cnt && !*abort_flag; ++j) {
                // the V group of both CTAs has landed and both streams' P are in tensor memory (the two streams finish
                // a group at about the same time: their scores arrive together)
                ok = ptx::mbar_wait(bar(BAR_VREADY + j % TC_STAGES), (j / TC_STAGES) & 1) &&
                     ptx::mbar_wait(bar(BAR_PREADY + (j & 1)), (j >> 1) & 1);
                if (!ok) break;
                ptx::tc_fence_after();
                if (j < 8) TRACE(48 + j);   // O += P V of group j issued
#pragma unroll
                for (int t = 0; t < 2; ++t) {   // stream t: keys [64 t, 64 t + 64) of the group
                    const uint64_t dv = dv0 + (uint64_t)(((j % TC_STAGES) * TC_V_BYTES + t * TC_HALF * 128) >> 4);
                    const uint32_t a = tmem + TM_S + (uint32_t)(j & 1) * 128 + (uint32_t)t * 64;
                    const uint32_t d = tmem + TM_O + (uint32_t)t * 128;
#pragma unroll
                    for (int kk = 0; kk < TC_HALF / 16; ++kk)
                        ptx::mma_pair_ts(d, a + kk * 8, dv + (uint64_t)((kk * 2048) >> 4), IDESC_PV, j > 0 || kk > 0);
                }
                ptx::tc_commit_pair(bar(BAR_ODONE + (j & 1)));
                ptx::tc_commit_pair(peer(BAR_ODONE + (j & 1)));
            }
            if (!ok || *abort_flag) give_up();
            // Every S group is read before its P is written and every P is consumed by one of the MMAs above, so when
            // these have completed all tensor-core work of the pair has (on the error path the other issuer's MMAs may
            // still run: the final cluster barrier is only passed by threads that have stopped signalling).
            ptx::tc_commit_pair(bar(BAR_FINAL));
            ptx::tc_commit_pair(peer(BAR_FINAL));
            if (!ok || *abort_flag) ptx::mbar_wait(bar(BAR_FINAL), 0);   // let what was issued finish
        }
        __syncwarp();
        ptx::cluster_arrive();
    } else {
        // ------------------------------------------------------------ softmax warps
        // Thread (row, st) owns query row `row` in stream st: keys [64 st, 64 st + 64) of every group.
        const int qd = warp & 3, st = warp >> 2;
        const int row = qd * 32 + lane;
        uint64_t alo = 0, ahi = 0;
        if (valid_row(row)) { alo = p.anc[(node0 + row / p.G) * 2]; ahi = p.anc[(node0 + row / p.G) * 2 + 1]; }
        const uint32_t lane_base = (uint32_t)(qd * 32) << 16;
        const uint32_t t_s = tmem + lane_base + TM_S + st * 64;   // + 128 for the odd groups; P goes over its first 32 columns
        const uint32_t t_o = tmem + lane_base + TM_O + st * 128;
        auto pair_sync = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(2 + qd) : "memory"); };   // the two warps that share these rows
        float m_used = -INFINITY, l = 0.f;
        bool ok = true;
        // visibility of the tree rows as 32-bit words: word w covers tree rows 32 w .. 32 w + 31
        auto anc_word = [&](int w) -> uint32_t {
            if (w < 0) return 0xffffffffu;     // prefix rows are visible to every node
            if (w == 0) return (uint32_t)alo;
            if (w == 1) return (uint32_t)(alo >> 32);
            if (w == 2) return (uint32_t)ahi;
            if (w == 3) return (uint32_t)(ahi >> 32);
            return 0u;                         // past the tree rows: nothing
        };
        const float2 sc2 = make_float2(p.scale_log2, p.scale_log2);
        for (int j = 0; j < cnt; ++j) {
            if (!ok || !ptx::mbar_wait(bar(BAR_SREADY + (j & 1)), (j >> 1) & 1)) { if (ok && lane == 0) give_up(); ok = false; }
            if (qd == 0 && j < 8) TRACE(8 + j * 4 + st * 2);       // S(j) ready
            ptx::tc_fence_after();
            uint32_t sr[64];
            ptx::tmem_ld32(t_s + (j & 1) * 128, *reinterpret_cast<uint32_t(*)[32]>(&sr[0]));
            ptx::tmem_ld32(t_s + (j & 1) * 128 + 32, *reinterpret_cast<uint32_t(*)[32]>(&sr[32]));
            // S of group j is complete: its K slot is free; so are (the S buffer was only refilled after them) both
            // streams' O += P V of group j - 2: that group's V slot is free
            if (lane == 0) {
                ptx::mbar_arrive(bar(BAR_KFREE + j % TC_STAGES));
                if (j >= 2) ptx::mbar_arrive(bar(BAR_VFREE + (j - 2) % TC_STAGES));
            }
            ptx::tmem_ld_wait_for(*reinterpret_cast<uint32_t(*)[32]>(&sr[0]));
            ptx::tmem_ld_wait_for(*reinterpret_cast<uint32_t(*)[32]>(&sr[32]));
            const int key0 = tile_of(j) * TC_BN + st * TC_HALF;
            if (key0 + TC_HALF > L) {
                // the tile overlaps the tree rows or the end of the cache: bit e of vis[h] is column 32 h + e
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int a0 = key0 + h * 32 - L;        // tree row of the half's first column
                    const int w = a0 >> 5, sh = a0 & 31;     // floor division
                    const uint32_t vis = __funnelshift_r(anc_word(w), anc_word(w + 1), sh);
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        if (!((vis >> e) & 1u)) sr[h * 32 + e] = 0xff800000u;   // -inf
                }
            }
            float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int e = 0; e < 64; e += 8)
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    mx[k] = ptx::fmax3(mx[k], __uint_as_float(sr[e + 2 * k]), __uint_as_float(sr[e + 2 * k + 1]));
            const float mxs = fmaxf(ptx::fmax3(mx[0], mx[1], mx[2]), mx[3]) * p.scale_log2;   // the scale is positive
            const float m_new = (j == 0 || mxs > m_used + TC_RESCALE_THRESHOLD) ? mxs : m_used;
            // O of this stream holds sums relative to m_used: rescale it when the reference moves (rare), once the
            // stream's O += P V of group j - 1 has completed
            const bool need = j > 0 && m_new != m_used && m_used != -INFINITY;
            if (__any_sync(0xffffffffu, need)) {
                if (ok && !ptx::mbar_wait(bar(BAR_ODONE + ((j - 1) & 1)), ((j - 1) >> 1) & 1)) { ok = false; if (lane == 0) give_up(); }
                ptx::tc_fence_after();
                const float alpha = need ? ex2(m_used - m_new) : 1.f;
#pragma unroll 1
                for (int h = 0; h < 4; ++h) {
                    uint32_t o[32];
                    ptx::tmem_ld32(t_o + h * 32, o);
                    ptx::tmem_ld_wait_for(o);
#pragma unroll
                    for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                    ptx::tmem_st32(t_o + h * 32, o);
                }
                ptx::tmem_st_wait();
                l *= alpha;
            }
            m_used = m_new;
            const float m_eff = m_used == -INFINITY ? 0.f : m_used;
            // ---- P = exp2(scale * S - m) with its row sum (two values per instruction where the instruction set
            //      has packed forms), bf16 P into tensor memory over this thread's own scores
            const float2 nm2 = make_float2(-m_eff, -m_eff);
            float2 la = make_float2(0.f, 0.f), lb = make_float2(0.f, 0.f);
            uint32_t pk[32];
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
                const float2 x01 = __ffma2_rn(make_float2(__uint_as_float(sr[2 * e]), __uint_as_float(sr[2 * e + 1])), sc2, nm2);
                const float2 x23 = __ffma2_rn(make_float2(__uint_as_float(sr[2 * e + 2]), __uint_as_float(sr[2 * e + 3])), sc2, nm2);
                float2 p01, p23;
                if (e % 8 == 6) {   // every fourth quadruple on the FMA pipes: the special-function unit is the bottleneck of a tile
                    p01 = exp2_poly2(x01);
                    p23 = exp2_poly2(x23);
                } else {
                    p01 = make_float2(ex2(x01.x), ex2(x01.y));
                    p23 = make_float2(ex2(x23.x), ex2(x23.y));
                }
                la = __fadd2_rn(la, p01);
                lb = __fadd2_rn(lb, p23);
                pk[e] = pack2_bf16(p01.x, p01.y);
                pk[e + 1] = pack2_bf16(p23.x, p23.y);
            }
            l += (la.x + la.y) + (lb.x + lb.y);
            ptx::tmem_st32(t_s + (j & 1) * 128, pk);
            ptx::tmem_st_wait();
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_remote(lead(BAR_PREADY + (j & 1)));
            if (qd == 0 && j < 8) TRACE(9 + j * 4 + st * 2);       // P(j) written by this warp
        }
        // ---- all tensor-core work of the pair is done
        if (cnt > 0) {
            if (*abort_flag) ok = false;
            if (ok && !ptx::mbar_wait(bar(BAR_FINAL), 0)) { ok = false; if (lane == 0) give_up(); }
            if (warp == 0) TRACE(40);
            ptx::tc_fence_after();
        }
        __syncwarp();
        ptx::cluster_arrive_relaxed();   // nothing more goes to the peer from this thread
        if (warp == 0) TRACE(3);
        // ---- the two streams of a row are merged: O = (w0 O0 + w1 O1) / (w0 l0 + w1 l1) with w_t = exp2(m_t - m);
        //      a stream that had no tile has (m, l) = (-inf, 0) and its accumulator is not read
        ml_x[st * 128 + row] = make_float2(m_used, l);
        pair_sync();
        if (warp == 0) TRACE(4);
        const float2 other = ml_x[(st ^ 1) * 128 + row];
        const float m_all = fmaxf(m_used, other.x);
        const float w_own = m_used == -INFINITY ? 0.f : ex2(m_used - m_all);
        const float w_oth = other.x == -INFINITY ? 0.f : ex2(other.x - m_all);
        const float l_all = w_own * l + w_oth * other.y;
        const float inv_l = ok && l_all > 0.f ? 1.f / l_all : 0.f;
        const float w0 = (st == 0 ? w_own : w_oth) * inv_l, w1 = (st == 0 ? w_oth : w_own) * inv_l;
        const bool have0 = ok && cnt > 0;   // both streams had a tile in every group
        // ---- this thread's 64 columns ([64 st, 64 st + 64)) as bf16 into the staging area (the Q tile is no longer
        //      needed): 16-byte chunk j of row r sits at chunk position j ^ (r & 15), so that both the one-row-per-lane
        //      stores here and the one-row-per-half-warp loads below are free of bank conflicts
        unsigned char *stage = gbase;
        {
            uint32_t o0[2][32], o1[2][32];   // this thread's 64 columns of O of stream 0 and of stream 1
            if (have0) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    ptx::tmem_ld32(tmem + lane_base + TM_O + (uint32_t)(st * 64 + h * 32), o0[h]);
                    ptx::tmem_ld32(tmem + lane_base + TM_O + 128 + (uint32_t)(st * 64 + h * 32), o1[h]);
                }
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    ptx::tmem_ld_wait_for(o0[h]);
                    ptx::tmem_ld_wait_for(o1[h]);
                }
            }
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                float v[32];
#pragma unroll
                for (int e = 0; e < 32; ++e)
                    v[e] = have0 ? fmaf(__uint_as_float(o1[h][e]), w1, __uint_as_float(o0[h][e]) * w0) : 0.f;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    uint4 u;
                    u.x = pack2_bf16(v[8 * e], v[8 * e + 1]);
                    u.y = pack2_bf16(v[8 * e + 2], v[8 * e + 3]);
                    u.z = pack2_bf16(v[8 * e + 4], v[8 * e + 5]);
                    u.w = pack2_bf16(v[8 * e + 6], v[8 * e + 7]);
                    *reinterpret_cast<uint4 *>(stage + row * 256 + (((st * 8 + h * 4 + e) ^ (row & 15)) << 4)) = u;
                }
            }
        }
        auto out_ptr = [&](int lrow) {   // the 128 output values of this CTA's row lrow
            const int node = node0 + lrow / p.G, hq = g * p.G + lrow % p.G;
            return p.out + (((size_t)b * p.T + node) * p.Hq + hq) * 128;
        };
        const int grp = blockIdx.z * gridDim.y + blockIdx.y;
        const size_t slab0 = (size_t)grp * p.nsplit;     // first slab (256 rows) of this query block
        const int slab_row0 = (int)rank * 128;
        const int ch = lane & 15, hs = lane >> 4;
        if (warp == 0) TRACE(5);
        pair_sync();   // the rows of this quarter of the tile are staged
        if (warp == 0) TRACE(6);
        // what the merge below needs, computed while the stores are on their way
        const int rows_per = (128 + p.nsplit - 1) / p.nsplit;
        const int row_begin = split * rows_per;
        const int n_my = max(0, min(128, row_begin + rows_per) - row_begin);
        if (have_rows && !over) {
            // ---- rows leave as whole 256-byte rows, two per warp instruction: warp (qd, st) takes rows 32 qd + 16 st ..
            uint4 v[8];
#pragma unroll
            for (int it = 0; it < 8; ++it) {
                const int srow = qd * 32 + st * 16 + it * 2 + hs;
                v[it] = *reinterpret_cast<const uint4 *>(stage + srow * 256 + ((ch ^ (srow & 15)) << 4));
            }
            if (p.nsplit == 1) {
#pragma unroll
                for (int it = 0; it < 8; ++it) {
                    const int srow = qd * 32 + st * 16 + it * 2 + hs;
                    if (valid_row(srow)) *reinterpret_cast<uint4 *>(out_ptr(srow) + ch * 8) = v[it];
                }
            } else {
                uint4 *dst = reinterpret_cast<uint4 *>(p.ws_o + ((slab0 + split) * 256 + slab_row0 + qd * 32 + st * 16 + hs) * 128 + ch * 8);
#pragma unroll
                for (int it = 0; it < 8; ++it) __stcg(dst + it * 2 * 16, v[it]);   // two rows of 16 chunks further each time
            }
        }
        if (warp == 0) TRACE(7);
        if (p.nsplit > 1 && have_rows && !over) {
            // ---- publish this split's rows, then combine a slice of the rows of all splits
            if (st == 0) __stcg(p.ws_ml + (slab0 + split) * 256 + slab_row0 + row, make_float2(m_all, l_all));
            softmax_sync();   // every softmax thread's stores precede the release below
            int32_t *arrive = p.arrive + grp * 2 + rank, *depart = p.depart + grp * 2 + rank;
            if (threadIdx.x == 0) {
                TRACE(44);   // partial written
                __threadfence();
                TRACE(41);   // fence done
                asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(arrive) : "memory");
                // relaxed polls (a round trip to L2 each), one acquire when the counter is full
                const long long t0 = clock64();
                while (*reinterpret_cast<volatile int32_t *>(arrive) < p.nsplit)
                    if (clock64() - t0 > ptx::WAIT_CYCLE_LIMIT) { atomicExch(p.dev_error, MTV_ERR_TIMEOUT); break; }
                (void)ld_acquire(arrive);
                TRACE(45);   // everybody arrived
            }
            softmax_sync();
            // This CTA has seen the counter full.  The last one to say so puts both counters back to zero at the end
            // (nobody polls them any more; the next call cannot start before this kernel has ended); the atomic is
            // issued here so that its round trip overlaps the merge.
            int departed = 0;
            if (threadIdx.x == 0) departed = atomicAdd(depart, 1);
            // half a warp per row, lane = 16-byte chunk of the row; all loads of a row first, then the arithmetic: one
            // round trip to L2 per pass, and with up to 16 rows per pass one pass for up to 8 splits
            for (int rl0 = warp * 2; rl0 < n_my; rl0 += 2 * TC_SOFTMAX_WARPS) {   // warp-uniform trip count: shuffles inside
                const bool mine = rl0 + hs < n_my;
                const int rl = mine ? rl0 + hs : rl0;            // the odd half warp may have no row: it repeats its neighbour's loads
                const int lrow = row_begin + rl;                 // row of this CTA
                const int srow = slab_row0 + lrow;               // row inside a slab
                const __nv_bfloat16 *src = p.ws_o + (slab0 * 256 + srow) * 128 + ch * 8;
                float acc[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[e] = 0.f;
                float m = -INFINITY, wsum = 0.f;
                for (int sp0 = 0; sp0 < p.nsplit; sp0 += 16) {   // (m, l) of up to 16 splits: lane ch holds split sp0 + ch
                    float2 ml = make_float2(-INFINITY, 0.f);
                    if (sp0 + ch < p.nsplit) ml = __ldcg(p.ws_ml + (slab0 + sp0 + ch) * 256 + srow);
                    uint4 v[16];
#pragma unroll
                    for (int u = 0; u < 16; ++u)
                        v[u] = sp0 + u < p.nsplit ? __ldcg(reinterpret_cast<const uint4 *>(src + (size_t)(sp0 + u) * 256 * 128))
                                                  : make_uint4(0u, 0u, 0u, 0u);
                    if (warp == 0 && sp0 == 0) TRACE(42);   // loads issued
                    // running maximum over the chunks of 16 splits (a second chunk rescales what has been summed)
                    float mc = ml.x;
#pragma unroll
                    for (int o = 8; o > 0; o >>= 1) mc = fmaxf(mc, __shfl_xor_sync(0xffffffffu, mc, o));
                    const float m_new = fmaxf(m, mc);
                    const float resc = m == -INFINITY ? 0.f : ex2(m - m_new);
                    const float w = ml.x == -INFINITY ? 0.f : ex2(ml.x - m_new) * ml.y;   // unnormalised weight of split sp0 + ch
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[e] *= resc;
                    m = m_new;
#pragma unroll
                    for (int u = 0; u < 16; ++u) {
                        const float wu = __shfl_sync(0xffffffffu, w, (lane & 16) | u);
                        const uint32_t vw[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            acc[2 * e] = fmaf(wu, __uint_as_float(vw[e] << 16), acc[2 * e]);
                            acc[2 * e + 1] = fmaf(wu, __uint_as_float(vw[e] & 0xffff0000u), acc[2 * e + 1]);
                        }
                    }
                    // the weights' sum rides along in every lane: sum over the half warp, folded into the same recurrence
                    float ws = w;
#pragma unroll
                    for (int o = 8; o > 0; o >>= 1) ws += __shfl_xor_sync(0xffffffffu, ws, o);
                    wsum = wsum * resc + ws;
                }
                if (warp == 0) TRACE(43);   // rows of all splits arrived and combined
                const float inv = wsum > 0.f ? 1.f / wsum : 0.f;
                if (mine && valid_row(lrow))
                    *reinterpret_cast<uint4 *>(out_ptr(lrow) + ch * 8) =
                        make_uint4(pack2_bf16(acc[0] * inv, acc[1] * inv), pack2_bf16(acc[2] * inv, acc[3] * inv),
                                   pack2_bf16(acc[4] * inv, acc[5] * inv), pack2_bf16(acc[6] * inv, acc[7] * inv));
            }
            if (threadIdx.x == 0 && departed == p.nsplit - 1) {
                *arrive = 0;
                *depart = 0;
                __threadfence();
            }
            if (warp == 0) TRACE(46);   // merge done
        }
    }

    // ---- nobody leaves while the pair's tensor-core work may still read its shared memory, write its
    //      tensor memory or arrive on its barriers: every thread arrived on the cluster barrier a second
    //      time when it had sent the peer its last signal, and waits here for the peer's threads
    ptx::tc_fence_before();
    cta_sync();
    ptx::cluster_wait();
    ptx::tc_fence_after();
    if (warp == TC_MMA_WARP) ptx::tmem_dealloc_pair(tmem, 512);
    if (warp == 0) TRACE(47);
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

// 4-D bf16 tensor map with a 128-byte-swizzled box whose innermost extent is 64 elements.  Encoding a map costs the host
// a microsecond or two and an attention call needs three, so encoded maps are kept in a small direct-mapped table keyed by
// everything that goes into them (a decode loop passes the same caches and strides step after step).
namespace {
struct MapKey {
    const void *base;
    cuuint64_t dims[4], strides[3];
    cuuint32_t box[4];
    int device;
};
struct MapSlot {
    MapKey key;
    CUtensorMap map;
    bool valid = false;
};
constexpr int MAP_SLOTS = 512;
MapSlot g_map_slots[MAP_SLOTS];
std::mutex g_map_mutex;
}  // namespace

static bool encode_map(CUtensorMap *map, const void *base, const cuuint64_t dims[4], const cuuint64_t strides_bytes[3],
                       const cuuint32_t box[4]) {
    MapKey key;
    memset(&key, 0, sizeof key);
    key.base = base;
    for (int i = 0; i < 4; ++i) { key.dims[i] = dims[i]; key.box[i] = box[i]; }
    for (int i = 0; i < 3; ++i) key.strides[i] = strides_bytes[i];
    if (cudaGetDevice(&key.device) != cudaSuccess) key.device = -1;
    const uint64_t h = ((uint64_t)(uintptr_t)base >> 8) * 0x9E3779B97F4A7C15ull + dims[1] * 0xC2B2AE3D27D4EB4Full + box[1] * 0x165667B19E3779F9ull;
    MapSlot &slot = g_map_slots[(h >> 40) % MAP_SLOTS];
    {
        std::lock_guard<std::mutex> lock(g_map_mutex);
        if (slot.valid && memcmp(&slot.key, &key, sizeof key) == 0) {
            *map = slot.map;
            return true;
        }
    }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint32_t ones[4] = {1, 1, 1, 1};
    if (fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides_bytes, box, ones,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    std::lock_guard<std::mutex> lock(g_map_mutex);
    slot.key = key;
    slot.map = *map;
    slot.valid = true;
    return true;
}

// order[r] = the sequence with the r-th largest length (ties: lower index first).  B is small: every thread ranks one
// sequence against all others.
__global__ void attn_order_kernel(const int32_t *seq_lens, int B, int32_t *order) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const int len = seq_lens[b];
    int rank = 0;
    for (int o = 0; o < B; ++o) {
        const int lo = seq_lens[o];
        rank += (lo > len || (lo == len && o < b)) ? 1 : 0;
    }
    order[rank] = b;
}
constexpr int TC_ORDER_MAX_B = 2048;

bool attn_tc_eligible(int D, int G) { return D == 128 && G >= 1 && G <= 8; }

static int tc_prepare() {
    static PerDeviceOnce once;
    bool *done = once.flag();
    if (!done || !*done) {
        MTV_CUDA_CHECK(cudaFuncSetAttribute(tree_attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_BYTES));
        if (done) *done = true;
    }
    return MTV_OK;
}

// Number of key splits of a problem: as many as keep the whole grid within one wave of CTA pairs (one CTA
// per SM), at most one per key tile, at most TC_MAX_SPLITS.  More than one split needs two merge counters
// per query block.
int attn_tc_plan(int T, int G, int B, int Hkv, int Lcap, int *n_blk_out) {
    const int npc = 128 / G;                      // tree nodes per CTA; a pair takes 2 npc
    const int n_blk = (T + 2 * npc - 1) / (2 * npc);
    const long base = (long)B * Hkv * n_blk;
    const int tiles = (Lcap + TC_BN - 1) / TC_BN;
    long ns = (sm_count() / 2) / base;
    if (ns > tiles) ns = tiles;
    if (ns > TC_MAX_SPLITS) ns = TC_MAX_SPLITS;
    if (ns < 1 || base * 2 > TC_MAX_COUNTERS) ns = 1;
    if (n_blk_out) *n_blk_out = n_blk;
    return (int)ns;
}

int launch_tree_attn_tc(const mtv_tree *tree, int B, int Hq, int Hkv, const __nv_bfloat16 *q, const __nv_bfloat16 *k,
                        const __nv_bfloat16 *v, int64_t sb, int64_t sh, int64_t st, int Lcap, const int32_t *seq_lens,
                        float scale_log2, __nv_bfloat16 *out, int32_t *status, void *ws_o, float *ws_ml, int32_t *ws_order,
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
        const cuuint32_t kbox[4] = {64, TC_BN / 2, 1, 1}, vbox[4] = {64, TC_BN, 1, 1};
        if (!encode_map(&k_map, k, dims, str, kbox) || !encode_map(&v_map, v, dims, str, vbox)) return MTV_ERR_CUDA;
    }
    if (tc_prepare() != MTV_OK) return MTV_ERR_CUDA;
    TcParams p;
    p.seq_lens = seq_lens; p.anc = tree->d_anc; p.out = out; p.status = status; p.dev_error = tree->d_error;
    p.ws_o = reinterpret_cast<__nv_bfloat16 *>(ws_o); p.ws_ml = reinterpret_cast<float2 *>(ws_ml);
    p.arrive = tree->d_counters; p.depart = tree->d_counters + TC_MAX_COUNTERS;
    p.scale_log2 = scale_log2;
    p.T = T; p.G = G; p.Hq = Hq; p.Hkv = Hkv; p.Lcap = Lcap;
    p.nsplit = attn_tc_plan(T, G, B, Hkv, Lcap, &p.n_blk);
    p.npc = 128 / G;
    p.R = p.npc * G;
    p.order = nullptr;
    if (p.nsplit == 1 && B > 1 && B <= TC_ORDER_MAX_B && (long)B * Hkv * p.n_blk > sm_count() / 2 && ws_order) {
        attn_order_kernel<<<(B + 255) / 256, 256, 0, stream>>>(seq_lens, B, ws_order);
        p.order = ws_order;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * p.nsplit, Hkv * p.n_blk, B);   // the kernel's cluster is (2, 1, 1): a CTA pair
    cfg.blockDim = dim3(TC_THREADS, 1, 1);
    cfg.dynamicSmemBytes = TC_SMEM_BYTES;
    cfg.stream = stream;
    // Launched as a programmatic dependent of the previous kernel in the stream (the kernel itself
    // waits for that kernel before it reads anything), which hides most of the launch latency when
    // attention calls follow each other.
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
