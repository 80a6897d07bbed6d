// Tree attention on the 5th-generation tensor cores (Section 3.2 / Fig. 2(b)), head_dim 128.
//
// One CTA owns up to 256 query rows (two 128-row tiles of the (node, head-in-group) block
// that shares one KV head) and a contiguous range of 128-key tiles.  Warp roles:
//   warps 0-3 / 4-7  softmax warpgroup of row tile 0 / 1: one thread per query row reads its
//                    row of S from tensor memory, applies the ancestor bitmask on the tiles that
//                    overlap the tree rows, keeps a running (max, sum), writes P (bf16) back to
//                    tensor memory over S, and finally writes the unnormalised partial
//                    (m, l, O) of its row to the workspace;
//   warp 8           issues tcgen05.mma: S_t = Q_t K^T (operands in shared memory) and
//                    O_t += P_t V (P from tensor memory, V from shared memory, N-major);
//   warp 9           TMA producer: Q once, then K and V tiles through a ring of 32 KB slots.
// Tensor memory: S0 | S1 | O0 | O1, 128 fp32 columns each; P_t overlays the first 64 columns
// of S_t.  The second kernel of attention.cu merges the partials of the key splits.
//
// The running max is only raised when the new row max exceeds it by more than 8 (in log2
// units), so O in tensor memory is rescaled rarely; P stays below 2^8.
#include <cuda.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace mtv {

constexpr int TC_BN = 128;
constexpr int TC_SLOTS = 5;
constexpr int TC_THREADS = 320;
constexpr uint32_t TC_TILE_BYTES = 128 * 128 * 2;   // one 128 x 128 bf16 tile: two 64-column halves
constexpr uint32_t TC_HALF_BYTES = TC_TILE_BYTES / 2;
constexpr uint32_t TC_Q_BYTES = 2 * TC_TILE_BYTES;
constexpr uint32_t TC_RING_BYTES = TC_SLOTS * TC_TILE_BYTES;
constexpr uint32_t TC_BAR_BYTES = 256;
constexpr uint32_t TC_SMEM_BYTES = 1024 + TC_Q_BYTES + TC_RING_BYTES + TC_BAR_BYTES;
constexpr float TC_RESCALE_THRESHOLD = 8.f;

// barrier slots (8 bytes each) inside the barrier region
enum { BAR_Q = 0, BAR_KV_FULL = 1, BAR_KV_EMPTY = BAR_KV_FULL + TC_SLOTS, BAR_S = BAR_KV_EMPTY + TC_SLOTS,
       BAR_P = BAR_S + 2, BAR_O = BAR_P + 2, BAR_FINAL = BAR_O + 2, BAR_COUNT = BAR_FINAL + 1 };
static_assert(BAR_COUNT * 8 + 8 <= TC_BAR_BYTES, "barrier region too small");

// instruction descriptors: bf16 x bf16 -> fp32, M = 128, N = 128
constexpr uint32_t IDESC_BASE = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t IDESC_QK = IDESC_BASE;               // A, B both K-major
constexpr uint32_t IDESC_PV = IDESC_BASE | (1u << 16);  // B (= V) N-major

struct TcParams {
    const int32_t *seq_lens;
    const uint64_t *anc;   // [T][2]
    float *ws_o, *ws_ml;
    int32_t *dev_error;
    float scale_log2;
    int T, G, Hkv, Lcap, nsplit, m_rows, n_rt, M_rows;
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

__global__ void __launch_bounds__(TC_THREADS, 1)
tree_attn_tc_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                    const __grid_constant__ CUtensorMap v_map, const TcParams p) {
    extern __shared__ unsigned char smem_raw[];
    const int split = blockIdx.x;
    const int g = blockIdx.y / p.n_rt, rt = blockIdx.y % p.n_rt;
    const int b = blockIdx.z;
    const int L = p.seq_lens[b];
    if (L + p.T > p.Lcap) return;   // reported by the combine kernel
    const int n_keys = L + p.T;
    const int tiles = (n_keys + TC_BN - 1) / TC_BN;
    const int base_cnt = tiles / p.nsplit, rem = tiles % p.nsplit;
    const int t_begin = split * base_cnt + min(split, rem);
    const int cnt = base_cnt + (split < rem ? 1 : 0);
    const int rows0 = rt * 256;
    const int nt = p.M_rows - rows0 > 128 ? 2 : 1;
    const size_t slab = (((size_t)b * p.Hkv + g) * p.nsplit + split) * p.m_rows + rows0;
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;

    if (cnt == 0) {   // no keys for this split: an empty partial
        for (int r = threadIdx.x; r < nt * 128; r += TC_THREADS)
            *reinterpret_cast<float2 *>(p.ws_ml + (slab + r) * 2) = make_float2(-INFINITY, 0.f);
        return;
    }

    // carve shared memory (tiles need 1024-byte alignment for the 128-byte swizzle)
    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
    const uint32_t q_smem = raw + pad;
    const uint32_t ring = q_smem + TC_Q_BYTES;
    const uint32_t bars = ring + TC_RING_BYTES;
    unsigned char *bar_region = smem_raw + pad + TC_Q_BYTES + TC_RING_BYTES;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(bar_region + BAR_COUNT * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bar_region + BAR_COUNT * 8 + 4);
    auto bar = [&](int i) { return bars + (uint32_t)i * 8u; };

    if (threadIdx.x == 0) {
        ptx::mbar_init(bar(BAR_Q), 1);
        for (int s = 0; s < TC_SLOTS; ++s) { ptx::mbar_init(bar(BAR_KV_FULL + s), 1); ptx::mbar_init(bar(BAR_KV_EMPTY + s), 1); }
        for (int t = 0; t < 2; ++t) {
            ptx::mbar_init(bar(BAR_S + t), 1);
            ptx::mbar_init(bar(BAR_P + t), 128);
            ptx::mbar_init(bar(BAR_O + t), 1);
        }
        ptx::mbar_init(bar(BAR_FINAL), 1);
        ptx::fence_mbar_init();
        *abort_flag = 0;
    }
    if (warp == 8) {
        ptx::tmem_alloc(ptx::smem_u32(const_cast<uint32_t *>(tmem_slot)), 512);
        ptx::tmem_relinquish();
    }
    if (warp == 9 && lane == 0) {
        ptx::prefetch_tensormap(&q_map);
        ptx::prefetch_tensormap(&k_map);
        ptx::prefetch_tensormap(&v_map);
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 9) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            ptx::mbar_arrive_expect_tx(bar(BAR_Q), nt * TC_TILE_BYTES);
            for (int t = 0; t < nt; ++t)
                for (int half = 0; half < 2; ++half)
                    ptx::tma_load_4d(q_smem + t * TC_TILE_BYTES + half * TC_HALF_BYTES, &q_map, bar(BAR_Q), half * 64,
                                     g * p.G, (rows0 + t * 128) / p.G, b);
        }
        for (int i = 0; i < 2 * cnt && !*abort_flag; ++i) {
            const int slot = i % TC_SLOTS, use = i / TC_SLOTS, j = i / 2;
            if (use > 0 && !ptx::mbar_wait(bar(BAR_KV_EMPTY + slot), (use - 1) & 1)) { *abort_flag = 1; break; }
            if (lane == 0) {
                const CUtensorMap *map = (i & 1) ? &v_map : &k_map;
                ptx::mbar_arrive_expect_tx(bar(BAR_KV_FULL + slot), TC_TILE_BYTES);
                for (int half = 0; half < 2; ++half)
                    ptx::tma_load_4d(ring + slot * TC_TILE_BYTES + half * TC_HALF_BYTES, map, bar(BAR_KV_FULL + slot),
                                     half * 64, (t_begin + j) * TC_BN, g, b);
            }
            __syncwarp();
        }
    } else if (warp == 8) {
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
        bool ok = ptx::mbar_wait(bar(BAR_Q), 0) && wait_kv(0);
        if (ok) {
            ptx::tc_fence_after();
            if (lane == 0) {
                issue_S(0, 0);
                ptx::tc_commit(bar(BAR_S + 0));
                if (nt == 2) { issue_S(1, 0); ptx::tc_commit(bar(BAR_S + 1)); }
                ptx::tc_commit(bar(BAR_KV_EMPTY + 0));
            }
            __syncwarp();
        }
        for (int j = 0; ok && j < cnt && !*abort_flag; ++j) {
            const bool more = j + 1 < cnt;
            ok = wait_kv(2 * j + 1) && ptx::mbar_wait(bar(BAR_P + 0), j & 1);
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
        if (!ok) *abort_flag = 1;
    } else if (warp / 4 < nt) {
        // ------------------------------------------------------------ softmax warpgroup of row tile t
        const int t = warp / 4;
        const int row = (warp % 4) * 32 + lane;
        const int r = rows0 + t * 128 + row;
        uint64_t alo = 0, ahi = 0;
        if (r < p.M_rows) { alo = p.anc[(r / p.G) * 2]; ahi = p.anc[(r / p.G) * 2 + 1]; }
        const uint32_t t_s = tmem + ((uint32_t)((warp % 4) * 32) << 16) + t * 128;
        const uint32_t t_o = tmem + ((uint32_t)((warp % 4) * 32) << 16) + 256 + t * 128;
        float m_used = -INFINITY, l = 0.f;
        bool ok = true;
        for (int j = 0; j < cnt && !*abort_flag; ++j) {
            ok = ptx::mbar_wait(bar(BAR_S + t), j & 1);
            if (!ok) break;
            ptx::tc_fence_after();
            uint32_t s[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c) ptx::tmem_ld32(t_s + c * 32, s[c]);
            ptx::tmem_ld_wait();
            const int key0 = (t_begin + j) * TC_BN;
            if (key0 + TC_BN > L) {
                // tile overlaps the tree rows (or the end of the cache): column c is key key0 + c
                const int off = L - key0;   // first tree row's column (may be negative)
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        const int a = c * 32 + e - off;
                        bool vis;
                        if (a < 0) vis = true;
                        else if (a < 64) vis = (alo >> a) & 1ull;
                        else if (a < 128) vis = (ahi >> (a - 64)) & 1ull;
                        else vis = false;
                        if (!vis) s[c][e] = 0xff800000u;   // -inf
                    }
            }
            float mx = -INFINITY;
#pragma unroll
            for (int c = 0; c < 4; ++c)
#pragma unroll
                for (int e = 0; e < 32; ++e) mx = fmaxf(mx, __uint_as_float(s[c][e]));
            const float mxs = mx * p.scale_log2;
            const float m_new = (j == 0 || mxs > m_used + TC_RESCALE_THRESHOLD) ? mxs : m_used;
            // O holds sums relative to m_used: rescale it when the reference moves (rare)
            const bool need = j > 0 && m_new != m_used && m_used != -INFINITY;
            if (__any_sync(0xffffffffu, need)) {
                ok = ptx::mbar_wait(bar(BAR_O + t), (j - 1) & 1);
                if (!ok) break;
                ptx::tc_fence_after();
                const float alpha = need ? ex2(m_used - m_new) : 1.f;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t o[32];
                    ptx::tmem_ld32(t_o + c * 32, o);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                    ptx::tmem_st32(t_o + c * 32, o);
                }
                ptx::tmem_st_wait();
                l *= alpha;
            }
            m_used = m_new;
            const float m_eff = m_used == -INFINITY ? 0.f : m_used;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t pk[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    const float p0 = ex2(fmaf(__uint_as_float(s[c][2 * e]), p.scale_log2, -m_eff));
                    const float p1 = ex2(fmaf(__uint_as_float(s[c][2 * e + 1]), p.scale_log2, -m_eff));
                    l += p0 + p1;
                    pk[e] = pack2_bf16(p0, p1);
                }
                ptx::tmem_st16(t_s + c * 16, pk);
            }
            ptx::tmem_st_wait();
            ptx::tc_fence_before();
            ptx::mbar_arrive(bar(BAR_P + t));
        }
        if (ok && !*abort_flag) ok = ptx::mbar_wait(bar(BAR_O + t), (cnt - 1) & 1);
        if (ok && !*abort_flag) {
            ptx::tc_fence_after();
            float *dst = p.ws_o + (slab + t * 128 + row) * 128;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t o[32];
                ptx::tmem_ld32(t_o + c * 32, o);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int e = 0; e < 32; e += 4)
                    *reinterpret_cast<uint4 *>(dst + c * 32 + e) = make_uint4(o[e], o[e + 1], o[e + 2], o[e + 3]);
            }
            *reinterpret_cast<float2 *>(p.ws_ml + (slab + t * 128 + row) * 2) = make_float2(m_used, l);
        }
        if (!ok) *abort_flag = 1;
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // A bounded wait ran out: raise the sticky error, give outstanding copies and tensor-core
        // work one more bounded chance to finish, then release tensor memory.
        if (threadIdx.x == 0) atomicExch(p.dev_error, MTV_ERR_TIMEOUT);
        if (warp == 9 && lane == 0) {
            ptx::mbar_wait(bar(BAR_Q), 0);
            for (int s = 0; s < TC_SLOTS; ++s) { ptx::mbar_wait(bar(BAR_KV_FULL + s), 0); ptx::mbar_wait(bar(BAR_KV_FULL + s), 1); }
        }
        if (warp == 8) {
            if (lane == 0) ptx::tc_commit(bar(BAR_FINAL));
            __syncwarp();
            ptx::mbar_wait(bar(BAR_FINAL), 0);
        }
        __syncthreads();
    }
    if (warp == 8) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem, 512);
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

int launch_tree_attn_tc(const mtv_tree *tree, int B, int Hq, int Hkv, const __nv_bfloat16 *q, const __nv_bfloat16 *k,
                        const __nv_bfloat16 *v, int64_t sb, int64_t sh, int64_t st, int Lcap, const int32_t *seq_lens,
                        float scale_log2, float *ws_o, float *ws_ml, int nsplit, int m_rows, cudaStream_t stream) {
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
    static bool attr_done = false;
    if (!attr_done) {
        MTV_CUDA_CHECK(cudaFuncSetAttribute(tree_attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_BYTES));
        attr_done = true;
    }
    TcParams p;
    p.seq_lens = seq_lens; p.anc = tree->d_anc; p.ws_o = ws_o; p.ws_ml = ws_ml; p.dev_error = tree->d_error;
    p.scale_log2 = scale_log2;
    p.T = T; p.G = G; p.Hkv = Hkv; p.Lcap = Lcap; p.nsplit = nsplit; p.m_rows = m_rows; p.n_rt = m_rows / 256;
    p.M_rows = T * G;
    const dim3 grid(nsplit, Hkv * p.n_rt, B);
    tree_attn_tc_kernel<<<grid, TC_THREADS, TC_SMEM_BYTES, stream>>>(q_map, k_map, v_map, p);
    return MTV_OK;
}

}  // namespace mtv
