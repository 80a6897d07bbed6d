// Pieces shared by the two vocabulary-projection kernels of the Medusa heads (Section 3.1): the
// parameter block, the ordering of candidates, and everything that follows the projection itself —
// merging the warps' candidate lists per CTA, the merge across the CTAs of a head by the last one to
// finish (atomic ticket, nobody waits), and the expansion into tree tokens by the last head (Section 3.2).
#pragma once
#include "common.cuh"

namespace mtv {

constexpr int HT_NB = 16;   // batch rows one pass of the tensor-core projection serves

// (value, id) ordering of the candidate lists: larger value first, equal values by smaller id.
__device__ __forceinline__ bool cand_before(float va, int ia, float vb, int ib) {
    return va > vb || (va == vb && ia < ib);
}

struct VocabParams {
    int B, H, V, K, T, C;
    const __nv_bfloat16 *W2;
    const float *hprime;
    const int32_t *kd_arr, *off_arr, *tree_indices, *root_tok;
    float *part_val;
    int32_t *part_idx;
    int32_t *counters;   // [btiles][K + 1], zeroed by the residual-block kernel
    int32_t *cand;
    float *cand_logit;
    int32_t *tree_tok;
    int32_t *dev_error;
    int rows_per_stage, n_stages, n_it;
    uint32_t stage_bytes, xs_off, lists_off, zbuf_off, bars_off;
};

// lval / lidx: [n_warps][NB][MTV_MAX_TOPK] sorted candidate lists in shared memory (unused slots hold
// (-inf, 0x7fffffff)); smem / scratch_bytes: shared memory free for the cross-CTA merge (at least
// per * MTV_MAX_TOPK * 8 bytes: one warp's staging area; more lets more warps merge batch rows side by side).
// Every thread of the CTA calls this.
__device__ __forceinline__ void vocab_tail(const VocabParams &p, const int NB, const int n_warps, const float *lval,
                                           const int32_t *lidx, unsigned char *smem, const int k, const int bz,
                                           const int b0, const int per, const int kd, const uint32_t scratch_bytes) {
    __shared__ int s_flag;
    // ---- merge the warps' lists: rank each entry among all CONS_WARPS*kd entries of its batch row
    for (int e = threadIdx.x; e < NB * n_warps * MTV_MAX_TOPK; e += (int)blockDim.x) {
        const int b = e / (n_warps * MTV_MAX_TOPK);
        const int w = (e / MTV_MAX_TOPK) % n_warps, sl = e % MTV_MAX_TOPK;
        if (sl >= kd || b0 + b >= p.B) continue;
        const float zz = lval[(w * NB + b) * MTV_MAX_TOPK + sl];
        const int id = lidx[(w * NB + b) * MTV_MAX_TOPK + sl];
        int rank = 0;
        for (int w2 = 0; w2 < n_warps; ++w2)
            for (int s2 = 0; s2 < kd; ++s2) {
                const float z2 = lval[(w2 * NB + b) * MTV_MAX_TOPK + s2];
                const int id2 = lidx[(w2 * NB + b) * MTV_MAX_TOPK + s2];
                // unused slots all carry the same sentinel: order them by position
                if (cand_before(z2, id2, zz, id) || (z2 == zz && id2 == id && (w2 * MTV_MAX_TOPK + s2) < (w * MTV_MAX_TOPK + sl)))
                    ++rank;
            }
        if (rank < kd) {
            const size_t o = (((size_t)k * p.B + b0 + b) * per + blockIdx.x) * MTV_MAX_TOPK + rank;
            p.part_val[o] = zz;
            p.part_idx[o] = id;
        }
    }
    // ---- last CTA of this head merges the CTAs' lists (ticket: nobody waits)
    int32_t *counters = p.counters + (size_t)bz * (p.K + 1);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_flag = atomicAdd(&counters[k], 1) == per - 1;
    __syncthreads();
    if (!s_flag) return;
    __threadfence();
    {
        // The CTAs' lists are sorted, so the best kd of all of them come out of a kd-round tournament over
        // the lists' heads.  Each warp takes one batch row at a time: it stages the row's lists in shared
        // memory, lane l plays for lists l, l + 32, ...
        const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
        const int off = p.off_arr[k];
        const uint32_t per_warp = (uint32_t)per * MTV_MAX_TOPK * 8;
        int n_w = (int)(scratch_bytes / per_warp);
        if (n_w > (int)blockDim.x / 32) n_w = (int)blockDim.x / 32;
        constexpr int MAXL = 8;                               // lists per lane: up to 256 CTAs per head
        if (warp < n_w) {
            float *mval = reinterpret_cast<float *>(smem + (size_t)warp * per_warp);   // [per][MTV_MAX_TOPK]
            int32_t *midx = reinterpret_cast<int32_t *>(mval + per * MTV_MAX_TOPK);
            for (int b = warp; b < NB && b0 + b < p.B; b += n_w) {
                const size_t base = ((size_t)k * p.B + b0 + b) * per * MTV_MAX_TOPK;
                __syncwarp();
                for (int e = lane; e < per * MTV_MAX_TOPK; e += 32) {
                    const bool used = e % MTV_MAX_TOPK < kd;
                    mval[e] = used ? __ldcg(p.part_val + base + e) : -INFINITY;
                    midx[e] = used ? __ldcg(p.part_idx + base + e) : 0x7fffffff;
                }
                __syncwarp();
                int head[MAXL];
#pragma unroll
                for (int q = 0; q < MAXL; ++q) head[q] = 0;
                for (int r = 0; r < kd; ++r) {
                    // this lane's best head
                    float bv = -INFINITY;
                    int bi = 0x7fffffff, bq = -1;
#pragma unroll
                    for (int q = 0; q < MAXL; ++q) {
                        const int c = lane + 32 * q;
                        if (c < per && head[q] < kd) {
                            const float v = mval[c * MTV_MAX_TOPK + head[q]];
                            const int id = midx[c * MTV_MAX_TOPK + head[q]];
                            if (bq < 0 || cand_before(v, id, bv, bi)) { bv = v; bi = id; bq = q; }
                        }
                    }
                    // the warp's best: value first, then id, then lane (equal sentinels)
                    float wv = bv;
                    int wi = bi, wl = bq < 0 ? 64 : lane;
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
                        const float ov = __shfl_xor_sync(0xffffffffu, wv, o);
                        const int oi = __shfl_xor_sync(0xffffffffu, wi, o);
                        const int ol = __shfl_xor_sync(0xffffffffu, wl, o);
                        const bool other = ol < 64 && (wl >= 64 || cand_before(ov, oi, wv, wi) || (ov == wv && oi == wi && ol < wl));
                        if (other) { wv = ov; wi = oi; wl = ol; }
                    }
                    if (lane == 0) {
                        p.cand[(size_t)(b0 + b) * p.C + off + r] = wi;
                        if (p.cand_logit) p.cand_logit[(size_t)(b0 + b) * (p.C - 1) + off - 1 + r] = wv;
                    }
                    if (lane == wl) {
#pragma unroll
                        for (int q = 0; q < MAXL; ++q)
                            if (q == bq) ++head[q];
                    }
                }
            }
        }
    }
    // ---- last head of this batch tile expands the candidates into the tree tokens
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_flag = atomicAdd(&counters[p.K], 1) == p.K - 1;
    __syncthreads();
    if (!s_flag) return;
    __threadfence();
    for (int e = threadIdx.x; e < NB * p.T; e += (int)blockDim.x) {
        const int b = b0 + e / p.T, i = e % p.T;
        if (b >= p.B) break;
        const int slot = p.tree_indices[i];
        if (!MTV_INDEX_OK(slot, p.C, p.dev_error)) continue;
        const int32_t root = p.root_tok[b];
        if (i == 0) p.cand[(size_t)b * p.C] = root;
        p.tree_tok[(size_t)b * p.T + i] = slot == 0 ? root : __ldcg(p.cand + (size_t)b * p.C + slot);
    }
}

}  // namespace mtv
