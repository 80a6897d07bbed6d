// Pieces that put one sequence's step back together when it was split over several GPUs (the paper runs on one
// device and has no counterpart; the split follows its structure: Section 3.1's heads are independent over the
// vocabulary, Section 3.2's tree attention is independent over KV heads).  Every rank runs the ordinary calls on its
// slice; a collective (outside this library) brings the slices into LOCAL buffers; the kernels here merge them.
// No kernel ever reads another GPU's memory.
#include "heads_common.cuh"

namespace mtv {

constexpr int MERGE_MAX_SHARDS = 16;

// grid = (K, B), one warp.  Head k of batch row b: the shards' lists (k_d entries each, sorted, ids local to the
// shard's vocabulary slab) -> the k_d best of all of them by (logit descending, global id ascending) — the order of
// the single-device lists, so equal inputs give identical candidates.  The last warp to finish a batch row expands
// the row's candidates into its tree tokens.
__global__ void __launch_bounds__(32)
heads_merge_shards_kernel(int B, int K, int C, int T, int n_shards, int v_slab, const int32_t *__restrict__ cand_shards,
                          const float *__restrict__ logit_shards, const int32_t *__restrict__ kd_arr,
                          const int32_t *__restrict__ off_arr, const int32_t *__restrict__ tree_indices,
                          const int32_t *__restrict__ root_tok, int32_t *__restrict__ cand, float *__restrict__ cand_logit,
                          int32_t *__restrict__ tree_tok, int32_t *__restrict__ tickets, int32_t *__restrict__ dev_error) {
    __shared__ float val[MERGE_MAX_SHARDS * MTV_MAX_TOPK];
    __shared__ int32_t idx[MERGE_MAX_SHARDS * MTV_MAX_TOPK];
    __shared__ int s_last;
    const int k = blockIdx.x, b = blockIdx.y, lane = threadIdx.x;
    const int kd = kd_arr[k], off = off_arr[k];
    const int n = n_shards * kd;
    for (int e = lane; e < n; e += 32) {
        const int r = e / kd, s = e % kd;
        val[e] = logit_shards[((size_t)r * B + b) * (C - 1) + off - 1 + s];
        idx[e] = cand_shards[((size_t)r * B + b) * C + off + s] + r * v_slab;
    }
    __syncwarp();
    // kd rounds: every lane proposes the best of its entries that are still in play, the warp takes the best proposal
    for (int s = 0; s < kd; ++s) {
        float bv = -INFINITY;
        int bi = 0x7fffffff, be = -1;
        for (int e = lane; e < n; e += 32)
            if (idx[e] >= 0 && (be < 0 || cand_before(val[e], idx[e], bv, bi))) { bv = val[e]; bi = idx[e]; be = e; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o), oe = __shfl_xor_sync(0xffffffffu, be, o);
            if (oe >= 0 && (be < 0 || cand_before(ov, oi, bv, bi))) { bv = ov; bi = oi; be = oe; }
        }
        if (lane == 0) {
            cand[(size_t)b * C + off + s] = bi;
            if (cand_logit) cand_logit[(size_t)b * (C - 1) + off - 1 + s] = bv;
            if (be >= 0) idx[be] = -1;                        // out of play
        }
        __syncwarp();
    }
    // ---- the last head of this batch row expands the candidates into the tree tokens
    __threadfence();
    if (lane == 0) s_last = atomicAdd(&tickets[b], 1) == K - 1;
    __syncwarp();
    if (!s_last) return;
    __threadfence();
    const int32_t root = root_tok[b];
    for (int i = lane; i < T; i += 32) {
        const int slot = tree_indices[i];
        if (!MTV_INDEX_OK(slot, C, dev_error)) continue;
        if (i == 0) cand[(size_t)b * C] = root;
        tree_tok[(size_t)b * T + i] = slot == 0 ? root : __ldcg(cand + (size_t)b * C + slot);
    }
    if (lane == 0) tickets[b] = 0;                            // ready for the next call
}

// out[row][r * Hq_local + h][:] = gathered[r][row][h][:]; one 16-byte chunk per thread.
__global__ void __launch_bounds__(256)
attn_interleave_shards_kernel(size_t rows, int n_shards, int Hq_local, int D, const uint4 *__restrict__ gathered,
                              uint4 *__restrict__ out) {
    const int vec = D / 8;
    const size_t per_row = (size_t)n_shards * Hq_local * vec;
    const size_t total = rows * per_row;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
        const size_t row = e / per_row;
        const int rem = (int)(e % per_row);
        const int r = rem / (Hq_local * vec), hc = rem % (Hq_local * vec);
        out[e] = gathered[((size_t)r * rows + row) * Hq_local * vec + hc];
    }
}

// keys[i] = max over shards of the shard's key with its slab offset folded into the index half (the low word is
// 0xffffffff - index, so the offset is subtracted); an all-zero key (nothing seen) stays zero.
__global__ void __launch_bounds__(256)
keys_merge_shards_kernel(int n, int n_shards, int v_slab, const unsigned long long *__restrict__ key_shards,
                         unsigned long long *__restrict__ keys) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    unsigned long long best = 0;
    for (int r = 0; r < n_shards; ++r) {
        unsigned long long kx = key_shards[(size_t)r * n + i];
        if (kx) kx -= (unsigned long long)r * (unsigned long long)v_slab;
        best = kx > best ? kx : best;
    }
    keys[i] = best;
}

}  // namespace mtv

extern "C" int heads_merge_shards(const mtv_tree_t *tree, int B, int n_shards, int v_slab, const int32_t *cand_shards,
                                  const float *logit_shards, const int32_t *root_tok, int32_t *cand, float *cand_logit,
                                  int32_t *tree_tok, void *ws, size_t ws_bytes, void *stream) {
    using namespace mtv;
    MTV_RANGE("heads_merge_shards");
    if (!tree || !tree->on_device || !cand_shards || !logit_shards || !root_tok || !cand || !tree_tok || !ws)
        return MTV_ERR_INVALID_ARG;
    if (B < 1 || n_shards < 1 || v_slab < 1) return MTV_ERR_INVALID_ARG;
    if (n_shards > MERGE_MAX_SHARDS || B > 65535) return MTV_ERR_UNSUPPORTED_SHAPE;
    if ((long long)(n_shards - 1) * v_slab + v_slab > 0x7fffffffLL) return MTV_ERR_UNSUPPORTED_SHAPE;
    for (int k = 0; k < tree->K; ++k)
        if (tree->k_d[k] > v_slab) return MTV_ERR_INVALID_ARG;     // a slab shorter than a head's top-k has no full list
    if (ws_bytes < (size_t)B * sizeof(int32_t)) return MTV_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    int32_t *tickets = static_cast<int32_t *>(ws);
    MTV_CUDA_CHECK(cudaMemsetAsync(tickets, 0, (size_t)B * sizeof(int32_t), st));
    heads_merge_shards_kernel<<<dim3(tree->K, B), 32, 0, st>>>(B, tree->K, tree->C, tree->T, n_shards, v_slab, cand_shards,
                                                               logit_shards, tree->d_kd, tree->d_cand_offset,
                                                               tree->d_tree_indices, root_tok, cand, cand_logit, tree_tok,
                                                               tickets, tree->d_error);
    MTV_CUDA_CHECK(cudaGetLastError());
    return MTV_OK;
}

extern "C" int attn_interleave_shards(int rows, int n_shards, int Hq_local, int D, const mtv_bf16 *gathered, mtv_bf16 *out,
                                      void *stream) {
    using namespace mtv;
    MTV_RANGE("attn_interleave_shards");
    if (!gathered || !out || rows < 1 || n_shards < 1 || Hq_local < 1 || D < 8 || D % 8) return MTV_ERR_INVALID_ARG;
    if (((uintptr_t)gathered | (uintptr_t)out) & 15) return MTV_ERR_INVALID_ARG;
    const size_t total = (size_t)rows * n_shards * Hq_local * (D / 8);
    const int blocks = (int)std::min<size_t>((total + 255) / 256, (size_t)sm_count() * 8);
    attn_interleave_shards_kernel<<<blocks, 256, 0, (cudaStream_t)stream>>>(
        (size_t)rows, n_shards, Hq_local, D, reinterpret_cast<const uint4 *>(gathered), reinterpret_cast<uint4 *>(out));
    MTV_CUDA_CHECK(cudaGetLastError());
    return MTV_OK;
}

extern "C" int keys_merge_shards(int n, int n_shards, int v_slab, const unsigned long long *key_shards,
                                 unsigned long long *keys, void *stream) {
    using namespace mtv;
    MTV_RANGE("keys_merge_shards");
    if (!key_shards || !keys || n < 1 || n_shards < 1 || v_slab < 1) return MTV_ERR_INVALID_ARG;
    if ((long long)n_shards * v_slab > 0x7fffffffLL) return MTV_ERR_UNSUPPORTED_SHAPE;
    keys_merge_shards_kernel<<<(n + 255) / 256, 256, 0, (cudaStream_t)stream>>>(n, n_shards, v_slab, key_shards, keys);
    MTV_CUDA_CHECK(cudaGetLastError());
    return MTV_OK;
}
