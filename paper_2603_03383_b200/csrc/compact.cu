// In-place KV compaction of the accepted path (Section 3.2, "Zero-Copy Retrieval",
// applied to the K/V rows): row seq_len + acc_nodes[j] -> row seq_len + j for
// j = 1..accept_len, every layer and KV head, then seq_len += accept_len + 1.
#include "common.cuh"

namespace mtv {

// grid = (Hkv, B, n_layers).  A source row of step j may be the destination of a later
// step j' (acc_nodes = [0,2,..]: j=1 reads slot 2, j=2 writes slot 2), so the block
// stages every source row in shared memory before it writes anything.
__global__ void __launch_bounds__(256)
kv_compact_kernel(int T, int K, int D, int Lcap, __nv_bfloat16 *const *__restrict__ k_caches,
                  __nv_bfloat16 *const *__restrict__ v_caches, int64_t sb, int64_t sh, int64_t st,
                  const int32_t *__restrict__ seq_lens, const int32_t *__restrict__ accept_len,
                  const int32_t *__restrict__ acc_nodes, int32_t *__restrict__ dev_error) {
    __shared__ uint4 stage[2 * MTV_MAX_K * 16];  // [k|v][j][D/8 <= 16]
    const int g = blockIdx.x, b = blockIdx.y, layer = blockIdx.z;
    const int L = seq_lens[b];
    const int n = accept_len[b];
    if (L + T > Lcap || n <= 0) return;
    if (!MTV_INDEX_OK(n, K + 1, dev_error)) return;      // accept_len comes from the caller's device memory
    const int vec = D / 8;
    __nv_bfloat16 *kc = k_caches[layer] + b * sb + g * sh;
    __nv_bfloat16 *vc = v_caches[layer] + b * sb + g * sh;
    const int total = 2 * n * vec;
    for (int e = threadIdx.x; e < total; e += blockDim.x) {
        const int which = e / (n * vec), j = (e / vec) % n, c = e % vec;
        const int node = acc_nodes[(size_t)b * (K + 1) + j + 1];
        const int src = L + node;
        const __nv_bfloat16 *base = which ? vc : kc;
        stage[e] = MTV_INDEX_OK(node, T, dev_error) ? *reinterpret_cast<const uint4 *>(base + (int64_t)src * st + c * 8)
                                                    : make_uint4(0, 0, 0, 0);
    }
    __syncthreads();
    for (int e = threadIdx.x; e < total; e += blockDim.x) {
        const int which = e / (n * vec), j = (e / vec) % n, c = e % vec;
        __nv_bfloat16 *base = which ? vc : kc;
        if (!MTV_INDEX_OK(acc_nodes[(size_t)b * (K + 1) + j + 1], T, dev_error)) continue;   // a row that was not read is not written
        *reinterpret_cast<uint4 *>(base + (int64_t)(L + j + 1) * st + c * 8) = stage[e];
    }
}

// Runs after every compaction block has read seq_lens (next kernel on the stream).
__global__ void seq_lens_advance_kernel(int B, int T, int Lcap, int32_t *seq_lens, const int32_t *accept_len,
                                        int32_t *status, int K, int32_t *dev_error) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const int L = seq_lens[b];
    if (L + T > Lcap) {
        if (status) status[b] = MTV_ERR_CAPACITY;
        return;
    }
    if (status) status[b] = MTV_OK;
    if (!MTV_INDEX_OK(accept_len[b], K + 1, dev_error)) return;
    seq_lens[b] = L + accept_len[b] + 1;
}

}  // namespace mtv

extern "C" int kv_compact_accepted(const mtv_tree_t *tree, int B, int Hkv, int D, int n_layers,
                                   mtv_bf16 *const *k_caches, mtv_bf16 *const *v_caches,
                                   int64_t stride_b, int64_t stride_h, int64_t stride_t, int Lcap,
                                   int32_t *seq_lens, const int32_t *accept_len, const int32_t *acc_nodes,
                                   int32_t *status, void *stream) {
    using namespace mtv;
    MTV_RANGE("kv_compact_accepted");
    if (!tree || !k_caches || !v_caches || !seq_lens || !accept_len || !acc_nodes || B < 1 || Hkv < 1 ||
        n_layers < 1 || Lcap < 1)
        return MTV_ERR_INVALID_ARG;
    if (D != 64 && D != 128) return MTV_ERR_UNSUPPORTED_SHAPE;
    if (stride_t % 8 || stride_h % 8 || stride_b % 8) return MTV_ERR_INVALID_ARG;
    if (B > 65535 || n_layers > 65535) return MTV_ERR_UNSUPPORTED_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    {
        TapScope tap(MTV_KERNEL_KV_COMPACT, st);
        kv_compact_kernel<<<dim3(Hkv, B, n_layers), 256, 0, st>>>(
        tree->T, tree->K, D, Lcap, reinterpret_cast<__nv_bfloat16 *const *>(k_caches),
        reinterpret_cast<__nv_bfloat16 *const *>(v_caches), stride_b, stride_h, stride_t, seq_lens, accept_len,
            acc_nodes, tree->d_error);
    }
    TapScope tap(MTV_KERNEL_SEQ_ADVANCE, st);
    seq_lens_advance_kernel<<<(B + 127) / 128, 128, 0, st>>>(B, tree->T, Lcap, seq_lens, accept_len, status, tree->K,
                                                                   tree->d_error);
    MTV_CUDA_CHECK(cudaGetLastError());
    return MTV_OK;
}
