// Tree K/V append with rotary embedding — the step just before the tree attention
// (Section 3.2: tree_indices maps the flattened tree nodes to their positions).  Node i of
// sequence b sits at position seq_lens[b] + depth[i]; its rotated K row and its V row go to cache
// row seq_lens[b] + i, its query is rotated in place.  Memory-bound and tiny (T rows per KV
// head): one block per (node, sequence); the angles of a node are computed once, in double
// precision (positions reach tens of thousands of radians), and reused by all heads.
#include "common.cuh"

namespace mtv {

// One layer (caches given directly) or, with blockIdx.z = layer, all layers of a step in one launch (caches through
// the device pointer arrays of kv_compact_accepted; q, k_new, v_new then hold the layers back to back).
__global__ void __launch_bounds__(128)
tree_kv_append_rope_kernel(int T, int Hq, int Hkv, int D, int Lcap, __nv_bfloat16 *__restrict__ q,
                           const __nv_bfloat16 *__restrict__ k_new, const __nv_bfloat16 *__restrict__ v_new,
                           __nv_bfloat16 *__restrict__ k_cache, __nv_bfloat16 *__restrict__ v_cache,
                           __nv_bfloat16 *const *__restrict__ k_caches, __nv_bfloat16 *const *__restrict__ v_caches,
                           int64_t sb, int64_t sh, int64_t st, const int32_t *__restrict__ seq_lens,
                           const int32_t *__restrict__ depth, double log2_theta, int32_t *__restrict__ status) {
    __shared__ float cs[64], sn[64];   // D / 2 <= 64
    const int i = blockIdx.x, b = blockIdx.y;
    if (k_caches) {
        const size_t layer = blockIdx.z, B = gridDim.y;
        k_cache = k_caches[layer];
        v_cache = v_caches[layer];
        q += layer * B * T * Hq * D;
        k_new += layer * B * T * Hkv * D;
        v_new += layer * B * T * Hkv * D;
    }
    const int L = seq_lens[b];
    if (L + T > Lcap) {
        if (status && i == 0 && threadIdx.x == 0) status[b] = MTV_ERR_CAPACITY;
        return;
    }
    if (status && i == 0 && threadIdx.x == 0) status[b] = MTV_OK;
    const int half = D / 2;
    if ((int)threadIdx.x < half) {
        const double pos = (double)L + (double)depth[i];
        const double ang = pos * exp2(-2.0 * threadIdx.x / D * log2_theta);
        double s, c;
        sincos(ang, &s, &c);
        cs[threadIdx.x] = (float)c;
        sn[threadIdx.x] = (float)s;
    }
    __syncthreads();
    // queries, in place
    for (int e = threadIdx.x; e < Hq * half; e += blockDim.x) {
        const int h = e / half, d = e % half;
        __nv_bfloat16 *row = q + (((size_t)b * T + i) * Hq + h) * D;
        const float x1 = __bfloat162float(row[d]), x2 = __bfloat162float(row[d + half]);
        row[d] = __float2bfloat16_rn(x1 * cs[d] - x2 * sn[d]);
        row[d + half] = __float2bfloat16_rn(x2 * cs[d] + x1 * sn[d]);
    }
    // keys (rotated) and values (copied) into cache row L + i
    for (int e = threadIdx.x; e < Hkv * half; e += blockDim.x) {
        const int h = e / half, d = e % half;
        const size_t src = (((size_t)b * T + i) * Hkv + h) * D;
        const int64_t dst = b * sb + h * sh + (int64_t)(L + i) * st;
        const float x1 = __bfloat162float(k_new[src + d]), x2 = __bfloat162float(k_new[src + d + half]);
        k_cache[dst + d] = __float2bfloat16_rn(x1 * cs[d] - x2 * sn[d]);
        k_cache[dst + d + half] = __float2bfloat16_rn(x2 * cs[d] + x1 * sn[d]);
        v_cache[dst + d] = v_new[src + d];
        v_cache[dst + d + half] = v_new[src + d + half];
    }
}

}  // namespace mtv

extern "C" int tree_kv_append_rope(const mtv_tree_t *tree, int B, int Hq, int Hkv, int D, mtv_bf16 *q,
                                   const mtv_bf16 *k_new, const mtv_bf16 *v_new, mtv_bf16 *k_cache, mtv_bf16 *v_cache,
                                   int64_t stride_b, int64_t stride_h, int64_t stride_t, int Lcap,
                                   const int32_t *seq_lens, float rope_theta, int32_t *status, void *stream) {
    using namespace mtv;
    MTV_RANGE("tree_kv_append_rope");
    if (!tree || !tree->on_device || !q || !k_new || !v_new || !k_cache || !v_cache || !seq_lens) return MTV_ERR_INVALID_ARG;
    if (B < 1 || Hq < 1 || Hkv < 1 || Lcap < tree->T || rope_theta < 0.f) return MTV_ERR_INVALID_ARG;
    if ((D != 64 && D != 128) || B > 65535) return MTV_ERR_UNSUPPORTED_SHAPE;
    const double theta = rope_theta == 0.f ? 10000.0 : (double)rope_theta;
    tree_kv_append_rope_kernel<<<dim3(tree->T, B), 128, 0, (cudaStream_t)stream>>>(
        tree->T, Hq, Hkv, D, Lcap, reinterpret_cast<__nv_bfloat16 *>(q), reinterpret_cast<const __nv_bfloat16 *>(k_new),
        reinterpret_cast<const __nv_bfloat16 *>(v_new), reinterpret_cast<__nv_bfloat16 *>(k_cache),
        reinterpret_cast<__nv_bfloat16 *>(v_cache), nullptr, nullptr, stride_b, stride_h, stride_t, seq_lens,
        tree->d_depth, log2(theta), status);
    MTV_CUDA_CHECK(cudaGetLastError());
    return MTV_OK;
}

extern "C" int tree_kv_append_rope_layers(const mtv_tree_t *tree, int B, int Hq, int Hkv, int D, int n_layers,
                                          mtv_bf16 *q_layers, const mtv_bf16 *k_new_layers, const mtv_bf16 *v_new_layers,
                                          mtv_bf16 *const *k_caches, mtv_bf16 *const *v_caches, int64_t stride_b,
                                          int64_t stride_h, int64_t stride_t, int Lcap, const int32_t *seq_lens,
                                          float rope_theta, int32_t *status, void *stream) {
    using namespace mtv;
    MTV_RANGE("tree_kv_append_rope_layers");
    if (!tree || !tree->on_device || !q_layers || !k_new_layers || !v_new_layers || !k_caches || !v_caches || !seq_lens)
        return MTV_ERR_INVALID_ARG;
    if (B < 1 || Hq < 1 || Hkv < 1 || n_layers < 1 || Lcap < tree->T || rope_theta < 0.f) return MTV_ERR_INVALID_ARG;
    if ((D != 64 && D != 128) || B > 65535 || n_layers > 65535) return MTV_ERR_UNSUPPORTED_SHAPE;
    const double theta = rope_theta == 0.f ? 10000.0 : (double)rope_theta;
    tree_kv_append_rope_kernel<<<dim3(tree->T, B, n_layers), 128, 0, (cudaStream_t)stream>>>(
        tree->T, Hq, Hkv, D, Lcap, reinterpret_cast<__nv_bfloat16 *>(q_layers),
        reinterpret_cast<const __nv_bfloat16 *>(k_new_layers), reinterpret_cast<const __nv_bfloat16 *>(v_new_layers),
        nullptr, nullptr, reinterpret_cast<__nv_bfloat16 *const *>(k_caches),
        reinterpret_cast<__nv_bfloat16 *const *>(v_caches), stride_b, stride_h, stride_t, seq_lens, tree->d_depth,
        log2(theta), status);
    MTV_CUDA_CHECK(cudaGetLastError());
    return MTV_OK;
}
