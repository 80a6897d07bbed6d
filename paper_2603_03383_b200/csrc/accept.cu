// Acceptance and token retrieval (Section 3.2, "Zero-Copy Retrieval"): per-node argmax
// of the base-model logits, greedy longest-prefix match over the static paths, and the
// gather of the accepted tokens through retrieve_indices — all on the device.
#include <atomic>
#include <cstdio>

#include <cuda_bf16.h>

#include "common.cuh"

namespace mtv {

constexpr int ARGMAX_THREADS = 256;

AcceptWs accept_ws_layout(const mtv_tree *t, int B, int V) {
    AcceptWs w;
    // split each logit row so that the scan fills the GPU: about 4 CTAs per SM in total,
    // but no chunk shorter than 2048 elements (8 per thread per iteration)
    long rows = (long)B * t->T;
    int ns = (int)((4L * sm_count() + rows - 1) / rows);
    int max_ns = (V + 2047) / 2048;
    if (ns > max_ns) ns = max_ns;
    if (ns < 1) ns = 1;
    w.nsplit = ns;
    w.part_off = 0;
    w.total = align_up((size_t)rows * ns * sizeof(unsigned long long), 256);
    return w;
}

// Order-preserving key: larger logit first, equal logits by lower index.  bf16 -> the
// usual sign-flip integer key; ~index in the low half so that max() prefers low indices.
__device__ __forceinline__ unsigned long long pack_key(uint32_t bf16_bits, uint32_t idx) {
    uint32_t k = bf16_bits & 0x8000u ? (~bf16_bits & 0xffffu) : (bf16_bits | 0x8000u);
    if ((bf16_bits & 0x7fffu) == 0) k = 0x8000u;  // -0.0 and +0.0 compare equal
    return ((unsigned long long)k << 32) | (0xffffffffu - idx);
}

__device__ __forceinline__ unsigned long long umax64(unsigned long long a, unsigned long long b) { return a > b ? a : b; }

// grid = (nsplit, B*T).  Partial argmax of one chunk of one row.
__global__ void __launch_bounds__(ARGMAX_THREADS)
node_argmax_partial_kernel(int V, const __nv_bfloat16 *__restrict__ logits, unsigned long long *__restrict__ part) {
    const int row = blockIdx.y, ns = gridDim.x;
    // chunk boundaries on multiples of 8 elements so that 16-byte loads stay aligned
    const int per = ((V + ns - 1) / ns + 7) / 8 * 8;
    const int begin = blockIdx.x * per;
    const int end = min(V, begin + per);
    const uint16_t *p = reinterpret_cast<const uint16_t *>(logits) + (size_t)row * V;
    unsigned long long best = 0;
    const bool aligned = (((size_t)row * V) % 8) == 0;
    if (aligned) {
        // Four independent 16-byte loads in flight per thread.  Per chunk of 8 logits only its maximum is formed
        // (packed bf16 max) and compared with the thread's running maximum; the chunk that first raised it is
        // looked at again at the end to find the element, so the scan costs about one instruction per logit.
        constexpr int U = 4;
        float smax = -INFINITY;
        int pos = -1;                      // first element of the chunk that holds the thread's maximum so far
        for (int i0 = begin + threadIdx.x * 8; i0 < end; i0 += U * ARGMAX_THREADS * 8) {
            uint4 u[U];
#pragma unroll
            for (int k = 0; k < U; ++k) {
                const int i = i0 + k * ARGMAX_THREADS * 8;
                u[k] = make_uint4(0u, 0u, 0u, 0u);
                if (i + 8 <= end)
                    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                                 : "=r"(u[k].x), "=r"(u[k].y), "=r"(u[k].z), "=r"(u[k].w) : "l"(p + i));
            }
#pragma unroll
            for (int k = 0; k < U; ++k) {
                const int i = i0 + k * ARGMAX_THREADS * 8;
                if (i + 8 <= end) {
                    const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&u[k]);
                    const __nv_bfloat162 m2 = __hmax2(__hmax2(h[0], h[1]), __hmax2(h[2], h[3]));
                    const float m = fmaxf(__low2float(m2), __high2float(m2));
                    if (pos < 0 || m > smax) { smax = m; pos = i; }     // strictly greater: the first chunk stays
                } else if (i < end) {
                    for (int j = i; j < end; ++j) best = umax64(best, pack_key(p[j], j));
                }
            }
        }
        if (pos >= 0) {
            // the first element of that chunk that equals the maximum (-0.0 == +0.0, as in the key)
            int j = 0;
            while (j < 7 && !(__uint_as_float((uint32_t)p[pos + j] << 16) == smax)) ++j;
            if (!(__uint_as_float((uint32_t)p[pos + j] << 16) == smax)) j = 0;   // a chunk of NaNs
            best = umax64(best, pack_key(p[pos + j], pos + j));
        }
    } else {
        for (int i = begin + threadIdx.x; i < end; i += ARGMAX_THREADS) best = umax64(best, pack_key(p[i], i));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) best = umax64(best, __shfl_xor_sync(0xffffffffu, best, o));
    __shared__ unsigned long long sm[ARGMAX_THREADS / 32];
    if (threadIdx.x % 32 == 0) sm[threadIdx.x / 32] = best;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < ARGMAX_THREADS / 32; ++w) best = umax64(best, sm[w]);
        part[(size_t)row * ns + blockIdx.x] = best;
    }
}

// grid = B, block = 128.  Finish the argmax, score every path, pick the best, gather.
__global__ void __launch_bounds__(128)
accept_finish_kernel(int T, int K, int P, int ns, const unsigned long long *__restrict__ part,
                     const int32_t *__restrict__ tree_tok, const int32_t *__restrict__ ri,
                     int32_t *__restrict__ accept_len, int32_t *__restrict__ best_path,
                     int32_t *__restrict__ acc_nodes, int32_t *__restrict__ acc_tok,
                     int32_t *__restrict__ next_root, int32_t *__restrict__ dev_error) {
    __shared__ int32_t am[MTV_MAX_T];
    __shared__ int32_t tok[MTV_MAX_T];
    __shared__ unsigned int best_key;
    const int b = blockIdx.x;
    for (int i = threadIdx.x; i < T; i += blockDim.x) {
        unsigned long long best = 0;
        for (int s = 0; s < ns; ++s) best = umax64(best, part[((size_t)b * T + i) * ns + s]);
        am[i] = (int32_t)(0xffffffffu - (uint32_t)(best & 0xffffffffu));
        tok[i] = tree_tok[(size_t)b * T + i];
    }
    if (threadIdx.x == 0) best_key = 0;
    __syncthreads();
    // key = len * 256 + (255 - p): max() picks the longest match, then the lowest path
    for (int p = threadIdx.x; p < P; p += blockDim.x) {
        const int32_t *path = ri + (size_t)p * (K + 1);
        int len = 0;
        for (int j = 1; j <= K; ++j) {
            const int node = path[j];
            if (node < 0) break;
            if (!MTV_INDEX_OK(node, T, dev_error) || !MTV_INDEX_OK(path[j - 1], T, dev_error)) break;
            if (tok[node] != am[path[j - 1]]) break;
            len = j;
        }
        atomicMax(&best_key, (unsigned)len * 256u + (255u - (unsigned)p));
    }
    __syncthreads();
    const int len = best_key / 256, p = 255 - (int)(best_key % 256);
    if ((int)threadIdx.x <= K) {
        const int j = threadIdx.x;
        int node = j <= len ? ri[(size_t)p * (K + 1) + j] : -1;
        if (node >= 0 && !MTV_INDEX_OK(node, T, dev_error)) node = -1;
        acc_nodes[(size_t)b * (K + 1) + j] = node;
        acc_tok[(size_t)b * (K + 1) + j] = node >= 0 ? tok[node] : -1;
        if (j == len && node >= 0) next_root[b] = am[node];
        if (j == 0) { accept_len[b] = len; best_path[b] = p; }
    }
}

}  // namespace mtv

extern "C" int tree_accept(const mtv_tree_t *tree, int B, int V, const mtv_bf16 *logits, const int32_t *tree_tok,
                           int32_t *accept_len, int32_t *best_path, int32_t *acc_nodes, int32_t *acc_tok,
                           int32_t *next_root, void *ws, size_t ws_bytes, void *stream) {
    using namespace mtv;
    MTV_RANGE("tree_accept");
    if (!tree || !tree->on_device || !logits || !tree_tok || !accept_len || !best_path || !acc_nodes ||
        !acc_tok || !next_root || !ws || B < 1 || V < 1)
        return MTV_ERR_INVALID_ARG;
    if (tree->P > 255) return MTV_ERR_UNSUPPORTED_SHAPE;
    if ((uintptr_t)logits & 15) return MTV_ERR_INVALID_ARG;   // the scan reads 16-byte chunks of the rows
    const AcceptWs L = accept_ws_layout(tree, B, V);
    if (ws_bytes < L.total) return MTV_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    auto *part = reinterpret_cast<unsigned long long *>((char *)ws + L.part_off);
    {
        TapScope tap(MTV_KERNEL_ARGMAX_PARTIAL, st);
        node_argmax_partial_kernel<<<dim3(L.nsplit, B * tree->T), ARGMAX_THREADS, 0, st>>>(
            V, reinterpret_cast<const __nv_bfloat16 *>(logits), part);
    }
    TapScope tap(MTV_KERNEL_ACCEPT_FINISH, st);
    accept_finish_kernel<<<B, 128, 0, st>>>(tree->T, tree->K, tree->P, L.nsplit, part, tree_tok, tree->d_retrieve,
                                            accept_len, best_path, acc_nodes, acc_tok, next_root, tree->d_error);
    MTV_CUDA_CHECK(cudaGetLastError());
    return MTV_OK;
}

// Per-node argmax keys of stored logits, in the form tree_accept_keys reads: what tree_accept computes before its path
// scan.  A rank that holds a vocabulary slab of the logits calls this on its slab; keys_merge_shards then folds the
// slab offsets in and takes the maximum over the ranks.
namespace mtv {
__global__ void argmax_keys_reduce_kernel(int rows, int ns, const unsigned long long *__restrict__ part,
                                          unsigned long long *__restrict__ keys) {
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= rows) return;
    unsigned long long best = 0;
    for (int s = 0; s < ns; ++s) best = umax64(best, part[(size_t)r * ns + s]);
    keys[r] = best;
}
}  // namespace mtv

extern "C" int node_argmax_keys(const mtv_tree_t *tree, int B, int V, const mtv_bf16 *logits, unsigned long long *keys,
                                void *ws, size_t ws_bytes, void *stream) {
    using namespace mtv;
    MTV_RANGE("node_argmax_keys");
    if (!tree || !tree->on_device || !logits || !keys || !ws || B < 1 || V < 1) return MTV_ERR_INVALID_ARG;
    if ((uintptr_t)logits & 15) return MTV_ERR_INVALID_ARG;
    const AcceptWs L = accept_ws_layout(tree, B, V);
    if (ws_bytes < L.total) return MTV_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    auto *part = reinterpret_cast<unsigned long long *>((char *)ws + L.part_off);
    const int rows = B * tree->T;
    {
        TapScope tap(MTV_KERNEL_ARGMAX_PARTIAL, st);
        node_argmax_partial_kernel<<<dim3(L.nsplit, rows), ARGMAX_THREADS, 0, st>>>(
            V, reinterpret_cast<const __nv_bfloat16 *>(logits), part);
    }
    argmax_keys_reduce_kernel<<<(rows + 127) / 128, 128, 0, st>>>(rows, L.nsplit, part, keys);
    MTV_CUDA_CHECK(cudaGetLastError());
    return MTV_OK;
}

// Acceptance from per-node argmax keys (what lm_head_argmax leaves): the finish kernel alone, with
// one key per node.
extern "C" int tree_accept_keys(const mtv_tree_t *tree, int B, const unsigned long long *keys, const int32_t *tree_tok,
                                int32_t *accept_len, int32_t *best_path, int32_t *acc_nodes, int32_t *acc_tok,
                                int32_t *next_root, void *stream) {
    using namespace mtv;
    MTV_RANGE("tree_accept_keys");
    if (!tree || !tree->on_device || !keys || !tree_tok || !accept_len || !best_path || !acc_nodes || !acc_tok ||
        !next_root || B < 1)
        return MTV_ERR_INVALID_ARG;
    if (tree->P > 255) return MTV_ERR_UNSUPPORTED_SHAPE;
    accept_finish_kernel<<<B, 128, 0, (cudaStream_t)stream>>>(tree->T, tree->K, tree->P, 1, keys, tree_tok,
                                                              tree->d_retrieve, accept_len, best_path, acc_nodes,
                                                              acc_tok, next_root, tree->d_error);
    MTV_CUDA_CHECK(cudaGetLastError());
    return MTV_OK;
}

// ---------------------------------------------------------------------------
// tree_accept for callers that must not allocate device memory (the paper has no counterpart).
// Its scratch — the per-chunk argmax keys that tree_accept keeps in the caller's workspace —
// lives in a fixed array inside the library image.
namespace mtv {

constexpr size_t ACCEPT_STATIC_SCRATCH_BYTES = 64 * 1024;
static __device__ __align__(256) unsigned char g_accept_scratch[ACCEPT_STATIC_SCRATCH_BYTES];

// Device address of g_accept_scratch on the current device.  In host code the array's name is
// only a handle for the runtime, not an address a kernel could use, so the address is asked for
// once per device (with that device current) and remembered.
static int accept_scratch_address(unsigned long long **out) {
    // (two host threads that meet on first use of a device both look the address up and store the same value;
    // the slots are atomics so that neither ever reads a half-written pointer)
    static std::atomic<unsigned long long *> cached[MTV_MAX_DEVICES];
    int dev = 0;
    MTV_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MTV_MAX_DEVICES) return MTV_ERR_UNSUPPORTED_SHAPE;
    unsigned long long *addr = cached[dev].load(std::memory_order_acquire);
    if (!addr) {
        void *ptr = nullptr;
        MTV_CUDA_CHECK(cudaGetSymbolAddress(&ptr, g_accept_scratch));
        addr = reinterpret_cast<unsigned long long *>(ptr);
        cached[dev].store(addr, std::memory_order_release);
    }
    *out = addr;
    return MTV_OK;
}

}  // namespace mtv

extern "C" size_t tree_accept_static_scratch_capacity(void) { return mtv::ACCEPT_STATIC_SCRATCH_BYTES; }

extern "C" int tree_accept_static_scratch(const mtv_tree_t *tree, int B, int V, const mtv_bf16 *logits,
                                          const int32_t *tree_tok, int32_t *accept_len, int32_t *best_path,
                                          int32_t *acc_nodes, int32_t *acc_tok, int32_t *next_root, void *stream) {
    using namespace mtv;
    MTV_RANGE("tree_accept_static_scratch");
    if (!tree || !tree->on_device || !logits || !tree_tok || !accept_len || !best_path || !acc_nodes ||
        !acc_tok || !next_root || B < 1 || V < 1)
        return MTV_ERR_INVALID_ARG;
    if (tree->P > 255) return MTV_ERR_UNSUPPORTED_SHAPE;
    if ((uintptr_t)logits & 15) return MTV_ERR_INVALID_ARG;   // the scan reads 16-byte chunks of the rows
    const AcceptWs L = accept_ws_layout(tree, B, V);
    if (L.total > ACCEPT_STATIC_SCRATCH_BYTES) {
        char msg[160];
        snprintf(msg, sizeof msg, "tree_accept_static_scratch: B*T = %ld logit rows need %zu bytes of scratch, "
                 "the built-in array holds %zu", (long)B * tree->T, L.total, ACCEPT_STATIC_SCRATCH_BYTES);
        set_last_error_text(msg);
        return MTV_ERR_WORKSPACE;
    }
    unsigned long long *part = nullptr;
    const int rc = accept_scratch_address(&part);
    if (rc != MTV_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    // every entry of `part` that the second kernel reads is written by the first one: nothing to clear
    node_argmax_partial_kernel<<<dim3(L.nsplit, B * tree->T), ARGMAX_THREADS, 0, st>>>(
        V, reinterpret_cast<const __nv_bfloat16 *>(logits), part);
    accept_finish_kernel<<<B, 128, 0, st>>>(tree->T, tree->K, tree->P, L.nsplit, part, tree_tok, tree->d_retrieve,
                                            accept_len, best_path, acc_nodes, acc_tok, next_root, tree->d_error);
    MTV_CUDA_CHECK(cudaGetLastError());
    return MTV_OK;
}
