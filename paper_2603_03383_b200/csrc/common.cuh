// Shared declarations of the CUDA library: the tree object, error plumbing and
// small device helpers.  Nothing here is used by the CPU checker.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "../../include/mtv.h"

struct mtv_tree {
    int T = 0, K = 0, P = 0, C = 0, anc_words = 0;
    int k_d[MTV_MAX_K] = {0};
    int cand_offset[MTV_MAX_K] = {0};
    std::vector<int32_t> node_ranks, parent, depth, rank, tree_indices, retrieve;
    std::vector<uint64_t> anc;
    std::vector<uint8_t> mask;
    // device copies (one allocation), valid when on_device
    bool on_device = false;
    int device = -1;
    void *d_blob = nullptr;
    const int32_t *d_tree_indices = nullptr;  // [T]
    const int32_t *d_retrieve = nullptr;      // [P][K+1]
    const uint64_t *d_anc = nullptr;          // [T][2]  (always two words per row on the device)
    const int32_t *d_kd = nullptr;            // [K]
    const int32_t *d_cand_offset = nullptr;   // [K]
    int32_t *d_error = nullptr;               // sticky device-side error word (0 = none)
    const int32_t *d_depth = nullptr;         // [T]
    int32_t *d_counters = nullptr;            // [512] merge counters of the attention kernel, zero between calls
};

namespace mtv {

void set_last_error(const char *what, cudaError_t e);
void set_last_error_text(const char *text);

#define MTV_CUDA_CHECK(expr)                                  \
    do {                                                      \
        cudaError_t e__ = (expr);                             \
        if (e__ != cudaSuccess) {                             \
            ::mtv::set_last_error(#expr, e__);                \
            return MTV_ERR_CUDA;                              \
        }                                                     \
    } while (0)

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Workspace carving shared by the entry points (all offsets 256-byte aligned).
struct HeadsWs {
    size_t hprime_off, part_val_off, part_idx_off, counters_off, xsplit_off, total;
    int ctas_per_head, n_counters;
    bool use_tc;   // several batch rows: vocabulary projection on the tcgen05 tensor cores
};
HeadsWs heads_ws_layout(const mtv_tree *t, int B, int H, int V);
bool heads_tc_eligible(int B, int H);
size_t heads_tc_xsplit_bytes(int K, int H);
int launch_heads_tc(const mtv_tree *t, int B, int H, int V, const __nv_bfloat16 *hidden, const __nv_bfloat16 *W1,
                    const __nv_bfloat16 *b1, const __nv_bfloat16 *W2, const int32_t *root_tok, int32_t *cand,
                    float *cand_logit, int32_t *tree_tok, const HeadsWs &L, char *ws, cudaStream_t st);

struct AttnWs {
    size_t o_off, ml_off, order_off = 0, total;
    int nsplit, m_rows;
    bool use_tc;   // head_dim 128 path on the tcgen05 tensor cores
};
AttnWs attn_ws_layout(const mtv_tree *t, int B, int Hq, int Hkv, int D, int Lcap);

struct AcceptWs {
    size_t part_off, total;
    int nsplit;
};
AcceptWs accept_ws_layout(const mtv_tree *t, int B, int V);

int sm_count();   // of the current device

// Set-up that has to happen once per device (kernel attributes, symbol addresses): one flag per device ordinal.
// Two host threads that meet on first use both do the set-up; it is idempotent.
constexpr int MTV_MAX_DEVICES = 64;
struct PerDeviceOnce {
    bool done[MTV_MAX_DEVICES] = {};
    // the current device's flag, or null if the device cannot be told (the caller then does the set-up every time)
    bool *flag() {
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MTV_MAX_DEVICES) return nullptr;
        return &done[dev];
    }
};

// Index checks of the -DMTV_DEBUG_BOUNDS build: MTV_INDEX_OK(i, n, err) is true when 0 <= i < n; otherwise it
// records MTV_ERR_BOUNDS in the device error word and is false, and the caller skips the access.  In normal builds
// it is the constant true and the checks vanish.
#ifdef MTV_DEBUG_BOUNDS
__device__ __forceinline__ bool index_ok(long long i, long long n, int32_t *err) {
    if (i >= 0 && i < n) return true;
    if (err) atomicExch(err, MTV_ERR_BOUNDS);
    return false;
}
#define MTV_INDEX_OK(i, n, err) ::mtv::index_ok((long long)(i), (long long)(n), (err))
#else
#define MTV_INDEX_OK(i, n, err) true
#endif

// NVTX range around a C-ABI call (visible in a timeline profiler; one indirect call when no tool is attached).
// -DMTV_NO_NVTX leaves them out.
#ifndef MTV_NO_NVTX
}  // namespace mtv
#include <nvtx3/nvToolsExt.h>
namespace mtv {
struct NvtxRange {
    explicit NvtxRange(const char *name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
    NvtxRange(const NvtxRange &) = delete;
    NvtxRange &operator=(const NvtxRange &) = delete;
};
#define MTV_RANGE(name) ::mtv::NvtxRange mtv_nvtx_range__(name)
#else
#define MTV_RANGE(name) do { } while (0)
#endif

// Optional per-kernel event taps (see mtv_set_kernel_taps).
struct Tap {
    cudaEvent_t *start = nullptr, *stop = nullptr;
    int cap = 0, n = 0;
};
extern Tap g_taps[MTV_KERNEL_COUNT];
struct TapScope {
    Tap &t;
    cudaStream_t st;
    bool on;
    TapScope(int id, cudaStream_t s) : t(g_taps[id]), st(s), on(t.start && t.n < t.cap) {
        if (on) cudaEventRecord(t.start[t.n], st);
    }
    ~TapScope() {
        if (on) cudaEventRecord(t.stop[t.n++], st);
    }
};

}  // namespace mtv
