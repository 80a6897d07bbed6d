// Whole verification step on one stream, and its host-buffer variant.
#include <mutex>

#include "common.cuh"
#include "sm100_ptx.cuh"

extern "C" size_t mtv_workspace_bytes(const mtv_tree_t *tree, int B, int H, int V, int Hq, int Hkv, int D, int Lcap) {
    using namespace mtv;
    if (!tree || B < 1) return 0;
    size_t need = 256;
    if (H > 0 && V > 0) {
        need = std::max(need, heads_ws_layout(tree, B, H, V).total);
        need = std::max(need, accept_ws_layout(tree, B, V).total);
    }
    if (Hq > 0 && Hkv > 0 && D > 0 && Lcap > 0 && Hq % Hkv == 0)
        need = std::max(need, attn_ws_layout(tree, B, Hq, Hkv, D, Lcap).total);
    return need;
}

// Acceptance of a step: from stored logits, or from the fused LM head when the caller gave its operands
// (the per-node keys then sit at the start of the workspace, which no other kernel uses at that point).
static int step_accept(const mtv_tree_t *tree, const mtv_step_args *a, void *stream) {
    if (a->x_final && a->W_lm) {
        if (!a->ws || a->ws_bytes < (size_t)a->B * tree->T * sizeof(unsigned long long)) return MTV_ERR_WORKSPACE;
        unsigned long long *keys = static_cast<unsigned long long *>(a->ws);
        const int rc = lm_head_argmax(tree, a->B, a->H, a->V, a->x_final, a->W_lm, nullptr, nullptr, keys, stream);
        if (rc != MTV_OK) return rc;
        return tree_accept_keys(tree, a->B, keys, a->tree_tok, a->accept_len, a->best_path, a->acc_nodes, a->acc_tok,
                                a->next_root, stream);
    }
    return tree_accept(tree, a->B, a->V, a->logits, a->tree_tok, a->accept_len, a->best_path, a->acc_nodes, a->acc_tok,
                       a->next_root, a->ws, a->ws_bytes, stream);
}

// One step; root_tok and the optional append are given separately so that a chain of steps can feed a step's root
// from the previous step's next_root without touching the caller's structs.
static int verify_step(const mtv_tree_t *tree, const mtv_step_args *a, const int32_t *root_tok,
                       const mtv_append_args *ap, void *stream) {
    if (!tree || !a || !a->k_caches_host || !a->v_caches_host || !root_tok) return MTV_ERR_INVALID_ARG;
    int rc = medusa_heads_topk(tree, a->B, a->H, a->V, a->hidden, a->W1, a->b1, a->W2, root_tok, a->cand,
                               a->cand_logit, a->tree_tok, a->ws, a->ws_bytes, stream);
    if (rc != MTV_OK) return rc;
    if (ap && (ap->k_new_layers || ap->v_new_layers)) {
        // the tree nodes' K/V rows of every layer, in one launch in front of the first attention (which starts its
        // set-up under this kernel's tail: programmatic dependent launch)
        rc = tree_kv_append_rope_layers(tree, a->B, a->Hq, a->Hkv, a->D, a->n_layers, const_cast<mtv_bf16 *>(a->q_layers),
                                        ap->k_new_layers, ap->v_new_layers, a->k_caches, a->v_caches, a->stride_b,
                                        a->stride_h, a->stride_t, a->Lcap, a->seq_lens, ap->rope_theta, a->status, stream);
        if (rc != MTV_OK) return rc;
    }
    const size_t per_layer = (size_t)a->B * tree->T * a->Hq * a->D;
    for (int l = 0; l < a->n_layers; ++l) {
        rc = tree_verify_attention(tree, a->B, a->Hq, a->Hkv, a->D, a->q_layers + l * per_layer, a->k_caches_host[l],
                                   a->v_caches_host[l], a->stride_b, a->stride_h, a->stride_t, a->Lcap, a->seq_lens,
                                   a->scale, a->out_layers + l * per_layer, a->status, a->ws, a->ws_bytes, stream);
        if (rc != MTV_OK) return rc;
    }
    rc = step_accept(tree, a, stream);
    if (rc != MTV_OK) return rc;
    return kv_compact_accepted(tree, a->B, a->Hkv, a->D, a->n_layers, a->k_caches, a->v_caches, a->stride_b,
                               a->stride_h, a->stride_t, a->Lcap, a->seq_lens, a->accept_len, a->acc_nodes, a->status,
                               stream);
}

extern "C" int mtv_verify_step(const mtv_tree_t *tree, const mtv_step_args *a, void *stream) {
    MTV_RANGE("mtv_verify_step");
    if (!a) return MTV_ERR_INVALID_ARG;
    return verify_step(tree, a, a->root_tok, nullptr, stream);
}

// n steps back to back on one stream.  Nothing is decided on the host between them: step s + 1 takes its root token
// from step s's next_root and its prefix lengths from the seq_lens that step s's compaction advanced, both on the device.
extern "C" int mtv_verify_steps(const mtv_tree_t *tree, const mtv_step_args *steps, const mtv_append_args *appends,
                                int n_steps, void *stream) {
    MTV_RANGE("mtv_verify_steps");
    if (!tree || !steps || n_steps < 1) return MTV_ERR_INVALID_ARG;
    for (int s = 0; s < n_steps; ++s) {      // the whole chain is looked at before anything is enqueued
        if (!steps[s].root_tok && (s == 0 || !steps[s - 1].next_root)) return MTV_ERR_INVALID_ARG;
        if (!steps[s].seq_lens || steps[s].seq_lens != steps[0].seq_lens) return MTV_ERR_INVALID_ARG;   // one chain, one set of lengths
        if (!steps[s].k_caches_host || !steps[s].v_caches_host) return MTV_ERR_INVALID_ARG;
    }
    for (int s = 0; s < n_steps; ++s) {
        const mtv_step_args *a = steps + s;
        const int32_t *root = a->root_tok ? a->root_tok : steps[s - 1].next_root;
        const int rc = verify_step(tree, a, root, appends ? appends + s : nullptr, stream);
        if (rc != MTV_OK) return rc;
    }
    return MTV_OK;
}

namespace {
// Copy streams and events of the host-buffer variant, created on first use, one set per device (the variant
// synchronises anyway, so it is not one of the allocation-free hot calls).  Calls on one device take turns.
struct HostStepAux {
    cudaStream_t up = nullptr, down = nullptr;
    cudaEvent_t start = nullptr, q_up = nullptr, logits_up = nullptr, down_done = nullptr;
    cudaEvent_t chunk[8] = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
    bool ready = false;
    std::mutex busy;
};
HostStepAux g_aux_table[mtv::MTV_MAX_DEVICES];
int host_step_aux(HostStepAux **out) {
    int dev = 0;
    MTV_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= mtv::MTV_MAX_DEVICES) return MTV_ERR_UNSUPPORTED_SHAPE;
    HostStepAux &g_aux = g_aux_table[dev];
    *out = &g_aux;
    std::lock_guard<std::mutex> lock(g_aux.busy);
    if (g_aux.ready) return MTV_OK;
    MTV_CUDA_CHECK(cudaStreamCreateWithFlags(&g_aux.up, cudaStreamNonBlocking));
    MTV_CUDA_CHECK(cudaStreamCreateWithFlags(&g_aux.down, cudaStreamNonBlocking));
    cudaEvent_t *ev[] = {&g_aux.start, &g_aux.q_up, &g_aux.logits_up, &g_aux.down_done, &g_aux.chunk[0], &g_aux.chunk[1],
                         &g_aux.chunk[2], &g_aux.chunk[3], &g_aux.chunk[4], &g_aux.chunk[5], &g_aux.chunk[6], &g_aux.chunk[7]};
    for (cudaEvent_t *e : ev) MTV_CUDA_CHECK(cudaEventCreateWithFlags(e, cudaEventDisableTiming));
    g_aux.ready = true;
    return MTV_OK;
}
}  // namespace

// The transfers overlap the compute: the queries and the base-model logits go up on a copy stream while the
// heads run (attention waits for the queries, acceptance for the logits), and the attention outputs come
// down on a second copy stream in up to sixteen groups of layers while later layers are still running.
extern "C" int mtv_verify_step_host(const mtv_tree_t *tree, const mtv_step_args *d, const mtv_step_args *h,
                                    void *stream) {
    MTV_RANGE("mtv_verify_step_host");
    if (!tree || !d || !h || !d->k_caches_host || !d->v_caches_host) return MTV_ERR_INVALID_ARG;
    HostStepAux *aux = nullptr;
    if (host_step_aux(&aux) != MTV_OK) return MTV_ERR_CUDA;
    HostStepAux &g_aux = *aux;
    std::lock_guard<std::mutex> turn(g_aux.busy);
    cudaStream_t st = (cudaStream_t)stream, up = g_aux.up, down = g_aux.down;
    const size_t B = d->B, T = tree->T, K = tree->K;
    const size_t per_layer = B * T * d->Hq * d->D;           // elements
    const size_t q_bytes = (size_t)d->n_layers * per_layer * 2;
    // uploads
    MTV_CUDA_CHECK(cudaEventRecord(g_aux.start, st));         // the copy streams start where the caller's stream is
    MTV_CUDA_CHECK(cudaStreamWaitEvent(up, g_aux.start, 0));
    MTV_CUDA_CHECK(cudaStreamWaitEvent(down, g_aux.start, 0));
    MTV_CUDA_CHECK(cudaMemcpyAsync((void *)d->hidden, h->hidden, B * d->H * 2, cudaMemcpyHostToDevice, st));
    MTV_CUDA_CHECK(cudaMemcpyAsync((void *)d->root_tok, h->root_tok, B * 4, cudaMemcpyHostToDevice, st));
    MTV_CUDA_CHECK(cudaMemcpyAsync((void *)d->q_layers, h->q_layers, q_bytes, cudaMemcpyHostToDevice, up));
    MTV_CUDA_CHECK(cudaEventRecord(g_aux.q_up, up));
    if (d->x_final && d->W_lm)
        MTV_CUDA_CHECK(cudaMemcpyAsync((void *)d->x_final, h->x_final, B * T * d->H * 2, cudaMemcpyHostToDevice, up));
    else
        MTV_CUDA_CHECK(cudaMemcpyAsync((void *)d->logits, h->logits, B * T * d->V * 2, cudaMemcpyHostToDevice, up));
    MTV_CUDA_CHECK(cudaEventRecord(g_aux.logits_up, up));
    // heads
    int rc = medusa_heads_topk(tree, d->B, d->H, d->V, d->hidden, d->W1, d->b1, d->W2, d->root_tok, d->cand, d->cand_logit,
                               d->tree_tok, d->ws, d->ws_bytes, stream);
    if (rc != MTV_OK) return rc;
    MTV_CUDA_CHECK(cudaMemcpyAsync(h->tree_tok, d->tree_tok, B * T * 4, cudaMemcpyDeviceToHost, st));
    // attention, its outputs leaving in groups of layers
    MTV_CUDA_CHECK(cudaStreamWaitEvent(st, g_aux.q_up, 0));
    const int per_group = (d->n_layers + 15) / 16;
    int sent = 0, n_sent = 0;
    for (int l = 0; l < d->n_layers; ++l) {
        rc = tree_verify_attention(tree, d->B, d->Hq, d->Hkv, d->D, d->q_layers + l * per_layer, d->k_caches_host[l],
                                   d->v_caches_host[l], d->stride_b, d->stride_h, d->stride_t, d->Lcap, d->seq_lens,
                                   d->scale, d->out_layers + l * per_layer, d->status, d->ws, d->ws_bytes, stream);
        if (rc != MTV_OK) return rc;
        if ((l + 1) % per_group == 0 || l + 1 == d->n_layers) {
            cudaEvent_t ev = g_aux.chunk[n_sent++ % 8];
            MTV_CUDA_CHECK(cudaEventRecord(ev, st));
            MTV_CUDA_CHECK(cudaStreamWaitEvent(down, ev, 0));
            MTV_CUDA_CHECK(cudaMemcpyAsync(h->out_layers + sent * per_layer, d->out_layers + sent * per_layer,
                                           (size_t)(l + 1 - sent) * per_layer * 2, cudaMemcpyDeviceToHost, down));
            sent = l + 1;
        }
    }
    // acceptance and compaction
    MTV_CUDA_CHECK(cudaStreamWaitEvent(st, g_aux.logits_up, 0));
    rc = step_accept(tree, d, stream);
    if (rc != MTV_OK) return rc;
    rc = kv_compact_accepted(tree, d->B, d->Hkv, d->D, d->n_layers, d->k_caches, d->v_caches, d->stride_b, d->stride_h,
                             d->stride_t, d->Lcap, d->seq_lens, d->accept_len, d->acc_nodes, d->status, stream);
    if (rc != MTV_OK) return rc;
    MTV_CUDA_CHECK(cudaMemcpyAsync(h->accept_len, d->accept_len, B * 4, cudaMemcpyDeviceToHost, st));
    MTV_CUDA_CHECK(cudaMemcpyAsync(h->best_path, d->best_path, B * 4, cudaMemcpyDeviceToHost, st));
    MTV_CUDA_CHECK(cudaMemcpyAsync(h->acc_nodes, d->acc_nodes, B * (K + 1) * 4, cudaMemcpyDeviceToHost, st));
    MTV_CUDA_CHECK(cudaMemcpyAsync(h->acc_tok, d->acc_tok, B * (K + 1) * 4, cudaMemcpyDeviceToHost, st));
    MTV_CUDA_CHECK(cudaMemcpyAsync(h->next_root, d->next_root, B * 4, cudaMemcpyDeviceToHost, st));
    MTV_CUDA_CHECK(cudaMemcpyAsync(h->seq_lens, d->seq_lens, B * 4, cudaMemcpyDeviceToHost, st));
    MTV_CUDA_CHECK(cudaEventRecord(g_aux.down_done, down));
    MTV_CUDA_CHECK(cudaStreamWaitEvent(st, g_aux.down_done, 0));
    MTV_CUDA_CHECK(cudaStreamSynchronize(st));
    return MTV_OK;
}

// ---------------------------------------------------------------------------
// Self-test of the bounded waits: a barrier nobody arrives on.
namespace {
__global__ void selftest_wait_timeout_kernel(int32_t *dev_error) {
    __shared__ __align__(8) unsigned long long bar_mem;
    const uint32_t bar = mtv::ptx::smem_u32(&bar_mem);
    if (threadIdx.x == 0) {
        mtv::ptx::mbar_init(bar, 1);
        mtv::ptx::fence_mbar_init();
    }
    __syncwarp();
    const bool ok = mtv::ptx::mbar_wait(bar, 0);      // gives up after WAIT_CYCLE_LIMIT cycles
    if (!ok && threadIdx.x == 0) atomicExch(dev_error, MTV_ERR_TIMEOUT);
}
}  // namespace

extern "C" int mtv_debug_bounds_enabled(void) {
#ifdef MTV_DEBUG_BOUNDS
    return 1;
#else
    return 0;
#endif
}

extern "C" int mtv_selftest_wait_timeout(const mtv_tree_t *tree, void *stream) {
    if (!tree || !tree->on_device) return MTV_ERR_INVALID_ARG;
    selftest_wait_timeout_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(tree->d_error);
    MTV_CUDA_CHECK(cudaGetLastError());
    return MTV_OK;
}
