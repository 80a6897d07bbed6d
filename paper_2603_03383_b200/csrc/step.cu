// Whole verification step on one stream, and its host-buffer variant.
#include "common.cuh"

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

extern "C" int mtv_verify_step(const mtv_tree_t *tree, const mtv_step_args *a, void *stream) {
    if (!tree || !a || !a->k_caches_host || !a->v_caches_host) return MTV_ERR_INVALID_ARG;
    int rc = medusa_heads_topk(tree, a->B, a->H, a->V, a->hidden, a->W1, a->b1, a->W2, a->root_tok, a->cand,
                               a->cand_logit, a->tree_tok, a->ws, a->ws_bytes, stream);
    if (rc != MTV_OK) return rc;
    const size_t per_layer = (size_t)a->B * tree->T * a->Hq * a->D;
    for (int l = 0; l < a->n_layers; ++l) {
        rc = tree_verify_attention(tree, a->B, a->Hq, a->Hkv, a->D, a->q_layers + l * per_layer, a->k_caches_host[l],
                                   a->v_caches_host[l], a->stride_b, a->stride_h, a->stride_t, a->Lcap, a->seq_lens,
                                   a->scale, a->out_layers + l * per_layer, a->status, a->ws, a->ws_bytes, stream);
        if (rc != MTV_OK) return rc;
    }
    rc = tree_accept(tree, a->B, a->V, a->logits, a->tree_tok, a->accept_len, a->best_path, a->acc_nodes, a->acc_tok,
                     a->next_root, a->ws, a->ws_bytes, stream);
    if (rc != MTV_OK) return rc;
    return kv_compact_accepted(tree, a->B, a->Hkv, a->D, a->n_layers, a->k_caches, a->v_caches, a->stride_b,
                               a->stride_h, a->stride_t, a->Lcap, a->seq_lens, a->accept_len, a->acc_nodes, a->status,
                               stream);
}

extern "C" int mtv_verify_step_host(const mtv_tree_t *tree, const mtv_step_args *d, const mtv_step_args *h,
                                    void *stream) {
    if (!tree || !d || !h) return MTV_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t B = d->B, T = tree->T, K = tree->K;
    const size_t q_bytes = (size_t)d->n_layers * B * T * d->Hq * d->D * 2;
    MTV_CUDA_CHECK(cudaMemcpyAsync((void *)d->hidden, h->hidden, B * d->H * 2, cudaMemcpyHostToDevice, st));
    MTV_CUDA_CHECK(cudaMemcpyAsync((void *)d->root_tok, h->root_tok, B * 4, cudaMemcpyHostToDevice, st));
    MTV_CUDA_CHECK(cudaMemcpyAsync((void *)d->q_layers, h->q_layers, q_bytes, cudaMemcpyHostToDevice, st));
    MTV_CUDA_CHECK(cudaMemcpyAsync((void *)d->logits, h->logits, B * T * d->V * 2, cudaMemcpyHostToDevice, st));
    int rc = mtv_verify_step(tree, d, stream);
    if (rc != MTV_OK) return rc;
    MTV_CUDA_CHECK(cudaMemcpyAsync(h->tree_tok, d->tree_tok, B * T * 4, cudaMemcpyDeviceToHost, st));
    MTV_CUDA_CHECK(cudaMemcpyAsync(h->out_layers, d->out_layers, q_bytes, cudaMemcpyDeviceToHost, st));
    MTV_CUDA_CHECK(cudaMemcpyAsync(h->accept_len, d->accept_len, B * 4, cudaMemcpyDeviceToHost, st));
    MTV_CUDA_CHECK(cudaMemcpyAsync(h->best_path, d->best_path, B * 4, cudaMemcpyDeviceToHost, st));
    MTV_CUDA_CHECK(cudaMemcpyAsync(h->acc_nodes, d->acc_nodes, B * (K + 1) * 4, cudaMemcpyDeviceToHost, st));
    MTV_CUDA_CHECK(cudaMemcpyAsync(h->acc_tok, d->acc_tok, B * (K + 1) * 4, cudaMemcpyDeviceToHost, st));
    MTV_CUDA_CHECK(cudaMemcpyAsync(h->next_root, d->next_root, B * 4, cudaMemcpyDeviceToHost, st));
    MTV_CUDA_CHECK(cudaMemcpyAsync(h->seq_lens, d->seq_lens, B * 4, cudaMemcpyDeviceToHost, st));
    MTV_CUDA_CHECK(cudaStreamSynchronize(st));
    return MTV_OK;
}
