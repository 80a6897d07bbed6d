"""TEST INFRASTRUCTURE — ctypes marshalling for ``mtv_oracle.c`` (no arithmetic).

Inputs are CPU torch tensors (bf16 data, int32 indices); outputs are float64 /
int32 CPU tensors.  The shared object is compiled on first use.
"""
import ctypes as C

import torch

from . import build as _build

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
    return _lib


def _p(t):
    if t is None:
        return None
    assert t.device.type == "cpu" and t.is_contiguous()
    return C.c_void_p(t.data_ptr())


def _i32(t):
    return torch.as_tensor(t, dtype=torch.int32).contiguous()


def heads_logits(hidden, W1, b1, W2):
    """Section 3.1 heads -> z [K,B,V] float64."""
    K, V, H = W2.shape
    B = hidden.shape[0]
    assert hidden.dtype == W1.dtype == W2.dtype == torch.bfloat16
    hidden, W1, W2 = hidden.contiguous(), W1.contiguous(), W2.contiguous()
    b1 = b1.contiguous() if b1 is not None else None
    z = torch.empty(K, B, V, dtype=torch.float64)
    lib().mtv_ref_heads_logits(K, B, H, V, _p(hidden), _p(W1), _p(b1), _p(W2), _p(z))
    return z


def topk(z_row, k):
    """(ids [k] int32, vals [k] float64, min gap among ranks 1..k+1)."""
    z_row = z_row.contiguous()
    assert z_row.dtype == torch.float64 and z_row.dim() == 1
    ids = torch.empty(k, dtype=torch.int32)
    vals = torch.empty(k, dtype=torch.float64)
    gap = C.c_double(0.0)
    lib().mtv_ref_topk(z_row.numel(), _p(z_row), k, _p(ids), _p(vals), C.byref(gap))
    return ids, vals, gap.value


def heads_candidates(z, root_tok, tb):
    """Flat candidate buffer and tree tokens from head logits z [K,B,V].

    cand[b] = [root_tok[b] | top-k_1 ids of head 1 | top-k_2 ids of head 2 | ...]
    tree_tok[b][i] = cand[b][tree_indices[i]].
    Returns cand [B,C] int32, cand_logit [B,C-1] float64, tree_tok [B,T] int32,
    min_gap (smallest rank gap met, for the seed-margin policy).
    """
    K, B, V = z.shape
    Cn, T = tb["C"], tb["T"]
    cand = torch.empty(B, Cn, dtype=torch.int32)
    cl = torch.empty(B, Cn - 1, dtype=torch.float64)
    min_gap = float("inf")
    for b in range(B):
        cand[b, 0] = int(root_tok[b])
        for d in range(K):
            kd = tb["k_d"][d]
            if kd == 0:
                continue
            ids, vals, gap = topk(z[d, b], kd)
            off = tb["offset"][d]
            cand[b, off:off + kd] = ids
            cl[b, off - 1:off - 1 + kd] = vals
            min_gap = min(min_gap, gap)
    ti = torch.tensor(tb["tree_indices"], dtype=torch.int64)
    tree_tok = cand[:, ti].contiguous()
    return cand, cl, tree_tok, min_gap


def _strides(cache):
    assert cache.dim() == 4 and cache.stride(3) == 1
    return cache.stride(0), cache.stride(1), cache.stride(2)


def tree_attention(q, k_cache, v_cache, seq_lens, mask, scale=None, rows=None):
    """Section 3.2 masked tree attention -> out float64.

    q [B,T,Hq,D]; caches [B,Hkv,Lcap,D]; mask [T][T] (medusa_attn_mask).
    rows: optional list of (b, i, h); then out is [len(rows), D].
    """
    B, T, Hq, D = q.shape
    Hkv = k_cache.shape[1]
    q = q.contiguous()
    sb, sh, st = _strides(k_cache)
    assert _strides(v_cache) == (sb, sh, st)
    seq_lens = _i32(seq_lens)
    m = torch.as_tensor(mask, dtype=torch.uint8).contiguous()
    assert m.shape == (T, T)
    scale = float(scale) if scale else 1.0 / float(D) ** 0.5
    args = (T, Hq, Hkv, D, _p(q), C.c_void_p(k_cache.data_ptr()), C.c_void_p(v_cache.data_ptr()),
            C.c_int64(sb), C.c_int64(sh), C.c_int64(st), _p(seq_lens), _p(m), C.c_double(scale))
    if rows is None:
        out = torch.empty(B, T, Hq, D, dtype=torch.float64)
        lib().mtv_ref_tree_attention(B, *args, _p(out))
    else:
        r = _i32(rows).reshape(-1, 3)
        out = torch.empty(r.shape[0], D, dtype=torch.float64)
        lib().mtv_ref_tree_attention_rows(*args, r.shape[0], _p(r), _p(out))
    return out


def node_argmax(logits):
    """am [B,T] int32: per-node argmax of base logits [B,T,V] bf16 (ties -> lowest id)."""
    B, T, V = logits.shape
    logits = logits.contiguous()
    am = torch.empty(B, T, dtype=torch.int32)
    lib().mtv_ref_node_argmax(B, T, V, _p(logits), _p(am))
    return am


def tree_accept(am, tree_tok, tb):
    """Greedy longest-prefix acceptance + token retrieval.  Returns a dict of int32 tensors."""
    B, T = am.shape
    K, P = tb["K"], tb["P"]
    am, tree_tok = _i32(am), _i32(tree_tok)
    ri = _i32(tb["retrieve"])
    out = dict(accept_len=torch.empty(B, dtype=torch.int32), best_path=torch.empty(B, dtype=torch.int32),
               acc_nodes=torch.empty(B, K + 1, dtype=torch.int32),
               acc_tok=torch.empty(B, K + 1, dtype=torch.int32),
               next_root=torch.empty(B, dtype=torch.int32))
    lib().mtv_ref_tree_accept(B, T, K, P, _p(am), _p(tree_tok), _p(ri), _p(out["accept_len"]),
                              _p(out["best_path"]), _p(out["acc_nodes"]), _p(out["acc_tok"]),
                              _p(out["next_root"]))
    return out


def kv_compact(cache, seq_lens, accept_len, acc_nodes):
    """Out-of-place compaction of one cache [B,Hkv,Lcap,D]; returns (new cache, new seq_lens)."""
    B, Hkv, Lcap, D = cache.shape
    assert cache.is_contiguous()
    sb, sh, st = _strides(cache)
    seq_lens, accept_len, acc_nodes = _i32(seq_lens), _i32(accept_len), _i32(acc_nodes)
    K = acc_nodes.shape[1] - 1
    dst = torch.empty_like(cache)
    lib().mtv_ref_kv_compact(B, Hkv, D, _p(cache), _p(dst), C.c_size_t(cache.numel()),
                             C.c_int64(sb), C.c_int64(sh), C.c_int64(st),
                             _p(seq_lens), _p(accept_len), _p(acc_nodes), K)
    return dst, seq_lens + accept_len + 1


def rope(q, k_new, seq_lens, depth, theta=10000.0):
    """Rotary embedding of the tree nodes' q [B,T,Hq,D] and k_new [B,T,Hkv,D] at positions seq_lens[b] + depth[i]
    (rotate-half pairing) -> (q_out, k_out) float64."""
    B, T, Hq, D = q.shape
    Hkv = k_new.shape[2]
    q, k_new = q.contiguous(), k_new.contiguous()
    seq_lens, depth = _i32(seq_lens), _i32(depth)
    q_out = torch.empty(B, T, Hq, D, dtype=torch.float64)
    k_out = torch.empty(B, T, Hkv, D, dtype=torch.float64)
    lib().mtv_ref_rope(B, T, Hq, Hkv, D, _p(q), _p(k_new), _p(seq_lens), _p(depth), C.c_double(theta), _p(q_out),
                       _p(k_out))
    return q_out, k_out


def lm_head_argmax(x, W, want_logits=False):
    """LM head + per-node argmax: x [M,H], W [V,H] bf16 -> (am int32 [M], zmax, z2 float64 [M][, z [M,V]])."""
    M, H = x.shape
    V = W.shape[0]
    assert x.dtype == W.dtype == torch.bfloat16 and W.shape[1] == H
    x, W = x.contiguous(), W.contiguous()
    am = torch.empty(M, dtype=torch.int32)
    zmax = torch.empty(M, dtype=torch.float64)
    z2 = torch.empty(M, dtype=torch.float64)
    z = torch.empty(M, V, dtype=torch.float64) if want_logits else None
    lib().mtv_ref_lm_head_argmax(M, H, V, _p(x), _p(W), _p(am), _p(zmax), _p(z2), _p(z))
    return (am, zmax, z2, z) if want_logits else (am, zmax, z2)
