"""ctypes binding of ``libmtv.so`` — argument marshalling only.

Every function has the name and argument order of its C declaration in
``include/mtv.h``; tensors are passed as device pointers, the current torch
stream is used unless one is given.  There is no fallback: if the CUDA library
is missing, loading fails with an error.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# MTV_LIB names another build of the same library (a variant of build.py, e.g. the bounds-checking one).
LIB_PATH = os.environ.get("MTV_LIB") or os.path.join(_HERE, "libmtv.so")

MTV_OK = 0
MTV_ERR_BOUNDS = -7
ERR = {-7: "MTV_ERR_BOUNDS", -1: "MTV_ERR_INVALID_ARG", -2: "MTV_ERR_UNSUPPORTED_SHAPE", -3: "MTV_ERR_WORKSPACE",
       -4: "MTV_ERR_CUDA", -5: "MTV_ERR_TIMEOUT", -6: "MTV_ERR_CAPACITY"}
MTV_ERR_TIMEOUT = -5
MTV_ERR_CAPACITY = -6
MAX_K = 8

EXPORTS = ["tree_build_static", "tree_gen_cartesian", "tree_gen_rank_prior", "tree_query", "tree_destroy",
           "mtv_workspace_bytes", "medusa_heads_topk", "tree_verify_attention", "tree_accept",
           "kv_compact_accepted", "mtv_verify_step", "mtv_verify_step_host", "mtv_last_error",
           "mtv_set_kernel_taps", "mtv_kernel_taps_used", "mtv_device_error",
           "tree_accept_static_scratch", "tree_accept_static_scratch_capacity", "tree_kv_append_rope",
           "lm_head_argmax", "tree_accept_keys", "mtv_selftest_wait_timeout", "tree_kv_append_rope_layers",
           "mtv_verify_steps", "mtv_debug_bounds_enabled", "heads_merge_shards", "attn_interleave_shards",
           "keys_merge_shards", "node_argmax_keys"]


class MtvError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        detail = ""
        if code == -4:
            detail = ": " + lib().mtv_last_error().decode()
        super().__init__("%s failed with %s%s" % (where, ERR.get(code, code), detail))


class TreeInfo(C.Structure):
    _fields_ = [("T", C.c_int32), ("K", C.c_int32), ("P", C.c_int32), ("C", C.c_int32),
                ("anc_words", C.c_int32), ("on_device", C.c_int32),
                ("k_d", C.c_int32 * MAX_K), ("cand_offset", C.c_int32 * MAX_K),
                ("node_ranks", C.POINTER(C.c_int32)), ("parent", C.POINTER(C.c_int32)),
                ("depth", C.POINTER(C.c_int32)), ("rank", C.POINTER(C.c_int32)),
                ("tree_indices", C.POINTER(C.c_int32)), ("retrieve_indices", C.POINTER(C.c_int32)),
                ("anc", C.POINTER(C.c_uint64)), ("medusa_attn_mask", C.POINTER(C.c_uint8))]


class StepArgs(C.Structure):
    _fields_ = [("B", C.c_int32), ("H", C.c_int32), ("V", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32),
                ("D", C.c_int32), ("n_layers", C.c_int32), ("Lcap", C.c_int32),
                ("stride_b", C.c_int64), ("stride_h", C.c_int64), ("stride_t", C.c_int64),
                ("scale", C.c_float),
                ("hidden", C.c_void_p), ("W1", C.c_void_p), ("b1", C.c_void_p), ("W2", C.c_void_p),
                ("root_tok", C.c_void_p), ("q_layers", C.c_void_p),
                ("k_caches", C.c_void_p), ("v_caches", C.c_void_p),
                ("k_caches_host", C.c_void_p), ("v_caches_host", C.c_void_p),
                ("logits", C.c_void_p), ("seq_lens", C.c_void_p),
                ("cand", C.c_void_p), ("cand_logit", C.c_void_p), ("tree_tok", C.c_void_p),
                ("out_layers", C.c_void_p),
                ("accept_len", C.c_void_p), ("best_path", C.c_void_p), ("acc_nodes", C.c_void_p),
                ("acc_tok", C.c_void_p), ("next_root", C.c_void_p), ("status", C.c_void_p),
                ("ws", C.c_void_p), ("ws_bytes", C.c_size_t),
                ("x_final", C.c_void_p), ("W_lm", C.c_void_p)]


class AppendArgs(C.Structure):
    _fields_ = [("k_new_layers", C.c_void_p), ("v_new_layers", C.c_void_p), ("rope_theta", C.c_float)]


_lib = None


def lib():
    """Load the CUDA library (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("CUDA library %s is missing: run paper_2603_03383_b200/build.py "
                               "(there is no CPU fallback)" % LIB_PATH)
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, sz = C.c_void_p, C.c_int, C.c_int64, C.c_size_t
        L.tree_build_static.argtypes = [i32, i32, vp, i32, C.POINTER(vp)]
        L.tree_gen_cartesian.argtypes = [i32, vp, i32, vp, C.POINTER(C.c_int)]
        L.tree_gen_rank_prior.argtypes = [i32, i32, i32, vp, C.POINTER(C.c_int)]
        L.tree_query.argtypes = [vp, C.POINTER(TreeInfo)]
        L.tree_destroy.argtypes = [vp]
        L.tree_destroy.restype = None
        L.mtv_workspace_bytes.argtypes = [vp] + [i32] * 7
        L.mtv_workspace_bytes.restype = sz
        L.medusa_heads_topk.argtypes = [vp, i32, i32, i32] + [vp] * 8 + [vp, sz, vp]
        L.tree_verify_attention.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, i64, i64, i64, i32, vp,
                                            C.c_float, vp, vp, vp, sz, vp]
        L.tree_accept.argtypes = [vp, i32, i32] + [vp] * 7 + [vp, sz, vp]
        L.kv_compact_accepted.argtypes = [vp, i32, i32, i32, i32, vp, vp, i64, i64, i64, i32, vp, vp, vp, vp, vp]
        L.mtv_verify_step.argtypes = [vp, C.POINTER(StepArgs), vp]
        L.mtv_verify_step_host.argtypes = [vp, C.POINTER(StepArgs), C.POINTER(StepArgs), vp]
        L.mtv_last_error.restype = C.c_char_p
        L.mtv_set_kernel_taps.argtypes = [i32, vp, vp, i32]
        L.mtv_kernel_taps_used.argtypes = [i32]
        L.mtv_device_error.argtypes = [vp, i32, C.POINTER(C.c_int32)]
        L.tree_accept_static_scratch.argtypes = [vp, i32, i32] + [vp] * 7 + [vp]
        L.tree_accept_static_scratch_capacity.restype = sz
        L.tree_kv_append_rope.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, i64, i64, i64, i32, vp, C.c_float,
                                          vp, vp]
        L.lm_head_argmax.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp, vp]
        L.tree_accept_keys.argtypes = [vp, i32] + [vp] * 7 + [vp]
        L.mtv_selftest_wait_timeout.argtypes = [vp, vp]
        L.tree_kv_append_rope_layers.argtypes = [vp, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, i64, i64, i64, i32, vp,
                                                 C.c_float, vp, vp]
        L.heads_merge_shards.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.attn_interleave_shards.argtypes = [i32, i32, i32, i32, vp, vp, vp]
        L.keys_merge_shards.argtypes = [i32, i32, i32, vp, vp, vp]
        L.node_argmax_keys.argtypes = [vp, i32, i32, vp, vp, vp, sz, vp]
        L.mtv_verify_steps.argtypes = [vp, C.POINTER(StepArgs), C.POINTER(AppendArgs), i32, vp]
        _lib = L
    return _lib


def _check(rc, where):
    if rc != MTV_OK:
        raise MtvError(rc, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def tree_gen_cartesian(topk: Sequence[int]):
    K = len(topk)
    tk = (C.c_int32 * K)(*topk)
    n = C.c_int(0)
    lib().tree_gen_cartesian(K, tk, 0, None, C.byref(n))
    buf = (C.c_int32 * (max(n.value, 1) * K))()
    _check(lib().tree_gen_cartesian(K, tk, n.value, buf, C.byref(n)), "tree_gen_cartesian")
    return [list(buf[i * K:(i + 1) * K]) for i in range(n.value)]


def tree_gen_rank_prior(K: int, T_total: int, R_max: int = 10):
    n = C.c_int(0)
    buf = (C.c_int32 * (max(T_total - 1, 1) * K))()
    _check(lib().tree_gen_rank_prior(K, T_total, R_max, buf, C.byref(n)), "tree_gen_rank_prior")
    return [list(buf[i * K:(i + 1) * K]) for i in range(n.value)]


class Tree:
    """Owner of one ``mtv_tree_t`` (built by ``tree_build_static``)."""

    def __init__(self, K: int, node_ranks, upload: bool = True):
        flat = []
        for row in node_ranks:
            row = list(row)
            flat += row + [-1] * (K - len(row))
        n = len(flat) // K
        arr = (C.c_int32 * max(len(flat), 1))(*flat)
        h = C.c_void_p()
        _check(lib().tree_build_static(K, n, arr, 1 if upload else 0, C.byref(h)), "tree_build_static")
        self.handle = h
        info = TreeInfo()
        _check(lib().tree_query(h, C.byref(info)), "tree_query")
        self.info = info
        self.T, self.K, self.P, self.C = info.T, info.K, info.P, info.C
        self.k_d = list(info.k_d[:self.K])
        self.cand_offset = list(info.cand_offset[:self.K])
        T, K1 = self.T, self.K + 1
        self.node_ranks = [list(info.node_ranks[i * K:(i + 1) * K]) for i in range(T)]
        self.parent = list(info.parent[:T])
        self.depth = list(info.depth[:T])
        self.rank = list(info.rank[:T])
        self.tree_indices = list(info.tree_indices[:T])
        self.retrieve_indices = [list(info.retrieve_indices[p * K1:(p + 1) * K1]) for p in range(self.P)]
        self.anc = [[info.anc[i * info.anc_words + w] for w in range(info.anc_words)] for i in range(T)]
        self.medusa_attn_mask = [[info.medusa_attn_mask[i * T + j] for j in range(T)] for i in range(T)]

    def __del__(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.tree_destroy(self.handle)
            self.handle = None


def tree_build_static(K, node_ranks, upload=True) -> Tree:
    return Tree(K, node_ranks, upload)


def mtv_device_error(tree: Tree, clear: bool = True) -> int:
    code = C.c_int32(0)
    _check(lib().mtv_device_error(tree.handle, 1 if clear else 0, C.byref(code)), "mtv_device_error")
    return code.value


def mtv_debug_bounds_enabled() -> bool:
    return bool(lib().mtv_debug_bounds_enabled())


def mtv_selftest_wait_timeout(tree: Tree, stream=None):
    """Enqueue a kernel whose bounded wait must run out (about a second); see include/mtv.h."""
    _check(lib().mtv_selftest_wait_timeout(tree.handle, _stream(stream)), "mtv_selftest_wait_timeout")


def mtv_workspace_bytes(tree: Tree, B, H, V, Hq, Hkv, D, Lcap) -> int:
    return lib().mtv_workspace_bytes(tree.handle, B, H, V, Hq, Hkv, D, Lcap)


def _ws(ws):
    return C.c_void_p(ws.data_ptr()), ws.numel() * ws.element_size()


def medusa_heads_topk(tree, hidden, W1, b1, W2, root_tok, cand, cand_logit, tree_tok, ws, stream=None):
    B, H = hidden.shape
    V = W2.shape[1]
    p, n = _ws(ws)
    _check(lib().medusa_heads_topk(tree.handle, B, H, V, _ptr(hidden), _ptr(W1), _ptr(b1), _ptr(W2),
                                   _ptr(root_tok), _ptr(cand), _ptr(cand_logit), _ptr(tree_tok), p, n,
                                   _stream(stream)), "medusa_heads_topk")


def tree_verify_attention(tree, q, k_cache, v_cache, seq_lens, out, ws, scale=0.0, status=None, stream=None,
                          Lcap=None):
    B, T, Hq, D = q.shape
    Hkv = k_cache.shape[1]
    Lcap = k_cache.shape[2] if Lcap is None else Lcap
    sb, sh, st = k_cache.stride(0), k_cache.stride(1), k_cache.stride(2)
    assert (v_cache.stride(0), v_cache.stride(1), v_cache.stride(2)) == (sb, sh, st)
    p, n = _ws(ws)
    _check(lib().tree_verify_attention(tree.handle, B, Hq, Hkv, D, _ptr(q), _ptr(k_cache), _ptr(v_cache),
                                       sb, sh, st, Lcap, _ptr(seq_lens), scale, _ptr(out), _ptr(status), p, n,
                                       _stream(stream)), "tree_verify_attention")


def tree_kv_append_rope(tree, q, k_new, v_new, k_cache, v_cache, seq_lens, rope_theta=0.0, status=None, stream=None,
                        Lcap=None):
    B, T, Hq, D = q.shape
    Hkv = k_new.shape[2]
    Lcap = k_cache.shape[2] if Lcap is None else Lcap
    sb, sh, st = k_cache.stride(0), k_cache.stride(1), k_cache.stride(2)
    assert (v_cache.stride(0), v_cache.stride(1), v_cache.stride(2)) == (sb, sh, st)
    _check(lib().tree_kv_append_rope(tree.handle, B, Hq, Hkv, D, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_cache),
                                     _ptr(v_cache), sb, sh, st, Lcap, _ptr(seq_lens), rope_theta, _ptr(status),
                                     _stream(stream)), "tree_kv_append_rope")


def tree_kv_append_rope_layers(tree, q_layers, k_new_layers, v_new_layers, k_ptrs, v_ptrs, strides, Lcap, seq_lens,
                               rope_theta=0.0, status=None, stream=None):
    """q_layers [n_layers][B][T][Hq][D], k_new_layers / v_new_layers [n_layers][B][T][Hkv][D]; k_ptrs / v_ptrs as for
    kv_compact_accepted."""
    n_layers, B, T, Hq, D = q_layers.shape
    Hkv = k_new_layers.shape[3]
    sb, sh, st = strides
    _check(lib().tree_kv_append_rope_layers(tree.handle, B, Hq, Hkv, D, n_layers, _ptr(q_layers), _ptr(k_new_layers),
                                            _ptr(v_new_layers), _ptr(k_ptrs), _ptr(v_ptrs), sb, sh, st, Lcap,
                                            _ptr(seq_lens), rope_theta, _ptr(status), _stream(stream)),
           "tree_kv_append_rope_layers")


def tree_accept(tree, logits, tree_tok, accept_len, best_path, acc_nodes, acc_tok, next_root, ws, stream=None):
    B, T, V = logits.shape
    p, n = _ws(ws)
    _check(lib().tree_accept(tree.handle, B, V, _ptr(logits), _ptr(tree_tok), _ptr(accept_len), _ptr(best_path),
                             _ptr(acc_nodes), _ptr(acc_tok), _ptr(next_root), p, n, _stream(stream)),
           "tree_accept")


def lm_head_argmax(tree, x, W, keys, am=None, am_val=None, stream=None):
    """x [B][T][H], W [V][H] bf16; keys [B*T] int64 storage for the uint64 keys (see include/mtv.h)."""
    B, T, H = x.shape
    _check(lib().lm_head_argmax(tree.handle, B, H, W.shape[0], _ptr(x), _ptr(W),
                                _ptr(am), _ptr(am_val), _ptr(keys), _stream(stream)), "lm_head_argmax")


def tree_accept_keys(tree, B, keys, tree_tok, accept_len, best_path, acc_nodes, acc_tok, next_root, stream=None):
    _check(lib().tree_accept_keys(tree.handle, B, _ptr(keys), _ptr(tree_tok), _ptr(accept_len), _ptr(best_path),
                                  _ptr(acc_nodes), _ptr(acc_tok), _ptr(next_root), _stream(stream)),
           "tree_accept_keys")


def tree_accept_static_scratch(tree, logits, tree_tok, accept_len, best_path, acc_nodes, acc_tok, next_root,
                               stream=None):
    """tree_accept for callers that may not allocate: no workspace argument (see include/mtv.h)."""
    B, T, V = logits.shape
    rc = lib().tree_accept_static_scratch(tree.handle, B, V, _ptr(logits), _ptr(tree_tok), _ptr(accept_len),
                                          _ptr(best_path), _ptr(acc_nodes), _ptr(acc_tok), _ptr(next_root),
                                          _stream(stream))
    if rc == -3:    # too large for the built-in array: the library says by how much
        raise MtvError(rc, "tree_accept_static_scratch [%s]" % lib().mtv_last_error().decode())
    _check(rc, "tree_accept_static_scratch")


def tree_accept_static_scratch_capacity() -> int:
    return lib().tree_accept_static_scratch_capacity()


def cache_pointer_array(caches, device=None):
    """int64 tensor holding the device addresses of a list of cache tensors."""
    t = torch.tensor([c.data_ptr() for c in caches], dtype=torch.int64)
    return t.to(device) if device is not None else t


def kv_compact_accepted(tree, k_ptrs, v_ptrs, n_layers, B, Hkv, D, strides, Lcap, seq_lens, accept_len, acc_nodes,
                        status=None, stream=None):
    sb, sh, st = strides
    _check(lib().kv_compact_accepted(tree.handle, B, Hkv, D, n_layers, _ptr(k_ptrs), _ptr(v_ptrs), sb, sh, st,
                                     Lcap, _ptr(seq_lens), _ptr(accept_len), _ptr(acc_nodes), _ptr(status),
                                     _stream(stream)), "kv_compact_accepted")


def mtv_verify_step(tree, args: StepArgs, stream=None):
    _check(lib().mtv_verify_step(tree.handle, C.byref(args), _stream(stream)), "mtv_verify_step")


def heads_merge_shards(tree, v_slab, cand_shards, logit_shards, root_tok, cand, cand_logit, tree_tok, ws, stream=None):
    """cand_shards [n][B][C], logit_shards [n][B][C-1] (every rank's medusa_heads_topk results, gathered)."""
    n, B, _ = cand_shards.shape
    p, nbytes = _ws(ws)
    _check(lib().heads_merge_shards(tree.handle, B, n, v_slab, _ptr(cand_shards), _ptr(logit_shards), _ptr(root_tok),
                                    _ptr(cand), _ptr(cand_logit), _ptr(tree_tok), p, nbytes, _stream(stream)),
           "heads_merge_shards")


def attn_interleave_shards(gathered, out, stream=None):
    """gathered [n][B][T][Hq_local][D] -> out [B][T][n * Hq_local][D]."""
    n, B, T, Hl, D = gathered.shape
    _check(lib().attn_interleave_shards(B * T, n, Hl, D, _ptr(gathered), _ptr(out), _stream(stream)),
           "attn_interleave_shards")


def node_argmax_keys(tree, logits, keys, ws, stream=None):
    """logits [B][T][V] bf16 -> keys [B*T] (int64 storage of the uint64 keys)."""
    B, T, V = logits.shape
    p, n = _ws(ws)
    _check(lib().node_argmax_keys(tree.handle, B, V, _ptr(logits), _ptr(keys), p, n, _stream(stream)), "node_argmax_keys")


def keys_merge_shards(v_slab, key_shards, keys, stream=None):
    """key_shards [n][B*T] (int64 storage of the uint64 keys) -> keys [B*T]."""
    n, m = key_shards.shape
    _check(lib().keys_merge_shards(m, n, v_slab, _ptr(key_shards), _ptr(keys), _stream(stream)), "keys_merge_shards")


def mtv_verify_steps(tree, steps: Sequence[StepArgs], appends: Optional[Sequence[AppendArgs]] = None, stream=None):
    """A chain of steps on one stream (see include/mtv.h); `steps` and `appends` are sequences of the structs."""
    n = len(steps)
    arr = (StepArgs * n)(*steps)
    app = None
    if appends is not None:
        assert len(appends) == n
        app = (AppendArgs * n)(*appends)
    _check(lib().mtv_verify_steps(tree.handle, arr, app, n, _stream(stream)), "mtv_verify_steps")


def mtv_verify_step_host(tree, dev: StepArgs, host: StepArgs, stream=None):
    _check(lib().mtv_verify_step_host(tree.handle, C.byref(dev), C.byref(host), _stream(stream)),
           "mtv_verify_step_host")


KERNELS = ["heads_resblock", "heads_vocab_topk", "heads_merge", "attn_partial", "attn_combine",
           "argmax_partial", "accept_finish", "kv_compact", "seq_advance"]


class KernelTaps:
    """Per-kernel device timing through ``mtv_set_kernel_taps`` (CUDA events on the launch stream)."""

    def __init__(self, capacity_per_kernel: int):
        self.cap = capacity_per_kernel
        self.ev = {}
        for kid, name in enumerate(KERNELS):
            st = [torch.cuda.Event(enable_timing=True) for _ in range(self.cap)]
            sp = [torch.cuda.Event(enable_timing=True) for _ in range(self.cap)]
            for e in st + sp:
                e.record()          # torch creates the CUDA event lazily: force it now
            a = (C.c_void_p * self.cap)(*[e.cuda_event for e in st])
            b = (C.c_void_p * self.cap)(*[e.cuda_event for e in sp])
            self.ev[kid] = (st, sp, a, b)

    def __enter__(self):
        for kid, (_, _, a, b) in self.ev.items():
            _check(lib().mtv_set_kernel_taps(kid, a, b, self.cap), "mtv_set_kernel_taps")
        return self

    def __exit__(self, *exc):
        self.used = {kid: lib().mtv_kernel_taps_used(kid) for kid in self.ev}
        for kid in self.ev:
            lib().mtv_set_kernel_taps(kid, None, None, 0)

    def times_ms(self):
        """{kernel name: [ms per recorded launch]} — call after a device synchronize."""
        out = {}
        for kid, (st, sp, _, _) in self.ev.items():
            n = self.used[kid]
            out[KERNELS[kid]] = [st[i].elapsed_time(sp[i]) for i in range(n)]
        return out
