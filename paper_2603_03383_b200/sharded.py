"""One sequence's verification step split over the ranks of a ``torch.distributed`` group.

The paper runs on one device; this split follows its structure.  The Medusa heads (Section 3.1) are independent
over the vocabulary: rank r projects onto the slab ``[r * v_slab, min(V, (r + 1) * v_slab))`` of every head's
``W2`` (``W1`` is replicated: it is 3 % of the heads' bytes) and keeps its own top-k lists.  The tree attention
(Section 3.2) is independent over KV heads: rank r holds the cache of KV heads ``[r * Hkv / n, (r + 1) * Hkv / n)``
and attends with their ``Hq / n`` query heads.  After each of the two, one all-gather brings every rank's result
into a LOCAL buffer and a small kernel of the library merges the pieces (``heads_merge_shards``: same candidate
order as on one device, so identical ids; ``attn_interleave_shards``; ``keys_merge_shards`` for the fused LM
head and for the acceptance over vocabulary slabs of stored logits).  No kernel is ever handed another GPU's memory; the collective is the group's backend (NCCL on GPUs).

This module holds the partition arithmetic and the collectives only; every step of the path itself runs in the
library's kernels through ``binding``.  Everything is enqueued on the current torch stream (the collectives of
``torch.distributed`` order themselves against that stream)."""
from __future__ import annotations

import dataclasses
from typing import Optional

import torch
import torch.distributed as dist

from . import binding


@dataclasses.dataclass(frozen=True)
class ShardPlan:
    rank: int
    world: int
    V: int
    v_slab: int       # rows of a full slab; slab r covers [r * v_slab, min(V, (r + 1) * v_slab))
    v_lo: int
    v_hi: int
    Hq: int
    Hkv: int
    hq_local: int
    hkv_local: int
    q_lo: int         # first query head of this rank
    kv_lo: int        # first KV head of this rank

    @property
    def v_local(self) -> int:
        return self.v_hi - self.v_lo


def plan(rank: int, world: int, V: int, Hq: int, Hkv: int, max_kd: int = 1, slab_multiple: int = 8) -> ShardPlan:
    """Partition of the vocabulary (slabs of equal size, rounded up to `slab_multiple` rows, the last one ragged) and of
    the heads (equal counts: `world` must divide Hkv).  Every slab must hold at least `max_kd` rows."""
    if not (0 <= rank < world):
        raise ValueError("rank %d outside a group of %d" % (rank, world))
    if world > 16:
        raise ValueError("at most 16 shards (the merge kernels' limit)")
    if Hkv % world or Hq % Hkv:
        raise ValueError("the group size %d must divide the %d KV heads (and Hkv must divide Hq)" % (world, Hkv))
    v_slab = -(-V // world)
    v_slab = -(-v_slab // slab_multiple) * slab_multiple
    v_lo, v_hi = min(V, rank * v_slab), min(V, (rank + 1) * v_slab)
    last = V - (world - 1) * v_slab
    if last < max_kd:
        raise ValueError("the last vocabulary slab would hold %d rows, fewer than the largest top-k %d" % (last, max_kd))
    g = Hq // Hkv
    hkv_local = Hkv // world
    return ShardPlan(rank, world, V, v_slab, v_lo, v_hi, Hq, Hkv, hkv_local * g, hkv_local, rank * hkv_local * g,
                     rank * hkv_local)


class Scratch:
    """Buffers of the calls below, allocated on first use and reused (a hot loop then allocates nothing)."""

    def __init__(self):
        self._bufs = {}

    def get(self, name, shape, dtype, device):
        key = (name, tuple(shape), dtype, str(device))
        buf = self._bufs.get(key)
        if buf is None:
            buf = self._bufs[key] = torch.empty(tuple(shape), dtype=dtype, device=device)
        return buf


_default_scratch = Scratch()


def gather(t: torch.Tensor, world: int, group=None, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """All ranks' `t` (same shape everywhere) as one local tensor ``[world, *t.shape]``."""
    t = t.contiguous()
    if out is None:
        out = t.new_empty((world,) + tuple(t.shape))
    if world == 1 and not dist.is_initialized():
        out[0].copy_(t)
        return out
    dist.all_gather_into_tensor(out.view(-1), t.view(-1), group=group)     # rank r's elements land in out[r]
    return out


def medusa_heads_topk_sharded(tree, p: ShardPlan, hidden, W1, b1, W2_slab, root_tok, cand, cand_logit, tree_tok, ws,
                              group=None, scratch: Optional[Scratch] = None):
    """W2_slab [K][v_local][H]: this rank's rows of every head.  cand, cand_logit, tree_tok as medusa_heads_topk
    on the whole vocabulary writes them (identical on every rank)."""
    B, dev = hidden.shape[0], hidden.device
    sc = scratch or _default_scratch
    assert W2_slab.shape[1] == p.v_local
    cand_l = sc.get("cand_l", (B, tree.C), torch.int32, dev)
    logit_l = sc.get("logit_l", (B, tree.C - 1), torch.float32, dev)
    tt_l = sc.get("tt_l", (B, tree.T), torch.int32, dev)
    binding.medusa_heads_topk(tree, hidden, W1, b1, W2_slab, root_tok, cand_l, logit_l, tt_l, ws)
    cand_all = gather(cand_l, p.world, group, sc.get("cand_all", (p.world, B, tree.C), torch.int32, dev))
    logit_all = gather(logit_l, p.world, group, sc.get("logit_all", (p.world, B, tree.C - 1), torch.float32, dev))
    binding.heads_merge_shards(tree, p.v_slab, cand_all, logit_all, root_tok, cand, cand_logit, tree_tok, ws)


def tree_verify_attention_sharded(tree, p: ShardPlan, q_local, k_local, v_local, seq_lens, out, ws, scale=0.0,
                                  status=None, group=None, Lcap=None, scratch: Optional[Scratch] = None):
    """q_local [B][T][hq_local][D], k_local / v_local [B][hkv_local][Lcap][D]: this rank's heads.  out
    [B][T][Hq][D]: all heads, identical on every rank."""
    sc = scratch or _default_scratch
    out_l = sc.get("out_l", q_local.shape, q_local.dtype, q_local.device)
    binding.tree_verify_attention(tree, q_local, k_local, v_local, seq_lens, out_l, ws, scale=scale, status=status,
                                  Lcap=Lcap)
    gathered = sc.get("out_all", (p.world,) + tuple(q_local.shape), q_local.dtype, q_local.device)
    binding.attn_interleave_shards(gather(out_l, p.world, group, gathered), out)


def lm_head_argmax_sharded(tree, p: ShardPlan, x, W_slab, keys, group=None, scratch: Optional[Scratch] = None):
    """W_slab [v_local][H]: this rank's rows of the LM head.  keys [B*T]: the input of tree_accept_keys."""
    sc = scratch or _default_scratch
    keys_l = sc.get("keys_l", keys.shape, keys.dtype, keys.device)
    binding.lm_head_argmax(tree, x, W_slab, keys_l)
    keys_all = sc.get("keys_all", (p.world,) + tuple(keys.shape), keys.dtype, keys.device)
    binding.keys_merge_shards(p.v_slab, gather(keys_l, p.world, group, keys_all), keys)


def tree_accept_sharded(tree, p: ShardPlan, logits_slab, tree_tok, accept_len, best_path, acc_nodes, acc_tok, next_root, ws,
                        group=None, scratch: Optional[Scratch] = None):
    """logits_slab [B][T][v_local]: this rank's vocabulary slab of the base-model logits (contiguous).  Per-node argmax
    of the slab, one all-gather of the (maximum, id) keys, the maximum over the ranks with the slab offsets folded in
    (ties to the lowest global id), then the ordinary path scan: identical outputs on every rank."""
    B, T, _ = logits_slab.shape
    sc, dev = scratch or _default_scratch, logits_slab.device
    keys_l = sc.get("akeys_l", (B * T,), torch.int64, dev)
    binding.node_argmax_keys(tree, logits_slab, keys_l, ws)
    keys = sc.get("akeys", (B * T,), torch.int64, dev)
    keys_all = sc.get("akeys_all", (p.world, B * T), torch.int64, dev)
    binding.keys_merge_shards(p.v_slab, gather(keys_l, p.world, group, keys_all), keys)
    binding.tree_accept_keys(tree, B, keys, tree_tok, accept_len, best_path, acc_nodes, acc_tok, next_root)
