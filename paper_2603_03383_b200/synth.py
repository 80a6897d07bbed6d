"""Seeded synthetic inputs for the static-tree verification path.

This module only produces *inputs* (hidden states, weights, Q/K/V, base-model
logits, prefix lengths).  It holds none of the method's arithmetic: no head
forward, no top-k, no attention, no acceptance rule.  Both the CUDA path and
the CPU checker are fed from here, and neither is imported here.

Generator
---------
Counter-based and device-independent: element ``i`` of tensor ``tid`` under
``seed`` is a pure function of ``(seed, tid, i)`` evaluated with wrapping
64-bit integer arithmetic only, so a CPU tensor and a CUDA tensor built from
the same arguments are bit-identical.

* three SplitMix64-style hashes give twelve 16-bit uniform fields ``u_j``;
* ``z = (2*sum(u_j) - 12*65535) / 131072`` is an Irwin-Hall(12) variate:
  mean 0, variance 1 - 2**-32, support (-6, 6), exact in fp32 (the integer
  numerator is below 2**24);
* the value is ``bf16_rne(fp32(z) * fp32(scale))`` (one IEEE multiply, one
  round-to-nearest-even conversion: the same on every device).

It stands in for the N(0,1) draws of the workloads' recipe.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Sequence

import torch

_GAMMA = -7046029254386353131  # 0x9E3779B97F4A7C15 as a signed 64-bit value
_M1 = -4658895280553007687     # 0xBF58476D1CE4E5B9
_M2 = -7723592293110705685     # 0x94D049BB133111EB

BASE_SEED = 260303383000


def _lsr(x: torch.Tensor, n: int) -> torch.Tensor:
    """Logical shift right of an int64 tensor."""
    return (x >> n) & ((1 << (64 - n)) - 1)


def _mix(x: torch.Tensor) -> torch.Tensor:
    x = (x ^ _lsr(x, 30)) * _M1
    x = (x ^ _lsr(x, 27)) * _M2
    return x ^ _lsr(x, 31)


def _wrap64(v: int) -> int:
    v &= (1 << 64) - 1
    return v - (1 << 64) if v >= (1 << 63) else v


def _key(seed: int, tid: int) -> int:
    return _wrap64(seed * 0x2545F4914F6CDD1D + (tid + 1) * 0x9E3779B97F4A7C15 * 0x10001)


def hash_u64(seed: int, tid: int, idx: torch.Tensor, lane: int = 0, lanes: int = 1) -> torch.Tensor:
    """64 hashed bits per counter ``lanes*idx + lane`` (int64 tensor, wrapping)."""
    c = idx * lanes + lane
    return _mix(c * _GAMMA + _key(seed, tid))


def normal_f32(seed: int, tid: int, start: int, count: int, device="cpu") -> torch.Tensor:
    """``count`` Irwin-Hall(12) variates for flat indices ``start..start+count``."""
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    s = torch.zeros(count, dtype=torch.int64, device=device)
    for lane in range(3):
        h = hash_u64(seed, tid, idx, lane, 3)
        for sh in (0, 16, 32, 48):
            s += (h >> sh) & 0xFFFF
    return (2 * s - 12 * 65535).to(torch.float32) / 131072.0


def normal_bf16(seed: int, tid: int, shape: Sequence[int], scale: float = 1.0,
                device="cpu", chunk: int = 1 << 24) -> torch.Tensor:
    """bf16 tensor of ``shape`` with entries ~ scale * N(0,1) (see module doc)."""
    n = 1
    for d in shape:
        n *= int(d)
    out = torch.empty(n, dtype=torch.bfloat16, device=device)
    sc = torch.tensor(scale, dtype=torch.float32, device=device)
    for s0 in range(0, n, chunk):
        c = min(chunk, n - s0)
        out[s0:s0 + c] = (normal_f32(seed, tid, s0, c, device) * sc).to(torch.bfloat16)
    return out.view(*shape)


def uniform_int(seed: int, tid: int, count: int, lo: int, hi: int, device="cpu") -> torch.Tensor:
    """``count`` integers in [lo, hi] (inclusive), int64."""
    idx = torch.arange(count, dtype=torch.int64, device=device)
    h = _lsr(hash_u64(seed, tid, idx), 11)  # 53 uniform bits, non-negative
    return lo + h % (hi - lo + 1)


def uniform_unit(seed: int, tid: int, count: int) -> List[float]:
    """``count`` floats in [0,1) as a Python list (CPU; for the planting walk)."""
    idx = torch.arange(count, dtype=torch.int64)
    h = _lsr(hash_u64(seed, tid, idx), 11)
    return [int(v) / float(1 << 53) for v in h.tolist()]


# tensor ids
TID_HIDDEN, TID_W1, TID_B1, TID_W2, TID_ROOT, TID_SEQ, TID_LOGITS, TID_WALK = range(8)
TID_Q, TID_K, TID_V = 100, 200, 300  # + layer


@dataclasses.dataclass(frozen=True)
class Workload:
    """Shapes of one benchmark configuration (H hidden size, V vocabulary, K heads, T tree nodes, L prefix length, Hq/Hkv query and KV heads, D head size)."""
    name: str
    cfg_id: int
    B: int
    L_lo: int
    L_hi: int           # prefix lengths uniform in [L_lo, L_hi]
    H: int
    Hq: int
    Hkv: int
    D: int
    V: int
    K: int
    tree: str           # "cartesian" | "rank_prior"
    topk: Sequence[int] = ()   # cartesian: top-k per depth
    T: int = 0          # rank_prior: total nodes including the root
    R_max: int = 10
    p_accept: Sequence[float] = (0.6,)

    @property
    def seed(self) -> int:
        return BASE_SEED + self.cfg_id


WORKLOADS = {
    "tiny": Workload("tiny", 1, 1, 128, 128, 512, 8, 2, 64, 1024, 3, "cartesian", (4, 2, 2), 29),
    "short": Workload("short", 2, 1, 512, 512, 4096, 32, 8, 128, 131072, 4, "rank_prior", (), 64),
    "long": Workload("long", 3, 1, 8192, 8192, 4096, 32, 8, 128, 131072, 4, "rank_prior", (), 64),
    "batched": Workload("batched", 4, 16, 1024, 4096, 4096, 32, 8, 128, 131072, 4, "rank_prior", (), 64,
                        p_accept=(0.3, 0.6, 0.9)),
    "stress": Workload("stress", 5, 4, 32768, 32768, 4096, 32, 8, 128, 131072, 5, "rank_prior", (), 128),
}


def seq_lens(w: Workload, seed: Optional[int] = None) -> torch.Tensor:
    seed = w.seed if seed is None else seed
    if w.L_lo == w.L_hi:
        return torch.full((w.B,), w.L_lo, dtype=torch.int32)
    return uniform_int(seed, TID_SEQ, w.B, w.L_lo, w.L_hi).to(torch.int32)


def head_inputs(B, H, V, K, seed, device="cpu", bias=True):
    """hidden [B,H], W1 [K,H,H], b1 [K,H], W2 [K,V,H], root_tok [B] (int32)."""
    hidden = normal_bf16(seed, TID_HIDDEN, (B, H), 1.0, device)
    W1 = normal_bf16(seed, TID_W1, (K, H, H), 1.0 / math.sqrt(H), device)
    b1 = normal_bf16(seed, TID_B1, (K, H), 0.1, device) if bias else None
    W2 = normal_bf16(seed, TID_W2, (K, V, H), 1.0 / math.sqrt(H), device)
    root = uniform_int(seed, TID_ROOT, B, 0, V - 1, device).to(torch.int32)
    return hidden, W1, b1, W2, root


def attention_inputs(B, T, Hq, Hkv, D, Lcap, seed, layer=0, device="cpu"):
    """q [B,T,Hq,D]; k_cache, v_cache [B,Hkv,Lcap,D]: every slot filled ~N(0,1).

    The caller's prefix occupies slots [0, L_b) and the tree nodes' K/V slots
    [L_b, L_b+T); slots beyond are filled too so that a kernel reading past
    the valid range shows up as an error instead of reading zeros.
    """
    q = normal_bf16(seed, TID_Q + layer, (B, T, Hq, D), 1.0, device)
    k = normal_bf16(seed, TID_K + layer, (B, Hkv, Lcap, D), 1.0, device)
    v = normal_bf16(seed, TID_V + layer, (B, Hkv, Lcap, D), 1.0, device)
    return q, k, v


def planted_logits(B, T, V, K, tree_tok, parent, rank, seed, p_accept=(0.6,), device="cpu"):
    """Base-model logits [B,T,V] bf16 ~N(0,1) with a planted greedy walk.

    Per sequence: start at the root; at a node with children draw
    Bernoulli(p_b).  Success: choose a child with probability proportional to
    1/(rank+1) and set the logit of that child's token at this node to 16.0.
    Failure (or a leaf): set 16.0 on the lowest token id that is not a child's
    token, and stop.  Returns (logits, planted_len [B] int32) where
    ``planted_len[b]`` is the number of successful draws.

    ``tree_tok`` [B,T], ``parent`` [T] and ``rank`` [T] are data supplied by
    the caller (host lists / CPU tensors); this function only places values.
    """
    logits = normal_bf16(seed, TID_LOGITS, (B, T, V), 1.0, device)
    tt = torch.as_tensor(tree_tok).cpu().tolist()
    parent = list(parent)
    rank = list(rank)
    children = [[] for _ in range(T)]
    for i in range(1, T):
        children[parent[i]].append(i)
    u = uniform_unit(seed, TID_WALK, B * 2 * (K + 1))
    planted = []
    for b in range(B):
        p = p_accept[b % len(p_accept)]
        node, n_ok = 0, 0
        for step in range(K + 1):
            ch = children[node]
            u_acc, u_pick = u[(b * (K + 1) + step) * 2], u[(b * (K + 1) + step) * 2 + 1]
            if ch and u_acc < p:
                wts = [1.0 / (rank[c] + 1) for c in ch]
                tot = sum(wts)
                acc, pick = 0.0, ch[-1]
                for c, wgt in zip(ch, wts):
                    acc += wgt / tot
                    if u_pick < acc:
                        pick = c
                        break
                logits[b, node, tt[b][pick]] = 16.0
                node = pick
                n_ok += 1
            else:
                taken = {tt[b][c] for c in ch}
                tok = 0
                while tok in taken:
                    tok += 1
                logits[b, node, tok] = 16.0
                break
        planted.append(n_ok)
    return logits, torch.tensor(planted, dtype=torch.int32)
