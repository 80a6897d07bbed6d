"""GPU parity of the fused LM-head projection + per-node argmax and of the acceptance that reads its keys."""
import pytest
import torch

from oracle import reference as ref
from paper_2603_03383_b200 import binding, synth
from tests._cases import make_tree

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _run(tree, x, W):
    B, T, H = x.shape
    M = B * T
    keys = torch.full((M,), -1, dtype=torch.int64, device=DEV)
    am = torch.full((M,), -7, dtype=torch.int32, device=DEV)
    val = torch.zeros(M, dtype=torch.float32, device=DEV)
    binding.lm_head_argmax(tree, x.to(DEV), W.to(DEV), keys, am, val)
    torch.cuda.synchronize()
    assert binding.mtv_device_error(tree) == 0
    return keys, am.cpu(), val.cpu()


def _check(x, W, am, val):
    """Index bit-exact where the fp64 maximum is decisive; elsewhere the chosen token must be a maximum within
    the accumulation error of fp32 sums.  Values within max|err| <= 1e-2 max|ref| + 1e-3."""
    M = am.numel()
    x2 = x.reshape(M, -1)
    want, zmax, z2 = ref.lm_head_argmax(x2, W)
    scale = zmax.abs().max().item()
    tol = 1e-4 * scale + 1e-6
    decisive = (zmax - z2) > tol
    assert torch.equal(am[decisive], want[decisive])
    assert decisive.float().mean() > 0.9
    for m in torch.nonzero(~decisive).flatten().tolist():
        z = (x2[m].double() * W[am[m].item()].double()).sum().item()
        assert z >= zmax[m].item() - tol
    assert (val.double() - zmax).abs().max().item() <= 1e-2 * scale + 1e-3
    return want


LM_CASES = [
    # B, tree (kind, K, topk, T), H, V
    (1, ("cartesian", 3, (4, 2, 2), 0), 512, 1024),        # 29 nodes: one partial pass of 64
    (1, ("rank_prior", 4, (), 64), 256, 3001),             # ragged vocabulary tail
    (2, ("rank_prior", 4, (), 64), 192, 2048),             # exactly 128 nodes
    (5, ("rank_prior", 4, (), 64), 128, 777),              # 320 nodes: three passes, the last one partial
    (3, ("cartesian", 1, (2,), 0), 64, 50),                # fewer vocabulary rows than one tile
    (1, ("rank_prior", 5, (), 128), 1024, 40000),          # more tile pairs than SMs
    (3, ("rank_prior", 4, (), 64), 256, 3001),             # 192 nodes: one partial pass of 256
    (9, ("rank_prior", 4, (), 64), 128, 20000),            # 576 nodes: three passes of 256, the last one partial
]


@pytest.mark.parametrize("B,tr,H,V", LM_CASES)
def test_lm_head_argmax(B, tr, H, V):
    tb, tree = make_tree(tr[0], tr[1], tr[2], tr[3])
    x = synth.normal_bf16(11, B + H, (B, tree.T, H))
    W = synth.normal_bf16(11, 1000 + V, (V, H))
    keys, am, val = _run(tree, x, W)
    _check(x, W, am, val)
    assert torch.equal((0xffffffff - (keys.cpu() & 0xffffffff)).to(torch.int32), am)


def test_lm_head_exact_ties_take_the_lowest_index():
    tb, tree = make_tree("rank_prior", 4, (), 64)
    H, V = 256, 5000
    W = synth.normal_bf16(12, 1, (V, H), scale=0.25)
    x = synth.normal_bf16(12, 2, (1, tree.T, H), scale=0.25)
    twins = [(7, 4999), (130, 131), (255, 256), (1000, 3000)]
    for m, (lo, hi) in enumerate(twins):
        W[hi] = W[lo]                                        # identical rows: identical fp32 sums
        x[0, m] = W[lo]                                      # ... and by far the largest at node m
    W[4000] = 0
    x[0, 10] = 0                                             # all logits zero: token 0
    keys, am, val = _run(tree, x, W)
    want = _check(x, W, am, val)
    for m, (lo, hi) in enumerate(twins):
        assert am[m].item() == lo == want[m].item()
    assert am[10].item() == 0 and val[10].item() == 0.0


def test_accept_from_lm_head_keys():
    B, H, V, K = 3, 256, 4096, 4
    tb, tree = make_tree("rank_prior", K, (), 64)
    T = tree.T
    g = torch.Generator().manual_seed(5)
    cand = torch.stack([torch.randperm(V, generator=g)[:tb["C"]] for _ in range(B)]).to(torch.int32)
    tree_tok = cand[:, torch.tensor(tb["tree_indices"])].contiguous()
    W = synth.normal_bf16(13, 1, (V, H))
    # the model's next token at node i: with probability 0.7 the token of i's first child (so that paths
    # get accepted), else a random one; x = the target's weight row plus noise makes it the argmax
    target = torch.randint(0, V, (B, T), generator=g)
    parent = tb["parent"]
    for i in range(1, T):
        if tb["rank"][i] == 0:
            take = torch.rand(B, generator=g) < 0.7
            target[take, parent[i]] = tree_tok[take, i].long()
    x = (W[target.flatten()].float().reshape(B, T, H) + 0.3 * torch.randn(B, T, H, generator=g)).to(torch.bfloat16)
    keys, am, val = _run(tree, x, W)
    want_am = _check(x, W, am, val)
    assert torch.equal(want_am.long(), target.flatten())
    want = ref.tree_accept(want_am.reshape(B, T), tree_tok, tb)
    assert want["accept_len"].max().item() >= 1
    outs = dict(accept_len=None, best_path=None, next_root=None)
    outs = {n: torch.full((B,), -7, dtype=torch.int32, device=DEV) for n in outs}
    outs["acc_nodes"] = torch.full((B, K + 1), -7, dtype=torch.int32, device=DEV)
    outs["acc_tok"] = torch.full((B, K + 1), -7, dtype=torch.int32, device=DEV)
    binding.tree_accept_keys(tree, B, keys, tree_tok.to(DEV), outs["accept_len"], outs["best_path"],
                             outs["acc_nodes"], outs["acc_tok"], outs["next_root"])
    torch.cuda.synchronize()
    for name, t in outs.items():
        assert torch.equal(t.cpu(), want[name]), name


@pytest.mark.parametrize("V", [32000, 131072])
def test_lm_head_full_size_7b(V):
    """64 nodes, H = 4096; V = 131072 is the vocabulary the step benchmark runs, V = 32000 one whose tiling has a
    ragged last slab."""
    tb, tree = make_tree("rank_prior", 4, (), 64)
    H = 4096
    x = synth.normal_bf16(14, 1, (1, tree.T, H))
    W = synth.normal_bf16(14, 2, (V, H), scale=0.02)
    keys, am, val = _run(tree, x, W)
    if V > 100000:      # the checker on every fourth node (its fp64 product over the whole vocabulary takes a second per node)
        sel = torch.arange(0, tree.T, 4)
        _check(x[:, sel], W, am[sel], val[sel])
    else:
        _check(x, W, am, val)
    keys2, am2, val2 = _run(tree, x, W)
    assert torch.equal(keys, keys2)                          # bitwise repeatable
