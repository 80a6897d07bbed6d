"""Helpers shared by the GPU parity tests: build the same tree on both sides, run the
checker on CPU tensors and the library on CUDA tensors."""
import torch

from oracle import reference as ref
from oracle import tree as otree
from paper_2603_03383_b200 import binding, synth

FLOAT_RTOL, FLOAT_ATOL = 1e-2, 1e-3          # max|err| <= 1e-2 * max|ref| + 1e-3
MARGIN = 1e-5                                 # seeds whose rank gaps fall below MARGIN * max|z| are rejected


def make_tree(kind, K, topk=(), T=0):
    nodes = otree.cartesian(topk) if kind == "cartesian" else otree.rank_prior(K, T)
    tb = otree.tables(nodes, K)
    tree = binding.tree_build_static(K, [list(n) for n in nodes], upload=True)
    assert tree.T == tb["T"] and tree.retrieve_indices == tb["retrieve"]
    return tb, tree


def workload_tree(w):
    return make_tree(w.tree, w.K, w.topk, w.T)


def assert_close(got, want, what=""):
    got, want = got.double().cpu(), want.double().cpu()
    err = (got - want).abs().max().item()
    bound = FLOAT_RTOL * want.abs().max().item() + FLOAT_ATOL
    assert err <= bound, "%s: max|err| %.3e > %.3e" % (what, err, bound)
    return err


def workspace(tree, B, H, V, Hq, Hkv, D, Lcap):
    n = binding.mtv_workspace_bytes(tree, B, H, V, Hq, Hkv, D, Lcap)
    assert n > 0
    return torch.empty(n, dtype=torch.uint8, device="cuda")


def oracle_heads_with_margin(B, H, V, K, tb, seed, bias=True, rows=None, device="cpu"):
    """Run the checker's heads; bump the seed (+1000) until every rank gap clears the margin.

    Inputs are generated on `device` (bit-identical on every device) and handed to the
    checker as CPU tensors.  rows: optional subset of batch rows to check.
    Returns (seed, inputs on CPU, cand, cand_logit, tree_tok) — the last three for `rows`.
    """
    for attempt in range(20):
        inp = synth.head_inputs(B, H, V, K, seed, device=device, bias=bias)
        cpu = [None if t is None else t.cpu() for t in inp]
        hidden, W1, b1, W2, root = cpu
        sel = list(range(B)) if rows is None else rows
        z = ref.heads_logits(hidden[sel], W1, b1, W2)
        cand, cl, tree_tok, gap = ref.heads_candidates(z, root[sel], tb)
        if gap > MARGIN * z.abs().max().item():
            return seed, inp, cpu, cand, cl, tree_tok
        seed += 1000
    raise AssertionError("no seed cleared the margin")
