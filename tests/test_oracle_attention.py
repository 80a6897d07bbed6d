"""Pins for the checker's masked tree attention (Section 3.2, Fig. 2(b))."""
import pytest
import torch
import torch.nn.functional as F

from oracle import reference as ref
from oracle import tree
from paper_2603_03383_b200 import synth


def _setup(tb, B, Hq, Hkv, D, lens, seed, Lcap=None):
    T = tb["T"]
    Lcap = Lcap or max(lens) + T + 3
    q, k, v = synth.attention_inputs(B, T, Hq, Hkv, D, Lcap, seed)
    return q, k, v, torch.tensor(lens, dtype=torch.int32)


def _path(tb, i):
    p = []
    while i >= 0:
        p.append(i)
        i = tb["parent"][i]
    return p[::-1]


@pytest.mark.parametrize("name,B,Hq,Hkv,D,lens", [
    ("cart", 2, 4, 2, 16, [5, 0]),
    ("prior", 1, 8, 2, 32, [37]),
    ("chain", 1, 2, 1, 8, [3]),
])
def test_equals_causal_attention_over_prefix_plus_path(name, B, Hq, Hkv, D, lens):
    """Each node's output == ordinary single-query attention (library routine) over the
    dense sequence [prefix K/V ; K/V of the nodes on the root-to-node path]."""
    nodes, K = {"cart": (tree.cartesian((3, 2, 2)), 3), "prior": (tree.rank_prior(4, 40), 4),
                "chain": ([(0,), (0, 0), (0, 0, 0)], 3)}[name]
    tb = tree.tables(nodes, K)
    q, k, v, sl = _setup(tb, B, Hq, Hkv, D, lens, seed=21)
    out = ref.tree_attention(q, k, v, sl, tb["mask"])
    G = Hq // Hkv
    for b in range(B):
        L = lens[b]
        for i in range(tb["T"]):
            slots = list(range(L)) + [L + a for a in _path(tb, i)]
            for h in range(Hq):
                kk = k[b, h // G, slots].double()[None, None]
                vv = v[b, h // G, slots].double()[None, None]
                qq = q[b, i, h].double()[None, None, None]
                want = F.scaled_dot_product_attention(qq, kk, vv)[0, 0, 0]
                assert torch.allclose(out[b, i, h], want, rtol=0, atol=1e-12), (b, i, h)


def test_root_only_tree_is_plain_decode_attention():
    tb = tree.tables([], 1)
    assert tb["T"] == 1
    q, k, v, sl = _setup(tb, 2, 4, 4, 16, [9, 4], seed=2)
    out = ref.tree_attention(q, k, v, sl, tb["mask"])
    for b, L in enumerate([9, 4]):
        kk = k[b, :, :L + 1].double()[None]
        vv = v[b, :, :L + 1].double()[None]
        qq = q[b, 0].double()[None, :, None, :]
        want = F.scaled_dot_product_attention(qq, kk, vv)[0, :, 0]
        assert torch.allclose(out[b, 0], want, rtol=0, atol=1e-12)


def test_empty_prefix_root_returns_its_own_value():
    tb = tree.tables(tree.cartesian((2, 2)), 2)
    q, k, v, sl = _setup(tb, 1, 2, 1, 8, [0], seed=4)
    out = ref.tree_attention(q, k, v, sl, tb["mask"])
    assert torch.equal(out[0, 0, 0], v[0, 0, 0].double())
    assert torch.equal(out[0, 0, 1], v[0, 0, 0].double())


def test_equal_keys_give_mean_of_visible_values():
    tb = tree.tables(tree.cartesian((2, 2)), 2)
    L = 6
    q, k, v, sl = _setup(tb, 1, 2, 2, 8, [L], seed=6)
    k[:] = k[0, 0, 0]                                   # every key identical -> uniform weights
    out = ref.tree_attention(q, k, v, sl, tb["mask"])
    for i in range(tb["T"]):
        slots = list(range(L)) + [L + a for a in _path(tb, i)]
        for h in range(2):
            want = v[0, h, slots].double().mean(0)
            assert torch.allclose(out[0, i, h], want, rtol=0, atol=1e-13)


def test_weights_sum_to_one_and_scale_is_used():
    tb = tree.tables(tree.cartesian((2,)), 1)
    q, k, v, sl = _setup(tb, 1, 1, 1, 8, [5], seed=8)
    ones = torch.ones_like(v)
    out = ref.tree_attention(q, k, ones, sl, tb["mask"])
    assert torch.allclose(out, torch.ones_like(out), rtol=0, atol=1e-14)
    a = ref.tree_attention(q, k, v, sl, tb["mask"], scale=0.5)
    b = ref.tree_attention(q, k, v, sl, tb["mask"])     # default 1/sqrt(D)
    assert not torch.allclose(a, b, atol=1e-3)
    kk, vv = k[0, 0, :6].double(), v[0, 0, :6].double()
    w = torch.softmax(0.5 * (kk @ q[0, 0, 0].double()), 0)
    assert torch.allclose(a[0, 0, 0], w @ vv, rtol=0, atol=1e-13)


def test_strided_cache_and_row_list():
    tb = tree.tables(tree.cartesian((2, 2)), 2)
    T, B, Hq, Hkv, D = tb["T"], 2, 4, 2, 16
    Lcap = 20
    q, k, v, sl = _setup(tb, B, Hq, Hkv, D, [7, 11], seed=10, Lcap=Lcap)
    big_k = torch.zeros(B, Hkv, Lcap + 5, D, dtype=torch.bfloat16)
    big_v = torch.zeros_like(big_k)
    big_k[:, :, :Lcap] = k
    big_v[:, :, :Lcap] = v
    full = ref.tree_attention(q, k, v, sl, tb["mask"])
    strided = ref.tree_attention(q, big_k[:, :, :Lcap], big_v[:, :, :Lcap], sl, tb["mask"])
    assert torch.equal(full, strided)
    rows = [(1, 3, 2), (0, 0, 0), (1, T - 1, 3)]
    some = ref.tree_attention(q, k, v, sl, tb["mask"], rows=rows)
    for r, (b, i, h) in enumerate(rows):
        assert torch.equal(some[r], full[b, i, h])
