"""CPU-side checks of the CUDA library: it loads, exports the declared C ABI, and its host
logic (static tree tensors, generators, argument validation) agrees with the checker."""
import ctypes as C
import os
import re

import pytest

from oracle import tree as otree
from paper_2603_03383_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def test_exports_every_declared_symbol():
    text = open(os.path.join(ROOT, "include", "mtv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"^\s*(?:const\s+)?(?:int|void|size_t|char)\s*\*?\s*(\w+)\s*\(", text, flags=re.M)
    assert set(names) == set(binding.EXPORTS), sorted(set(names) ^ set(binding.EXPORTS))
    lib = binding.lib()
    for n in names:
        assert hasattr(lib, n), n


def _same_tables(t, tb):
    assert (t.T, t.K, t.P, t.C) == (tb["T"], tb["K"], tb["P"], tb["C"])
    assert t.k_d == tb["k_d"] and t.cand_offset == tb["offset"]
    assert t.parent == tb["parent"] and t.depth == tb["depth"] and t.rank == tb["rank"]
    assert t.tree_indices == tb["tree_indices"]
    assert t.retrieve_indices == tb["retrieve"]
    assert t.medusa_attn_mask == tb["mask"]
    for i in range(t.T):
        bits = sum(w << (64 * j) for j, w in enumerate(t.anc[i]))
        assert [(bits >> j) & 1 for j in range(t.T)] == tb["mask"][i]
        assert [r for r in t.node_ranks[i] if r >= 0] == list(tb["nodes"][i])


@pytest.mark.parametrize("K,T", [(4, 64), (4, 65), (5, 128), (3, 20), (1, 5), (2, 2)])
def test_rank_prior_tree_matches_checker(K, T):
    nodes = binding.tree_gen_rank_prior(K, T)
    want = otree.rank_prior(K, T)
    assert [tuple(r for r in n if r >= 0) for n in nodes] == want      # same nodes, same admission order
    _same_tables(binding.tree_build_static(K, nodes, upload=False), otree.tables(want, K))


@pytest.mark.parametrize("topk", [(4, 2, 2), (3,), (2, 2, 2, 2), (10, 3)])
def test_cartesian_tree_matches_checker(topk):
    nodes = binding.tree_gen_cartesian(topk)
    want = otree.cartesian(topk)
    assert sorted(tuple(r for r in n if r >= 0) for n in nodes) == sorted(want)
    _same_tables(binding.tree_build_static(len(topk), nodes, upload=False), otree.tables(want, len(topk)))


def test_node_order_is_free_and_root_only_tree():
    a = binding.tree_build_static(2, [[1, -1], [0, 0], [0, -1]], upload=False)
    b = binding.tree_build_static(2, [[0, -1], [1, -1], [0, 0]], upload=False)
    assert a.retrieve_indices == b.retrieve_indices == [[0, 2, -1], [0, 1, 3]]
    r = binding.tree_build_static(1, [], upload=False)
    assert (r.T, r.P, r.C) == (1, 1, 1) and r.retrieve_indices == [[0, -1]]


@pytest.mark.parametrize("nodes,code", [
    ([[0, -1], [1, 0]], -1),          # orphan: parent (1,) missing
    ([[0, -1], [0, -1]], -1),         # duplicate
    ([[-1, 0]], -1),                  # rank after padding
    ([[-1, -1]], -1),                 # empty tuple
    ([[16, -1]], -2),                 # top-k beyond the limit
])
def test_bad_trees_are_rejected(nodes, code):
    with pytest.raises(binding.MtvError) as e:
        binding.tree_build_static(2, nodes, upload=False)
    assert e.value.code == code


def test_limits():
    with pytest.raises(binding.MtvError) as e:
        binding.tree_build_static(9, [], upload=False)
    assert e.value.code == -2
    chain = [[0] * d + [-1] * (8 - d) for d in range(1, 9)]
    assert binding.tree_build_static(8, chain, upload=False).T == 9
    many = binding.tree_gen_rank_prior(4, 129)                  # 129 nodes > MTV_MAX_T
    with pytest.raises(binding.MtvError) as e:
        binding.tree_build_static(4, many, upload=False)
    assert e.value.code == -2
    with pytest.raises(binding.MtvError):
        binding.tree_gen_rank_prior(7, 10, R_max=16)            # comparison would not fit 128 bits


def test_hot_calls_validate_before_touching_the_device():
    lib = binding.lib()
    t = binding.tree_build_static(2, [[0, -1]], upload=False)   # host-only tree: hot calls must refuse it
    one = C.c_void_p(16)
    rc = lib.medusa_heads_topk(t.handle, 1, 8, 8, one, one, None, one, one, one, None, one, one, 1 << 20, None)
    assert rc == -1
    rc = lib.tree_verify_attention(t.handle, 1, 4, 2, 64, one, one, one, 64, 64, 64, 16, one, 0.0, one, None,
                                   one, 1 << 20, None)
    assert rc == -1
    rc = lib.tree_accept(t.handle, 1, 8, one, one, one, one, one, one, one, one, 1 << 20, None)
    assert rc == -1
    assert lib.kv_compact_accepted(t.handle, 1, 2, 96, 1, one, one, 8, 8, 8, 16, one, one, one, None, None) == -2
    assert lib.kv_compact_accepted(t.handle, 1, 2, 64, 1, one, one, 8, 8, 7, 16, one, one, one, None, None) == -1
    assert lib.mtv_workspace_bytes(None, 1, 8, 8, 4, 2, 64, 16) == 0
    assert lib.mtv_last_error() is not None
