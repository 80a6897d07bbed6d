"""Pins for the checker's static tree tables (Section 3.2, Tensorization of Tree Topology)."""
import heapq
from collections import Counter
from fractions import Fraction

import pytest

from oracle import tree


def test_hand_example():
    # root, two depth-1 candidates, one depth-2 candidate under the first.
    tb = tree.tables([(1,), (0, 0), (0,)], K=2)
    assert tb["nodes"] == [(), (0,), (1,), (0, 0)]
    assert tb["parent"] == [-1, 0, 0, 1]
    assert tb["depth"] == [0, 1, 1, 2]
    assert tb["k_d"] == [2, 1] and tb["C"] == 4
    assert tb["tree_indices"] == [0, 1, 2, 3]
    assert tb["mask"] == [[1, 0, 0, 0], [1, 1, 0, 0], [1, 0, 1, 0], [1, 1, 0, 1]]
    assert tb["retrieve"] == [[0, 2, -1], [0, 1, 3]]      # leaves 2 and 3, ascending
    assert tb["P"] == 2


def test_orphan_rejected():
    with pytest.raises(ValueError):
        tree.tables([(0,), (1, 0)], K=2)


@pytest.mark.parametrize("K,T,per_depth,P,k_d", [
    (4, 64, [1, 10, 36, 16, 1], 42, [10, 10, 5, 1]),
    (4, 65, [1, 10, 37, 16, 1], 43, [10, 10, 5, 1]),
    (5, 128, [1, 10, 57, 50, 9, 1], 84, [10, 10, 10, 3, 1]),
    (5, 129, [1, 10, 57, 51, 9, 1], 85, [10, 10, 10, 3, 1]),
])
def test_rank_prior_sizes(K, T, per_depth, P, k_d):
    # sizes fixed by the mathematics of p(r) = 1/((r+1) H_10) and the stated tie-break
    tb = tree.tables(tree.rank_prior(K, T), K)
    cnt = Counter(tb["depth"])
    assert [cnt[d] for d in range(K + 1)] == per_depth
    assert tb["T"] == T and tb["P"] == P and tb["k_d"] == k_d


def test_rank_prior_cut_inside_tie_group():
    n64, n65 = tree.rank_prior(4, 64), tree.rank_prior(4, 65)
    assert n64[-1] == (1, 7) and n65[-1] == (3, 3)        # equal scores 1/16: tie-break decides
    n128, n129 = tree.rank_prior(5, 128), tree.rank_prior(5, 129)
    assert n128[-1] == (1, 4, 0) and n129[-1] == (4, 0, 1)


@pytest.mark.parametrize("K,T", [(4, 64), (5, 128), (3, 20)])
def test_rank_prior_equals_greedy_frontier_growth(K, T):
    """Second formulation: grow the tree one best frontier node at a time."""
    Z = sum(Fraction(1, r + 1) for r in range(10))

    def score(t):
        s = Fraction(1)
        for r in t:
            s *= Fraction(1, r + 1) / Z
        return s

    chosen, frontier = [], [(-score((0,)), 1, (0,))]
    while len(chosen) < T - 1:
        _, d, t = heapq.heappop(frontier)
        chosen.append(t)
        if t[-1] + 1 < 10:                                  # right sibling
            s = t[:-1] + (t[-1] + 1,)
            heapq.heappush(frontier, (-score(s), d, s))
        if d < K:                                           # first child
            c = t + (0,)
            heapq.heappush(frontier, (-score(c), d + 1, c))
    assert sorted(chosen) == sorted(tree.rank_prior(K, T))


def test_cartesian_422():
    tb = tree.tables(tree.cartesian((4, 2, 2)), 3)
    cnt = Counter(tb["depth"])
    assert [cnt[d] for d in range(4)] == [1, 4, 8, 16]
    assert tb["T"] == 29 and tb["P"] == 16 and tb["C"] == 9
    for i, t in enumerate(tb["nodes"]):
        if t:
            assert tb["tree_indices"][i] == [1, 5, 7][len(t) - 1] + t[-1]


@pytest.mark.parametrize("make", [lambda: (tree.rank_prior(4, 64), 4), lambda: (tree.rank_prior(5, 128), 5),
                                  lambda: (tree.cartesian((4, 2, 2)), 3), lambda: ([(0,), (0, 0), (0, 0, 0)], 3)])
def test_table_invariants(make):
    nodes, K = make()
    tb = tree.tables(nodes, K)
    T, order = tb["T"], tb["nodes"]
    for i in range(T):
        for j in range(T):
            # independent definition: j visible from i iff j's tuple is a prefix of i's
            assert tb["mask"][i][j] == int(order[i][:len(order[j])] == order[j])
            if j > i:
                assert tb["mask"][i][j] == 0
        assert tb["mask"][i][i] == 1 and tb["mask"][i][0] == 1
        assert sum(tb["mask"][i]) == tb["depth"][i] + 1
    seen = Counter()
    for p, path in enumerate(tb["retrieve"]):
        assert len(path) == K + 1
        real = [x for x in path if x >= 0]
        assert path[:len(real)] == real                     # padding only at the end
        for j, node in enumerate(real):
            assert tb["depth"][node] == j and node >= j
            if j:
                assert tb["parent"][node] == real[j - 1]
        seen[real[-1]] += 1
        if p:
            assert real[-1] > [x for x in tb["retrieve"][p - 1] if x >= 0][-1]
    children = Counter(tb["parent"][1:])
    leaves = [i for i in range(T) if children[i] == 0]
    assert sorted(seen) == leaves and all(v == 1 for v in seen.values())
    # candidate slots: every (depth, rank) pair maps to its own slot
    for i in range(1, T):
        d, r = tb["depth"][i], tb["rank"][i]
        assert tb["tree_indices"][i] == 1 + sum(tb["k_d"][:d - 1]) + r
        assert 0 <= r < tb["k_d"][d - 1]
