"""TEST INFRASTRUCTURE — static tree tables by direct definition (pure Python).

Section 3.2, "Tensorization of Tree Topology": the verification tree is fixed
offline and mapped to static tensors — ``medusa_attn_mask`` [T][T] (which
nodes each node may attend to: the parent-child dependencies of the candidate
paths), ``tree_indices`` (flattened node -> position) and, "Zero-Copy
Retrieval", ``retrieve_indices`` [N_paths][K+1].

A node is the tuple of per-depth ranks on the way from the root: (r_1..r_d);
head d (1-based) supplies its rank-r_d candidate (head k predicts token
t+k+1, the base model predicts t+1, so depth = head index).  Readings fixed
here because the paper is silent:
  * flattened order: root first, then by (depth, rank tuple) ascending;
  * tree_indices[i]: slot in the flat candidate buffer
    [root | top-k_1 of head 1 | top-k_2 of head 2 | ...], k_d = 1 + largest
    rank used at depth d; the KV slot of node i is L_b + i;
  * one path per leaf, ordered by ascending leaf index, padded with -1.

Pins: tests/test_oracle_tree.py.
"""
from fractions import Fraction
from itertools import product


def tables(nodes, K):
    """nodes: iterable of rank tuples (root excluded).  Returns a dict."""
    nodes = sorted(set(tuple(n) for n in nodes), key=lambda t: (len(t), t))
    order = [()] + nodes
    index = {t: i for i, t in enumerate(order)}
    T = len(order)
    for t in nodes:
        if not (1 <= len(t) <= K) or min(t) < 0:
            raise ValueError("bad node %r" % (t,))
        if t[:-1] not in index:
            raise ValueError("node %r has no parent in the tree" % (t,))
    parent = [-1] + [index[t[:-1]] for t in nodes]
    depth = [len(t) for t in order]
    rank = [-1] + [t[-1] for t in nodes]
    k_d = [0] * K
    for t in nodes:
        k_d[len(t) - 1] = max(k_d[len(t) - 1], t[-1] + 1)
    offset = [1]
    for d in range(K):
        offset.append(offset[-1] + k_d[d])
    C = offset[-1]
    tree_indices = [0] + [offset[len(t) - 1] + t[-1] for t in nodes]
    # ancestors-or-self by walking parent links
    anc = []
    for i in range(T):
        s, j = set(), i
        while j >= 0:
            s.add(j)
            j = parent[j]
        anc.append(s)
    mask = [[1 if j in anc[i] else 0 for j in range(T)] for i in range(T)]
    has_child = [False] * T
    for i in range(1, T):
        has_child[parent[i]] = True
    leaves = [i for i in range(T) if not has_child[i]]
    retrieve = []
    for leaf in leaves:
        path, j = [], leaf
        while j >= 0:
            path.append(j)
            j = parent[j]
        path.reverse()
        retrieve.append(path + [-1] * (K + 1 - len(path)))
    return dict(T=T, K=K, P=len(leaves), C=C, k_d=k_d, offset=offset[:-1], nodes=order,
                parent=parent, depth=depth, rank=rank, tree_indices=tree_indices,
                mask=mask, retrieve=retrieve)


def cartesian(topk):
    """Full Cartesian tree: every rank tuple with r_d < topk[d]."""
    nodes = []
    for d in range(1, len(topk) + 1):
        nodes += list(product(*[range(topk[j]) for j in range(d)]))
    return nodes


_memo = {}


def rank_prior(K, T_total, R_max=10):
    """Root plus the T_total-1 best nodes of the full R_max-ary depth-K tree.

    Score of a node = product over its depths of p(r) = 1/((r+1) Z) with
    Z = sum_{r<R_max} 1/(r+1), compared exactly; ties broken by depth
    ascending, then rank tuple ascending.
    """
    if (K, R_max) not in _memo:         # the full sorted list, computed once per (K, R_max)
        Z = sum(Fraction(1, r + 1) for r in range(R_max))
        scored = []
        for d in range(1, K + 1):
            for t in product(range(R_max), repeat=d):
                s = Fraction(1)
                for r in t:
                    s *= Fraction(1, r + 1) / Z
                scored.append((-s, d, t))
        scored.sort()
        _memo[(K, R_max)] = [t for _, _, t in scored]
    return list(_memo[(K, R_max)][:T_total - 1])
