"""Pins for the checker's acceptance / retrieval and KV compaction (Section 3.2, Zero-Copy Retrieval)."""
import pytest
import torch

from oracle import reference as ref
from oracle import tree
from paper_2603_03383_b200 import synth


def test_hand_example():
    # nodes: 0 root, 1=(0), 2=(1), 3=(0,0); paths [0,2,-1] and [0,1,3]
    tb = tree.tables([(0,), (1,), (0, 0)], 2)
    tree_tok = torch.tensor([[10, 20, 21, 30]], dtype=torch.int32)
    out = ref.tree_accept(torch.tensor([[20, 30, 5, 6]], dtype=torch.int32), tree_tok, tb)
    assert out["accept_len"].tolist() == [2] and out["best_path"].tolist() == [1]
    assert out["acc_nodes"].tolist() == [[0, 1, 3]] and out["acc_tok"].tolist() == [[10, 20, 30]]
    assert out["next_root"].tolist() == [6]
    out = ref.tree_accept(torch.tensor([[21, 30, 5, 6]], dtype=torch.int32), tree_tok, tb)
    assert out["accept_len"].tolist() == [1] and out["best_path"].tolist() == [0]
    assert out["acc_nodes"].tolist() == [[0, 2, -1]] and out["acc_tok"].tolist() == [[10, 21, -1]]
    assert out["next_root"].tolist() == [5]
    out = ref.tree_accept(torch.tensor([[99, 30, 5, 6]], dtype=torch.int32), tree_tok, tb)
    assert out["accept_len"].tolist() == [0] and out["best_path"].tolist() == [0]   # tie -> lowest path
    assert out["acc_nodes"].tolist() == [[0, -1, -1]] and out["next_root"].tolist() == [99]


def test_node_argmax_ties_take_lowest_id():
    lg = torch.zeros(1, 2, 9, dtype=torch.bfloat16)
    lg[0, 0, [3, 6]] = 2.0
    lg[0, 1, 8] = -1.0
    assert ref.node_argmax(lg).tolist() == [[3, 0]]
    lg = synth.normal_bf16(3, 1, (2, 3, 500))
    am = ref.node_argmax(lg)
    for b in range(2):
        for i in range(3):
            row = lg[b, i].float().tolist()
            assert am[b, i].item() == min(v for v in range(500) if row[v] == max(row))


def _toy_logits(seq, V, seed):
    """Toy 'model': logits over V tokens as a seeded function of the whole token sequence."""
    hsh = seed
    for t in seq:
        hsh = (hsh * 1000003 + t + 1) % (1 << 40)
    return synth.normal_bf16(hsh, 0, (V,))


@pytest.mark.parametrize("topk,V", [((3, 2, 2), 6), ((2, 2, 2, 2), 5), ((4,), 8)])
def test_equals_sequential_greedy_decoding(topk, V):
    """Accepted tokens are a prefix of brute-force greedy decoding and the length is maximal."""
    K = len(topk)
    tb = tree.tables(tree.cartesian(topk), K)
    T = tb["T"]
    seen_lens = set()
    for trial in range(300):
        seed = 1000 + trial
        prefix = [1, 2, 3]
        # candidates: root token, then k_d distinct tokens per head
        cand = [int(synth.uniform_int(seed, 1, 1, 0, V - 1))]
        for d in range(K):
            perm = sorted(range(V), key=lambda t: int(synth.uniform_int(seed, 10 + d, V, 0, 1 << 30)[t]))
            cand += perm[:topk[d]]
        tree_tok = [cand[tb["tree_indices"][i]] for i in range(T)]
        logits = torch.empty(1, T, V, dtype=torch.bfloat16)
        for i in range(T):
            path, j = [], i
            while j >= 0:
                path.append(tree_tok[j])
                j = tb["parent"][j]
            logits[0, i] = _toy_logits(prefix + path[::-1], V, seed)
        am = ref.node_argmax(logits)
        out = ref.tree_accept(am, torch.tensor([tree_tok], dtype=torch.int32), tb)
        n = out["accept_len"].item()
        # brute force: decode K+1 tokens one at a time after prefix + root
        seq, greedy = prefix + [tree_tok[0]], []
        for _ in range(K + 1):
            row = _toy_logits(seq, V, seed).float().tolist()
            nxt = min(v for v in range(V) if row[v] == max(row))
            greedy.append(nxt)
            seq.append(nxt)
        assert out["acc_tok"][0, :n + 1].tolist() == [tree_tok[0]] + greedy[:n]
        assert out["next_root"].item() == greedy[n]
        last = out["acc_nodes"][0, n].item()
        kids = [tree_tok[c] for c in range(T) if tb["parent"][c] == last]
        assert n == K or greedy[n] not in kids                # maximal
        assert out["acc_nodes"][0, n + 1:].tolist() == [-1] * (K - n)
        # second formulation: walk from the root along the child that carries am[current]
        walk, cur = [0], 0
        while True:
            nxt = [c for c in range(T) if tb["parent"][c] == cur and tree_tok[c] == am[0, cur].item()]
            if not nxt:
                break
            assert len(nxt) == 1
            cur = nxt[0]
            walk.append(cur)
        assert out["acc_nodes"][0, :n + 1].tolist() == walk
        assert out["best_path"].item() == min(p for p, r in enumerate(tb["retrieve"]) if r[:n + 1] == walk)
        seen_lens.add(n)
    assert seen_lens == set(range(K + 1))


def test_planted_walk_is_reproduced_and_matches_closed_form():
    K, topk, V, B = 3, (4, 2, 2), 1024, 400
    tb = tree.tables(tree.cartesian(topk), K)
    T = tb["T"]
    cand = torch.stack([torch.randperm(V, generator=torch.Generator().manual_seed(b))[:tb["C"]] for b in range(B)])
    tree_tok = cand[:, torch.tensor(tb["tree_indices"])].to(torch.int32)
    logits, planted = synth.planted_logits(B, T, V, K, tree_tok, tb["parent"], tb["rank"], seed=77, p_accept=(0.6,))
    out = ref.tree_accept(ref.node_argmax(logits), tree_tok, tb)
    assert torch.equal(out["accept_len"], planted)
    want = 0.6 + 0.36 + 0.216                               # E[len] = sum_j p^j on a full tree
    got = planted.double().mean().item()
    assert abs(got - want) < 4 * (1.0 / B) ** 0.5           # ~4 sigma (sd of len < 1.2)


# ------------------------------------------------------------- compaction
def _append_one_at_a_time(cache, L, nodes):
    """Prefix-only cache, then append the accepted nodes' rows at L, L+1, ..."""
    new = cache.clone()
    for j, node in enumerate(nodes):
        new[:, L + j] = cache[:, L + node]
    return new


@pytest.mark.parametrize("acc", [[0, 2, 5, -1], [0, 1, 2, 3], [0, -1, -1, -1], [0, 3, 9, 12]])
def test_compaction_equals_appending_accepted_rows(acc):
    K, B, Hkv, D, Lcap, T = 3, 2, 2, 8, 40, 13
    lens = [11, 6]
    cache = synth.normal_bf16(5, 1, (B, Hkv, Lcap, D))
    n = sum(1 for a in acc if a >= 0) - 1
    accept_len = torch.tensor([n, 0], dtype=torch.int32)
    acc_nodes = torch.tensor([acc, [0, -1, -1, -1]], dtype=torch.int32)
    got, new_len = ref.kv_compact(cache, lens, accept_len, acc_nodes)
    assert new_len.tolist() == [lens[0] + n + 1, lens[1] + 1]
    for b in range(B):
        nodes = [a for a in acc_nodes[b].tolist() if a >= 0]
        want = _append_one_at_a_time(cache[b], lens[b], nodes)
        keep = new_len[b].item()
        assert torch.equal(got[b, :, :keep], want[:, :keep])          # rows >= new seq_len are don't-care
        assert torch.equal(got[b, :, :lens[b]], cache[b, :, :lens[b]])  # prefix untouched
