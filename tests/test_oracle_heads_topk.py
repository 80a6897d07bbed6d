"""Pins for the checker's Medusa heads (Section 3.1) and per-head top-k."""
import itertools

import pytest
import torch

from oracle import reference as ref
from oracle import tree
from paper_2603_03383_b200 import synth

SIG1 = 0.7310585786300049   # sigmoid(1), textbook constant
SIG2 = 0.8807970779778823   # sigmoid(2)


def bf(x):
    return torch.tensor(x, dtype=torch.float64).to(torch.bfloat16)


def test_hand_case_sigmoid_constants():
    # y = W1 h (+b1) = [2, -1]; silu(2) = 2 sigmoid(2); silu(-1) = -(1 - sigmoid(1))
    h = bf([[1.0, 2.0]])
    W1 = bf([[[0.0, 1.0], [-1.0, 0.0]]])          # asymmetric: W1^T would give y = [-2, 1]
    W2 = bf([[[1.0, 2.0], [0.0, 1.0]]])           # asymmetric: W2^T would give z = [h0, 2 h0 + h1]
    hp0 = 1.0 + 2.0 * SIG2
    hp1 = 2.0 - (1.0 - SIG1)
    z = ref.heads_logits(h, W1, None, W2)
    assert z.shape == (1, 1, 2)
    assert z[0, 0].tolist() == pytest.approx([hp0 + 2 * hp1, hp1], rel=0, abs=1e-14)
    # with a bias: y = [2, -1] + [-1, 2] = [1, 1]
    z = ref.heads_logits(h, W1, bf([[-1.0, 2.0]]), W2)
    hp0, hp1 = 1.0 + SIG1, 2.0 + SIG1
    assert z[0, 0].tolist() == pytest.approx([hp0 + 2 * hp1, hp1], rel=0, abs=1e-14)


def test_zero_block_reduces_to_matvec():
    # W1 = 0, b1 = 0  =>  SiLU(0) = 0, h' = h, z = W2 h : a plain library matrix-vector product
    B, H, V, K = 3, 96, 200, 2
    hidden, W1, b1, W2, _ = synth.head_inputs(B, H, V, K, seed=11)
    z = ref.heads_logits(hidden, torch.zeros_like(W1), torch.zeros_like(b1), W2)
    want = torch.einsum("kvh,bh->kbv", W2.double(), hidden.double())
    assert torch.allclose(z, want, rtol=0, atol=1e-12)


def test_heads_and_batch_rows_are_independent():
    B, H, V, K = 2, 64, 50, 3
    hidden, W1, b1, W2, _ = synth.head_inputs(B, H, V, K, seed=5)
    z = ref.heads_logits(hidden, W1, b1, W2)
    for k, b in itertools.product(range(K), range(B)):
        zk = ref.heads_logits(hidden[b:b + 1], W1[k:k + 1], b1[k:k + 1], W2[k:k + 1])
        assert torch.equal(zk[0, 0], z[k, b])
    assert not torch.equal(z[0, 0], z[1, 0]) and not torch.equal(z[0, 0], z[0, 1])


def test_general_case_against_library_ops():
    B, H, V, K = 2, 128, 300, 2
    hidden, W1, b1, W2, _ = synth.head_inputs(B, H, V, K, seed=7)
    z = ref.heads_logits(hidden, W1, b1, W2)
    y = torch.einsum("koh,bh->kbo", W1.double(), hidden.double()) + b1.double()[:, None, :]
    hp = hidden.double()[None] + torch.nn.functional.silu(y)
    want = torch.einsum("kvh,kbh->kbv", W2.double(), hp)
    assert torch.allclose(z, want, rtol=0, atol=1e-12)
    # the residual term matters (a dropped "h +" must not pass)
    assert not torch.allclose(z, torch.einsum("kvh,kbh->kbv", W2.double(), torch.nn.functional.silu(y)), atol=1e-3)


def test_doubling_w2_doubles_logits():
    hidden, W1, b1, W2, _ = synth.head_inputs(1, 64, 40, 1, seed=3)
    z1 = ref.heads_logits(hidden, W1, b1, W2)
    z2 = ref.heads_logits(hidden, W1, b1, (W2.float() * 2).to(torch.bfloat16))
    assert torch.equal(z2, 2 * z1)


# ------------------------------------------------------------------ top-k
def test_topk_brute_force():
    V = 16
    z = synth.normal_f32(1, 50, 0, V).double()
    z[5] = z[11]                                     # an exact tie
    for k in range(1, V + 1):
        ids, vals, gap = ref.topk(z, k)
        order = sorted(range(V), key=lambda v: (-float(z[v]), v))
        assert ids.tolist() == order[:k]
        assert vals.tolist() == [float(z[v]) for v in order[:k]]
        assert gap >= 0
        assert len(set(ids.tolist())) == k
    assert ref.topk(z, 1)[0].item() == int(torch.argmax(z))


def test_topk_equal_values_lowest_id_first():
    z = torch.zeros(1000, dtype=torch.float64)
    z[900] = 3.0
    z[7] = 3.0
    ids, _, gap = ref.topk(z, 3)
    assert ids.tolist() == [7, 900, 0] and gap == 0.0


def test_duplicate_rows_of_w2_rank_by_id():
    B, H, V, K = 1, 64, 1024, 1
    hidden, W1, b1, W2, root = synth.head_inputs(B, H, V, K, seed=9)
    z = ref.heads_logits(hidden, W1, b1, W2)
    top = int(torch.argmax(z[0, 0]))
    W2[0, 7] = W2[0, top]
    W2[0, 900] = W2[0, top]
    z = ref.heads_logits(hidden, W1, b1, W2)
    ids, _, _ = ref.topk(z[0, 0], 3)
    assert ids.tolist() == sorted({7, 900, top})


def test_candidate_buffer_layout():
    tb = tree.tables(tree.cartesian((3, 2)), 2)
    z = torch.zeros(2, 1, 10, dtype=torch.float64)
    z[0, 0, [4, 8, 2]] = torch.tensor([3.0, 2.0, 1.0], dtype=torch.float64)
    z[1, 0, [9, 0]] = torch.tensor([5.0, 4.0], dtype=torch.float64)
    cand, cl, tree_tok, gap = ref.heads_candidates(z, torch.tensor([77]), tb)
    assert cand.tolist() == [[77, 4, 8, 2, 9, 0]]
    assert cl.tolist() == [[3.0, 2.0, 1.0, 5.0, 4.0]]
    # nodes: root, (0) (1) (2), then (0,0) (0,1) (1,0) (1,1) (2,0) (2,1)
    assert tree_tok.tolist() == [[77, 4, 8, 2, 9, 0, 9, 0, 9, 0]]
    assert gap == 1.0
