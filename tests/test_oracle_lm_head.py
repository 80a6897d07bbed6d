"""Pins of the checker's LM-head projection with per-node argmax."""
import torch

from oracle import reference as ref


def _bf16(x):
    return torch.tensor(x, dtype=torch.float32).to(torch.bfloat16)


def test_hand_computed_case():
    # z = x W^T with x = [[1, 2, -1], [0.5, 0, 4]] and four vocabulary rows
    x = _bf16([[1.0, 2.0, -1.0], [0.5, 0.0, 4.0]])
    W = _bf16([[1.0, 0.0, 0.0], [0.0, 1.0, 1.0], [2.0, -1.0, 3.0], [0.0, 2.0, 0.5]])
    am, zmax, z2, z = ref.lm_head_argmax(x, W, want_logits=True)
    assert z.tolist() == [[1.0, 1.0, -3.0, 3.5], [0.5, 4.0, 13.0, 2.0]]
    assert am.tolist() == [3, 2]
    assert zmax.tolist() == [3.5, 13.0] and z2.tolist() == [1.0, 4.0]


def test_one_hot_hidden_state_selects_a_weight_column():
    # x[m] = e_j makes z[m][v] = W[v][j]: the answer is the argmax of a stored column (a transposed operand
    # or a wrong stride would pick from a row instead)
    g = torch.Generator().manual_seed(3)
    V, H = 37, 11
    W = torch.randn(V, H, generator=g).to(torch.bfloat16)
    x = torch.zeros(H, H, dtype=torch.bfloat16)
    for j in range(H):
        x[j, j] = 1.0
    am, zmax, z2 = ref.lm_head_argmax(x, W)
    col = W.double()
    for j in range(H):
        c = col[:, j]
        assert am[j].item() == int(torch.argmax(c)) and zmax[j].item() == c.max().item()
        assert z2[j].item() == torch.sort(c, descending=True).values[1].item()


def test_ties_go_to_the_lowest_index_and_the_runner_up_equals_the_maximum():
    W = _bf16([[1.0, 1.0], [3.0, 0.0], [0.0, 3.0], [3.0, 0.0], [2.0, 2.0]])
    x = _bf16([[1.0, 0.0], [0.0, 1.0], [1.0, 1.0], [-1.0, -1.0]])
    am, zmax, z2 = ref.lm_head_argmax(x, W)
    assert am.tolist() == [1, 2, 4, 0]
    assert zmax.tolist() == [3.0, 3.0, 4.0, -2.0]
    assert z2.tolist() == [3.0, 2.0, 3.0, -3.0]      # row 0: rows 1 and 3 tie, the runner-up is the twin


def test_single_vocabulary_row():
    am, zmax, z2 = ref.lm_head_argmax(_bf16([[2.0, 3.0]]), _bf16([[1.0, -1.0]]))
    assert am.tolist() == [0] and zmax.tolist() == [-1.0] and z2[0].item() == float("-inf")


def test_against_a_library_matrix_product():
    g = torch.Generator().manual_seed(4)
    M, H, V = 9, 96, 301
    x = torch.randn(M, H, generator=g).to(torch.bfloat16)
    W = torch.randn(V, H, generator=g).to(torch.bfloat16)
    am, zmax, z2, z = ref.lm_head_argmax(x, W, want_logits=True)
    lib = x.double() @ W.double().T
    assert torch.allclose(z, lib, rtol=0, atol=1e-11)
    assert torch.equal(am.long(), lib.argmax(dim=1))
    # scaling a node's hidden state by a positive power of two keeps its argmax, negating it turns it into the argmin
    am2, _, _ = ref.lm_head_argmax((x.float() * 4).to(torch.bfloat16), W)
    assert torch.equal(am2, am)
    am3, _, _ = ref.lm_head_argmax((-x.float()).to(torch.bfloat16), W)
    assert torch.equal(am3.long(), lib.argmin(dim=1))
