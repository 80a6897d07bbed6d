"""Pins of the checker's rotary embedding for the tree nodes (positions seq_len + depth)."""
import math

import torch

from oracle import reference as ref


def _bf16(x):
    return torch.tensor(x, dtype=torch.float32).to(torch.bfloat16)


def test_hand_computed_rotation():
    # D = 4: pairs (0, 2) and (1, 3); theta = 100 -> inverse frequencies 1 and 100^(-1/2) = 0.1
    q = _bf16([[[[1.0, 2.0, 0.0, 0.0]]]])          # B = T = Hq = 1
    k = _bf16([[[[0.0, 0.0, 1.0, 4.0]]]])
    q_out, k_out = ref.rope(q, k, [2], [1], theta=100.0)     # position 3
    c0, s0, c1, s1 = math.cos(3.0), math.sin(3.0), math.cos(0.3), math.sin(0.3)
    assert torch.allclose(q_out.flatten(), torch.tensor([c0, 2 * c1, s0, 2 * s1], dtype=torch.float64), atol=1e-12)
    assert torch.allclose(k_out.flatten(), torch.tensor([-s0, -4 * s1, c0, 4 * c1], dtype=torch.float64), atol=1e-12)


def test_position_zero_is_the_identity_and_norms_are_kept():
    g = torch.Generator().manual_seed(1)
    q = torch.randn(2, 5, 3, 8, generator=g).to(torch.bfloat16)
    k = torch.randn(2, 5, 1, 8, generator=g).to(torch.bfloat16)
    q0, k0 = ref.rope(q, k, [0, 0], [0] * 5)
    assert torch.equal(q0, q.double()) and torch.equal(k0, k.double())
    q1, k1 = ref.rope(q, k, [7, 1000], [0, 1, 1, 2, 3])
    for a, b in ((q1, q.double()), (k1, k.double())):
        for d in range(4):                                    # each rotated pair keeps its length
            assert torch.allclose(a[..., d] ** 2 + a[..., d + 4] ** 2, b[..., d] ** 2 + b[..., d + 4] ** 2, atol=1e-9)


def test_scores_depend_on_the_position_difference_only():
    g = torch.Generator().manual_seed(2)
    q = torch.randn(1, 1, 1, 16, generator=g).to(torch.bfloat16)
    k = torch.randn(1, 1, 1, 16, generator=g).to(torch.bfloat16)
    dots = []
    for base in (0, 5, 1234):
        qa, _ = ref.rope(q, k, [base + 9], [0])               # query at base + 9
        _, kb = ref.rope(q, k, [base], [2])                   # key at base + 2
        dots.append(float((qa * kb).sum()))
    assert abs(dots[0] - dots[1]) < 1e-9 and abs(dots[0] - dots[2]) < 1e-6


def test_depth_sets_the_position_not_the_node_index():
    q = _bf16([[[[1.0, 0.0]], [[1.0, 0.0]], [[1.0, 0.0]]]])   # T = 3 nodes, D = 2
    k = q.clone()
    q_out, _ = ref.rope(q, k, [10], [0, 1, 1])                # nodes 1 and 2 are siblings: same depth
    assert torch.equal(q_out[0, 1], q_out[0, 2]) and not torch.equal(q_out[0, 0], q_out[0, 1])
    assert abs(float(q_out[0, 1, 0, 0]) - math.cos(11.0)) < 1e-12
