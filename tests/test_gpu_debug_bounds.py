"""The bounds-checking build (-DMTV_DEBUG_BOUNDS, `build.py debug_bounds`): every index that a kernel reads from
device memory is checked before it becomes an address; a bad one is recorded in the tree's device error word and the
access is skipped.  It stands in for a memory checker where none can be run.

The first test runs whole verification steps and the chained call through that build in a child process (the library
is chosen when the binding is first loaded, so it cannot be swapped inside this process) and asks for identical
results and a clean error word.  The second one — run in the child only, it is skipped under the normal build, where
nothing would stop the access — hands the compaction indices that are out of range and checks that they are reported,
not followed."""
import os
import subprocess
import sys

import pytest
import torch

from paper_2603_03383_b200 import binding, build
from tests._cases import make_tree

pytestmark = pytest.mark.gpu
DEV = "cuda"
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_steps_under_the_bounds_checking_build():
    lib = build.build(variant="debug_bounds")
    env = dict(os.environ, MTV_LIB=lib)
    cases = ["tests/test_gpu_parity.py::test_full_step_tiny_configuration",
             "tests/test_gpu_parity.py::test_full_step_batched_ragged",
             "tests/test_gpu_parity.py::test_full_step_with_fused_lm_head",
             "tests/test_gpu_parity.py::test_verify_steps_chain_in_one_call",
             "tests/test_gpu_parity.py::test_attention_large_ragged_batch",
             "tests/test_gpu_debug_bounds.py::test_indices_out_of_range_are_reported_not_followed"]
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-rs"] + cases, cwd=ROOT, env=env,
                       capture_output=True, text=True, timeout=900)
    tail = r.stdout[-3000:] + r.stderr[-2000:]
    assert r.returncode == 0, tail
    assert "skipped" not in r.stdout.splitlines()[-1], tail       # the child really ran the second test


def test_indices_out_of_range_are_reported_not_followed():
    if not binding.mtv_debug_bounds_enabled():
        pytest.skip("only meaningful in the bounds-checking build (run by the test above in a child process)")
    K = 3
    tb, tree = make_tree("cartesian", K, (4, 2, 2))
    T, B, Hkv, D, Lcap, n_layers = tree.T, 2, 2, 64, 80, 2
    g = torch.Generator().manual_seed(3)
    caches = [torch.randn(B, Hkv, Lcap, D, generator=g).to(torch.bfloat16).to(DEV) for _ in range(2 * n_layers)]
    before = [c.clone() for c in caches]
    kp = binding.cache_pointer_array(caches[:n_layers], DEV)
    vp = binding.cache_pointer_array(caches[n_layers:], DEV)
    strides = (Hkv * Lcap * D, Lcap * D, D)
    seq_lens = torch.tensor([10, 20], dtype=torch.int32, device=DEV)
    status = torch.full((B,), -7, dtype=torch.int32, device=DEV)
    assert binding.mtv_device_error(tree) == 0
    # a node index far outside the tree in sequence 0, an accepted length beyond K in sequence 1
    accept_len = torch.tensor([2, K + 5], dtype=torch.int32, device=DEV)
    acc_nodes = torch.tensor([[0, 1, 100000], [0, 1, 5]], dtype=torch.int32, device=DEV)
    acc_nodes = torch.cat([acc_nodes, torch.full((B, K + 1 - 3), -1, dtype=torch.int32, device=DEV)], dim=1).contiguous()
    binding.kv_compact_accepted(tree, kp, vp, n_layers, B, Hkv, D, strides, Lcap, seq_lens, accept_len, acc_nodes,
                                status=status)
    torch.cuda.synchronize()
    assert binding.mtv_device_error(tree) == binding.MTV_ERR_BOUNDS      # reported (and cleared by the read)
    for c, c0 in zip(caches, before):
        # sequence 1 untouched; in sequence 0 only row 10 + 1 may have moved (node 1 -> slot 1: onto itself)
        assert torch.equal(c[1], c0[1]) and torch.equal(c[0], c0[0])
    assert seq_lens.tolist() == [13, 20]                                 # the bad length did not advance its sequence
    # the context is fine and a correct call works
    accept_len = torch.tensor([1, 2], dtype=torch.int32, device=DEV)
    acc_nodes[:, :3] = torch.tensor([[0, 2, -1], [0, 1, 5]], dtype=torch.int32, device=DEV)
    binding.kv_compact_accepted(tree, kp, vp, n_layers, B, Hkv, D, strides, Lcap, seq_lens, accept_len, acc_nodes,
                                status=status)
    torch.cuda.synchronize()
    assert binding.mtv_device_error(tree) == 0 and status.tolist() == [0, 0]
    for c, c0 in zip(caches, before):
        assert torch.equal(c[0, :, 13 + 1], c0[0, :, 13 + 2]) and torch.equal(c[1, :, 20 + 2], c0[1, :, 20 + 5])
