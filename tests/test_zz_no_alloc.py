"""tree_accept_static_scratch: the workspace-free variant of tree_accept.

Some users of this library run where device allocation is off limits (inside a serving runtime that
owns the device heap, or in a decode loop where an allocator call is banned).  For them tree_accept
exists in a form whose scratch is a fixed array inside the library.  This file checks, through the
C ABI, that it returns exactly what tree_accept and the CPU checker return — on two calls in a row, because
the array keeps whatever the previous call left in it —, that a call allocates no device memory, and that a
problem too large for the array, or logits the scan cannot read in 16-byte chunks, are refused with nothing
launched.  The file name keeps it last in pytest's collection order."""
import pytest
import torch

from oracle import reference as ref
from paper_2603_03383_b200 import binding, synth
from tests._cases import make_tree, workspace

pytestmark = pytest.mark.gpu
DEV = "cuda"
NAMES = ["accept_len", "best_path", "acc_nodes", "acc_tok", "next_root"]


def _outputs(B, K):
    f = lambda *s: torch.full(s, -7, dtype=torch.int32, device=DEV)
    return [f(B), f(B), f(B, K + 1), f(B, K + 1), f(B)]


def _inputs(tb, B, T, V, K, seed, p):
    g = torch.Generator().manual_seed(seed)
    cand = torch.stack([torch.randperm(V, generator=g)[:tb["C"]] for _ in range(B)]).to(torch.int32)
    tree_tok = cand[:, torch.tensor(tb["tree_indices"])].contiguous()
    logits, _ = synth.planted_logits(B, T, V, K, tree_tok, tb["parent"], tb["rank"], seed=seed, p_accept=p)
    return logits.to(DEV), tree_tok.to(DEV)


def test_matches_tree_accept_on_two_calls_in_a_row():
    K = 4
    tb, tree = make_tree("rank_prior", K, (), 64)
    T = tree.T
    # two different problems back to back: the second call finds the first one's keys in the array
    for B, V, seed, p in [(4, 20000, 11, (0.9, 0.3)), (2, 5003, 12, (0.6,))]:
        logits, tree_tok = _inputs(tb, B, T, V, K, seed, p)
        want = _outputs(B, K)
        binding.tree_accept(tree, logits, tree_tok, *want, workspace(tree, B, 8, V, 0, 0, 0, 0))
        got = _outputs(B, K)
        for attempt in range(3):    # free device memory as the driver reports it: unchanged across a call (a second look
            torch.cuda.synchronize()    # if something else on the device moved it meanwhile)
            free_before, allocated_before = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
            binding.tree_accept_static_scratch(tree, logits, tree_tok, *got)
            torch.cuda.synchronize()
            if torch.cuda.mem_get_info()[0] == free_before:
                break
        assert torch.cuda.mem_get_info()[0] == free_before and torch.cuda.memory_allocated() == allocated_before
        checker = ref.tree_accept(ref.node_argmax(logits.cpu()), tree_tok.cpu(), tb)
        for name, a, b in zip(NAMES, got, want):
            assert torch.equal(a, b), name          # integer outputs: bit-exact, as in the other accept tests
            assert torch.equal(a.cpu(), checker[name]), name
        assert int(want[0].max()) >= 1              # the planted walks were found, not an all-zero coincidence


def test_replays_from_a_cuda_graph():
    """The call only enqueues two kernels: captured into a CUDA graph and replayed (no allocation, no synchronisation
    inside), it gives the outputs of the plain call."""
    K = 4
    tb, tree = make_tree("rank_prior", K, (), 64)
    B, V = 3, 9000
    logits, tree_tok = _inputs(tb, B, tree.T, V, K, 21, (0.8, 0.4, 0.6))
    want = _outputs(B, K)
    binding.tree_accept_static_scratch(tree, logits, tree_tok, *want)     # also the first use on this device: outside capture
    torch.cuda.synchronize()
    got = _outputs(B, K)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            binding.tree_accept_static_scratch(tree, logits, tree_tok, *got, stream=side)
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(2):
        for t in got:
            t.fill_(-7)
        graph.replay()
        torch.cuda.synchronize()
        for name, a, b in zip(NAMES, got, want):
            assert torch.equal(a, b), name
    assert int(want[0].max()) >= 1


def test_refuses_logits_that_are_not_16_byte_aligned():
    """The row scan reads 16-byte chunks; a view that starts at an odd element is turned away on the host (an error
    code, no launch) by both entry points."""
    K = 3
    tb, tree = make_tree("cartesian", K, (4, 2, 2))
    B, T, V = 2, tree.T, 512
    backing = torch.zeros(B * T * V + 8, dtype=torch.bfloat16, device=DEV)
    logits = backing[1:1 + B * T * V].view(B, T, V)          # two bytes past a 16-byte boundary
    assert logits.data_ptr() % 16 == 2
    tree_tok = torch.zeros(B, T, dtype=torch.int32, device=DEV)
    for call in (lambda o: binding.tree_accept_static_scratch(tree, logits, tree_tok, *o),
                 lambda o: binding.tree_accept(tree, logits, tree_tok, *o, workspace(tree, B, 8, V, 0, 0, 0, 0))):
        outs = _outputs(B, K)
        with pytest.raises(binding.MtvError) as e:
            call(outs)
        assert e.value.code == -1
        torch.cuda.synchronize()
        assert all(bool((t == -7).all()) for t in outs)


def test_refuses_more_rows_than_the_array_can_serve():
    tb, tree = make_tree("rank_prior", 5, (), 128)
    B, V = 65, 8                                    # 65 * 128 rows * 8 bytes > 65536
    assert B * tree.T * 8 > binding.tree_accept_static_scratch_capacity()
    logits = torch.zeros(B, tree.T, V, dtype=torch.bfloat16, device=DEV)
    tree_tok = torch.zeros(B, tree.T, dtype=torch.int32, device=DEV)
    outs = _outputs(B, 5)
    with pytest.raises(binding.MtvError) as e:
        binding.tree_accept_static_scratch(tree, logits, tree_tok, *outs)
    assert e.value.code == -3 and "65536" in str(e.value)
    torch.cuda.synchronize()
    assert all(bool((t == -7).all()) for t in outs)  # nothing was launched
