"""GPU parity at the full sizes of the five benchmark configurations, in the launch configuration
that bench.py times.  Attention is compared on every row where the checker finishes in seconds, else on rows
that cover every sequence, KV head and row tile; integer outputs are compared in full (top-k ids for sampled
batch rows, acceptance for every sequence)."""
import pytest
import torch

from oracle import reference as ref
from paper_2603_03383_b200 import binding, synth
from tests._cases import assert_close, oracle_heads_with_margin, workload_tree, workspace

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _covering_rows(B, T, Hq, Hkv, per_cell, seed):
    """(sequence, node, head) rows that reach every (sequence, KV head, 128-row tile of the (node, head-in-group)
    block) at least `per_cell` times, plus the corners."""
    G = Hq // Hkv
    tiles = (T * G + 127) // 128
    g = torch.Generator().manual_seed(seed)
    rows = []
    for b in range(B):
        for kv in range(Hkv):
            for t in range(tiles):
                lo, hi = t * 128, min(T * G, t * 128 + 128)
                for r in torch.randint(lo, hi, (per_cell,), generator=g).tolist():
                    rows.append([b, r // G, kv * G + r % G])
    rows += [[0, 0, 0], [B - 1, T - 1, Hq - 1], [0, T - 1, 0], [B - 1, 0, Hq - 1]]     # root and last node, first and last head
    return rows


@pytest.mark.parametrize("name,per_cell", [("tiny", 0), ("short", 0), ("long", 0), ("batched", 2), ("stress", 4)])
def test_attention_full_size(name, per_cell):
    """Every output row at `tiny`, `short` and `long`; at `batched` and `stress` (where the checker would take minutes)
    at least 512 rows that reach every sequence, KV head and row tile."""
    w = synth.WORKLOADS[name]
    tb, tree = workload_tree(w)
    T, B = tree.T, w.B
    lens = synth.seq_lens(w)
    Lcap = int(w.L_hi) + T
    q, k, v = synth.attention_inputs(B, T, w.Hq, w.Hkv, w.D, Lcap, w.seed, device=DEV)
    out = torch.zeros(B, T, w.Hq, w.D, dtype=torch.bfloat16, device=DEV)
    status = torch.full((B,), -7, dtype=torch.int32, device=DEV)
    ws = workspace(tree, B, 0, 0, w.Hq, w.Hkv, w.D, Lcap)
    binding.tree_verify_attention(tree, q, k, v, lens.to(DEV), out, ws, status=status)
    torch.cuda.synchronize()
    assert status.tolist() == [0] * B
    assert binding.mtv_device_error(tree) == 0
    if per_cell == 0:
        want = ref.tree_attention(q.cpu(), k.cpu(), v.cpu(), lens, tb["mask"])
        assert_close(out, want, "%s attention, every row" % name)
    else:
        rows = _covering_rows(B, T, w.Hq, w.Hkv, per_cell, w.cfg_id)
        assert len(rows) >= 512
        want = ref.tree_attention(q.cpu(), k.cpu(), v.cpu(), lens, tb["mask"], rows=rows)
        idx = torch.tensor(rows)
        got = out.cpu()[idx[:, 0], idx[:, 1], idx[:, 2]]
        assert_close(got, want, "%s attention, %d rows" % (name, len(rows)))
    # a property that holds for every row: each output is a convex combination of V rows
    vmax = v.float().abs().max().item()
    assert out.float().abs().max().item() <= vmax * 1.01 and bool(torch.isfinite(out.float()).all())


@pytest.mark.parametrize("name,rows", [("long", None), ("batched", [0, 9, 15]), ("stress", [2])])
def test_heads_full_size(name, rows):
    w = synth.WORKLOADS[name]
    tb, tree = workload_tree(w)
    B = w.B
    seed, inp, _, cand_ref, cl_ref, tt_ref = oracle_heads_with_margin(B, w.H, w.V, w.K, tb, w.seed, rows=rows, device=DEV)
    hidden, W1, b1, W2, root = inp
    ws = workspace(tree, B, w.H, w.V, 0, 0, 0, 0)
    cand = torch.full((B, tree.C), -7, dtype=torch.int32, device=DEV)
    cl = torch.zeros(B, tree.C - 1, device=DEV)
    tt = torch.full((B, tree.T), -7, dtype=torch.int32, device=DEV)
    binding.medusa_heads_topk(tree, hidden, W1, b1, W2, root, cand, cl, tt, ws)
    torch.cuda.synchronize()
    assert binding.mtv_device_error(tree) == 0
    sel = list(range(B)) if rows is None else rows
    assert torch.equal(cand.cpu()[sel], cand_ref), seed
    assert torch.equal(tt.cpu()[sel], tt_ref)
    assert_close(cl.cpu()[sel], cl_ref, "cand_logit")
    # every row, cheap properties: ids in range and distinct within a head, logits descending
    c = cand.cpu()
    assert int(c.min()) >= 0 and int(c.max()) < w.V
    for d in range(w.K):
        off, kd = tb["offset"][d], tb["k_d"][d]
        seg = c[:, off:off + kd]
        assert all(len(set(r.tolist())) == kd for r in seg)
        lg = cl.cpu()[:, off - 1:off - 1 + kd]
        assert bool((lg[:, :-1] >= lg[:, 1:]).all())


@pytest.mark.parametrize("name", ["short", "batched", "stress"])
def test_accept_full_size(name):
    w = synth.WORKLOADS[name]
    tb, tree = workload_tree(w)
    T, B, K = tree.T, w.B, w.K
    g = torch.Generator().manual_seed(w.cfg_id)
    cand = torch.stack([torch.randperm(w.V, generator=g)[:tb["C"]] for _ in range(B)]).to(torch.int32)
    tree_tok = cand[:, torch.tensor(tb["tree_indices"])].contiguous()
    logits, planted = synth.planted_logits(B, T, w.V, K, tree_tok, tb["parent"], tb["rank"], w.seed,
                                           p_accept=w.p_accept, device=DEV)
    want = ref.tree_accept(ref.node_argmax(logits.cpu()), tree_tok, tb)
    assert torch.equal(want["accept_len"], planted)
    f = lambda *s: torch.full(s, -7, dtype=torch.int32, device=DEV)
    outs = dict(accept_len=f(B), best_path=f(B), acc_nodes=f(B, K + 1), acc_tok=f(B, K + 1), next_root=f(B))
    ws = workspace(tree, B, 8, w.V, 0, 0, 0, 0)
    binding.tree_accept(tree, logits, tree_tok.to(DEV), outs["accept_len"], outs["best_path"], outs["acc_nodes"],
                        outs["acc_tok"], outs["next_root"], ws)
    torch.cuda.synchronize()
    for name_, t in outs.items():
        assert torch.equal(t.cpu(), want[name_]), name_


@pytest.mark.parametrize("name,reps", [("long", 300), ("short", 300), ("stress", 20)])
def test_attention_is_bitwise_repeatable(name, reps):
    """The key splits of a query block meet through counters and the workspace inside one launch; the merge order
    is fixed, so repeated calls must give bit-identical output.  A missing fence in that exchange would show up
    here as a rare difference."""
    w = synth.WORKLOADS[name]
    tb, tree = workload_tree(w)
    T, B = tree.T, w.B
    lens = synth.seq_lens(w).to(DEV)
    Lcap = int(w.L_hi) + T
    q, k, v = synth.attention_inputs(B, T, w.Hq, w.Hkv, w.D, Lcap, w.seed + 5, device=DEV)
    ws = workspace(tree, B, 0, 0, w.Hq, w.Hkv, w.D, Lcap)
    first = torch.zeros(B, T, w.Hq, w.D, dtype=torch.bfloat16, device=DEV)
    binding.tree_verify_attention(tree, q, k, v, lens, first, ws)
    outs = [torch.zeros_like(first) for _ in range(4)]
    bad = torch.zeros((), dtype=torch.int64, device=DEV)
    for i in range(reps):
        o = outs[i % 4]
        o.fill_(float("nan"))
        binding.tree_verify_attention(tree, q, k, v, lens, o, ws)
        bad += (o.view(torch.int16) != first.view(torch.int16)).sum()
    torch.cuda.synchronize()
    assert binding.mtv_device_error(tree) == 0
    assert int(bad) == 0


def test_heads_are_bitwise_repeatable():
    w = synth.WORKLOADS["long"]
    tb, tree = workload_tree(w)
    hidden, W1, b1, W2, root = synth.head_inputs(4, w.H, 32768, w.K, 99, device=DEV)    # four rows: the tensor-core path
    ws = workspace(tree, 4, w.H, 32768, 0, 0, 0, 0)
    ref_c = torch.zeros(4, tree.C, dtype=torch.int32, device=DEV)
    ref_l = torch.zeros(4, tree.C - 1, device=DEV)
    tt = torch.zeros(4, tree.T, dtype=torch.int32, device=DEV)
    binding.medusa_heads_topk(tree, hidden, W1, b1, W2, root, ref_c, ref_l, tt, ws)
    for _ in range(30):
        c, l = torch.zeros_like(ref_c), torch.zeros_like(ref_l)
        binding.medusa_heads_topk(tree, hidden, W1, b1, W2, root, c, l, tt, ws)
        assert torch.equal(c, ref_c) and torch.equal(l, ref_l)
    assert binding.mtv_device_error(tree) == 0
