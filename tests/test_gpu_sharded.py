"""One sequence's step split over several GPUs, checked on one: the ranks' slices are computed one after the other
on the same device (ordinary launches, nothing waits on anything), laid out as the all-gather would deliver them,
and merged by the library's kernels.  Results must equal the CPU checker on the whole problem, and the integer
outputs must be bit-identical to the single-device call."""
import pytest
import torch

from oracle import reference as ref
from paper_2603_03383_b200 import binding, sharded, synth
from tests._cases import assert_close, make_tree, oracle_heads_with_margin, workspace

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _i32(*shape, fill=-7):
    return torch.full(shape, fill, dtype=torch.int32, device=DEV)


@pytest.mark.parametrize("world,B,H,V,kind,K,topk,T", [
    (2, 1, 512, 1024, "cartesian", 3, (4, 2, 2), 0),          # the small configuration's heads, one row per rank pass
    (4, 3, 256, 3001, "rank_prior", 4, (), 64),               # ragged last slab, tensor-core path (B > 1)
    (3, 2, 256, 2000, "rank_prior", 4, (), 64),               # slabs of 672, 672, 656
    (16, 1, 64, 1000, "rank_prior", 5, (), 128),               # the largest group the merge takes
])
def test_heads_by_vocabulary_slab(world, B, H, V, kind, K, topk, T):
    tb, tree = make_tree(kind, K, topk, T)
    seed, inp, _, cand_ref, cl_ref, tt_ref = oracle_heads_with_margin(B, H, V, K, tb, 300 + world)
    hidden, W1, b1, W2, root = [t.to(DEV) for t in inp]
    ws = workspace(tree, B, H, V, 0, 0, 0, 0)
    cand_all, logit_all = _i32(world, B, tree.C), torch.zeros(world, B, tree.C - 1, device=DEV)
    v_slab = None
    for r in range(world):
        p = sharded.plan(r, world, V, 48, 48, max_kd=max(tb["k_d"]))       # (the head counts play no part here)
        v_slab = p.v_slab
        W2_slab = W2[:, p.v_lo:p.v_hi].contiguous()
        tt = _i32(B, tree.T)
        binding.medusa_heads_topk(tree, hidden, W1, b1, W2_slab, root, cand_all[r], logit_all[r], tt, ws)
    cand, cl, tt = _i32(B, tree.C), torch.zeros(B, tree.C - 1, device=DEV), _i32(B, tree.T)
    binding.heads_merge_shards(tree, v_slab, cand_all, logit_all, root, cand, cl, tt, ws)
    torch.cuda.synchronize()
    assert binding.mtv_device_error(tree) == 0
    assert torch.equal(cand.cpu(), cand_ref), seed
    assert torch.equal(tt.cpu(), tt_ref)
    assert (cl.double().cpu() - cl_ref).abs().max().item() <= 2e-5 * cl_ref.abs().max().item()
    # and against the single-device call: same ids, same logits to the last bit (a row's sum does not depend on the slab)
    cand1, cl1, tt1 = _i32(B, tree.C), torch.zeros(B, tree.C - 1, device=DEV), _i32(B, tree.T)
    binding.medusa_heads_topk(tree, hidden, W1, b1, W2, root, cand1, cl1, tt1, ws)
    assert torch.equal(cand1, cand) and torch.equal(tt1, tt) and torch.equal(cl1, cl)
    # a second merge right after the first (the tickets reset themselves)
    cand2, tt2 = _i32(B, tree.C), _i32(B, tree.T)
    binding.heads_merge_shards(tree, v_slab, cand_all, logit_all, root, cand2, None, tt2, ws)
    assert torch.equal(cand2, cand) and torch.equal(tt2, tt)


def test_heads_merge_ties_across_slabs_take_the_lowest_global_id():
    K = 2
    tb, tree = make_tree("cartesian", K, (4, 3))
    B, V, world = 2, 64, 4
    p0 = sharded.plan(0, world, V, 8, 4, max_kd=4)
    cand_all, logit_all = _i32(world, B, tree.C, fill=0), torch.zeros(world, B, tree.C - 1, device=DEV)
    # every slab reports the same logits 5, 4, 3, 2 for head 0 with local ids 3, 2, 1, 0: the winners are the four copies
    # of logit 5, ordered by global id; head 1: distinct logits, the best three overall
    for r in range(world):
        cand_all[r, :, 1:5] = torch.tensor([3, 2, 1, 0], dtype=torch.int32)
        logit_all[r, :, 0:4] = torch.tensor([5., 4., 3., 2.])
        cand_all[r, :, 5:8] = torch.tensor([7, 6, 5], dtype=torch.int32)
        logit_all[r, :, 4:7] = torch.tensor([10. - r, 1., 0.5])
    root = torch.tensor([11, 12], dtype=torch.int32, device=DEV)
    cand, cl, tt = _i32(B, tree.C), torch.zeros(B, tree.C - 1, device=DEV), _i32(B, tree.T)
    ws = torch.zeros(256, dtype=torch.uint8, device=DEV)
    binding.heads_merge_shards(tree, p0.v_slab, cand_all, logit_all, root, cand, cl, tt, ws)
    torch.cuda.synchronize()
    s = p0.v_slab
    for b in range(B):
        assert cand[b].tolist() == [root[b].item(), 3, 3 + s, 3 + 2 * s, 3 + 3 * s, 7, 7 + s, 7 + 2 * s]
        assert cl[b].tolist() == [5., 5., 5., 5., 10., 9., 8.]
        assert tt[b].tolist() == [cand[b, i].item() for i in tb["tree_indices"]]


@pytest.mark.parametrize("world,B,Hq,Hkv,D,lens,kind,K,topk,T", [
    (2, 1, 32, 8, 128, [1000], "rank_prior", 4, (), 64),
    (4, 3, 16, 4, 128, [300, 0, 77], "rank_prior", 4, (), 64),
    (2, 2, 8, 2, 64, [128, 5], "cartesian", 3, (4, 2, 2), 0),
])
def test_attention_by_kv_head(world, B, Hq, Hkv, D, lens, kind, K, topk, T):
    tb, tree = make_tree(kind, K, topk, T)
    T = tree.T
    Lcap = max(lens) + T
    q, k, v = synth.attention_inputs(B, T, Hq, Hkv, D, Lcap, 41)
    sl = torch.tensor(lens, dtype=torch.int32)
    want = ref.tree_attention(q, k, v, sl, tb["mask"])
    gathered = None
    for r in range(world):
        p = sharded.plan(r, world, 1000, Hq, Hkv)
        ql = q[:, :, p.q_lo:p.q_lo + p.hq_local].contiguous().to(DEV)
        kl = k[:, p.kv_lo:p.kv_lo + p.hkv_local].contiguous().to(DEV)
        vl = v[:, p.kv_lo:p.kv_lo + p.hkv_local].contiguous().to(DEV)
        if gathered is None:
            gathered = torch.zeros(world, B, T, p.hq_local, D, dtype=torch.bfloat16, device=DEV)
        ws = workspace(tree, B, 0, 0, p.hq_local, p.hkv_local, D, Lcap)
        status = _i32(B)
        binding.tree_verify_attention(tree, ql, kl, vl, sl.to(DEV), gathered[r], ws, status=status)
        assert status.tolist() == [0] * B
    out = torch.zeros(B, T, Hq, D, dtype=torch.bfloat16, device=DEV)
    binding.attn_interleave_shards(gathered, out)
    torch.cuda.synchronize()
    assert binding.mtv_device_error(tree) == 0
    assert_close(out, want, "attention by KV head")
    # the single-device call on all heads: heads are independent, so the same bits
    out1 = torch.zeros_like(out)
    ws = workspace(tree, B, 0, 0, Hq, Hkv, D, Lcap)
    binding.tree_verify_attention(tree, q.to(DEV), k.to(DEV), v.to(DEV), sl.to(DEV), out1, ws)
    assert_close(out1, want)
    assert (out.float() - out1.float()).abs().max().item() <= 1e-2 * want.abs().max().item()


def test_lm_head_by_vocabulary_slab():
    tb, tree = make_tree("rank_prior", 4, (), 64)
    B, H, V, world = 2, 256, 3001, 4
    x = synth.normal_bf16(21, 1, (B, tree.T, H))
    W = synth.normal_bf16(21, 2, (V, H))
    W[2999] = W[5]                                                # a tie between the first and the last slab
    x[0, 3] = W[5]
    xd, Wd = x.to(DEV), W.to(DEV)
    M = B * tree.T
    key_all = torch.zeros(world, M, dtype=torch.int64, device=DEV)
    for r in range(world):
        p = sharded.plan(r, world, V, 8, 4)
        binding.lm_head_argmax(tree, xd, Wd[p.v_lo:p.v_hi].contiguous(), key_all[r])
    keys = torch.zeros(M, dtype=torch.int64, device=DEV)
    binding.keys_merge_shards(p.v_slab, key_all, keys)
    keys1 = torch.zeros(M, dtype=torch.int64, device=DEV)
    binding.lm_head_argmax(tree, xd, Wd, keys1)
    torch.cuda.synchronize()
    am = (0xffffffff - (keys.cpu() & 0xffffffff)).to(torch.int32)
    want, zmax, z2 = ref.lm_head_argmax(x.reshape(M, H), W)
    decisive = (zmax - z2) > 1e-4 * zmax.abs().max()
    assert torch.equal(am[decisive], want[decisive]) and decisive.float().mean() > 0.9
    assert am[3].item() == 5 == want[3].item()
    assert torch.equal(keys, keys1)                               # the same keys as the single-device call, bit for bit


def test_sharded_calls_with_a_group_of_one():
    """The module's own entry points (local call, gather, merge) with one rank and no process group."""
    tb, tree = make_tree("rank_prior", 4, (), 64)
    B, H, V, Hq, Hkv, D = 2, 256, 2000, 8, 2, 128
    seed, inp, _, cand_ref, cl_ref, tt_ref = oracle_heads_with_margin(B, H, V, 4, tb, 55)
    hidden, W1, b1, W2, root = [t.to(DEV) for t in inp]
    p = sharded.plan(0, 1, V, Hq, Hkv, max_kd=max(tb["k_d"]))
    assert (p.v_lo, p.v_hi, p.hq_local, p.hkv_local) == (0, V, Hq, Hkv)
    lens = [200, 31]
    Lcap = max(lens) + tree.T
    ws = workspace(tree, B, H, V, Hq, Hkv, D, Lcap)
    cand, cl, tt = _i32(B, tree.C), torch.zeros(B, tree.C - 1, device=DEV), _i32(B, tree.T)
    sharded.medusa_heads_topk_sharded(tree, p, hidden, W1, b1, W2, root, cand, cl, tt, ws)
    q, k, v = synth.attention_inputs(B, tree.T, Hq, Hkv, D, Lcap, 56)
    sl = torch.tensor(lens, dtype=torch.int32)
    out = torch.zeros(B, tree.T, Hq, D, dtype=torch.bfloat16, device=DEV)
    sharded.tree_verify_attention_sharded(tree, p, q.to(DEV), k.to(DEV), v.to(DEV), sl.to(DEV), out, ws)
    torch.cuda.synchronize()
    assert torch.equal(cand.cpu(), cand_ref) and torch.equal(tt.cpu(), tt_ref)
    assert_close(out, ref.tree_attention(q, k, v, sl, tb["mask"]))


@pytest.mark.parametrize("world,V", [(2, 1024), (4, 3001), (3, 777)])
def test_accept_by_vocabulary_slab(world, V):
    """Stored logits split by vocabulary slab: per-slab argmax keys, merged, give the acceptance of the whole vocabulary
    (planted walks, natural ties across slabs included: the rows outside the walk are rounded N(0,1) draws)."""
    K = 4
    tb, tree = make_tree("rank_prior", K, (), 64)
    B, T = 3, tree.T
    g = torch.Generator().manual_seed(world)
    cand = torch.stack([torch.randperm(V, generator=g)[:tb["C"]] for _ in range(B)]).to(torch.int32)
    tree_tok = cand[:, torch.tensor(tb["tree_indices"])].contiguous()
    logits, planted = synth.planted_logits(B, T, V, K, tree_tok, tb["parent"], tb["rank"], seed=40 + world, p_accept=(0.9, 0.5, 0.7))
    logits[0, 5, V - 1] = logits[0, 5].max()          # an exact tie between a low id and the last id of the last slab
    want = ref.tree_accept(ref.node_argmax(logits), tree_tok, tb)
    ws = workspace(tree, B, 8, V, 0, 0, 0, 0)
    key_all = torch.zeros(world, B * T, dtype=torch.int64, device=DEV)
    for r in range(world):
        p = sharded.plan(r, world, V, 48, 48)
        binding.node_argmax_keys(tree, logits[:, :, p.v_lo:p.v_hi].contiguous().to(DEV), key_all[r], ws)
    keys = torch.zeros(B * T, dtype=torch.int64, device=DEV)
    binding.keys_merge_shards(p.v_slab, key_all, keys)
    outs = dict(accept_len=_i32(B), best_path=_i32(B), acc_nodes=_i32(B, K + 1), acc_tok=_i32(B, K + 1), next_root=_i32(B))
    binding.tree_accept_keys(tree, B, keys, tree_tok.to(DEV), outs["accept_len"], outs["best_path"], outs["acc_nodes"],
                             outs["acc_tok"], outs["next_root"])
    torch.cuda.synchronize()
    am = (0xffffffff - (keys.cpu() & 0xffffffff)).to(torch.int32).reshape(B, T)
    assert torch.equal(am, ref.node_argmax(logits))
    for name, t in outs.items():
        assert torch.equal(t.cpu(), want[name]), name
    # the whole vocabulary in one call gives the same keys' indices, and tree_accept the same outputs
    keys1 = torch.zeros(B * T, dtype=torch.int64, device=DEV)
    binding.node_argmax_keys(tree, logits.to(DEV), keys1, ws)
    assert torch.equal(keys1 & 0xffffffff, keys & 0xffffffff)
