"""GPU parity: every C-ABI call against the fp64 checker, element by element, on the same
seeded inputs.  Integer outputs bit-exact; floats within max|err| <= 1e-2*max|ref| + 1e-3."""
import ctypes as C

import pytest
import torch

from oracle import reference as ref
from paper_2603_03383_b200 import binding, synth
from tests._cases import assert_close, make_tree, oracle_heads_with_margin, workspace

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _i32(*shape, fill=-7):
    return torch.full(shape, fill, dtype=torch.int32, device=DEV)


# ------------------------------------------------------------------ heads
HEAD_CASES = [
    # B, H, V, K, tree
    (1, 512, 1024, 3, ("cartesian", (4, 2, 2), 0)),       # the tiny configuration
    (2, 520, 1000, 3, ("cartesian", (4, 2, 2), 0)),       # H, V not multiples of the tile sizes
    (3, 256, 3001, 4, ("rank_prior", (), 64)),
    (5, 1024, 5000, 4, ("rank_prior", (), 64)),
    (16, 512, 2048, 2, ("cartesian", (16, 3), 0)),
    (1, 8, 20, 1, ("cartesian", (16,), 0)),               # V barely above top-k
    (2, 512, 2048, 3, ("cartesian", (4, 2, 2), 0)),       # two rows, H a multiple of 64: the tensor-core kernels
    (9, 256, 3001, 4, ("rank_prior", (), 64)),            # an odd number of rows above 8
    (4, 64, 50, 1, ("cartesian", (16,), 0)),              # one K chunk, slabs far shorter than a 128-row tile
    (16, 192, 777, 5, ("rank_prior", (), 128)),           # three K chunks (fewer than the four accumulators)
]


@pytest.mark.parametrize("B,H,V,K,tr", HEAD_CASES)
@pytest.mark.parametrize("bias", [True, False])
def test_heads_topk(B, H, V, K, tr, bias):
    tb, tree = make_tree(tr[0], K, tr[1], tr[2])
    seed, inp, _, cand_ref, cl_ref, tt_ref = oracle_heads_with_margin(B, H, V, K, tb, 100 + B + H, bias=bias)
    hidden, W1, b1, W2, root = [None if t is None else t.to(DEV) for t in inp]
    ws = workspace(tree, B, H, V, 0, 0, 0, 0)
    cand, cl, tt = _i32(B, tree.C), torch.zeros(B, tree.C - 1, device=DEV), _i32(B, tree.T)
    binding.medusa_heads_topk(tree, hidden, W1, b1, W2, root, cand, cl, tt, ws)
    torch.cuda.synchronize()
    assert torch.equal(cand.cpu(), cand_ref), seed
    assert torch.equal(tt.cpu(), tt_ref)
    assert_close(cl, cl_ref, "cand_logit")
    assert (cl.double().cpu() - cl_ref).abs().max().item() <= 2e-5 * cl_ref.abs().max().item()   # fp32 carry
    # cand_logit is optional
    cand2, tt2 = _i32(B, tree.C), _i32(B, tree.T)
    binding.medusa_heads_topk(tree, hidden, W1, b1, W2, root, cand2, None, tt2, ws)
    assert torch.equal(cand2, cand) and torch.equal(tt2, tt)


def test_heads_exact_ties_take_lowest_id():
    B, H, V, K = 2, 256, 4096, 2
    tb, tree = make_tree("cartesian", K, (4, 3))
    hidden, W1, b1, W2, root = synth.head_inputs(B, H, V, K, seed=77)
    z = ref.heads_logits(hidden, W1, b1, W2)
    top = int(torch.argmax(z[0, 0]))
    for dup in (7, 900, 4095):                # bit-identical rows in different warps / blocks
        W2[0, dup] = W2[0, top]
    z = ref.heads_logits(hidden, W1, b1, W2)
    cand_ref, _, tt_ref, _ = ref.heads_candidates(z, root, tb)
    assert cand_ref[0, 1:5].tolist() == sorted({7, 900, 4095, top})
    ws = workspace(tree, B, H, V, 0, 0, 0, 0)
    cand, tt = _i32(B, tree.C), _i32(B, tree.T)
    binding.medusa_heads_topk(tree, hidden.to(DEV), W1.to(DEV), b1.to(DEV), W2.to(DEV), root.to(DEV), cand, None,
                              tt, ws)
    assert torch.equal(cand.cpu(), cand_ref) and torch.equal(tt.cpu(), tt_ref)


# -------------------------------------------------------------- attention
def _attention_case(tb, tree, B, Hq, Hkv, D, lens, seed, Lcap=None, pad=0):
    T = tree.T
    Lcap = Lcap or max(lens) + T + 5
    q, k, v = synth.attention_inputs(B, T, Hq, Hkv, D, Lcap + pad, seed)
    k, v = k[:, :, :Lcap], v[:, :, :Lcap]                 # pad > 0: a strided view of a larger cache
    sl = torch.tensor(lens, dtype=torch.int32)
    want = ref.tree_attention(q, k, v, sl, tb["mask"])
    kd = k.to(DEV) if pad == 0 else synth.attention_inputs(B, T, Hq, Hkv, D, Lcap + pad, seed, device=DEV)[1][:, :, :Lcap]
    vd = v.to(DEV) if pad == 0 else synth.attention_inputs(B, T, Hq, Hkv, D, Lcap + pad, seed, device=DEV)[2][:, :, :Lcap]
    out = torch.zeros(B, T, Hq, D, dtype=torch.bfloat16, device=DEV)
    status = _i32(B)
    ws = workspace(tree, B, 0, 0, Hq, Hkv, D, Lcap)
    binding.tree_verify_attention(tree, q.to(DEV), kd, vd, sl.to(DEV), out, ws, status=status, Lcap=Lcap)
    torch.cuda.synchronize()
    assert status.tolist() == [0] * B
    return assert_close(out, want, "tree attention")


@pytest.mark.parametrize("L", [0, 1, 35, 63, 64, 65, 127, 128, 129, 700])
def test_attention_prefix_lengths_tiny_tree(L):
    tb, tree = make_tree("cartesian", 3, (4, 2, 2))
    _attention_case(tb, tree, 1, 8, 2, 64, [L], seed=L + 1)


@pytest.mark.parametrize("kind,K,topk,T,Hq,Hkv,D,lens", [
    ("rank_prior", 4, (), 64, 32, 8, 128, [517]),                  # 7B head shape, 64-node tree
    ("rank_prior", 4, (), 65, 8, 2, 128, [200, 131]),              # T = 65: second mask word
    ("rank_prior", 5, (), 128, 8, 2, 128, [300]),                  # 128-node tree, 512 query rows / KV head
    ("rank_prior", 5, (), 128, 16, 2, 64, [97, 0, 260]),           # group of 8, ragged batch
    ("cartesian", 1, (1,), 0, 4, 4, 64, [50]),                     # T = 2, no grouping
    ("cartesian", 1, (), 0, 2, 1, 128, [40, 3]),                   # root-only tree
    ("cartesian", 3, (4, 2, 2), 0, 8, 2, 64, [128]),               # the tiny configuration
    ("rank_prior", 4, (), 64, 28, 4, 128, [3000]),                 # groups of 7 heads (18 nodes per CTA, 126 of 128 rows), key splits
    ("rank_prior", 5, (), 128, 21, 3, 128, [200, 0, 77]),          # groups of 7, four row blocks, ragged batch
    ("rank_prior", 4, (), 65, 12, 4, 128, [517, 64]),              # groups of 3
    ("rank_prior", 4, (), 64, 10, 2, 128, [1100]),                 # groups of 5 (25 nodes per CTA, 125 rows)
    ("cartesian", 2, (3, 2), 0, 12, 2, 128, [90, 300, 5]),         # groups of 6, a ten-node tree
])
def test_attention_shapes(kind, K, topk, T, Hq, Hkv, D, lens):
    tb, tree = make_tree(kind, K, topk, T)
    _attention_case(tb, tree, len(lens), Hq, Hkv, D, lens, seed=5)


def test_attention_ragged_batch_many_splits_and_strided_cache():
    tb, tree = make_tree("rank_prior", 4, (), 64)
    _attention_case(tb, tree, 3, 8, 2, 128, [1500, 40, 777], seed=9, Lcap=1600, pad=24)


def test_attention_large_ragged_batch():
    """More query blocks than half the SMs: one CTA per block and no key splits, sequences from empty to full."""
    tb, tree = make_tree("rank_prior", 4, (), 64)
    g = torch.Generator().manual_seed(77)
    lens = torch.randint(0, 1100, (40,), generator=g).tolist()
    lens[3], lens[17] = 0, 1099
    _attention_case(tb, tree, 40, 8, 2, 128, lens, seed=12, Lcap=1100 + tree.T)


@pytest.mark.parametrize("D", [64, 128])
def test_attention_capacity_is_reported_not_faulted(D):
    tb, tree = make_tree("cartesian", 2, (2, 2))
    T, B, Hq, Hkv, Lcap = tree.T, 2, 4, 2, 40
    q, k, v = synth.attention_inputs(B, T, Hq, Hkv, D, Lcap, 3, device=DEV)
    sl = torch.tensor([Lcap - T + 1, 10], dtype=torch.int32, device=DEV)       # first sequence does not fit
    out = torch.full((B, T, Hq, D), 3.0, dtype=torch.bfloat16, device=DEV)
    status = _i32(B)
    ws = workspace(tree, B, 0, 0, Hq, Hkv, D, Lcap)
    binding.tree_verify_attention(tree, q, k, v, sl, out, ws, status=status)
    torch.cuda.synchronize()
    assert status.tolist() == [binding.MTV_ERR_CAPACITY, 0]
    assert bool((out[0] == 3.0).all())                                          # untouched
    want = ref.tree_attention(q[1:].cpu(), k[1:].cpu(), v[1:].cpu(), sl[1:].cpu(), tb["mask"])
    assert_close(out[1:], want)
    # and the next call on the same device works (nothing was left allocated or half-synchronised)
    sl2 = torch.tensor([5, 10], dtype=torch.int32, device=DEV)
    binding.tree_verify_attention(tree, q, k, v, sl2, out, ws, status=status)
    torch.cuda.synchronize()
    assert status.tolist() == [0, 0] and binding.mtv_device_error(tree) == 0
    assert_close(out, ref.tree_attention(q.cpu(), k.cpu(), v.cpu(), sl2.cpu(), tb["mask"]))


@pytest.mark.parametrize("Hq,Hkv,D", [(8, 2, 128), (8, 2, 64)])
def test_attention_never_reads_past_the_tree_rows(Hq, Hkv, D):
    """Cache rows behind the tree rows are uninitialised memory in real use: NaN there must not leak."""
    tb, tree = make_tree("rank_prior", 4, (), 64)
    T, B, Lcap = tree.T, 2, 400
    lens = [200, 77]
    q, k, v = synth.attention_inputs(B, T, Hq, Hkv, D, Lcap, 21)
    sl = torch.tensor(lens, dtype=torch.int32)
    want = ref.tree_attention(q, k, v, sl, tb["mask"])
    kd, vd = k.to(DEV), v.to(DEV)
    for b, L in enumerate(lens):
        kd[b, :, L + T:] = float("nan")
        vd[b, :, L + T:] = float("nan")
    out = torch.zeros(B, T, Hq, D, dtype=torch.bfloat16, device=DEV)
    ws = workspace(tree, B, 0, 0, Hq, Hkv, D, Lcap)
    binding.tree_verify_attention(tree, q.to(DEV), kd, vd, sl.to(DEV), out, ws)
    assert_close(out, want)


def test_attention_explicit_scale():
    tb, tree = make_tree("cartesian", 2, (2, 2))
    T, D = tree.T, 64
    q, k, v = synth.attention_inputs(1, T, 2, 1, D, 64, 4)
    sl = torch.tensor([30], dtype=torch.int32)
    want = ref.tree_attention(q, k, v, sl, tb["mask"], scale=0.05)
    out = torch.zeros(1, T, 2, D, dtype=torch.bfloat16, device=DEV)
    ws = workspace(tree, 1, 0, 0, 2, 1, D, 64)
    binding.tree_verify_attention(tree, q.to(DEV), k.to(DEV), v.to(DEV), sl.to(DEV), out, ws, scale=0.05)
    assert_close(out, want)


# ----------------------------------------------------------------- accept
@pytest.mark.parametrize("B,V,kind,K,topk,T,p", [
    (1, 1024, "cartesian", 3, (4, 2, 2), 0, (0.6,)),
    (7, 1001, "cartesian", 3, (4, 2, 2), 0, (0.3, 0.6, 0.9)),      # odd V: rows not 16-byte aligned
    (4, 20000, "rank_prior", 4, (), 64, (0.9,)),
    (3, 4096, "rank_prior", 5, (), 128, (0.6,)),
    (2, 50, "cartesian", 1, (), 0, (0.5,)),                        # root-only tree
])
def test_accept(B, V, kind, K, topk, T, p):
    tb, tree = make_tree(kind, K, topk, T)
    T = tree.T
    g = torch.Generator().manual_seed(V)
    cand = torch.stack([torch.randperm(V, generator=g)[:tb["C"]] for _ in range(B)]).to(torch.int32)
    tree_tok = cand[:, torch.tensor(tb["tree_indices"])].contiguous()
    logits, planted = synth.planted_logits(B, T, V, K, tree_tok, tb["parent"], tb["rank"], seed=V + B, p_accept=p)
    logits[0, T - 1, :] = 0.5                                      # a row of exact ties -> id 0
    want = ref.tree_accept(ref.node_argmax(logits), tree_tok, tb)
    assert torch.equal(want["accept_len"], planted)
    outs = dict(accept_len=_i32(B), best_path=_i32(B), acc_nodes=_i32(B, K + 1), acc_tok=_i32(B, K + 1),
                next_root=_i32(B))
    ws = workspace(tree, B, 8, V, 0, 0, 0, 0)
    binding.tree_accept(tree, logits.to(DEV), tree_tok.to(DEV), outs["accept_len"], outs["best_path"],
                        outs["acc_nodes"], outs["acc_tok"], outs["next_root"], ws)
    torch.cuda.synchronize()
    for name, t in outs.items():
        assert torch.equal(t.cpu(), want[name]), name


def test_accept_negative_zero_and_negative_rows():
    tb, tree = make_tree("cartesian", 1, (2,))
    B, T, V = 1, tree.T, 64
    logits = torch.full((B, T, V), -3.0, dtype=torch.bfloat16)
    logits[0, 0, 9] = -0.0
    logits[0, 0, 20] = 0.0                                         # -0.0 == +0.0: lowest id wins
    logits[0, 1, 33] = -1.5
    logits[0, 2, :] = float("-inf")
    tree_tok = torch.tensor([[5, 9, 20]], dtype=torch.int32)
    am = ref.node_argmax(logits)
    assert am.tolist() == [[9, 33, 0]]
    want = ref.tree_accept(am, tree_tok, tb)
    outs = [_i32(B), _i32(B), _i32(B, 2), _i32(B, 2), _i32(B)]
    ws = workspace(tree, B, 8, V, 0, 0, 0, 0)
    binding.tree_accept(tree, logits.to(DEV), tree_tok.to(DEV), *outs, ws)
    for t, name in zip(outs, ["accept_len", "best_path", "acc_nodes", "acc_tok", "next_root"]):
        assert torch.equal(t.cpu(), want[name]), name


# ------------------------------------------------------------- compaction
@pytest.mark.parametrize("D,n_layers,B,Hkv", [(128, 3, 4, 2), (64, 1, 2, 8)])
def test_kv_compaction(D, n_layers, B, Hkv):
    K = 4
    tb, tree = make_tree("rank_prior", K, (), 64)
    T, Lcap = tree.T, 300
    lens = [100, 0, 236, 237][:B]                                  # 237 + 64 > 300: reported, skipped
    paths = [[0, 2, 12, 13, -1], [0, -1, -1, -1, -1], [0, 1, 11, 47, 63], [0, 1, -1, -1, -1]][:B]
    alen = torch.tensor([sum(1 for x in p if x >= 0) - 1 for p in paths], dtype=torch.int32)
    acc = torch.tensor(paths, dtype=torch.int32)
    ks = [synth.normal_bf16(3, 10 + l, (B, Hkv, Lcap, D)) for l in range(n_layers)]
    vs = [synth.normal_bf16(3, 50 + l, (B, Hkv, Lcap, D)) for l in range(n_layers)]
    kd, vd = [t.to(DEV) for t in ks], [t.to(DEV) for t in vs]
    kp, vp = binding.cache_pointer_array(kd, DEV), binding.cache_pointer_array(vd, DEV)
    sl = torch.tensor(lens, dtype=torch.int32, device=DEV)
    status = _i32(B)
    binding.kv_compact_accepted(tree, kp, vp, n_layers, B, Hkv, D, (Hkv * Lcap * D, Lcap * D, D), Lcap, sl,
                                alen.to(DEV), acc.to(DEV), status=status)
    torch.cuda.synchronize()
    fits = [l + T <= Lcap for l in lens]
    assert status.tolist() == [0 if f else binding.MTV_ERR_CAPACITY for f in fits]
    for layer in range(n_layers):
        for cache, got in ((ks[layer], kd[layer]), (vs[layer], vd[layer])):
            want, new_len = ref.kv_compact(cache, lens, alen, acc)
            for b in range(B):
                if not fits[b]:
                    assert torch.equal(got[b].cpu(), cache[b]) and sl[b].item() == lens[b]
                    continue
                keep = new_len[b].item()
                assert sl[b].item() == keep
                assert torch.equal(got[b, :, :keep].cpu(), want[b, :, :keep])
                assert torch.equal(got[b, :, lens[b] + T:].cpu(), cache[b, :, lens[b] + T:])   # nothing past the tree rows


# -------------------------------------------------------------- full step
def _step_case(B, H, V, Hq, Hkv, D, n_layers, kind, K, topk, T, lens, seed, host=False, lm_head=False):
    tb, tree = make_tree(kind, K, topk, T)
    T = tree.T
    Lcap = max(lens) + T
    seed, inp, cpu, cand_ref, cl_ref, tt_ref = oracle_heads_with_margin(B, H, V, K, tb, seed)
    logits, planted = synth.planted_logits(B, T, V, K, tt_ref, tb["parent"], tb["rank"], seed, p_accept=(0.6, 0.9))
    acc_ref = ref.tree_accept(ref.node_argmax(logits), tt_ref, tb)
    assert torch.equal(acc_ref["accept_len"], planted)
    if lm_head:
        # the same planted next tokens, this time as the argmax of an LM head: the hidden state of node i is
        # the weight row of its token plus noise; the step gets (x_final, W_lm) and no logits
        target = ref.node_argmax(logits).long()
        W_lm = synth.normal_bf16(seed, 901, (V, H))
        x_final = (W_lm[target.flatten()].float().reshape(B, T, H) +
                   0.3 * synth.normal_bf16(seed, 902, (B, T, H)).float()).to(torch.bfloat16)
        am, zmax, z2 = ref.lm_head_argmax(x_final.reshape(B * T, H), W_lm)
        assert torch.equal(am.long(), target.flatten()) and ((zmax - z2) > 1e-3 * zmax.abs().max()).all()
    sl = torch.tensor(lens, dtype=torch.int32)
    layers = [synth.attention_inputs(B, T, Hq, Hkv, D, Lcap, seed, layer=l) for l in range(n_layers)]
    out_ref = torch.stack([ref.tree_attention(q, k, v, sl, tb["mask"]) for q, k, v in layers])
    kd, vd = [l[1].to(DEV) for l in layers], [l[2].to(DEV) for l in layers]
    q_all = torch.stack([l[0] for l in layers])
    hidden, W1, b1, W2, root = inp
    a = binding.StepArgs()
    a.B, a.H, a.V, a.Hq, a.Hkv, a.D, a.n_layers, a.Lcap = B, H, V, Hq, Hkv, D, n_layers, Lcap
    a.stride_b, a.stride_h, a.stride_t, a.scale = Hkv * Lcap * D, Lcap * D, D, 0.0
    kp, vp = binding.cache_pointer_array(kd, DEV), binding.cache_pointer_array(vd, DEV)
    kph, vph = binding.cache_pointer_array(kd), binding.cache_pointer_array(vd)
    dev = dict(hidden=hidden.to(DEV), W1=W1.to(DEV), b1=b1.to(DEV), W2=W2.to(DEV), root_tok=root.to(DEV),
               q_layers=q_all.to(DEV), logits=logits.to(DEV), seq_lens=sl.to(DEV),
               cand=_i32(B, tree.C), cand_logit=torch.zeros(B, tree.C - 1, device=DEV), tree_tok=_i32(B, T),
               out_layers=torch.zeros(n_layers, B, T, Hq, D, dtype=torch.bfloat16, device=DEV),
               accept_len=_i32(B), best_path=_i32(B), acc_nodes=_i32(B, K + 1), acc_tok=_i32(B, K + 1),
               next_root=_i32(B), status=_i32(B), k_caches=kp, v_caches=vp, k_caches_host=kph, v_caches_host=vph,
               ws=workspace(tree, B, H, V, Hq, Hkv, D, Lcap))
    up = ["hidden", "root_tok", "q_layers", "logits"]
    src = dict(hidden=hidden, root_tok=root, q_layers=q_all, logits=logits)
    if lm_head:
        del dev["logits"]                                          # never read on this path
        dev["x_final"], dev["W_lm"] = x_final.to(DEV), W_lm.to(DEV)
        up[3], src["x_final"] = "x_final", x_final
        del src["logits"]
    for name, t in dev.items():
        setattr(a, name, t.data_ptr())
    a.ws_bytes = dev["ws"].numel()
    if host:
        hb = binding.StepArgs()
        names = up + ["tree_tok", "out_layers", "accept_len", "best_path", "acc_nodes", "acc_tok", "next_root",
                      "seq_lens"]
        hostbuf = {n: (src[n].clone() if n in src else torch.empty_like(dev[n], device="cpu")).pin_memory()
                   for n in names}
        for n in up:                                               # the device copies start out wrong
            dev[n].zero_()
        for n, t in hostbuf.items():
            setattr(hb, n, t.data_ptr())
        binding.mtv_verify_step_host(tree, a, hb)
        got = {n: hostbuf[n] for n in names}
    else:
        binding.mtv_verify_step(tree, a)
        torch.cuda.synchronize()
        got = {n: t.cpu() for n, t in dev.items() if n not in ("ws",)}
    assert got.get("status", torch.zeros(B)).tolist() == [0] * B if not host else True
    assert torch.equal(got["tree_tok"], tt_ref)
    if not host:
        assert torch.equal(got["cand"], cand_ref)
    for l in range(n_layers):
        assert_close(got["out_layers"][l], out_ref[l], "layer %d" % l)
    for name in ("accept_len", "best_path", "acc_nodes", "acc_tok", "next_root"):
        assert torch.equal(got[name], acc_ref[name]), name
    assert torch.equal(got["seq_lens"], sl + acc_ref["accept_len"] + 1)
    for l in range(n_layers):
        for cache, gotc in ((layers[l][1], kd[l]), (layers[l][2], vd[l])):
            want, new_len = ref.kv_compact(cache, lens, acc_ref["accept_len"], acc_ref["acc_nodes"])
            for b in range(B):
                assert torch.equal(gotc[b, :, :new_len[b]].cpu(), want[b, :, :new_len[b]])
    return acc_ref["accept_len"]


def test_full_step_tiny_configuration():
    w = synth.WORKLOADS["tiny"]
    _step_case(w.B, w.H, w.V, w.Hq, w.Hkv, w.D, 3, w.tree, w.K, w.topk, w.T, [w.L_lo], w.seed)


def test_full_step_batched_ragged():
    _step_case(5, 256, 3000, 8, 2, 128, 2, "rank_prior", 4, (), 64, [300, 17, 0, 129, 64], seed=31)


def test_full_step_from_host_buffers():
    _step_case(2, 256, 2000, 8, 2, 64, 2, "cartesian", 3, (4, 2, 2), 0, [90, 33], seed=8, host=True)


def test_full_step_with_fused_lm_head():
    _step_case(5, 256, 3000, 8, 2, 128, 2, "rank_prior", 4, (), 64, [300, 17, 0, 129, 64], seed=31, lm_head=True)


def test_full_step_with_fused_lm_head_from_host_buffers():
    _step_case(2, 256, 2000, 8, 2, 64, 2, "cartesian", 3, (4, 2, 2), 0, [90, 33], seed=8, host=True, lm_head=True)


def test_full_step_at_the_long_shapes():
    """Hidden size, vocabulary, heads and prefix of the `long` configuration (two layers: the checker's attention
    takes seconds per layer), every output and the compacted caches against the checker."""
    w = synth.WORKLOADS["long"]
    _step_case(w.B, w.H, w.V, w.Hq, w.Hkv, w.D, 2, w.tree, w.K, w.topk, w.T, [w.L_lo], w.seed)


def test_full_step_from_host_buffers_with_more_layers_than_download_groups():
    """Twenty layers: the attention outputs leave in groups of two layers (sixteen groups at most)."""
    _step_case(2, 256, 2000, 8, 2, 128, 20, "rank_prior", 4, (), 64, [70, 33], seed=9, host=True)


def test_three_chained_steps():
    """Step, compaction, append of the next tree's K/V with the rotary embedding, step again: attention of a later
    step reads the cache that this library's own compaction and append produced, and the whole chain equals the
    checker stepping the same way (the accepted path's K/V are what sequential decoding would have appended)."""
    B, H, V, Hq, Hkv, D, K, n_layers = 2, 256, 2000, 8, 2, 128, 4, 2
    tb, tree = make_tree("rank_prior", K, (), 64)
    T = tree.T
    lens0 = [150, 37]
    Lcap = max(lens0) + 3 * (K + 1) + T
    seed = 77
    f = lambda *s_: torch.full(s_, -7, dtype=torch.int32, device=DEV)
    # state: caches and lengths, on both sides
    kc = [synth.normal_bf16(seed, 500 + l, (B, Hkv, Lcap, D)) for l in range(n_layers)]
    vc = [synth.normal_bf16(seed, 600 + l, (B, Hkv, Lcap, D)) for l in range(n_layers)]
    kd, vd = [t.to(DEV) for t in kc], [t.to(DEV) for t in vc]
    sl_ref = torch.tensor(lens0, dtype=torch.int32)
    sl_dev = sl_ref.to(DEV)
    root_ref = synth.uniform_int(seed, 7, B, 0, V - 1).to(torch.int32)
    root_dev = root_ref.to(DEV)
    ws = workspace(tree, B, H, V, Hq, Hkv, D, Lcap)
    kp, vp = binding.cache_pointer_array(kd, DEV), binding.cache_pointer_array(vd, DEV)
    strides = (Hkv * Lcap * D, Lcap * D, D)
    for step in range(3):
        # ---- inputs of this step (same values on both sides); the heads' seed is bumped until the checker's rank
        #      gaps clear the margin
        s_in = seed + 10 * step
        for attempt in range(20):
            hidden, W1, b1, W2, _ = synth.head_inputs(B, H, V, K, s_in)
            z = ref.heads_logits(hidden, W1, b1, W2)
            cand_ref, _, tt_ref, gap = ref.heads_candidates(z, root_ref, tb)
            if gap > 1e-5 * z.abs().max().item():
                break
            s_in += 1000
        q = [synth.normal_bf16(s_in, 700 + l, (B, T, Hq, D)) for l in range(n_layers)]
        kn = [synth.normal_bf16(s_in, 800 + l, (B, T, Hkv, D)) for l in range(n_layers)]
        vn = [synth.normal_bf16(s_in, 900 + l, (B, T, Hkv, D)) for l in range(n_layers)]
        logits, planted = synth.planted_logits(B, T, V, K, tt_ref, tb["parent"], tb["rank"], s_in, p_accept=(0.9, 0.6))
        # ---- the checker's step
        out_ref = []
        for l in range(n_layers):
            q_rot, k_rot = ref.rope(q[l], kn[l], sl_ref.tolist(), tb["depth"])
            for b in range(B):
                L = int(sl_ref[b])
                kc[l][b, :, L:L + T] = k_rot[b].to(torch.bfloat16).permute(1, 0, 2)
                vc[l][b, :, L:L + T] = vn[l][b].permute(1, 0, 2)
            out_ref.append(ref.tree_attention(q_rot.to(torch.bfloat16), kc[l], vc[l], sl_ref, tb["mask"]))
        acc_ref = ref.tree_accept(ref.node_argmax(logits), tt_ref, tb)
        assert torch.equal(acc_ref["accept_len"], planted)
        new_len = None
        for l in range(n_layers):
            kc[l], new_len = ref.kv_compact(kc[l], sl_ref, acc_ref["accept_len"], acc_ref["acc_nodes"])
            vc[l], _ = ref.kv_compact(vc[l], sl_ref, acc_ref["accept_len"], acc_ref["acc_nodes"])
        # ---- this library's step, call by call
        cand, tt = f(B, tree.C), f(B, T)
        binding.medusa_heads_topk(tree, hidden.to(DEV), W1.to(DEV), b1.to(DEV), W2.to(DEV), root_dev, cand, None, tt, ws)
        assert torch.equal(tt.cpu(), tt_ref) and torch.equal(cand.cpu(), cand_ref)
        status = f(B)
        for l in range(n_layers):
            qd = q[l].to(DEV)
            binding.tree_kv_append_rope(tree, qd, kn[l].to(DEV), vn[l].to(DEV), kd[l], vd[l], sl_dev, status=status)
            out = torch.zeros(B, T, Hq, D, dtype=torch.bfloat16, device=DEV)
            binding.tree_verify_attention(tree, qd, kd[l], vd[l], sl_dev, out, ws, status=status)
            torch.cuda.synchronize()
            assert status.tolist() == [0] * B
            assert_close(out, out_ref[l], "step %d layer %d" % (step, l))
        outs = dict(accept_len=f(B), best_path=f(B), acc_nodes=f(B, K + 1), acc_tok=f(B, K + 1), next_root=f(B))
        binding.tree_accept(tree, logits.to(DEV), tt, outs["accept_len"], outs["best_path"], outs["acc_nodes"],
                            outs["acc_tok"], outs["next_root"], ws)
        binding.kv_compact_accepted(tree, kp, vp, n_layers, B, Hkv, D, strides, Lcap, sl_dev, outs["accept_len"],
                                    outs["acc_nodes"], status=status)
        torch.cuda.synchronize()
        for name, t in outs.items():
            assert torch.equal(t.cpu(), acc_ref[name]), (step, name)
        assert status.tolist() == [0] * B and torch.equal(sl_dev.cpu(), new_len)
        for l in range(n_layers):
            for b in range(B):
                # V rows are copies: bit-exact.  The appended K rows were rotated in fp32 here and in fp64 by the
                # checker before the rounding to bf16: equal to the float tolerance, and bit-exact below the first
                # appended row
                n, n0 = int(new_len[b]), lens0[b]
                assert torch.equal(vd[l][b, :, :n].cpu(), vc[l][b, :, :n])
                assert torch.equal(kd[l][b, :, :n0].cpu(), kc[l][b, :, :n0])
                assert_close(kd[l][b, :, :n], kc[l][b, :, :n], "compacted K rows")
        # ---- the next step starts from the token after the accepted path
        sl_ref = new_len
        root_ref = acc_ref["next_root"]
        root_dev = outs["next_root"]
    assert binding.mtv_device_error(tree) == 0
    assert int(sl_ref.min()) > min(lens0)


def test_generator_is_identical_on_cpu_and_gpu():
    a = synth.normal_bf16(123, 5, (1 << 16,), 0.37)
    b = synth.normal_bf16(123, 5, (1 << 16,), 0.37, device=DEV)
    assert torch.equal(a, b.cpu())
    assert torch.equal(synth.uniform_int(9, 1, 100, 5, 5000), synth.uniform_int(9, 1, 100, 5, 5000, device=DEV).cpu())


def test_full_step_replays_from_a_cuda_graph():
    """The whole step only enqueues work (no host synchronisation, no allocation): it can be captured once
    and replayed, and the replay gives what the oracle gives."""
    w = synth.WORKLOADS["tiny"]
    tb, tree = make_tree(w.tree, w.K, w.topk, w.T)
    T, B, K, n_layers = tree.T, 2, w.K, 2
    lens = [100, 37]
    Lcap = max(lens) + T
    seed, inp, cpu, cand_ref, cl_ref, tt_ref = oracle_heads_with_margin(B, 256, 2000, K, tb, 41)
    logits, planted = synth.planted_logits(B, T, 2000, K, tt_ref, tb["parent"], tb["rank"], seed, p_accept=(0.9,))
    acc_ref = ref.tree_accept(ref.node_argmax(logits), tt_ref, tb)
    sl = torch.tensor(lens, dtype=torch.int32)
    layers = [synth.attention_inputs(B, T, 8, 2, 128, Lcap, seed, layer=l) for l in range(n_layers)]
    out_ref = torch.stack([ref.tree_attention(q, k, v, sl, tb["mask"]) for q, k, v in layers])
    kd, vd = [l[1].to(DEV) for l in layers], [l[2].to(DEV) for l in layers]
    k0, v0 = [t.clone() for t in kd], [t.clone() for t in vd]
    hidden, W1, b1, W2, root = inp
    a = binding.StepArgs()
    a.B, a.H, a.V, a.Hq, a.Hkv, a.D, a.n_layers, a.Lcap = B, 256, 2000, 8, 2, 128, n_layers, Lcap
    a.stride_b, a.stride_h, a.stride_t, a.scale = 2 * Lcap * 128, Lcap * 128, 128, 0.0
    dev = dict(hidden=hidden.to(DEV), W1=W1.to(DEV), b1=b1.to(DEV), W2=W2.to(DEV), root_tok=root.to(DEV),
               q_layers=torch.stack([l[0] for l in layers]).to(DEV), logits=logits.to(DEV), seq_lens=sl.to(DEV),
               cand=_i32(B, tree.C), cand_logit=torch.zeros(B, tree.C - 1, device=DEV), tree_tok=_i32(B, T),
               out_layers=torch.zeros(n_layers, B, T, 8, 128, dtype=torch.bfloat16, device=DEV),
               accept_len=_i32(B), best_path=_i32(B), acc_nodes=_i32(B, K + 1), acc_tok=_i32(B, K + 1),
               next_root=_i32(B), status=_i32(B), k_caches=binding.cache_pointer_array(kd, DEV),
               v_caches=binding.cache_pointer_array(vd, DEV), k_caches_host=binding.cache_pointer_array(kd),
               v_caches_host=binding.cache_pointer_array(vd), ws=workspace(tree, B, 256, 2000, 8, 2, 128, Lcap))
    for name, t in dev.items():
        setattr(a, name, t.data_ptr())
    a.ws_bytes = dev["ws"].numel()
    sl0 = sl.to(DEV)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        binding.mtv_verify_step(tree, a)             # once outside capture: first-use set-up happens here
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            binding.mtv_verify_step(tree, a)
    for _ in range(2):                               # restore the inputs the step consumed, then replay
        dev["seq_lens"].copy_(sl0)
        for l in range(n_layers):
            kd[l].copy_(k0[l]); vd[l].copy_(v0[l])
        for n in ("tree_tok", "accept_len", "acc_nodes", "next_root"):
            dev[n].fill_(-7)
        dev["out_layers"].zero_()
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(dev["tree_tok"].cpu(), tt_ref)
        for name in ("accept_len", "best_path", "acc_nodes", "acc_tok", "next_root"):
            assert torch.equal(dev[name].cpu(), acc_ref[name]), name
        assert torch.equal(dev["seq_lens"].cpu(), sl + acc_ref["accept_len"] + 1)
        for l in range(n_layers):
            assert_close(dev["out_layers"][l], out_ref[l], "layer %d" % l)
    assert binding.mtv_device_error(tree) == 0


# ------------------------------------------------------------ append + RoPE
@pytest.mark.parametrize("Hq,Hkv,D,lens,theta", [(32, 8, 128, [8192], 0.0), (8, 2, 64, [0, 517, 30000], 500000.0)])
def test_tree_kv_append_rope(Hq, Hkv, D, lens, theta):
    tb, tree = make_tree("rank_prior", 4, (), 64)
    T, B = tree.T, len(lens)
    Lcap = max(lens) + T + 3
    q = synth.normal_bf16(5, 1, (B, T, Hq, D))
    k_new = synth.normal_bf16(5, 2, (B, T, Hkv, D))
    v_new = synth.normal_bf16(5, 3, (B, T, Hkv, D))
    kc = synth.normal_bf16(5, 4, (B, Hkv, Lcap, D))
    vc = synth.normal_bf16(5, 5, (B, Hkv, Lcap, D))
    q_ref, k_ref = ref.rope(q, k_new, lens, tb["depth"], theta or 10000.0)
    qd, kd, vd = q.to(DEV), kc.to(DEV), vc.to(DEV)
    status = _i32(B)
    sl = torch.tensor(lens, dtype=torch.int32, device=DEV)
    binding.tree_kv_append_rope(tree, qd, k_new.to(DEV), v_new.to(DEV), kd, vd, sl, rope_theta=theta, status=status)
    torch.cuda.synchronize()
    assert status.tolist() == [0] * B and sl.cpu().tolist() == lens
    assert_close(qd, q_ref, "rotated q")
    # one bf16 rounding of an fp32 result whose angle came from double precision: within an ulp of the checker
    assert (qd.double().cpu() - q_ref).abs().max().item() <= 2.0 ** -7 * q_ref.abs().max().item()
    for b, L in enumerate(lens):
        got_k = kd[b, :, L:L + T].cpu().permute(1, 0, 2)            # [T][Hkv][D]
        assert_close(got_k, k_ref[b], "rotated k in the cache")
        assert torch.equal(vd[b, :, L:L + T].cpu().permute(1, 0, 2), v_new[b])          # V copied bit-exactly
        assert torch.equal(kd[b, :, :L].cpu(), kc[b, :, :L]) and torch.equal(kd[b, :, L + T:].cpu(), kc[b, :, L + T:])
        assert torch.equal(vd[b, :, :L].cpu(), vc[b, :, :L]) and torch.equal(vd[b, :, L + T:].cpu(), vc[b, :, L + T:])


def test_tree_kv_append_rope_capacity():
    tb, tree = make_tree("cartesian", 2, (2, 2))
    T, B, Lcap = tree.T, 2, 20
    q = synth.normal_bf16(6, 1, (B, T, 4, 64), device=DEV)
    q0 = q.clone()
    kn, vn = synth.normal_bf16(6, 2, (B, T, 2, 64), device=DEV), synth.normal_bf16(6, 3, (B, T, 2, 64), device=DEV)
    kc, vc = torch.zeros(B, 2, Lcap, 64, dtype=torch.bfloat16, device=DEV), torch.zeros(B, 2, Lcap, 64, dtype=torch.bfloat16, device=DEV)
    status = _i32(B)
    binding.tree_kv_append_rope(tree, q, kn, vn, kc, vc, torch.tensor([Lcap - T + 1, 3], dtype=torch.int32, device=DEV),
                                status=status)
    torch.cuda.synchronize()
    assert status.tolist() == [binding.MTV_ERR_CAPACITY, 0]
    assert torch.equal(q[0], q0[0]) and not torch.equal(q[1], q0[1]) and bool((kc[0] == 0).all())


# ------------------------------------------------------- failure detection
def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    """No fault is provoked: a barrier nobody arrives on makes the kernels' bounded wait give up after about a
    second; the error word says so, clearing it works, and the next hot call runs and matches the oracle."""
    tb, tree = make_tree("cartesian", 2, (2, 2))
    assert binding.mtv_device_error(tree) == 0
    binding.mtv_selftest_wait_timeout(tree)
    torch.cuda.synchronize()
    assert binding.mtv_device_error(tree, clear=False) == binding.MTV_ERR_TIMEOUT     # sticky until cleared
    assert binding.mtv_device_error(tree) == binding.MTV_ERR_TIMEOUT
    assert binding.mtv_device_error(tree) == 0
    _attention_case(tb, tree, 1, 8, 2, 128, [300], seed=3)
    assert binding.mtv_device_error(tree) == 0


@pytest.mark.parametrize("lm_head", [False, True])
def test_verify_steps_chain_in_one_call(lm_head):
    """Three steps through mtv_verify_steps, enqueued by ONE call with every step's inputs laid out beforehand: each
    step appends its tree's K/V rows (all layers in one launch, rotary embedding at seq_lens + depth), attends,
    accepts and compacts; the next step's root token and prefix lengths reach it on the device only.  Every
    step's outputs and the final caches equal the checker stepping the same way."""
    B, H, V, Hq, Hkv, D, K, n_layers, n_steps = 2, 256, 2000, 8, 2, 128, 4, 3, 3
    tb, tree = make_tree("rank_prior", K, (), 64)
    T = tree.T
    lens0 = [131, 20]
    Lcap = max(lens0) + n_steps * (K + 1) + T
    seed = 177
    kc = [synth.normal_bf16(seed, 500 + l, (B, Hkv, Lcap, D)) for l in range(n_layers)]
    vc = [synth.normal_bf16(seed, 600 + l, (B, Hkv, Lcap, D)) for l in range(n_layers)]
    kd, vd = [t.to(DEV) for t in kc], [t.to(DEV) for t in vc]
    sl_ref = torch.tensor(lens0, dtype=torch.int32)
    sl_dev = sl_ref.to(DEV)
    root_ref = synth.uniform_int(seed, 7, B, 0, V - 1).to(torch.int32)
    root0_dev = root_ref.to(DEV)
    ws = workspace(tree, B, H, V, Hq, Hkv, D, Lcap)
    kp, vp = binding.cache_pointer_array(kd, DEV), binding.cache_pointer_array(vd, DEV)
    kph, vph = binding.cache_pointer_array(kd), binding.cache_pointer_array(vd)
    W_lm = synth.normal_bf16(seed, 901, (V, H))
    W_lm_dev = W_lm.to(DEV)
    steps, appends, keep, want = [], [], [], []
    for s in range(n_steps):
        # ---- the checker's step s, which also fixes the inputs of step s
        s_in = seed + 10 * s
        for attempt in range(20):
            hidden, W1, b1, W2, _ = synth.head_inputs(B, H, V, K, s_in)
            z = ref.heads_logits(hidden, W1, b1, W2)
            cand_ref, _, tt_ref, gap = ref.heads_candidates(z, root_ref, tb)
            if gap > 1e-5 * z.abs().max().item():
                break
            s_in += 1000
        q = torch.stack([synth.normal_bf16(s_in, 700 + l, (B, T, Hq, D)) for l in range(n_layers)])
        kn = torch.stack([synth.normal_bf16(s_in, 800 + l, (B, T, Hkv, D)) for l in range(n_layers)])
        vn = torch.stack([synth.normal_bf16(s_in, 900 + l, (B, T, Hkv, D)) for l in range(n_layers)])
        logits, planted = synth.planted_logits(B, T, V, K, tt_ref, tb["parent"], tb["rank"], s_in, p_accept=(0.9, 0.6))
        am_ref = ref.node_argmax(logits)
        out_ref = []
        for l in range(n_layers):
            q_rot, k_rot = ref.rope(q[l], kn[l], sl_ref.tolist(), tb["depth"])
            for b in range(B):
                L = int(sl_ref[b])
                kc[l][b, :, L:L + T] = k_rot[b].to(torch.bfloat16).permute(1, 0, 2)
                vc[l][b, :, L:L + T] = vn[l][b].permute(1, 0, 2)
            out_ref.append(ref.tree_attention(q_rot.to(torch.bfloat16), kc[l], vc[l], sl_ref, tb["mask"]))
        acc_ref = ref.tree_accept(am_ref, tt_ref, tb)
        assert torch.equal(acc_ref["accept_len"], planted)
        for l in range(n_layers):
            kc[l], new_len = ref.kv_compact(kc[l], sl_ref, acc_ref["accept_len"], acc_ref["acc_nodes"])
            vc[l], _ = ref.kv_compact(vc[l], sl_ref, acc_ref["accept_len"], acc_ref["acc_nodes"])
        want.append(dict(tree_tok=tt_ref, cand=cand_ref, out=out_ref, acc=acc_ref, seq_lens=new_len))
        # ---- this library's step s: buffers and the struct, nothing launched yet
        dev = dict(hidden=hidden.to(DEV), W1=W1.to(DEV), b1=b1.to(DEV), W2=W2.to(DEV), q_layers=q.to(DEV),
                   seq_lens=sl_dev, cand=_i32(B, tree.C), tree_tok=_i32(B, T),
                   out_layers=torch.zeros(n_layers, B, T, Hq, D, dtype=torch.bfloat16, device=DEV),
                   accept_len=_i32(B), best_path=_i32(B), acc_nodes=_i32(B, K + 1), acc_tok=_i32(B, K + 1),
                   next_root=_i32(B), status=_i32(B), k_caches=kp, v_caches=vp, k_caches_host=kph, v_caches_host=vph, ws=ws)
        if lm_head:     # the same next tokens as the argmax of an LM head over hidden states built around its rows
            x_final = (W_lm[am_ref.flatten().long()].float().reshape(B, T, H) +
                       0.3 * synth.normal_bf16(s_in, 902, (B, T, H)).float()).to(torch.bfloat16)
            am, zmax, z2 = ref.lm_head_argmax(x_final.reshape(B * T, H), W_lm)
            assert torch.equal(am.long(), am_ref.flatten().long()) and ((zmax - z2) > 1e-3 * zmax.abs().max()).all()
            dev["x_final"], dev["W_lm"] = x_final.to(DEV), W_lm_dev
        else:
            dev["logits"] = logits.to(DEV)
        if s == 0:
            dev["root_tok"] = root0_dev      # later steps: NULL = the previous step's next_root, on the device
        a = binding.StepArgs()
        a.B, a.H, a.V, a.Hq, a.Hkv, a.D, a.n_layers, a.Lcap = B, H, V, Hq, Hkv, D, n_layers, Lcap
        a.stride_b, a.stride_h, a.stride_t, a.scale = Hkv * Lcap * D, Lcap * D, D, 0.0
        for name, t in dev.items():
            setattr(a, name, t.data_ptr())
        a.ws_bytes = ws.numel()
        ap = binding.AppendArgs()
        kn_d, vn_d = kn.to(DEV), vn.to(DEV)
        ap.k_new_layers, ap.v_new_layers, ap.rope_theta = kn_d.data_ptr(), vn_d.data_ptr(), 0.0
        steps.append(a)
        appends.append(ap)
        keep.append((dev, kn_d, vn_d))
        sl_ref, root_ref = new_len, acc_ref["next_root"]
    # ---- one call, then everything is compared
    torch.cuda.synchronize()
    binding.mtv_verify_steps(tree, steps, appends)
    torch.cuda.synchronize()
    assert binding.mtv_device_error(tree) == 0
    for s in range(n_steps):
        dev, w = keep[s][0], want[s]
        assert dev["status"].tolist() == [0] * B
        assert torch.equal(dev["tree_tok"].cpu(), w["tree_tok"]) and torch.equal(dev["cand"].cpu(), w["cand"]), s
        for l in range(n_layers):
            assert_close(dev["out_layers"][l], w["out"][l], "step %d layer %d" % (s, l))
        for name in ("accept_len", "best_path", "acc_nodes", "acc_tok", "next_root"):
            assert torch.equal(dev[name].cpu(), w["acc"][name]), (s, name)
    assert torch.equal(sl_dev.cpu(), sl_ref) and int(sl_ref.min()) > min(lens0)
    for l in range(n_layers):
        for b in range(B):
            n, n0 = int(sl_ref[b]), lens0[b]
            assert torch.equal(vd[l][b, :, :n].cpu(), vc[l][b, :, :n])
            assert torch.equal(kd[l][b, :, :n0].cpu(), kc[l][b, :, :n0])
            assert_close(kd[l][b, :, :n], kc[l][b, :, :n], "compacted K rows")


def test_verify_steps_refuses_a_chain_without_a_first_root_or_with_two_length_arrays():
    tb, tree = make_tree("cartesian", 3, (4, 2, 2))
    a, b = binding.StepArgs(), binding.StepArgs()
    two = torch.zeros(2, 4, dtype=torch.int32, device=DEV)
    ptrs = torch.zeros(1, dtype=torch.int64)
    for x in (a, b):
        x.k_caches_host = x.v_caches_host = ptrs.data_ptr()
        x.seq_lens = two[0].data_ptr()
    with pytest.raises(binding.MtvError) as e:
        binding.mtv_verify_steps(tree, [a])                       # root_tok NULL in the first step
    assert e.value.code == -1
    a.root_tok = a.next_root = two[1].data_ptr()
    b.seq_lens = two[1].data_ptr()                                # the second step names other lengths
    with pytest.raises(binding.MtvError) as e:
        binding.mtv_verify_steps(tree, [a, b])                    # refused before the first step is enqueued
    assert e.value.code == -1
    torch.cuda.synchronize()
    assert binding.mtv_device_error(tree) == 0


def test_verify_steps_chain_replayed_from_a_cuda_graph():
    """The chain of steps is one static sequence of launches: captured once into a CUDA graph and replayed, it gives
    the results of the plain call (compared here) — no launch depends on anything the host would have to look at."""
    B, H, V, Hq, Hkv, D, K, n_layers, n_steps = 2, 256, 2000, 8, 2, 128, 4, 2, 2
    tb, tree = make_tree("rank_prior", K, (), 64)
    T = tree.T
    lens0 = torch.tensor([90, 33], dtype=torch.int32)
    Lcap = int(lens0.max()) + n_steps * (K + 1) + T
    seed = 211
    hidden, W1, b1, W2, root = [t.to(DEV) for t in synth.head_inputs(B, H, V, K, seed)]
    kc0 = [synth.normal_bf16(seed, 500 + l, (B, Hkv, Lcap, D)).to(DEV) for l in range(n_layers)]
    vc0 = [synth.normal_bf16(seed, 600 + l, (B, Hkv, Lcap, D)).to(DEV) for l in range(n_layers)]
    kd, vd = [t.clone() for t in kc0], [t.clone() for t in vc0]
    q0 = torch.stack([synth.normal_bf16(seed, 700 + l, (B, T, Hq, D)) for l in range(n_layers)]).to(DEV)
    kn = torch.stack([synth.normal_bf16(seed, 800 + l, (B, T, Hkv, D)) for l in range(n_layers)]).to(DEV)
    vn = torch.stack([synth.normal_bf16(seed, 900 + l, (B, T, Hkv, D)) for l in range(n_layers)]).to(DEV)
    logits = synth.normal_bf16(seed, 950, (B, T, V)).to(DEV)
    sl = lens0.to(DEV)
    ws = workspace(tree, B, H, V, Hq, Hkv, D, Lcap)
    kp, vp = binding.cache_pointer_array(kd, DEV), binding.cache_pointer_array(vd, DEV)
    kph, vph = binding.cache_pointer_array(kd), binding.cache_pointer_array(vd)
    steps, appends, bufs = [], [], []
    for s in range(n_steps):
        dev = dict(hidden=hidden, W1=W1, b1=b1, W2=W2, q_layers=q0.clone(), logits=logits, seq_lens=sl,
                   cand=_i32(B, tree.C), tree_tok=_i32(B, T),
                   out_layers=torch.zeros(n_layers, B, T, Hq, D, dtype=torch.bfloat16, device=DEV),
                   accept_len=_i32(B), best_path=_i32(B), acc_nodes=_i32(B, K + 1), acc_tok=_i32(B, K + 1),
                   next_root=_i32(B), status=_i32(B), k_caches=kp, v_caches=vp, k_caches_host=kph, v_caches_host=vph, ws=ws)
        if s == 0:
            dev["root_tok"] = root
        a = binding.StepArgs()
        a.B, a.H, a.V, a.Hq, a.Hkv, a.D, a.n_layers, a.Lcap = B, H, V, Hq, Hkv, D, n_layers, Lcap
        a.stride_b, a.stride_h, a.stride_t, a.scale = Hkv * Lcap * D, Lcap * D, D, 0.0
        for name, t in dev.items():
            setattr(a, name, t.data_ptr())
        a.ws_bytes = ws.numel()
        ap = binding.AppendArgs()
        ap.k_new_layers, ap.v_new_layers, ap.rope_theta = kn.data_ptr(), vn.data_ptr(), 0.0
        steps.append(a), appends.append(ap), bufs.append(dev)

    def reset():
        sl.copy_(lens0)
        for l in range(n_layers):
            kd[l].copy_(kc0[l]), vd[l].copy_(vc0[l])
        for dev in bufs:
            dev["q_layers"].copy_(q0)            # the append rotates the queries in place
    names = ("cand", "tree_tok", "out_layers", "accept_len", "best_path", "acc_nodes", "acc_tok", "next_root")
    reset()
    binding.mtv_verify_steps(tree, steps, appends)
    torch.cuda.synchronize()
    want = [{n: dev[n].clone() for n in names} for dev in bufs]
    want_sl, want_k = sl.clone(), [t.clone() for t in kd]
    assert int(want_sl.min()) > int(lens0.min()) and binding.mtv_device_error(tree) == 0
    # the same chain, captured and replayed
    reset()
    for dev in bufs:
        for n in names:
            dev[n].zero_()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            binding.mtv_verify_steps(tree, steps, appends, stream=side)
    torch.cuda.current_stream().wait_stream(side)
    reset()                                      # (capture launches nothing, but keep the state explicit)
    graph.replay()
    torch.cuda.synchronize()
    assert binding.mtv_device_error(tree) == 0
    for dev, w_ in zip(bufs, want):
        for n in names:
            assert torch.equal(dev[n], w_[n]), n    # the same kernels on the same inputs: bit-identical
    assert torch.equal(sl, want_sl)
    for l in range(n_layers):
        assert torch.equal(kd[l], want_k[l])


def _random_tree(g, K, T_target):
    """A random ancestor-closed tree with up to T_target nodes (root included): nodes are added one at a time as the next
    unused rank under a random existing node of depth < K."""
    nodes, children = [()], {(): 0}
    while len(nodes) < T_target:
        cand = [n for n in nodes if len(n) < K and children[n] < 10]
        if not cand:
            break
        parent = cand[int(torch.randint(0, len(cand), (1,), generator=g))]
        child = parent + (children[parent],)
        children[parent] += 1
        children[child] = 0
        nodes.append(child)
    return [list(n) for n in nodes[1:]]


@pytest.mark.parametrize("case", range(20))
def test_attention_random_shapes(case):
    """Seeded random problems: tree shape and size, head counts and head size, batch, prefix lengths (empty ones
    included), cache capacity and a padded (strided) cache — the shapes no hand-picked case covers."""
    from oracle import tree as otree
    g = torch.Generator().manual_seed(1000 + case)
    pick = lambda xs: xs[int(torch.randint(0, len(xs), (1,), generator=g))]
    D = pick([64, 128, 128])
    Hkv = pick([1, 2, 4, 8])
    G = pick([1, 2, 4, 8])
    if case >= 16:
        G = [3, 5, 6, 7][case - 16]              # group sizes that do not divide the 128 rows of a tile
        D, Hkv = 128, pick([1, 2, 4])
    Hq = Hkv * G
    K = pick([1, 2, 3, 4, 5])
    T_target = pick([2, 5, 17, 33, 64, 65, 97, 128])
    nodes = _random_tree(g, K, T_target)
    tb = otree.tables([tuple(n) for n in nodes], K)
    tree = binding.tree_build_static(K, nodes, upload=True)
    T = tree.T
    assert T == tb["T"]
    B = pick([1, 1, 2, 3, 5])
    hi = pick([40, 300, 1300])
    lens = [int(torch.randint(0, hi + 1, (1,), generator=g)) for _ in range(B)]
    if case % 4 == 0:
        lens[0] = 0
    pad = pick([0, 0, 8, 40])
    Lcap = max(lens) + T + pick([0, 1, 77])
    _attention_case(tb, tree, B, Hq, Hkv, D, lens, seed=2000 + case, Lcap=Lcap, pad=pad)
    assert binding.mtv_device_error(tree) == 0


@pytest.mark.parametrize("case", range(8))
def test_heads_accept_compaction_random_trees(case):
    """The integer part of a step on random trees (shapes the two generators never produce: uneven fan-out, leaves at
    every depth): candidates and tree tokens from the heads, acceptance of planted walks, compaction of the accepted rows;
    all bit-exact against the checker."""
    from oracle import tree as otree
    g = torch.Generator().manual_seed(3000 + case)
    pick = lambda xs: xs[int(torch.randint(0, len(xs), (1,), generator=g))]
    K = pick([2, 3, 4, 5])
    nodes = _random_tree(g, K, pick([7, 20, 64, 100, 128]))
    tb = otree.tables([tuple(n) for n in nodes], K)
    tree = binding.tree_build_static(K, nodes, upload=True)
    T, B = tree.T, pick([1, 2, 4, 7])
    H, V = pick([64, 192, 520]), pick([300, 1001, 4096])
    # ---- heads
    seed, inp, _, cand_ref, cl_ref, tt_ref = oracle_heads_with_margin(B, H, V, K, tb, 3100 + case)
    hidden, W1, b1, W2, root = [t.to(DEV) for t in inp]
    ws = workspace(tree, B, H, V, 8, 2, 64, 64 + T)
    cand, tt = _i32(B, tree.C), _i32(B, T)
    binding.medusa_heads_topk(tree, hidden, W1, b1, W2, root, cand, None, tt, ws)
    assert torch.equal(cand.cpu(), cand_ref) and torch.equal(tt.cpu(), tt_ref), seed
    # ---- acceptance of planted walks
    logits, planted = synth.planted_logits(B, T, V, K, tt_ref, tb["parent"], tb["rank"], seed, p_accept=(0.85, 0.5))
    want = ref.tree_accept(ref.node_argmax(logits), tt_ref, tb)
    assert torch.equal(want["accept_len"], planted)
    outs = dict(accept_len=_i32(B), best_path=_i32(B), acc_nodes=_i32(B, K + 1), acc_tok=_i32(B, K + 1), next_root=_i32(B))
    binding.tree_accept(tree, logits.to(DEV), tt, outs["accept_len"], outs["best_path"], outs["acc_nodes"], outs["acc_tok"],
                        outs["next_root"], ws)
    for name, t in outs.items():
        assert torch.equal(t.cpu(), want[name]), name
    # ---- compaction of those rows, two layers
    Hkv, D = 2, 64
    lens = [int(torch.randint(0, 60, (1,), generator=g)) for _ in range(B)]
    Lcap = 64 + T
    caches = [synth.normal_bf16(seed, 40 + l, (B, Hkv, Lcap, D)) for l in range(4)]
    dev_c = [c.to(DEV) for c in caches]
    kp, vp = binding.cache_pointer_array(dev_c[:2], DEV), binding.cache_pointer_array(dev_c[2:], DEV)
    sl = torch.tensor(lens, dtype=torch.int32, device=DEV)
    status = _i32(B)
    binding.kv_compact_accepted(tree, kp, vp, 2, B, Hkv, D, (Hkv * Lcap * D, Lcap * D, D), Lcap, sl, outs["accept_len"],
                                outs["acc_nodes"], status=status)
    torch.cuda.synchronize()
    assert status.tolist() == [0] * B and binding.mtv_device_error(tree) == 0
    for c, dc in zip(caches, dev_c):
        want_c, new_len = ref.kv_compact(c, lens, want["accept_len"], want["acc_nodes"])
        for b in range(B):
            assert torch.equal(dc[b, :, :new_len[b]].cpu(), want_c[b, :, :new_len[b]])
    assert torch.equal(sl.cpu(), torch.tensor(lens, dtype=torch.int32) + want["accept_len"] + 1)
