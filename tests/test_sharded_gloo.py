"""The split of one sequence's step over ranks, on CPU: two gloo ranks (world size 2) run the partition arithmetic
and the collectives of `paper_2603_03383_b200.sharded`; each rank's slice is computed by the CPU checker (the
library's kernels need a GPU), the gathered pieces are merged by the rule the merge kernels implement, written out
here by definition, and the result must equal the checker on the whole problem: identical candidate ids, identical
attention rows."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _merge_by_definition(cand_all, logit_all, v_slab, tb, root):
    """Per head: all shards' (logit, global id) entries, the k_d best by (logit descending, id ascending)."""
    world, B, C = cand_all.shape
    cand = torch.zeros(B, C, dtype=torch.int32)
    cand[:, 0] = root
    for b in range(B):
        for d, (kd, off) in enumerate(zip(tb["k_d"], tb["offset"])):
            entries = [(-logit_all[r, b, off - 1 + s].item(), cand_all[r, b, off + s].item() + r * v_slab)
                       for r in range(world) for s in range(kd)]
            entries.sort()
            cand[b, off:off + kd] = torch.tensor([e[1] for e in entries[:kd]], dtype=torch.int32)
    return cand


def _worker(rank, world, port):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    from oracle import reference as ref, tree as otree
    from paper_2603_03383_b200 import sharded, synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    K, B, H, V, Hq, Hkv, D = 4, 2, 64, 1001, 8, 4, 64
    tb = otree.tables(otree.rank_prior(K, 64), K)
    p = sharded.plan(rank, world, V, Hq, Hkv, max_kd=max(tb["k_d"]))
    # ---- heads by vocabulary slab
    hidden, W1, b1, W2, root = synth.head_inputs(B, H, V, K, seed=91)
    z_local = ref.heads_logits(hidden, W1, b1, W2[:, p.v_lo:p.v_hi].contiguous())
    cand_l, logit_l, _, _ = ref.heads_candidates(z_local, root, tb)
    cand_all = sharded.gather(cand_l, world)
    logit_all = sharded.gather(torch.as_tensor(logit_l, dtype=torch.float64), world)
    cand = _merge_by_definition(cand_all, logit_all, p.v_slab, tb, root)
    z = ref.heads_logits(hidden, W1, b1, W2)
    cand_full, _, tt_full, _ = ref.heads_candidates(z, root, tb)
    tree_tok = cand[:, torch.tensor(tb["tree_indices"])]
    # ---- attention by KV head
    lens = [70, 9]
    Lcap = max(lens) + tb["T"]
    q, k, v = synth.attention_inputs(B, tb["T"], Hq, Hkv, D, Lcap, 92)
    sl = torch.tensor(lens, dtype=torch.int32)
    out_l = ref.tree_attention(q[:, :, p.q_lo:p.q_lo + p.hq_local].contiguous(),
                               k[:, p.kv_lo:p.kv_lo + p.hkv_local].contiguous(),
                               v[:, p.kv_lo:p.kv_lo + p.hkv_local].contiguous(), sl, tb["mask"])
    gathered = sharded.gather(out_l, world)                         # [world][B][T][hq_local][D]
    out = gathered.permute(1, 2, 0, 3, 4).reshape(B, tb["T"], Hq, D)
    out_full = ref.tree_attention(q, k, v, sl, tb["mask"])
    dist.barrier()
    res = dict(plan=(p.v_lo, p.v_hi, p.v_slab, p.q_lo, p.hq_local, p.kv_lo, p.hkv_local),
               cand_equal=bool(torch.equal(cand, cand_full)), tt_equal=bool(torch.equal(tree_tok, tt_full)),
               attn_equal=bool(torch.equal(out, out_full)), cand=cand.tolist())
    _RESULTS[rank] = res
    dist.destroy_process_group()


_RESULTS = {}


def _entry(rank, world, port, shared):
    _worker(rank, world, port)
    shared[rank] = _RESULTS[rank]


def test_two_ranks_split_heads_and_attention_and_agree_with_the_whole():
    world = 2
    with mp.Manager() as mgr:
        shared = mgr.dict()
        mp.spawn(_entry, args=(world, 29541, shared), nprocs=world, join=True)
        res = dict(shared)
    assert res[0]["plan"] == (0, 504, 504, 0, 4, 0, 2) and res[1]["plan"] == (504, 1001, 504, 4, 4, 2, 2)
    for r in range(world):
        assert res[r]["cand_equal"] and res[r]["tt_equal"] and res[r]["attn_equal"], r
    assert res[0]["cand"] == res[1]["cand"]                        # every rank ends with the same candidates


def test_plan_partitions_and_refuses_what_cannot_be_split():
    sys.path.insert(0, ROOT)
    from paper_2603_03383_b200 import sharded
    V, world = 131072, 8
    plans = [sharded.plan(r, world, V, 32, 8, max_kd=10) for r in range(world)]
    assert [p.v_lo for p in plans] == [r * 16384 for r in range(world)] and plans[-1].v_hi == V
    assert sorted(h for p in plans for h in range(p.q_lo, p.q_lo + p.hq_local)) == list(range(32))
    assert sorted(h for p in plans for h in range(p.kv_lo, p.kv_lo + p.hkv_local)) == list(range(8))
    # ragged: slabs rounded up to 8 rows, the last one shorter, all rows covered exactly once
    plans = [sharded.plan(r, 3, 2000, 12, 6) for r in range(3)]
    assert [(p.v_lo, p.v_hi) for p in plans] == [(0, 672), (672, 1344), (1344, 2000)]
    with pytest.raises(ValueError):
        sharded.plan(0, 3, 1000, 32, 8)                            # three ranks do not divide eight KV heads
    with pytest.raises(ValueError):
        sharded.plan(0, 4, 25, 8, 4, max_kd=10)                    # last slab: 1 row < top-10
    with pytest.raises(ValueError):
        sharded.plan(0, 32, 100000, 32, 32)                        # beyond the merge kernels' limit
