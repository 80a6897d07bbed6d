"""Benchmark of the static-tree verification step (tree-verify steps/s, 7B shape, 8k context).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload long] [--layers 32]
    python bench.py --impl reference ...      # the fp64 CPU checker, timed on the host cores

A step is one pass of the whole path over one batch of synthetic input: Medusa heads +
top-k + tree expansion, tree attention for each of `layers` distinct KV caches, acceptance,
in-place KV compaction (followed by a device-side reset of seq_lens so shapes stay fixed).
With N > 1 (torchrun) every rank verifies its own independent sequences: no collective on
the data path, weak scaling.  Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "tree_verify_steps_per_s"
UNIT = "steps/s"
PAPER_CONTEXT = "paper: 1.35x end-to-end speedup on its NPU at sequence length 128 (context, not comparable)"


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="long")
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-taps", action="store_true", help="skip per-kernel event timing")
    ap.add_argument("--launch", default="graph", choices=["graph", "stream"],
                    help="timed steps: replay of one captured CUDA graph per step, or plain stream launches")
    ap.add_argument("--repeats", type=int, default=5, help="timed repeats of --steps; the median is reported")
    ap.add_argument("--no-other-workloads", action="store_true", help="skip the short runs of the other four configurations")
    ap.add_argument("--no-parity-gate", action="store_true", help="skip the checks against the CPU checker before timing")
    ap.add_argument("--shard", default="sequence", choices=["sequence", "kvhead"],
                    help="how N GPUs share the work: 'sequence' = every rank verifies its own sequences (no collective, "
                         "weak scaling); 'kvhead' = all ranks work on the SAME sequences, heads split by vocabulary slab "
                         "and attention by KV head with an all-gather after each (strong scaling)")
    ap.add_argument("--overhead-sweep", action="store_true",
                    help="instead of the step benchmark: time tree attention (T nodes) against single-token decode "
                         "attention (a root-only tree) over prefix lengths, the attention part of the paper's overhead ratio")
    return ap.parse_args()


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"], source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, source="fallback")


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu captures summarised under
# profiles/, keyed by tap name, with the hash of the kernel's source at capture time: a changed kernel reports null.
NCU_TRAFFIC = {
    "attn_partial": ("attention_tc.cu", "3b39f055e83c8c7d", 34.4122e6 + 0.0003e6),
    "heads_vocab_topk": ("heads.cu", "914e411d83fc386f", 4.2995e9),
    "lm_head_argmax": ("lm_head.cu", "8eac35b20edf1166", 1.0795e9),
}


def measured_traffic(kernel):
    import hashlib
    if kernel not in NCU_TRAFFIC:
        return None
    fname, digest, traffic = NCU_TRAFFIC[kernel]
    path = os.path.join(ROOT, "paper_2603_03383_b200", "csrc", fname)
    try:
        with open(path, "rb") as f:
            now = hashlib.sha256(f.read()).hexdigest()[:16]
    except OSError:
        return None
    return traffic if now == digest else None


def algorithmic_bytes(w, tree, n_layers, lens):
    """Bytes the method itself must move per step (weights, K/V rows, Q, O, logits)."""
    K, H, V, B, T = w.K, w.H, w.V, w.B, tree.T
    heads = K * (H * H + H + V * H) * 2
    vocab = K * V * H * 2
    attn = 0
    for L in lens:
        attn += 2 * (L + T) * w.Hkv * w.D * 2 + 2 * T * w.Hq * w.D * 2
    accept = B * T * V * 2
    compact = n_layers * B * w.Hkv * 2 * K * w.D * 2 * 2
    return dict(heads=heads, heads_vocab=vocab, attn_per_layer=attn, accept=accept, compact=compact,
                step=heads + n_layers * attn + accept + compact)


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.QUERY,
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        self.thread.join(timeout=2)
        sm = [float(r[1]) for r in self.rows if len(r) >= 9 and r[1].replace(".", "").isdigit()]
        mx = [float(r[2]) for r in self.rows if len(r) >= 9 and r[2].replace(".", "").isdigit()]
        reasons = set()
        for r in self.rows:
            if len(r) < 9:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


def rank_seed(w, rank):
    """Seed of the sequences rank `rank` verifies (ranks work on independent sequences)."""
    return w.seed + 7919 * rank


def max_over_ranks(value, world, device=None):
    """Largest `value` over all ranks (the job is as slow as its slowest rank)."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.item()


def build_problem(w, n_layers, device, seed=None):
    """Everything one rank needs, resident on `device`.  Returns a dict."""
    import torch
    from paper_2603_03383_b200 import binding, synth
    nodes = (binding.tree_gen_cartesian(list(w.topk)) if w.tree == "cartesian"
             else binding.tree_gen_rank_prior(w.K, w.T, w.R_max))
    tree = binding.tree_build_static(w.K, nodes, upload=True)
    T, B = tree.T, w.B
    seed = w.seed if seed is None else seed
    lens = synth.seq_lens(w, seed=seed)
    Lcap = int(w.L_hi) + T
    seed = w.seed if seed is None else seed
    hidden, W1, b1, W2, root = synth.head_inputs(B, w.H, w.V, w.K, seed, device=device)
    ws = torch.empty(binding.mtv_workspace_bytes(tree, B, w.H, w.V, w.Hq, w.Hkv, w.D, Lcap), dtype=torch.uint8,
                     device=device)
    i32 = lambda *s: torch.zeros(*s, dtype=torch.int32, device=device)
    d = dict(tree=tree, lens=lens, Lcap=Lcap, hidden=hidden, W1=W1, b1=b1, W2=W2, root_tok=root, ws=ws,
             cand=i32(B, tree.C), cand_logit=torch.zeros(B, tree.C - 1, device=device), tree_tok=i32(B, T),
             accept_len=i32(B), best_path=i32(B), acc_nodes=i32(B, w.K + 1), acc_tok=i32(B, w.K + 1),
             next_root=i32(B), status=i32(B), seq_lens=lens.to(device), seq_lens0=lens.to(device))
    # tree tokens from one heads pass, then the planted base-model logits
    binding.medusa_heads_topk(tree, hidden, W1, b1, W2, root, d["cand"], d["cand_logit"], d["tree_tok"], ws)
    torch.cuda.synchronize()
    logits, planted = synth.planted_logits(B, T, w.V, w.K, d["tree_tok"].cpu(), tree.parent, tree.rank, seed,
                                           p_accept=w.p_accept, device=device)
    d["logits"], d["planted"] = logits, planted
    qs, ks, vs = [], [], []
    for l in range(n_layers):
        q, k, v = synth.attention_inputs(B, T, w.Hq, w.Hkv, w.D, Lcap, seed, layer=l, device=device)
        qs.append(q), ks.append(k), vs.append(v)
    d["q_layers"] = torch.stack(qs)
    d["k_list"], d["v_list"] = ks, vs
    d["out_layers"] = torch.zeros_like(d["q_layers"])
    d["k_caches"], d["v_caches"] = binding.cache_pointer_array(ks, device), binding.cache_pointer_array(vs, device)
    d["k_caches_host"], d["v_caches_host"] = binding.cache_pointer_array(ks), binding.cache_pointer_array(vs)
    a = binding.StepArgs()
    a.B, a.H, a.V, a.Hq, a.Hkv, a.D, a.n_layers, a.Lcap = B, w.H, w.V, w.Hq, w.Hkv, w.D, n_layers, Lcap
    a.stride_b, a.stride_h, a.stride_t, a.scale = w.Hkv * Lcap * w.D, Lcap * w.D, w.D, 0.0
    for name in ("hidden", "W1", "b1", "W2", "root_tok", "q_layers", "k_caches", "v_caches", "k_caches_host",
                 "v_caches_host", "logits", "seq_lens", "cand", "cand_logit", "tree_tok", "out_layers", "accept_len",
                 "best_path", "acc_nodes", "acc_tok", "next_root", "status", "ws"):
        setattr(a, name, d[name].data_ptr())
    a.ws_bytes = ws.numel()
    d["args"] = a
    return d


LAUNCHES_PER_STEP = lambda n_layers: 2 + n_layers + 2 + 2


def workload_string(w, T, n_layers):
    """The description of a workload, identical in both arms."""
    return "%s: B=%d prefix=%s H=%d Hq/Hkv=%d/%d D=%d V=%d K=%d T=%d layers=%d" % (
        w.name, w.B, w.L_lo if w.L_lo == w.L_hi else "U[%d,%d]" % (w.L_lo, w.L_hi), w.H, w.Hq, w.Hkv, w.D, w.V,
        w.K, T, n_layers)


class ParityError(RuntimeError):
    pass


def parity_gate(w, P, n_layers, rows=96):
    """Checks of this run's own results against the CPU checker, before anything is timed: sampled attention rows
    of one layer, the tree tokens of the heads pass, and the acceptance outputs of one whole step.  Raises ParityError."""
    import torch
    from oracle import reference as ref
    from oracle import tree as otree
    from paper_2603_03383_b200 import binding
    tree, B, T = P["tree"], w.B, P["tree"].T
    nodes = otree.cartesian(w.topk) if w.tree == "cartesian" else otree.rank_prior(w.K, w.T, w.R_max)
    tb = otree.tables(nodes, w.K)
    t0 = time.perf_counter()
    report = {}
    # attention: sampled (sequence, node, head) rows of the last layer, against the cache as it is now
    l = n_layers - 1
    total = B * T * w.Hq
    sel = sorted({(i * 2654435761) % total for i in range(rows)})
    rws = [(r // (T * w.Hq), (r // w.Hq) % T, r % w.Hq) for r in sel]
    out = torch.zeros_like(P["q_layers"][l])
    binding.tree_verify_attention(tree, P["q_layers"][l], P["k_list"][l], P["v_list"][l], P["seq_lens0"], out, P["ws"])
    torch.cuda.synchronize()
    want = ref.tree_attention(P["q_layers"][l].cpu(), P["k_list"][l].cpu(), P["v_list"][l].cpu(), P["lens"], tb["mask"],
                              rows=rws)
    got = torch.stack([out[b, i, h].cpu() for b, i, h in rws]).double()
    err = (got - want).abs().max().item()
    tol = 1e-2 * want.abs().max().item() + 1e-3
    if not err <= tol:
        raise ParityError("attention rows: max |err| %.3e above %.3e" % (err, tol))
    report["attention"] = "%d rows of layer %d: max |err| %.2e <= %.2e" % (len(rws), l, err, tol)
    # one whole step on the device
    P["seq_lens"].copy_(P["seq_lens0"])
    binding.mtv_verify_step(tree, P["args"])
    torch.cuda.synchronize()
    if any(P["status"].cpu().tolist()):
        raise ParityError("status %s" % P["status"].cpu().tolist())
    # tree tokens: the checker's heads + top-k + expansion on the same inputs
    z = ref.heads_logits(P["hidden"].cpu(), P["W1"].cpu(), P["b1"].cpu(), P["W2"].cpu())
    _, _, tt_ref, _ = ref.heads_candidates(z, P["root_tok"].cpu(), tb)
    del z
    if not torch.equal(P["tree_tok"].cpu(), tt_ref):
        raise ParityError("tree_tok differs from the checker's")
    report["tree_tok"] = "bit-exact (%d x %d)" % (B, T)
    # acceptance: the checker on the stored logits, and the planted lengths
    acc_ref = ref.tree_accept(ref.node_argmax(P["logits"].cpu()), tt_ref, tb)
    for name in ("accept_len", "best_path", "acc_nodes", "acc_tok", "next_root"):
        if not torch.equal(P[name].cpu(), acc_ref[name]):
            raise ParityError("%s differs from the checker's" % name)
    if not torch.equal(P["accept_len"].cpu(), P["planted"].to(torch.int32).cpu()):
        raise ParityError("accept_len differs from the planted lengths")
    if not torch.equal(P["seq_lens"].cpu(), P["lens"] + acc_ref["accept_len"] + 1):
        raise ParityError("seq_lens not advanced by accept_len + 1")
    report["acceptance"] = "bit-exact, equals the planted lengths %s" % P["planted"].tolist()
    report["seconds"] = round(time.perf_counter() - t0, 2)
    return report


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2603_03383_b200 import binding, synth
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    w = synth.WORKLOADS[args.workload]
    n_layers = args.layers
    P = build_problem(w, n_layers, dev, seed=rank_seed(w, rank))
    tree, a = P["tree"], P["args"]
    K_steps, W_steps = args.steps, max(args.warmup, 3)
    gate = None
    if rank == 0 and not args.no_parity_gate:
        # nothing is timed, and no value printed, unless this run's own results match the CPU checker
        try:
            gate = parity_gate(w, P, n_layers)
        except ParityError as e:
            print(json.dumps({"metric": METRIC, "value": None, "unit": UNIT, "error": "parity gate failed: %s" % e,
                              "config": {"workload": workload_string(w, tree.T, n_layers)}}))
            sys.exit(1)

    def step():
        P["seq_lens"].copy_(P["seq_lens0"])          # shapes stay fixed from step to step
        binding.mtv_verify_step(tree, a)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(W_steps):
        step()
    barrier()
    sampler = ClockSampler(local)     # nvidia-smi takes a while to start: it runs from here to the end of the timed steps
    if rank == 0:
        sampler.start()
    # per-kernel durations: an untimed pass of stream launches with the library's event taps
    taps = None
    tap_steps = min(K_steps, 10)
    if not args.no_taps:
        taps = binding.KernelTaps(tap_steps * n_layers)
        taps.__enter__()
        for _ in range(tap_steps):
            step()
        barrier()
        taps.__exit__()
    # the timed steps
    run_step = step
    if args.launch == "graph":
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                step()
        torch.cuda.current_stream().wait_stream(side)
        run_step = graph.replay
        for _ in range(2):
            run_step()
        barrier()
    # the attention calls of one step back to back, as they run in the timed steps (no events in between)
    attn_block_ms = None
    if not args.no_taps:
        def attn_block():
            for l in range(n_layers):
                binding.tree_verify_attention(tree, P["q_layers"][l], P["k_list"][l], P["v_list"][l], P["seq_lens0"],
                                              P["out_layers"][l], P["ws"])
        attn_block()
        barrier()
        b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        b0.record()
        for _ in range(tap_steps):
            attn_block()
        b1.record()
        barrier()
        attn_block_ms = b0.elapsed_time(b1) / (tap_steps * n_layers)
    # the timed region: `repeats` runs of exactly K_steps steps, each bracketed by a barrier and a device synchronise;
    # the reported time is the median run (max over ranks per run)
    runs_ms = []
    for _ in range(max(1, args.repeats)):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        for _ in range(K_steps):
            run_step()
        e1.record()
        barrier()
        runs_ms.append(max_over_ranks(e0.elapsed_time(e1), world, dev))
    clocks = sampler.stop() if rank == 0 else None
    ms_total = statistics.median(runs_ms)
    ms_step = ms_total / K_steps
    value = world * 1000.0 / ms_step
    mean_tokens = (P["accept_len"].float().mean().item() + 1.0)

    # end to end: per-step tensors start in pinned host memory, results end there
    names_in = ["hidden", "root_tok", "q_layers", "logits"]
    names_out = ["tree_tok", "out_layers", "accept_len", "best_path", "acc_nodes", "acc_tok", "next_root", "seq_lens"]
    hb = binding.StepArgs()
    host = {n: P[n].cpu().pin_memory() for n in names_in + names_out}
    for n, t in host.items():
        setattr(hb, n, t.data_ptr())
    h2d = sum(host[n].numel() * host[n].element_size() for n in names_in)
    d2h = sum(host[n].numel() * host[n].element_size() for n in names_out)
    e2e_steps = max(3, min(K_steps, 20))
    for _ in range(2):
        P["seq_lens"].copy_(P["seq_lens0"])
        binding.mtv_verify_step_host(tree, a, hb)
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        P["seq_lens"].copy_(P["seq_lens0"])
        binding.mtv_verify_step_host(tree, a, hb)
    torch.cuda.synchronize()
    e2e_s = (time.perf_counter() - t0) / e2e_steps
    e2e_s = max_over_ranks(e2e_s, world, dev)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    pk = peaks()
    alg = algorithmic_bytes(w, tree, n_layers, P["lens"].tolist())
    lm = time_lm_head(tree, w, P, dev)
    lm_step_ms = time_step_with_lm_head(tree, w, P, dev, args.launch, max(3, min(K_steps, 20)))
    chain_ms = time_chained_steps(tree, w, P, dev, args.launch, max(3, min(K_steps, 10)))
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K_steps, "warmup": W_steps,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": workload_string(w, tree.T, n_layers),
            "timing": "median of %d runs of %d steps (%s ms each)" % (
                len(runs_ms), K_steps, ", ".join("%.1f" % r for r in runs_ms)),
            "l2": "inputs larger than L2: %.2f GB streamed per step, %d distinct KV caches" % (alg["step"] / 1e9, n_layers),
            "launch": ("one CUDA graph per step (captured mtv_verify_step), replayed" if args.launch == "graph"
                       else "stream launches through mtv_verify_step"), "seed": w.seed,
            "mean_tokens_per_step": mean_tokens, "context": PAPER_CONTEXT},
        "clocks": clocks,
        "e2e": {"value": world / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps},
        "gpu_launches": K_steps * LAUNCHES_PER_STEP(n_layers),
        "device_error": binding.mtv_device_error(tree, clear=False),
        "parity_gate": gate if gate is not None else "skipped",
        "step_roofline": {"algorithmic_bytes": alg["step"], "achieved_gbs": alg["step"] / ms_step / 1e6,
                          "frac_of_measured": alg["step"] / ms_step / 1e6 / pk["hbm_gbs"],
                          "frac_of_8tbs": alg["step"] / ms_step / 1e6 / 8000.0},
    }
    if taps:
        tm = taps.times_ms()
        avg = {k: (sum(v) / len(v) if v else None) for k, v in tm.items()}
        per_step = {k: (sum(v) / tap_steps if v else 0.0) for k, v in tm.items()}
        out["kernel_ms_per_step"] = per_step
        dom = max(per_step, key=per_step.get)
        bytes_of = {"heads_vocab_topk": alg["heads_vocab"], "attn_partial": alg["attn_per_layer"],
                    "argmax_partial": alg["accept"], "heads_resblock": alg["heads"] - alg["heads_vocab"]}
        ach = bytes_of.get(dom, 0) / avg[dom] / 1e6
        out["roofline"] = {"kernel": dom, "bound": "hbm", "achieved": ach, "peak": pk["hbm_gbs"], "unit": "GB/s",
                           "frac": ach / pk["hbm_gbs"], "traffic": measured_traffic(dom), "peak_source": pk["source"],
                           "algorithmic_bytes_per_launch": bytes_of.get(dom, 0), "avg_launch_ms": avg[dom]}
        a_ms = (avg["attn_partial"] or 0.0) + (avg["attn_combine"] or 0.0)
        if attn_block_ms is not None:
            # per-launch duration of the attention call inside a run of back-to-back launches (events around
            # the run, not around each launch: a pair of events per launch adds several microseconds)
            out["attn_us_per_call_back_to_back"] = attn_block_ms * 1e3
            if attn_block_ms < a_ms:
                a_ms = attn_block_ms
                if dom == "attn_partial":
                    ach = bytes_of[dom] / a_ms / 1e6
                    out["roofline"].update(achieved=ach, frac=ach / pk["hbm_gbs"], avg_launch_ms=a_ms,
                                           timing="CUDA events around %d back-to-back launches" % (tap_steps * n_layers))
        out["gpu_launches"] = sum(len(v) for v in tm.values()) * K_steps // tap_steps
        ach = alg["attn_per_layer"] / a_ms / 1e6
        out["roofline_attn"] = {"kernel": "tree_verify_attention (all its launches)", "bound": "hbm", "achieved": ach,
                                "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": ach / pk["hbm_gbs"],
                                "frac_of_8tbs": ach / 8000.0, "avg_call_us": a_ms * 1e3,
                                "algorithmic_bytes_per_launch": alg["attn_per_layer"]}
    lm_bytes = w.V * w.H * 2 + 2 * w.B * tree.T * w.H
    out["beyond_the_step"] = {"lm_head_argmax": {
        "what": "LM head with fused per-node argmax + acceptance from its keys (not part of the timed step)",
        "us_per_call": lm * 1e3, "algorithmic_bytes": lm_bytes, "achieved_gbs": lm_bytes / lm / 1e6,
        "frac_of_measured_hbm": lm_bytes / lm / 1e6 / pk["hbm_gbs"],
        "tflops": 2.0 * w.B * tree.T * w.V * w.H / lm / 1e9},
        "step_with_lm_head": {
            "what": "the same step with the acceptance fed by the fused LM head (x_final, W_lm) instead of stored logits",
            "ms_per_step": lm_step_ms, "steps_per_s": 1000.0 / lm_step_ms,
            "algorithmic_bytes": alg["step"] - alg["accept"] + lm_bytes,
            "frac_of_measured_hbm": (alg["step"] - alg["accept"] + lm_bytes) / lm_step_ms / 1e6 / pk["hbm_gbs"]},
        "chained_steps_with_append": {
            "what": "mtv_verify_steps: chains of two steps per call, each step first appending its tree's K/V rows with the "
                    "rotary embedding (all layers, one launch); root token and prefix lengths pass between the steps on the device; "
                    "the chain starts K + 1 rows short of the configured prefix so that both links fit the caches",
            "ms_per_step": chain_ms, "steps_per_s": 1000.0 / chain_ms}}
    if not args.no_cpu_baseline and world == 1:
        out["cpu_baseline"] = cpu_baseline(w, P, n_layers, budget_s=20.0)
    if not args.no_other_workloads and world == 1:
        del P
        torch.cuda.empty_cache()
        out["other_workloads"] = {}
        for name in ("tiny", "short", "batched", "stress"):
            if name != w.name:
                out["other_workloads"][name] = quick_workload(name, n_layers, dev, pk)
    elif not args.no_cpu_baseline:
        out["cpu_baseline"] = None
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def run_sharded(args):
    """--shard kvhead: all ranks verify the same sequences.  Rank r projects the heads onto its vocabulary slab and
    attends with its KV heads; one all-gather after each brings the pieces into local memory, where the library's
    merge kernels put them together; acceptance runs on every rank (the logits are replicated), compaction on the
    rank's own caches.  Total work is fixed as N grows: "scaling": "strong"."""
    import torch
    import torch.distributed as dist
    from paper_2603_03383_b200 import binding, sharded, synth
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    use_dist = world > 1 or "RANK" in os.environ      # under torchrun the collectives are NCCL's even with one rank
    if use_dist:
        dist.init_process_group("nccl", device_id=dev)
    w = synth.WORKLOADS[args.workload]
    n_layers = args.layers
    P = build_problem(w, n_layers, dev, seed=w.seed)             # the same sequences on every rank
    tree, B, T = P["tree"], w.B, P["tree"].T
    K_steps, W_steps = args.steps, max(args.warmup, 3)
    gate = None
    if rank == 0 and not args.no_parity_gate:
        try:
            gate = parity_gate(w, P, n_layers)                    # the unsplit path against the CPU checker
        except ParityError as e:
            print(json.dumps({"metric": METRIC, "value": None, "unit": UNIT, "error": "parity gate failed: %s" % e,
                              "config": {"workload": workload_string(w, T, n_layers)}}))
            sys.exit(1)
    else:
        P["seq_lens"].copy_(P["seq_lens0"])
        binding.mtv_verify_step(tree, P["args"])
    torch.cuda.synchronize()
    whole = {n: P[n].clone() for n in ("cand", "tree_tok", "accept_len", "best_path", "acc_nodes", "acc_tok", "next_root",
                                       "seq_lens")}
    # the unsplit attention of the last layer on the caches as that step's compaction left them (the state the slices
    # below are cut from)
    whole_out = torch.zeros_like(P["out_layers"][n_layers - 1])
    binding.tree_verify_attention(tree, P["q_layers"][n_layers - 1], P["k_list"][n_layers - 1], P["v_list"][n_layers - 1],
                                  P["seq_lens0"], whole_out, P["ws"])
    torch.cuda.synchronize()
    # ---- this rank's slices (a rank of a real job would load only these)
    pl = sharded.plan(rank, world, w.V, w.Hq, w.Hkv, max_kd=max(tree.k_d))
    W2_slab = P["W2"][:, pl.v_lo:pl.v_hi].contiguous()
    q_l = P["q_layers"][:, :, :, pl.q_lo:pl.q_lo + pl.hq_local].contiguous()
    k_l = [k[:, pl.kv_lo:pl.kv_lo + pl.hkv_local].contiguous() for k in P["k_list"]]
    v_l = [v[:, pl.kv_lo:pl.kv_lo + pl.hkv_local].contiguous() for v in P["v_list"]]
    if world > 1:
        del P["W2"], P["k_list"], P["v_list"]
        torch.cuda.empty_cache()
    kp, vp = binding.cache_pointer_array(k_l, dev), binding.cache_pointer_array(v_l, dev)
    Lcap = P["Lcap"]
    strides = (pl.hkv_local * Lcap * w.D, Lcap * w.D, w.D)
    out_layers = torch.zeros(n_layers, B, T, w.Hq, w.D, dtype=torch.bfloat16, device=dev)

    def step():
        P["seq_lens"].copy_(P["seq_lens0"])
        sharded.medusa_heads_topk_sharded(tree, pl, P["hidden"], P["W1"], P["b1"], W2_slab, P["root_tok"], P["cand"],
                                          P["cand_logit"], P["tree_tok"], P["ws"])
        for l in range(n_layers):
            sharded.tree_verify_attention_sharded(tree, pl, q_l[l], k_l[l], v_l[l], P["seq_lens"], out_layers[l], P["ws"],
                                                  status=P["status"])
        binding.tree_accept(tree, P["logits"], P["tree_tok"], P["accept_len"], P["best_path"], P["acc_nodes"],
                            P["acc_tok"], P["next_root"], P["ws"])
        binding.kv_compact_accepted(tree, kp, vp, n_layers, B, pl.hkv_local, w.D, strides, Lcap, P["seq_lens"],
                                    P["accept_len"], P["acc_nodes"], status=P["status"])

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # the split step must give what the unsplit one gave (integers bit-exact; attention within the float tolerance:
    # the key splits of a call depend on how many heads it serves)
    step()
    barrier()
    for n, t in whole.items():
        if not torch.equal(P[n], t):
            print(json.dumps({"metric": METRIC, "value": None, "unit": UNIT,
                              "error": "split step: %s differs from the unsplit step on rank %d" % (n, rank)}))
            sys.exit(1)
    err = (out_layers[n_layers - 1].float() - whole_out.float()).abs().max().item()
    tol = 1e-2 * whole_out.float().abs().max().item() + 1e-3
    if not err <= tol:
        print(json.dumps({"metric": METRIC, "value": None, "unit": UNIT,
                          "error": "split step: attention differs from the unsplit step by %.3e on rank %d" % (err, rank)}))
        sys.exit(1)
    sampler = ClockSampler(local)     # nvidia-smi takes a while to start: it runs from here to the end of the timed steps
    if rank == 0:
        sampler.start()
    for _ in range(W_steps):
        step()
    barrier()
    run_step, launch = step, "stream launches"
    if args.launch == "graph":
        # the whole split step, collectives included, as one CUDA graph (every rank captures the same sequence)
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(graph, stream=side):
                    step()
            torch.cuda.current_stream().wait_stream(side)
            for _ in range(2):
                graph.replay()
            run_step, launch = graph.replay, "one CUDA graph per step, replayed"
        except Exception as e:      # a collective that cannot be captured: plain launches
            launch = "stream launches (graph capture failed: %s)" % type(e).__name__
        barrier()
    runs_ms = []
    for _ in range(max(1, args.repeats)):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(K_steps):
            run_step()
        e1.record()
        barrier()
        runs_ms.append(max_over_ranks(e0.elapsed_time(e1), world, dev))
    clocks = sampler.stop() if rank == 0 else None
    ms_step = statistics.median(runs_ms) / K_steps
    # end to end: the step's inputs from pinned host memory, its results back to the host, every step
    host = {n: P[n].cpu().pin_memory() for n in ("hidden", "root_tok", "logits")}
    host["q"] = q_l.cpu().pin_memory()
    back = {n: torch.empty_like(P[n], device="cpu").pin_memory() for n in ("tree_tok", "accept_len", "best_path",
                                                                          "acc_nodes", "acc_tok", "next_root", "seq_lens")}
    back["out"] = torch.empty_like(out_layers, device="cpu").pin_memory()

    def e2e_step():
        for n in ("hidden", "root_tok", "logits"):
            P[n].copy_(host[n], non_blocking=True)
        q_l.copy_(host["q"], non_blocking=True)
        step()
        for n in back:
            back[n].copy_(out_layers if n == "out" else P[n], non_blocking=True)
        torch.cuda.synchronize()

    e2e_steps = max(3, min(K_steps, 20))
    e2e_step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    barrier()
    e2e_s = max_over_ranks((time.perf_counter() - t0) / e2e_steps, world, dev)
    h2d = sum(t.numel() * t.element_size() for t in host.values())
    d2h = sum(t.numel() * t.element_size() for t in back.values())
    if rank == 0:
        pk = peaks()
        alg = algorithmic_bytes(w, tree, n_layers, P["lens"].tolist())
        gathered = 2 * B * (tree.C * 4 + (tree.C - 1) * 4) + n_layers * B * T * w.Hq * w.D * 2
        out = {
            "metric": METRIC, "value": 1000.0 / ms_step, "unit": UNIT, "n_gpus": world, "steps": K_steps, "warmup": W_steps,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": workload_string(w, T, n_layers),
                       "parallelism": "one sequence set on %d GPU(s): heads by vocabulary slab (%d rows each), attention "
                                      "by KV head (%d of %d each), all-gather + merge kernel after each" % (
                                          world, pl.v_slab, pl.hkv_local, w.Hkv),
                       "timing": "median of %d runs of %d steps (%s ms each), %s" % (
                           len(runs_ms), K_steps, ", ".join("%.1f" % r for r in runs_ms), launch),
                       "l2": "inputs larger than L2: %.2f GB streamed per step over all ranks" % (alg["step"] / 1e9),
                       "collective_bytes_per_step_per_rank": gathered, "seed": w.seed, "context": PAPER_CONTEXT},
            "clocks": clocks,
            "e2e": {"value": 1.0 / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": e2e_steps},
            "gpu_launches": K_steps * (LAUNCHES_PER_STEP(n_layers) + 2 + n_layers),
            "device_error": binding.mtv_device_error(tree, clear=False),
            "parity_gate": dict(gate or {}, split="integers bit-exact, attention max |diff| %.2e <= %.2e against the unsplit "
                                "step" % (err, tol)) if gate is not None else "skipped",
            "step_roofline": {"algorithmic_bytes": alg["step"], "achieved_gbs": alg["step"] / ms_step / 1e6,
                              "frac_of_measured": alg["step"] / ms_step / 1e6 / (pk["hbm_gbs"] * world)},
        }
        print(json.dumps(out))
    if use_dist:
        dist.destroy_process_group()


def quick_workload(name, n_layers, dev, pk, steps=5, repeats=3):
    """A short measurement of one of the other configurations: whole steps (graph replay and plain stream launches:
    their difference is the launch overhead), the attention call alone, and the roofline fractions that go with them.
    Checked before timing: statuses, and the accepted lengths against the planted ones."""
    import torch
    from paper_2603_03383_b200 import binding, synth
    w = synth.WORKLOADS[name]
    P = build_problem(w, n_layers, dev)
    tree, a = P["tree"], P["args"]

    def step():
        P["seq_lens"].copy_(P["seq_lens0"])
        binding.mtv_verify_step(tree, a)

    for _ in range(3):
        step()
    torch.cuda.synchronize()
    checks = (not any(P["status"].cpu().tolist())) and torch.equal(P["accept_len"].cpu(), P["planted"].to(torch.int32).cpu())
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            step()
    torch.cuda.current_stream().wait_stream(side)

    def timed(fn, n):
        best = []
        for _ in range(repeats):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(n):
                fn()
            e1.record()
            torch.cuda.synchronize()
            best.append(e0.elapsed_time(e1) / n)
        return statistics.median(best)

    graph.replay()
    ms_graph = timed(graph.replay, steps)
    ms_stream = timed(step, steps)

    def attn_block():
        for l in range(n_layers):
            binding.tree_verify_attention(tree, P["q_layers"][l], P["k_list"][l], P["v_list"][l], P["seq_lens0"],
                                          P["out_layers"][l], P["ws"])
    attn_block()
    attn_us = timed(attn_block, 3) * 1e3 / n_layers
    alg = algorithmic_bytes(w, tree, n_layers, P["lens"].tolist())
    T = tree.T
    attn_flops = sum(4.0 * (L + T) * T * w.Hq * w.D for L in P["lens"].tolist())
    res = {
        "workload": workload_string(w, T, n_layers), "checks_passed": bool(checks),
        "steps_per_s": 1000.0 / ms_graph, "ms_per_step": ms_graph, "ms_per_step_stream_launches": ms_stream,
        "launch_overhead_share": max(0.0, (ms_stream - ms_graph) / ms_stream),
        "step_frac_of_measured_hbm": alg["step"] / ms_graph / 1e6 / pk["hbm_gbs"],
        "attn_us_per_call": attn_us,
        "attn_frac_of_measured_hbm": alg["attn_per_layer"] / attn_us / 1e3 / pk["hbm_gbs"],
        "attn_tflops": attn_flops / attn_us / 1e6,
        "attn_frac_of_measured_bf16": attn_flops / attn_us / 1e6 / pk["bf16_tflops"],
        "device_error": binding.mtv_device_error(tree, clear=False),
    }
    del P
    torch.cuda.empty_cache()
    return res


def time_lm_head(tree, w, P, dev, iters=20):
    """ms per call of lm_head_argmax + tree_accept_keys on the workload's B, T, H, V (the first Medusa head's
    vocabulary matrix stands in for the LM head: same shape, same distribution), back-to-back launches."""
    import torch
    from paper_2603_03383_b200 import binding, synth
    B, T, K = w.B, tree.T, w.K
    x = synth.normal_bf16(w.seed, 77, (B, T, w.H), device=dev)
    W = P["W2"][0]
    keys = torch.zeros(B * T, dtype=torch.int64, device=dev)
    i32 = lambda *s: torch.zeros(*s, dtype=torch.int32, device=dev)
    outs = [i32(B), i32(B), i32(B, K + 1), i32(B, K + 1), i32(B)]
    def call():
        binding.lm_head_argmax(tree, x, W, keys)
        binding.tree_accept_keys(tree, B, keys, P["tree_tok"], *outs)
    for _ in range(3):
        call()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(iters):
        call()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def time_step_with_lm_head(tree, w, P, dev, launch, steps):
    """ms per step of mtv_verify_step when the acceptance takes the argmax from the fused LM head (same inputs
    otherwise; the first Medusa head's vocabulary matrix stands in for the LM head)."""
    import torch
    from paper_2603_03383_b200 import binding, synth
    a2 = binding.StepArgs.from_buffer_copy(P["args"])
    x = synth.normal_bf16(w.seed, 77, (w.B, tree.T, w.H), device=dev)
    W = P["W2"][0]
    a2.x_final, a2.W_lm, a2.logits = x.data_ptr(), W.data_ptr(), None

    def step():
        P["seq_lens"].copy_(P["seq_lens0"])
        binding.mtv_verify_step(tree, a2)
    for _ in range(3):
        step()
    torch.cuda.synchronize()
    run = step
    if launch == "graph":
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                step()
        torch.cuda.current_stream().wait_stream(side)
        run = graph.replay
        run()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(steps):
        run()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


def time_chained_steps(tree, w, P, dev, launch, steps, n_chain=2):
    """ms per step of mtv_verify_steps: chains of `n_chain` steps in one call, each step first appending its tree's
    K/V rows (rotary embedding, all layers in one launch), the next step's root token and prefix lengths passed on the
    device.  Same per-step inputs for every link of the chain (the timing does not depend on the values)."""
    import torch
    from paper_2603_03383_b200 import binding, synth
    n_layers = P["q_layers"].shape[0]
    kn = synth.normal_bf16(w.seed, 78, (n_layers, w.B, tree.T, w.Hkv, w.D), device=dev)
    vn = synth.normal_bf16(w.seed, 79, (n_layers, w.B, tree.T, w.Hkv, w.D), device=dev)
    chain, appends = [], []
    for s in range(n_chain):
        a = binding.StepArgs.from_buffer_copy(P["args"])
        if s > 0:
            a.root_tok = None                       # = the previous step's next_root
        ap = binding.AppendArgs()
        ap.k_new_layers, ap.v_new_layers, ap.rope_theta = kn.data_ptr(), vn.data_ptr(), 0.0
        chain.append(a)
        appends.append(ap)

    # every link must fit the caches' capacity (prefix + tree rows): the chain starts (n_chain - 1) (K + 1) rows short of
    # the configured prefix
    start = (P["seq_lens0"] - (n_chain - 1) * (w.K + 1)).clamp_(min=0)

    def run_chain():
        P["seq_lens"].copy_(start)
        binding.mtv_verify_steps(tree, chain, appends)
    for _ in range(2):
        run_chain()
    torch.cuda.synchronize()
    if any(P["status"].cpu().tolist()) or int((P["seq_lens"] - start).min()) < n_chain:
        raise RuntimeError("chained steps: a link was refused (status %s)" % P["status"].cpu().tolist())
    run = run_chain
    if launch == "graph":
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                run_chain()
        torch.cuda.current_stream().wait_stream(side)
        run = graph.replay
        run()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(steps):
        run()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / (steps * n_chain)


def _sample_plan(w, T, n_layers, est_full_s, budget_s):
    """How much of one step the checker runs so that it takes about budget_s seconds."""
    f = min(1.0, budget_s / max(est_full_s, 1e-9))
    n_heads = max(1, min(w.K, int(round(w.K * f))))
    vocab_rows = w.V if n_heads > 1 else min(w.V, max(2048, int(w.V * w.K * f)))
    layers = max(1, min(n_layers, int(round(n_layers * f))))
    total_rows = w.B * T * w.Hq
    attn_rows = total_rows if layers > 1 else min(total_rows, max(8, int(total_rows * n_layers * f)))
    logit_rows = max(1, min(T, int(round(T * f))))
    return dict(n_heads=n_heads, vocab_rows=vocab_rows, layers=layers, attn_rows=attn_rows, logit_rows=logit_rows)


def _sample_inputs_from_problem(w, P, plan):
    """CPU copies of the slices the checker's sample needs (same values the CUDA arm uses)."""
    nh, vr, nl, nr = plan["n_heads"], plan["vocab_rows"], plan["layers"], plan["logit_rows"]
    return dict(hidden=P["hidden"].cpu(), W1=P["W1"][:nh].cpu(), b1=P["b1"][:nh].cpu(),
                W2=P["W2"][:nh, :vr].cpu(), q=[P["q_layers"][l].cpu() for l in range(nl)],
                k=[P["k_list"][l].cpu() for l in range(nl)], v=[P["v_list"][l].cpu() for l in range(nl)],
                logits=P["logits"][:, :nr].cpu(), lens=P["lens"], mask=P["tree"].medusa_attn_mask, T=P["tree"].T)


def _sample_inputs_on_cpu(w, plan):
    """The same slices generated on the host (the generator is counter-based: a prefix of a
    tensor has the same values as the whole tensor's prefix).  No CUDA code involved."""
    import math
    import torch
    from oracle import tree as otree
    from paper_2603_03383_b200 import synth
    nh, vr, nl, nr = plan["n_heads"], plan["vocab_rows"], plan["layers"], plan["logit_rows"]
    nodes = otree.cartesian(w.topk) if w.tree == "cartesian" else otree.rank_prior(w.K, w.T, w.R_max)
    tb = otree.tables(nodes, w.K)
    T, seed, Lcap = tb["T"], w.seed, int(w.L_hi) + tb["T"]
    qkv = [synth.attention_inputs(w.B, T, w.Hq, w.Hkv, w.D, Lcap, seed, layer=l) for l in range(nl)]
    W2 = torch.stack([synth.normal_bf16(seed, synth.TID_W2, (h + 1, w.V, w.H), 1.0 / math.sqrt(w.H))[h, :vr]
                      for h in range(nh)]) if nh > 1 else \
        synth.normal_bf16(seed, synth.TID_W2, (1, vr, w.H), 1.0 / math.sqrt(w.H))
    logits = synth.normal_bf16(seed, synth.TID_LOGITS, (w.B, T, w.V))[:, :nr].contiguous() if w.B > 1 else \
        synth.normal_bf16(seed, synth.TID_LOGITS, (1, nr, w.V))
    return dict(hidden=synth.normal_bf16(seed, synth.TID_HIDDEN, (w.B, w.H)),
                W1=synth.normal_bf16(seed, synth.TID_W1, (nh, w.H, w.H), 1.0 / math.sqrt(w.H)),
                b1=synth.normal_bf16(seed, synth.TID_B1, (nh, w.H), 0.1), W2=W2,
                q=[t[0] for t in qkv], k=[t[1] for t in qkv], v=[t[2] for t in qkv], logits=logits,
                lens=synth.seq_lens(w), mask=tb["mask"], T=T)


def _oracle_step_sample(w, S, n_layers, plan):
    """Run the checker on the planned sample; returns (seconds, estimated seconds for a whole step, description)."""
    from oracle import reference as ref
    T, B = S["T"], w.B
    nh, vr, nl, ar, nr = plan["n_heads"], plan["vocab_rows"], plan["layers"], plan["attn_rows"], plan["logit_rows"]
    total_rows = B * T * w.Hq
    rows = None if ar >= total_rows else [(r % B, (r * 7) % T, (r * 13) % w.Hq) for r in range(ar)]
    t0 = time.perf_counter()
    ref.heads_logits(S["hidden"], S["W1"], S["b1"], S["W2"])
    t_head = time.perf_counter() - t0
    t0 = time.perf_counter()
    for l in range(nl):
        ref.tree_attention(S["q"][l], S["k"][l], S["v"][l], S["lens"], S["mask"], rows=rows)
    t_attn = time.perf_counter() - t0
    t0 = time.perf_counter()
    ref.node_argmax(S["logits"])
    t_arg = time.perf_counter() - t0
    full = (t_head * (w.K / nh) * (w.V / vr) + t_attn * (n_layers / nl) * (total_rows / min(ar, total_rows))
            + t_arg * (T / nr))
    desc = ("%d of %d heads on %d of %d vocabulary rows, %d of %d attention rows of %d of %d layers, argmax of %d of %d "
            "logit rows per sequence; each part's time scaled to a whole step" % (
                nh, w.K, vr, w.V, min(ar, total_rows), total_rows, nl, n_layers, nr, T))
    return t_head + t_attn + t_arg, full, desc


_CALIBRATION = dict(n_heads=1, vocab_rows=2048, layers=1, attn_rows=8, logit_rows=1)


def cpu_baseline(w, P, n_layers, budget_s):
    cores = os.cpu_count() or 1
    # calibrate on a small sample, then size the real one to the budget
    cal = dict(_CALIBRATION, vocab_rows=min(w.V, 2048))
    _, full, _ = _oracle_step_sample(w, _sample_inputs_from_problem(w, P, cal), n_layers, cal)
    plan = _sample_plan(w, P["tree"].T, n_layers, full, budget_s)
    s, full, desc = _oracle_step_sample(w, _sample_inputs_from_problem(w, P, plan), n_layers, plan)
    return {"value": 1.0 / full, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc,
            "sample_seconds": s}


def run_reference(args):
    """The fp64 CPU checker as it stands, on the host cores, each step a bounded sample."""
    if int(os.environ.get("RANK", 0)) != 0:
        return
    from paper_2603_03383_b200 import synth
    w = synth.WORKLOADS[args.workload]
    n_layers = args.layers
    K_steps, W_steps = args.steps, args.warmup
    per_step_budget = min(5.0, 150.0 / max(1, K_steps + W_steps))
    cal = dict(_CALIBRATION, vocab_rows=min(w.V, 2048))
    S = _sample_inputs_on_cpu(w, cal)
    _, full, _ = _oracle_step_sample(w, S, n_layers, cal)
    plan = _sample_plan(w, S["T"], n_layers, full, per_step_budget)
    S = _sample_inputs_on_cpu(w, plan)
    for _ in range(W_steps):
        _oracle_step_sample(w, S, n_layers, plan)
    fulls, desc = [], ""
    t0 = time.perf_counter()
    for _ in range(K_steps):
        _, full, desc = _oracle_step_sample(w, S, n_layers, plan)
        fulls.append(full)
    wall = time.perf_counter() - t0
    full = sum(fulls) / len(fulls)
    value = 1.0 / full
    cores = os.cpu_count() or 1
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": K_steps, "warmup": W_steps, "ms_per_step": full * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_string(w, S["T"], n_layers)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": desc + "; timed wall %.1f s" % wall},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def run_overhead_sweep(args):
    """Attention part of the paper's Overhead = Time_speculative / Time_autoregressive (Eq. 3) on this GPU:
    the T-node tree attention call against the same call with a root-only tree (one query token), per
    prefix length, on 32 rotating KV caches (median of five runs of 5 x 32 calls).  One JSON line per length."""
    import torch
    from paper_2603_03383_b200 import binding, synth
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    w = synth.WORKLOADS["long"]
    nodes = binding.tree_gen_rank_prior(w.K, w.T, w.R_max)
    trees = {"tree": binding.tree_build_static(w.K, nodes), "single": binding.tree_build_static(w.K, [])}
    layers, reps = 32, 5
    for L in (128, 512, 1024, 2048, 4096, 8192, 16384, 32768):
        res = {}
        for name, tree in trees.items():
            T = tree.T
            Lcap = L + T
            qs = [synth.normal_bf16(7, synth.TID_Q + l, (1, T, w.Hq, w.D), device=dev) for l in range(layers)]
            ks = [synth.normal_bf16(7, synth.TID_K + l, (1, w.Hkv, Lcap, w.D), device=dev) for l in range(layers)]
            vs = [synth.normal_bf16(7, synth.TID_V + l, (1, w.Hkv, Lcap, w.D), device=dev) for l in range(layers)]
            out = torch.zeros_like(qs[0])
            sl = torch.tensor([L], dtype=torch.int32, device=dev)
            ws = torch.empty(binding.mtv_workspace_bytes(tree, 1, 0, 0, w.Hq, w.Hkv, w.D, Lcap), dtype=torch.uint8,
                             device=dev)
            for l in range(layers):
                binding.tree_verify_attention(tree, qs[l], ks[l], vs[l], sl, out, ws)
            torch.cuda.synchronize()
            runs = []
            for _ in range(5):      # the median of five timed runs: single runs of a call this short scatter by a microsecond
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(reps):
                    for l in range(layers):
                        binding.tree_verify_attention(tree, qs[l], ks[l], vs[l], sl, out, ws)
                e1.record()
                torch.cuda.synchronize()
                runs.append(e0.elapsed_time(e1) * 1e3 / (reps * layers))
            res[name] = statistics.median(runs)
            del qs, ks, vs
        print(json.dumps({"prefix": L, "tree_nodes": trees["tree"].T, "us_tree_attention": res["tree"],
                          "us_single_token_attention": res["single"],
                          "attention_overhead_ratio": res["tree"] / res["single"]}))


if __name__ == "__main__":
    a = parse()
    if a.overhead_sweep:
        run_overhead_sweep(a)
        sys.exit(0)
    if a.impl == "reference":
        run_reference(a)
    elif a.shard == "kvhead":
        run_sharded(a)
    else:
        run_ours(a)
