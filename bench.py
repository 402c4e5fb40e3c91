#!/usr/bin/env python
"""Benchmark of the tree-verification step (tree attention + node top-k + accept walk + KV compaction).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl ours|reference]

One "step" is one pass of the whole hot path over one batch of seeded synthetic input of the chosen
workload (default: the 33B-shaped config).  Prints ONE JSON line (rank 0):
  value      tree-verify steps/s, inputs resident in HBM, CUDA-graph replay, L2-cold by rotating replicas
  e2e        the same metric through goose_verify_step_host (pinned host buffers, copies inside the timing)
  roofline   the attention kernel alone: algorithmic bytes / CUDA-event time vs the measured HBM copy peak
  cpu_baseline  the fp64 oracle on the host cores, on a bounded sample of the same workload
N > 1: the path does not shard across GPUs (one GPU per the benchmark spec), so every rank runs an independent
replica of the same workload ("replicas only", weak scaling, no data-path collective).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "tree_verify_steps_per_s"
UNIT = "steps/s"
L2_BYTES = 126 * 1024 * 1024
# DRAM traffic per attention launch from the ncu capture summarised under profiles/ (bytes), per config
# name; None = not captured for that workload.
NCU_TRAFFIC_BYTES = {"33b": 227_470_000,    # tree_attn_umma_kernel: 223.29 MB read + 4.2 MB written per launch
                     "13b": 89_450_000,
                     "gqa8b": 169_570_000}  # 165.0 MB read + 3.2-5.8 MB written per launch (two launches averaged)     # 86.42 MB read + 3.0 MB written


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.samples = []
        self._stop = threading.Event()
        self._t = None

    def _run(self):
        while not self._stop.is_set():
            try:
                r = subprocess.run(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.FIELDS,
                                    "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=5)
                if r.returncode == 0 and r.stdout.strip():
                    self.samples.append([t.strip() for t in r.stdout.strip().split(",")])
            except Exception:
                pass
            self._stop.wait(0.1)

    def __enter__(self):
        self._t = threading.Thread(target=self._run, daemon=True)
        self._t.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._t.join(timeout=6)

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for s in self.samples:
            try:
                sm.append(float(s[0])); mx.append(float(s[1]))
            except Exception:
                continue
            for n, v in zip(names, s[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm)}


# ----------------------------------------------------------------------------- distributed plumbing
def dist_max(x: float, device) -> float:
    """Max over ranks of a python float (no-op without an initialised process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return x
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def dist_barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def aggregate_steps_per_s(steps: int, local_ms: float, world: int, device) -> tuple:
    """Whole-job throughput of `world` independent replicas: all ranks' steps / slowest rank's time."""
    ms = dist_max(local_ms, device)
    return world * steps / (ms * 1e-3), ms / steps


# ----------------------------------------------------------------------------- CPU oracle legs
def oracle_sample(x, budget_s: float = 12.0):
    """Time the oracle, as it stands, on a bounded sample of workload x; scale to one whole step."""
    import oracle
    oracle.build()
    rng = np.random.default_rng(0)
    total_rows = x.S * x.B * x.H
    # calibrate on a few rows, then size the sample for about `budget_s` of attention work
    n0 = min(total_rows, max(16, oracle.num_threads()))
    pick = lambda n: (rng.integers(0, x.S, n), rng.integers(0, x.B, n), rng.integers(0, x.H, n))
    ss, si, sh = pick(n0)
    t0 = time.perf_counter()
    oracle.tree_attn_rows(x.q, x.k_cache, x.v_cache, x.row_off, x.ctx_len, x.parent, x.scale, ss, si, sh)
    per_row = (time.perf_counter() - t0) / n0
    n_attn = int(min(total_rows, max(n0, budget_s * 0.8 / max(per_row, 1e-9))))
    ss, si, sh = pick(n_attn)
    t0 = time.perf_counter()
    oracle.tree_attn_rows(x.q, x.k_cache, x.v_cache, x.row_off, x.ctx_len, x.parent, x.scale, ss, si, sh)
    t_attn = time.perf_counter() - t0
    # weight rows by their sequence's key count so the scaling is right for ragged batches
    keys = (x.ctx_len.astype(np.float64) + x.B)
    scale_attn = (keys.sum() * x.B * x.H) / keys[ss].sum()
    n_topk = min(x.S * x.B, max(oracle.num_threads(), 16))
    rows = rng.choice(x.S * x.B, n_topk, replace=False)
    t0 = time.perf_counter()
    am_s, _, _ = oracle.node_topk(x.logits[rows], x.k)
    t_topk = time.perf_counter() - t0
    am, _, _ = oracle.node_topk(x.logits, 1) if x.S * x.B <= 256 else (None, None, None)
    if am is None:                                    # argmax only (cheap, numpy) to feed the walk on big batches
        from paper_2604_02047_b200 import synth
        am = np.argmax(synth.bf16_bits_to_f32(x.logits), axis=1).astype(np.int32)
    t0 = time.perf_counter()
    path, alen, _ = oracle.accept(x.draft_tok, x.parent, am.reshape(x.S, x.B))
    t_acc = time.perf_counter() - t0
    t0 = time.perf_counter()
    oracle.kv_compact(x.k_cache, x.v_cache, x.row_off, x.ctx_len, path, alen)
    t_cmp = time.perf_counter() - t0
    step_s = t_attn * scale_attn + t_topk * (x.S * x.B / n_topk) + t_acc + t_cmp
    sample = ("attention on %d of %d (seq,node,head) rows + top-k on %d of %d logits rows + full accept walk and "
              "KV compaction, scaled to one step" % (n_attn, total_rows, n_topk, x.S * x.B))
    return {"value": 1.0 / step_s, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample,
            "step_s": step_s, "sampled_s": t_attn + t_topk + t_acc + t_cmp}


def run_reference(args, x, cfg_name):
    """--impl reference: the oracle (the only reference there is), on the host cores, rank 0 only."""
    res = None
    for i in range(args.warmup + args.steps):
        # bounded sample per step so that warm-up + K steps stay within a few minutes of host time
        r = oracle_sample(x, budget_s=max(0.15, min(12.0, 100.0 / max(1, args.warmup + args.steps))))
        if i >= args.warmup:
            res = r if res is None else {**r, "step_s": res["step_s"] + r["step_s"]}
    step_s = res["step_s"] / args.steps
    line = {
        "impl": "reference", "metric": METRIC, "value": 1.0 / step_s, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_s * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg_name, "S": x.S, "H": x.H, "Hkv": x.Hkv, "B": x.B, "V": x.V, "k": x.k,
                   "note": "fp64 CPU oracle on a bounded sample per step, scaled to a whole step"},
        "cpu_baseline": {"value": 1.0 / step_s, "unit": UNIT, "cores": res["cores"], "kind": "oracle",
                         "sample": res["sample"]},
        "e2e": {"value": 1.0 / step_s, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------- GPU legs
def quick_step_timing(config_id, dev, steps, peak):
    """Whole-step and attention timing of another workload of the table, same method as the main line (CUDA-graph replay
    over rotating replicas, CUDA events), without the CPU and end-to-end legs: context for the main line, not a bench line."""
    import torch
    from paper_2604_02047_b200 import binding, synth
    x = synth.make_config(config_id)
    g = binding.Goose(max_S=x.S, max_B=128, max_H=max(64, x.H), device=dev.index)
    base = binding.to_device(x, dev)
    footprint = sum(t.numel() * t.element_size() for t in base.values())
    R = int(max(2, min(64, -(-max(2 * L2_BYTES, 1 << 30) // footprint))))
    reps = [base] + [{k: v.clone() for k, v in base.items()} for _ in range(R - 1)]
    outs = [g.alloc_step_outputs(x.S, x.B, x.H, x.D, x.k, dev) for _ in range(R)]
    stream = torch.cuda.Stream(device=dev)

    def step(i):
        d = reps[i % R]
        g.verify_step(d["q"], d["k_cache"], d["v_cache"], d["row_off"], d["ctx_len"], d["parent"], d["draft_tok"],
                      d["logits"], x.k, x.scale, outs=outs[i % R])

    def attn(i):
        d = reps[i % R]
        g.tree_attn(d["q"], d["k_cache"], d["v_cache"], d["row_off"], d["ctx_len"], d["parent"], x.scale, out=outs[i % R]["out"])

    res = {}
    with torch.cuda.stream(stream):
        for i in range(3):
            step(i)
        stream.synchronize()
        for name, fn in (("step", step), ("attn", attn)):
            gr = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gr, stream=stream, capture_error_mode="thread_local"):
                for i in range(R):
                    fn(i)
            rounds = max(3, -(-steps // R))
            for _ in range(2):
                gr.replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(rounds):
                gr.replay()
            e1.record(stream)
            e1.synchronize()
            res[name] = e0.elapsed_time(e1) / (rounds * R)       # ms per call
    ab = synth.algorithmic_bytes(x.S, x.H, x.B, x.D, x.V, x.ctx_len, Hkv=x.Hkv)
    g.close()
    return {"steps_per_s": 1e3 / res["step"], "us_per_step": res["step"] * 1e3, "tree_attn_us": res["attn"] * 1e3,
            "tree_attn_frac_of_peak": ab["attn"] / (res["attn"] * 1e-3) / 1e9 / peak}


def run_ours(args, x, cfg, rank, world, local_rank):
    import torch
    from paper_2604_02047_b200 import binding, build, synth

    if local_rank == 0:                  # one builder per node (a no-op when the shipped library matches the sources)
        build.build()
    dist_barrier()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    g = binding.Goose(max_S=x.S, max_B=128, max_H=max(64, x.H), device=local_rank)
    if args.attn_impl:
        g.set_attn_impl({"mma": binding.ATTN_MMA, "umma": binding.ATTN_UMMA}[args.attn_impl])

    base = binding.to_device(x, dev)
    ab = synth.algorithmic_bytes(x.S, x.H, x.B, x.D, x.V, x.ctx_len, Hkv=x.Hkv)
    gqa = x.Hkv != x.H          # grouped-query workload: the *_gqa entry points
    verify_step = g.verify_step_gqa if gqa else g.verify_step
    tree_attn = g.tree_attn_gqa if gqa else g.tree_attn
    verify_step_host = g.verify_step_host_gqa if gqa else g.verify_step_host
    footprint = sum(t.numel() * t.element_size() for t in base.values())
    R = int(max(2, min(64, -(-max(2 * L2_BYTES, 1 << 30) // footprint))))
    reps = [base] + [{k: v.clone() for k, v in base.items()} for _ in range(R - 1)]
    outs = [g.alloc_step_outputs(x.S, x.B, x.H, x.D, x.k, dev) for _ in range(R)]
    stream = torch.cuda.Stream(device=dev)

    def step(i):
        d, o = reps[i % R], outs[i % R]
        verify_step(d["q"], d["k_cache"], d["v_cache"], d["row_off"], d["ctx_len"], d["parent"], d["draft_tok"],
                    d["logits"], x.k, x.scale, outs=o)

    def attn(i):
        d, o = reps[i % R], outs[i % R]
        tree_attn(d["q"], d["k_cache"], d["v_cache"], d["row_off"], d["ctx_len"], d["parent"], x.scale, out=o["out"])

    def topk(i):
        d = reps[i % R]
        g.node_topk(d["logits"], x.k)

    adj_ids = torch.full((x.V, x.k), -1, dtype=torch.int32, device=dev)
    adj_scores = torch.zeros((x.V, x.k), dtype=torch.float32, device=dev)

    def harvest(i):          # adjacent row of the path (not part of the step metric): top-k + lse + table scatter
        d = reps[i % R]
        g.harvest(d["logits"], x.k, d["draft_tok"].view(-1), adj_ids, adj_scores)

    def step_harvest(i):     # the step and the harvest of its logits in one call (the logits are read once)
        d, o = reps[i % R], outs[i % R]
        g.verify_step_harvest(d["q"], d["k_cache"], d["v_cache"], d["row_off"], d["ctx_len"], d["parent"], d["draft_tok"],
                              d["logits"], x.k, x.scale, adj_ids, adj_scores, outs=o)

    with torch.cuda.stream(stream):
        for i in range(max(3, args.warmup)):
            step(i)
        stream.synchronize()
        # one CUDA graph per leg: a full rotation over the replicas
        def capture(fn, n=R):
            gr = torch.cuda.CUDAGraph()
            n0 = g.launch_count()
            with torch.cuda.graph(gr, stream=stream, capture_error_mode="thread_local"):
                for i in range(n):
                    fn(i)
            return gr, (g.launch_count() - n0) // n
        g_step, launches_per_step = capture(step)
        # K steps = whole rotations plus one partial rotation, which gets a graph of its own
        g_tail = capture(step, args.steps % R)[0] if args.steps % R else None
        g_attn, _ = capture(attn)
        g_topk, _ = capture(topk)
        g_harv, _ = capture(harvest)
        g_sh, _ = capture(step_harvest)

        def time_graph(gr, rounds):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(rounds):
                gr.replay()
            e1.record(stream)
            e1.synchronize()
            return e0.elapsed_time(e1)

        # warm-up replays, then the timed region: barrier + synchronize on both sides
        for _ in range(max(1, -(-args.warmup // R))):
            g_step.replay()
        torch.cuda.synchronize(dev)
        dist_barrier()
        with ClockSampler(local_rank) as clk:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            done = 0
            while args.steps - done >= R:                 # exactly K steps: whole rotations, then the partial one
                g_step.replay(); done += R
            if g_tail is not None:
                g_tail.replay(); done += args.steps % R
            e1.record(stream)
            torch.cuda.synchronize(dev)
            dist_barrier()
            local_ms = e0.elapsed_time(e1)
            # per-kernel legs, inside the same sampled region
            attn_rounds = max(3, min(200, int(0.3e3 / max(local_ms / args.steps, 1e-3)) // R + 1))
            time_graph(g_attn, 1)
            attn_ms = time_graph(g_attn, attn_rounds) / (attn_rounds * R)
            time_graph(g_topk, 1)
            topk_ms = time_graph(g_topk, attn_rounds) / (attn_rounds * R)
            time_graph(g_harv, 1)
            harv_ms = time_graph(g_harv, attn_rounds) / (attn_rounds * R)
            time_graph(g_sh, 1)
            sh_ms = time_graph(g_sh, attn_rounds) / (attn_rounds * R)
        clocks = clk.summary()
    value, ms_per_step = aggregate_steps_per_s(args.steps, local_ms, world, dev)

    # ---- end to end: pinned host buffers through goose_verify_step_host
    d0 = reps[0]
    hin = {k: d0[k].cpu().pin_memory() for k in ("q", "row_off", "ctx_len", "parent", "draft_tok", "logits")}
    rows = np.concatenate([np.arange(x.row_off[s] + x.ctx_len[s], x.row_off[s] + x.ctx_len[s] + x.B) for s in range(x.S)])
    rows_t = torch.from_numpy(rows).to(dev)
    k_new = d0["k_cache"][rows_t].reshape(x.S, x.B, x.Hkv, x.D).cpu().pin_memory()
    v_new = d0["v_cache"][rows_t].reshape(x.S, x.B, x.Hkv, x.D).cpu().pin_memory()
    houts = {k: v.pin_memory() for k, v in g.alloc_step_outputs(x.S, x.B, x.H, x.D, x.k, device="cpu").items()}
    h2d = sum(t.numel() * t.element_size() for t in hin.values()) + 2 * k_new.numel() * 2
    d2h = sum(t.numel() * t.element_size() for t in houts.values())
    e2e_steps = max(3, min(args.steps, 50))
    e2e_ms = float("nan")
    if not args.no_e2e:
        with torch.cuda.stream(stream):
            def host_step(i):
                d = reps[i % R]
                verify_step_host(d["k_cache"], d["v_cache"], hin["q"], k_new, v_new, hin["row_off"],
                                 hin["ctx_len"], hin["parent"], hin["draft_tok"], hin["logits"], x.k, x.scale, houts)
            for i in range(3):
                host_step(i)
            torch.cuda.synchronize(dev)
            dist_barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for i in range(e2e_steps):
                host_step(i)
            e1.record(stream)
            torch.cuda.synchronize(dev)
            e2e_ms = e0.elapsed_time(e1)
    e2e_value, _ = aggregate_steps_per_s(e2e_steps, e2e_ms, world, dev)

    status = g.last_status(x.S)
    if status.any():
        raise RuntimeError("device status words set: %s" % status.tolist())

    peak, peak_kind = _peaks()
    attn_gbs = ab["attn"] / (attn_ms * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg.name, "S": x.S, "H": x.H, "Hkv": x.Hkv, "B": x.B, "D": x.D, "V": x.V, "k": x.k,
                   "ctx_len": [int(c) for c in x.ctx_len] if x.S > 1 else int(x.ctx_len[0]),
                   "l2": "rotating %d input replicas (%.2f GB total, > 2x L2)" % (R, R * footprint / 1e9),
                   "timing": "CUDA graph replay of whole steps, CUDA events, max over ranks",
                   "multi_gpu": "replicas only"},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                "steps": e2e_steps, "note": "goose_verify_step_host: per-step inputs/outputs in pinned host memory; "
                                           "the prefix KV cache is device-resident state"},
        "gpu_launches": int(launches_per_step * args.steps),
        "clocks": clocks,
        "roofline": {"kernel": "tree_attn", "bound": "hbm", "achieved": attn_gbs, "peak": peak, "unit": "GB/s",
                     "frac": attn_gbs / peak, "peak_kind": peak_kind,
                     "traffic": NCU_TRAFFIC_BYTES.get(cfg.name), "algorithmic_bytes": ab["attn"],
                     "us_per_launch": attn_ms * 1e3},
        "kernels": {"tree_attn_us": attn_ms * 1e3, "node_topk_us": topk_ms * 1e3, "harvest_us": harv_ms * 1e3,
                    "step_with_harvest_us": sh_ms * 1e3,
                    "node_topk_gbs": ab["topk"] / (topk_ms * 1e-3) / 1e9,
                    "step_gbs": ab["total"] / (ms_per_step * 1e-3) / 1e9,
                    "step_frac_of_peak": ab["total"] / (ms_per_step * 1e-3) / 1e9 / peak},
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cb = oracle_sample(x)
        line["cpu_baseline"] = {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")}
    g.close()
    # context for the single-GPU default line: the other batch-1 workloads of the table, timed the same way
    if rank == 0 and world == 1 and args.config == 3 and not args.no_others and not args.attn_impl:
        del reps, outs, base
        torch.cuda.empty_cache()
        line["other_workloads"] = {synth.CONFIGS[cid].name: quick_step_timing(cid, dev, args.steps, peak) for cid in (1, 2)}
    if rank == 0:
        print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", type=int, default=3, help="index into the workload table (0..4 the benchmark table, 5 the grouped-query workload); default 33B")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--attn-impl", choices=["mma", "umma"], default=None)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--no-others", action="store_true",
                    help="skip the short timings of the 7b and 13b workloads that the default line carries as context")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    from paper_2604_02047_b200 import synth
    cfg = synth.CONFIGS[args.config]

    if args.impl == "reference":
        if rank != 0:
            return
        x = synth.make_config(args.config, seed=args.seed)
        run_reference(args, x, cfg.name)
        return

    if world > 1:
        import torch
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    x = synth.make_config(args.config, seed=args.seed)
    run_ours(args, x, cfg, rank, world, local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
