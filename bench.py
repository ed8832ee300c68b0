#!/usr/bin/env python
"""Benchmark of the budgeted MoE verify layer (MoE-Spec, Algorithm 1) on B200.

A "step" is one pass of the whole hot path (router -> shortlist -> re-routing ->
gather -> expert FFNs over the kept experts -> combine) over one draft tree.
Workload at N=1: the OLMoE-shaped single layer (d=2048, N=64, k=8, f=1024,
bf16 weights, fp32 accumulation), M=63 tree tokens, budget B=32; the other
budgets of that configuration are reported in "sweep".  Inputs are seeded and
synthetic.  L2 reuse is defeated by rotating over independently seeded copies
of the layer (each step streams ~400 MB; 126 MB of L2 cannot hold a copy).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Prints one JSON line.  With --gpus N > 1 (under torchrun) every rank runs an
independent replica of the same workload on its own GPU (the layer has no
data-path collective); time is the max over ranks.  --impl reference times the
CPU oracle on the host cores instead.

  --mode ep   (with --gpus N under torchrun) expert-parallel instead of replicas: rank r holds the weights of
              its block of the experts only, every rank routes the same tree (replicated router, no exchange),
              streams its resident kept experts and the partial outputs [M, d] fp32 are summed by one NCCL
              all-reduce per layer, inside the timed region.  The job then processes K layers in total
              ("scaling": "strong").
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2602_16052_b200 import synth

METRIC = "us per budgeted MoE verify layer and achieved HBM GB/s (% roofline) vs M, B"
WORKLOAD = "olmoe"
M_TOKENS = 63
B_HEADLINE = 32
N_COPIES = 4
FALLBACK_HBM_GBS = 6650.0
# DRAM counters of the expert-FFN launch of one verify layer of this workload, from a profiler capture:
# a small key = value file kept beside the capture's summary
TRAFFIC_FILE = os.path.join("profiles", "ffn_tc_kernel_olmoe_M63_B32.counters.txt")


def read_counters(path=None):
    """key = value lines of a counters file -> dict of floats (None when the file is missing)."""
    path = path or os.path.join(ROOT, TRAFFIC_FILE)
    if not os.path.exists(path):
        return None
    out = {}
    for line in open(path):
        line = line.split("#", 1)[0].strip()
        if "=" in line:
            k_, v_ = line.split("=", 1)
            try:
                out[k_.strip()] = float(v_.strip())
            except ValueError:
                pass
    return out


def dram_traffic_per_launch():
    c = read_counters()
    if not c or "dram__bytes_read.sum" not in c or "dram__bytes_write.sum" not in c:
        return None
    return c["dram__bytes_read.sum"] + c["dram__bytes_write.sum"]


def workload_name(cfg):
    return (f"{WORKLOAD} single layer d={cfg.d} N={cfg.n_experts} k={cfg.k} f={cfg.f} M={M_TOKENS} B={B_HEADLINE} "
            f"substitution renormalised, bf16 weights, fp32 accumulate and output")


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def mark(self):
        return time.time()

    def stop(self, t0=None, t1=None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        rows = [l for (t, l) in self.lines if (t0 is None or t >= t0 - 0.05) and (t1 is None or t <= t1 + 0.15)]
        if not rows:
            rows = [l for _, l in self.lines]
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in rows:
            parts = [x.strip() for x in l.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0])); smax.append(float(parts[1])); power.append(float(parts[2]))
            except ValueError:
                continue
            for n, v in zip(names, parts[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def algorithmic_bytes(cfg, M, n_active, out_bytes):
    """Bytes the method itself must move for one layer: kept experts' weights, the router, hidden in, out."""
    w = 4 if cfg.dtype == "fp32" else 2
    return n_active * 3 * cfg.d * cfg.f * w + cfg.n_experts * cfg.d * w + M * cfg.d * w + M * cfg.d * out_bytes


def build_layers(cfg, M, n_copies, device, out_dtype, resident=None):
    """resident = (first, count): only that block of every copy's experts is generated and held (expert-parallel)."""
    from paper_2602_16052_b200 import moespec
    layers, hiddens = [], []
    experts = None if resident is None else range(resident[0], resident[0] + resident[1])
    for c in range(n_copies):
        L = synth.gen_layer(cfg, seed=1000 + c, layer=0, device=device, experts=experts)
        hiddens.append(synth.gen_hidden(cfg, M, seed=1000 + c, layer=0, device=device))
        layers.append(moespec.Layer(L["router_w"], L["router_bias"], L["w_gate"], L["w_up"], L["w_down"], max_M=M,
                                    max_k=cfg.k, policy=moespec.SUBSTITUTION, shortlist=moespec.FROM_ALL,
                                    renormalize=True, out_dtype=out_dtype, resident=resident))
    return layers, hiddens


def run_expert_parallel(args, dist, device, rank, world, barrier):
    """--mode ep: one layer split by experts over the ranks; per step every rank runs its shard and the partial
    outputs are summed with one all-reduce.  Prints the benchmark line (rank 0)."""
    from paper_2602_16052_b200 import ep
    cfg = synth.CONFIGS[WORKLOAD]
    M, k, B = M_TOKENS, cfg.k, B_HEADLINE
    resident = ep.expert_range(rank, world, cfg.n_experts)
    layers, hiddens = build_layers(cfg, M, args.copies, device, torch.float32, resident if world > 1 else None)
    outs = [torch.empty((M, cfg.d), dtype=torch.float32, device=device) for _ in layers]
    n = len(layers)
    stream = torch.cuda.current_stream()

    def step(i):
        layers[i % n].verify_layer(hiddens[i % n], k, B, outs[i % n], stream)
        if world > 1:
            dist.all_reduce(outs[i % n])          # sum of the shards' partial outputs, on every rank

    sampler = ClockSampler(device.index or 0)
    sampler.start()
    time.sleep(0.3)
    for i in range(args.warmup):
        step(i)
    barrier()
    torch.cuda.synchronize()
    t0m = sampler.mark()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(args.steps):
        step(i)
    e1.record(stream)
    torch.cuda.synchronize()
    barrier()
    clocks = sampler.stop(t0m, sampler.mark())
    ms_total = job_time_ms(e0.elapsed_time(e1), dist, device)
    # end to end: the step's hidden states come from pinned host memory and the reduced output goes back
    h_host = [h.cpu().pin_memory() for h in hiddens]
    o_host = [torch.empty((M, cfg.d), dtype=torch.float32).pin_memory() for _ in layers]
    def step_e2e(i):
        hiddens[i % n].copy_(h_host[i % n], non_blocking=True)
        step(i)
        o_host[i % n].copy_(outs[i % n], non_blocking=True)
        torch.cuda.current_stream().synchronize()
    for i in range(args.warmup):
        step_e2e(i)
    barrier()
    t0 = time.perf_counter()
    for i in range(args.steps):
        step_e2e(i)
    e2e_ms = job_time_ms((time.perf_counter() - t0) * 1e3, dist, device)
    act = torch.tensor([float(sum(L.get_stats()["n_active"] for L in layers)) / n], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(act)
    n_active = float(act.item())                 # kept experts with rows, summed over the shards
    peak, peak_kind = measured_peaks()
    us = ms_total * 1e3 / args.steps             # the job processes `steps` layers in total
    layer_bytes = algorithmic_bytes(cfg, M, n_active, 4)
    agg = layer_bytes / (us * 1e-6) / 1e9
    if rank == 0:
        line = {
            "metric": METRIC, "value": us, "unit": "us", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_total / args.steps, "higher_is_better": False, "scaling": "strong", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": workload_name(cfg), "parallelism": f"ep{world}: experts split in contiguous blocks, "
                       "router replicated, one NCCL all-reduce of out[M,d] fp32 per layer inside the timed region",
                       "l2": f"rotating over {args.copies} independently seeded layer copies", "n_active": n_active},
            "clocks": clocks,
            "e2e": {"value": e2e_ms * 1e3 / args.steps, "unit": "us", "h2d_bytes_per_step": h_host[0].numel() * 2,
                    "d2h_bytes_per_step": o_host[0].numel() * 4},
            "gpu_launches": layers[0].last_launch_count() * args.steps,
            "roofline": {"bound": "hbm", "kernel": "ffn_tc_kernel on every rank (its resident kept experts)",
                         "achieved": agg, "peak": peak * world, "unit": "GB/s", "frac": agg / (peak * world),
                         "peak_kind": f"of {peak_kind} x {world} GPUs", "traffic": None,
                         "basis": "algorithmic bytes of the whole layer / step time incl. the all-reduce"},
            "cpu_baseline": None,
        }
        print(json.dumps(line), flush=True)
    for L in layers:
        L.destroy()


def time_steps(layers, hiddens, outs, k, B, steps, warmup, barrier):
    """W untimed steps, then exactly K steps between two events on the launching stream."""
    n = len(layers)
    stream = torch.cuda.current_stream()
    for i in range(warmup):
        layers[i % n].verify_layer(hiddens[i % n], k, B, outs[i % n], stream)
    barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(steps):
        layers[i % n].verify_layer(hiddens[i % n], k, B, outs[i % n], stream)
    e1.record(stream)
    torch.cuda.synchronize()
    barrier()
    return e0.elapsed_time(e1)  # ms


def time_batches(layers, hiddens, outs, k, B, n_batches, per_batch):
    """Distribution of the step time: n_batches batches of per_batch steps, each batch between two events on
    the launching stream (an event after every single step would break the overlap of consecutive layers).
    Returns microseconds per step of every batch."""
    n = len(layers)
    stream = torch.cuda.current_stream()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(n_batches + 1)]
    for i in range(per_batch):
        layers[i % n].verify_layer(hiddens[i % n], k, B, outs[i % n], stream)
    torch.cuda.synchronize()
    ev[0].record(stream)
    i = 0
    for b in range(n_batches):
        for _ in range(per_batch):
            layers[i % n].verify_layer(hiddens[i % n], k, B, outs[i % n], stream)
            i += 1
        ev[b + 1].record(stream)
    torch.cuda.synchronize()
    return [ev[b].elapsed_time(ev[b + 1]) * 1e3 / per_batch for b in range(n_batches)]


def time_e2e(layers, hiddens, k, B, steps, warmup, out_dtype):
    """Same metric through the host-buffer entry point: H2D of the step's hidden states and D2H of its
    result are inside the timed region of every step."""
    n = len(layers)
    h_host = [h.cpu().pin_memory() for h in hiddens]
    o_host = [torch.empty(h.shape, dtype=out_dtype).pin_memory() for h in hiddens]
    for i in range(warmup):
        layers[i % n].verify_layer_host(h_host[i % n], k, B, o_host[i % n])
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for i in range(steps):
        layers[i % n].verify_layer_host(h_host[i % n], k, B, o_host[i % n])   # synchronises inside
    t1 = time.perf_counter()
    h2d = h_host[0].numel() * h_host[0].element_size()
    d2h = o_host[0].numel() * o_host[0].element_size()
    return (t1 - t0) * 1e3, h2d, d2h


def kernel_profile(layers, hiddens, outs, k, B, reps):
    """Average per-kernel duration with the library's event bracketing (separate from the timed region)."""
    n = len(layers)
    acc = {}
    for L in layers:
        L.set_profiling(True)
    for i in range(reps + 3):
        L = layers[i % n]
        L.verify_layer(hiddens[i % n], k, B, outs[i % n])
        t = L.get_kernel_times()
        if i >= 3:
            for name, ms in t.items():
                acc.setdefault(name, []).append(ms)
    for L in layers:
        L.set_profiling(False)
    return {name: sum(v) / len(v) for name, v in acc.items()}


def run_analysis(cfg, layer0, hidden, M, device):
    """Reconstruction error ||O_S - O*||^2 / ||O*||^2 (Section 4.5) of router-based, static and oracle (Eq. 6)
    shortlists at several budgets, truncation outputs, on one layer of the benchmark workload; and the time
    of the oracle ranking itself (an unpruned pass, the Gram matrices and the greedy loop)."""
    from paper_2602_16052_b200 import moespec
    rw, rb, wg, wu, wd = layer0._keep
    mk = lambda mode: moespec.Layer(rw, rb, wg, wu, wd, max_M=128, max_k=cfg.k, policy=moespec.TRUNCATION,
                                    shortlist=mode, renormalize=True, out_dtype=torch.float32)
    router, static, oracle = mk(moespec.FROM_ALL), mk(moespec.STATIC), mk(moespec.STATIC)
    O_star = torch.empty((M, cfg.d), dtype=torch.float32, device=device)
    order, obj, gold = router.oracle_ranking(hidden, cfg.k, cfg.n_experts, O_star)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(5):
        router.oracle_ranking(hidden, cfg.k, cfg.n_experts, O_star)
    rank_us = (time.perf_counter() - t0) / 5 * 1e6
    for j in range(4):
        static.calibrate(synth.gen_hidden(cfg, 128, seed=7000 + j, device=device), cfg.k)
    static.set_static_ranking()
    oracle.set_static_ranking(order)
    rows = []
    for B in (8, 16, 24, 32, 48):
        row = {"B": B}
        for name, lay in (("router", router), ("static", static), ("oracle", oracle)):
            O_S = lay.verify_layer(hidden, cfg.k, B)
            row[name] = router.reconstruction_error(O_S, O_star)[0]
        rows.append(row)
    for lay in (router, static, oracle):
        lay.destroy()
    return {"M": M, "policy": "truncation", "reconstruction_error": rows, "oracle_ranking_us": rank_us,
            "note": "synthetic router and experts: the curves show the mechanism, not the paper's trained-model values"}


def time_stack(cfg, M, B, device, reps):
    """L-layer residual stack (bf16 stream): microseconds per layer through the stack entry point (one graph
    launch per pass), through the same entry point enqueuing kernel by kernel, and as L separate layer
    calls; plus the share of the event-bracketed kernel time that goes to choosing experts."""
    from paper_2602_16052_b200 import moespec
    L = cfg.n_layers
    weights = [synth.gen_layer(cfg, seed=2000, layer=l, device=device) for l in range(L)]
    layers = [moespec.Layer(w["router_w"], w["router_bias"], w["w_gate"], w["w_up"], w["w_down"], max_M=M,
                            max_k=cfg.k, policy=moespec.SUBSTITUTION, shortlist=moespec.FROM_ALL, renormalize=True,
                            residual=True) for w in weights]
    stack = moespec.Stack(layers)
    x0 = synth.gen_hidden(cfg, M, seed=2000, layer=0, device=device)
    out = torch.empty_like(x0)
    bufs = [torch.empty_like(x0) for _ in range(2)]
    budgets = [B] * L

    def by_calls():
        cur = x0
        for l, lay in enumerate(layers):
            lay.verify_layer(cur, cfg.k, B, bufs[l % 2])
            cur = bufs[l % 2]

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / (reps * L)

    us_graph = timed(lambda: stack.verify_stack(x0, cfg.k, budgets, out))
    # host-side cost of enqueuing one pass (the call returns once the work is queued)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    stack.verify_stack(x0, cfg.k, budgets, out)
    enqueue_graph_us = (time.perf_counter() - t0) * 1e6
    torch.cuda.synchronize()
    stack.set_graph(False)
    us_plain = timed(lambda: stack.verify_stack(x0, cfg.k, budgets, out))
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    stack.verify_stack(x0, cfg.k, budgets, out)
    enqueue_plain_us = (time.perf_counter() - t0) * 1e6
    torch.cuda.synchronize()
    stack.set_graph(True)
    us_calls = timed(by_calls)
    act = sum(lay.get_stats()["n_active"] for lay in layers) / L
    # per-kernel times of one pass with event bracketing (outside the timed runs)
    acc = {}
    for lay in layers:
        lay.set_profiling(True)
    for _ in range(3):
        cur = x0
        for l, lay in enumerate(layers):
            lay.verify_layer(cur, cfg.k, B, bufs[l % 2])
            cur = bufs[l % 2]
            for name, ms_ in lay.get_kernel_times().items():
                acc[name] = acc.get(name, 0.0) + ms_
    tot = sum(acc.values())
    line = {"layers": L, "M": M, "B": B, "us_per_layer_graph": us_graph, "us_per_layer_kernel_by_kernel": us_plain,
            "us_per_layer_separate_calls": us_calls, "host_enqueue_us_per_pass_graph": enqueue_graph_us,
            "host_enqueue_us_per_pass_kernel_by_kernel": enqueue_plain_us, "gpu_launches_per_pass": stack.last_launch_count(),
            "n_active_mean": act, "kernel_share": {n: v / tot for n, v in acc.items()},
            "selection_share_of_layer": (tot - acc.get("ffn", 0.0)) / tot}
    stack.destroy()
    for lay in layers:
        lay.destroy()
    del layers, weights
    torch.cuda.empty_cache()
    return line


def run_tables(args, device):
    """Sweeps over every workload shape (not part of the default run): one JSON line per point."""
    from paper_2602_16052_b200 import moespec
    peak, peak_kind = measured_peaks()
    names = args.tables.split(",")
    for name in names:
        cfg = synth.CONFIGS[name]
        L = cfg.n_layers
        n_copies = L if L > 1 else (2 if name == "mixtral" else 4)
        Ms, Bs = synth.SWEEPS[name]["M"], synth.SWEEPS[name]["B"]
        if args.only_M:          # one point (or a few) instead of the sweep, e.g. for a profiler capture
            Ms = [int(x) for x in args.only_M.split(",")]
        if args.only_B:
            Bs = [int(x) for x in args.only_B.split(",")]
        max_M = max(Ms)
        weights = [synth.gen_layer(cfg, seed=2000, layer=l, device=device) for l in range(n_copies)]
        out_dtype = torch.bfloat16 if L > 1 else torch.float32
        layers = [moespec.Layer(w["router_w"], w["router_bias"], w["w_gate"], w["w_up"], w["w_down"], max_M=max_M,
                                max_k=cfg.k, policy=moespec.SUBSTITUTION, shortlist=moespec.FROM_ALL, renormalize=True,
                                residual=L > 1, out_dtype=out_dtype) for w in weights]
        stack = moespec.Stack(layers) if L > 1 else None
        for M in Ms:
            x0 = synth.gen_hidden(cfg, M, seed=2000, layer=0, device=device)
            bufs = [torch.empty_like(x0, dtype=out_dtype) for _ in range(2)]
            for B in Bs:
                def one_pass():
                    if L > 1:        # stack: x <- dtype(x + MoE_l(x)), all layers as one graph launch
                        stack.verify_stack(x0, cfg.k, [B] * L, bufs[0])
                    else:            # single layer: rotate over independently seeded copies
                        for lay in layers:
                            lay.verify_layer(x0, cfg.k, B, bufs[0])
                reps = max(3, args.steps // len(layers))
                for _ in range(2):
                    one_pass()
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(reps):
                    one_pass()
                e1.record()
                torch.cuda.synchronize()
                us = e0.elapsed_time(e1) * 1e3 / (reps * len(layers))
                st = [lay.get_stats() for lay in layers]
                act = sum(s_["n_active"] for s_ in st) / len(st)
                uni = sum(s_["n_union"] for s_ in st) / len(st)
                by = algorithmic_bytes(cfg, M, act, 2 if out_dtype == torch.bfloat16 else 4)
                cpu_us = None
                if args.tables_cpu:        # the oracle on one layer of this point, once (host cores)
                    case = oracle_case(cfg, M, seed=2000, device=device)
                    cpu_us, cpu_cores, _ = time_oracle(cfg, M, B, 0.0, 1, case)
                    del case
                print(json.dumps({"table": name, "layers": L, "M": M, "B": B, "us_per_layer": round(us, 2),
                                  "cpu_oracle_us": None if cpu_us is None else round(cpu_us),
                                  "n_active": round(act, 2), "n_union": round(uni, 2), "MB": round(by / 1e6, 1),
                                  "GBs": round(by / us / 1e3, 1), "frac_of_" + peak_kind: round(by / us / 1e3 / peak, 3),
                                  "ideal_us": round(by / peak / 1e3, 1)}), flush=True)
        if stack is not None:
            stack.destroy()
        for lay in layers:
            lay.destroy()
        del layers, weights
        torch.cuda.empty_cache()


def job_time_ms(local_ms: float, dist=None, device=None) -> float:
    """Job time of a replicated run: the slowest rank's device time (max over ranks)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return local_ms
    t = torch.tensor([local_ms], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_us_per_layer(job_ms: float, steps: int, world: int) -> float:
    """Whole-job metric of N independent replicas: every rank ran `steps` layers in `job_ms`."""
    return job_ms * 1e3 / (steps * world)


def oracle_case(cfg, M, seed, device="cpu"):
    """Inputs of one layer as fp64 numpy arrays (generated on `device`: the generator gives the same bits)."""
    L = synth.gen_layer(cfg, seed=seed, layer=0, device=device)
    h = synth.gen_hidden(cfg, M, seed=seed, layer=0, device=device)
    f64 = lambda t: t.to("cpu").to(torch.float64).numpy()
    return {k: f64(v) for k, v in L.items()}, f64(h)


def time_oracle(cfg, M, B, min_seconds, max_reps, case=None, threads=None):
    """The CPU oracle as it stands on the host cores: whole layers of the same workload until the
    sample has used about `min_seconds` of wall time (at most max_reps layers).  threads=1 limits the
    numerical library under numpy to one thread (the oracle itself is not changed)."""
    from oracle import moespec_oracle as orc
    L, h = case or oracle_case(cfg, M, seed=1000)
    try:
        from threadpoolctl import threadpool_info, threadpool_limits
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] or [os.cpu_count() or 1])
    except Exception:
        threadpool_limits = None
        cores = os.cpu_count() or 1

    def run():
        times = []
        t_start = time.perf_counter()
        while len(times) < max_reps and (not times or time.perf_counter() - t_start < min_seconds):
            t0 = time.perf_counter()
            orc.verify_layer(h, L["router_w"], L["router_bias"], L["w_gate"], L["w_up"], L["w_down"], cfg.k, B,
                             orc.SUBSTITUTION, orc.FROM_ALL, True)
            times.append(time.perf_counter() - t0)
        return times

    if threads is not None and threadpool_limits is not None:
        with threadpool_limits(limits=threads):
            times = run()
        cores = threads
    else:
        times = run()
    return statistics.median(times) * 1e6, cores, len(times)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = synth.CONFIGS[WORKLOAD]
    case = oracle_case(cfg, M_TOKENS, seed=1000)
    warm = min(args.warmup, 3)
    for _ in range(warm):
        time_oracle(cfg, M_TOKENS, B_HEADLINE, 0.0, 1, case)
    steps = max(1, min(args.steps, 200))       # a layer takes ~50 ms on the host cores: K steps as asked, up to ~10 s
    us, cores, reps = time_oracle(cfg, M_TOKENS, B_HEADLINE, 1e9, steps, case)
    sample = f"{reps} whole verify layers (M={M_TOKENS}, B={B_HEADLINE}) of the same workload, median"
    line = {
        "impl": "reference", "metric": METRIC, "value": us, "unit": "us", "n_gpus": args.gpus, "steps": reps,
        "warmup": warm, "ms_per_step": us / 1e3, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(cfg)},
        "cpu_baseline": {"value": us, "unit": "us", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": us, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="moespec", choices=["moespec", "reference"])
    ap.add_argument("--mode", default="replicas", choices=["replicas", "ep"],
                    help="multi-GPU mode: independent replicas (default) or one layer split by experts")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--copies", type=int, default=N_COPIES, help="independently seeded layer copies rotated over")
    ap.add_argument("--tables", default="", help="comma-separated workload names (tiny is excluded): sweep M and B "
                    "of each and print one JSON line per point instead of the benchmark line")
    ap.add_argument("--tables-cpu", action="store_true",
                    help="with --tables: also time the CPU oracle once per point (one layer, host cores)")
    ap.add_argument("--only-M", default="", help="with --tables: tree sizes to run instead of the workload's sweep")
    ap.add_argument("--only-B", default="", help="with --tables: budgets to run instead of the workload's sweep")
    ap.add_argument("--timed-only", action="store_true",
                    help="run only the warm-up and the timed steps (for profiler captures); prints a short line")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    args.warmup = max(args.warmup, 3)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    else:
        torch.cuda.set_device(0)
        local_rank = 0
    device = torch.device("cuda", local_rank)

    def barrier():
        if dist is not None:
            dist.barrier()

    def max_over_ranks(x: float) -> float:
        return job_time_ms(x, dist, device)

    if args.tables:
        return run_tables(args, device)
    if args.mode == "ep":
        run_expert_parallel(args, dist, device, rank, world, barrier)
        if dist is not None:
            dist.destroy_process_group()
        return

    cfg = synth.CONFIGS[WORKLOAD]
    M, k, B = M_TOKENS, cfg.k, B_HEADLINE
    out_dtype = torch.float32          # unrounded fp32 accumulators, the output the 2e-2*RMS bar is stated on
    layers, hiddens = build_layers(cfg, M, args.copies, device, out_dtype)
    outs = [torch.empty((M, cfg.d), dtype=out_dtype, device=device) for _ in layers]

    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    t_mark0 = sampler.mark()
    ms_total = time_steps(layers, hiddens, outs, k, B, args.steps, args.warmup, barrier)
    t_mark1 = sampler.mark()
    clocks = sampler.stop(t_mark0, t_mark1)
    ms_total = max_over_ranks(ms_total)
    launches_per_step = layers[0].last_launch_count()
    stats = layers[0].get_stats()
    assert stats["status"] == 0, stats

    if args.timed_only:
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": ms_total * 1e3 / (args.steps * world), "unit": "us",
                              "steps": args.steps, "warmup": args.warmup, "timed_only": True,
                              "gpu_launches": launches_per_step * args.steps}), flush=True)
        return

    # distribution over at least 100 further steps, whatever --steps was
    per_batch = 10
    batch_us = time_batches(layers, hiddens, outs, k, B, max(10, (args.steps + per_batch - 1) // per_batch), per_batch)
    median_us, min_us = statistics.median(batch_us), min(batch_us)

    e2e_ms, h2d, d2h = time_e2e(layers, hiddens, k, B, args.steps, args.warmup, out_dtype)
    e2e_ms = max_over_ranks(e2e_ms)

    # value: job-wide microseconds per verify layer (all ranks' layers / max time over ranks)
    us_per_layer = job_us_per_layer(ms_total, args.steps, world)
    e2e_us = job_us_per_layer(e2e_ms, args.steps, world)

    # Roofline.  The dominant kernel is the expert-FFN weight stream (ffn_tc_kernel, one launch per layer).  In
    # the product its launch overlaps the routing kernels (it starts on the shortlist while they finish), so a
    # duration of that kernel alone exists only when events between the kernels serialise them.  The top-level
    # figure is therefore the conservative one: all algorithmic bytes of the layer over the un-bracketed step
    # time of the timed region; the event-bracketed kernel alone is reported under "kernel_only".
    peak, peak_kind = measured_peaks()
    kt = kernel_profile(layers, hiddens, outs, k, B, reps=40)
    n_active = [L.get_stats()["n_active"] for L in layers]
    mean_active = sum(n_active) / len(n_active)
    ffn_bytes = mean_active * cfg.expert_weight_bytes()
    ffn_ms = kt["ffn"]
    achieved = ffn_bytes / (ffn_ms * 1e-3) / 1e9
    layer_bytes = algorithmic_bytes(cfg, M, mean_active, 4)
    layer_gbs = layer_bytes / (us_per_layer * world * 1e-6) / 1e9
    roofline = {
        "bound": "hbm", "kernel": "ffn_tc_kernel (gate/up units, down units and the combine in one launch; "
                                  "overlaps the routing kernels)",
        "achieved": layer_gbs, "peak": peak, "unit": "GB/s", "frac": layer_gbs / peak, "peak_kind": f"of {peak_kind}",
        "frac_of_nominal_8TBs": layer_gbs / 8000.0,
        "basis": "algorithmic bytes of the whole layer / un-bracketed step time of the timed region",
        "traffic": dram_traffic_per_launch(), "traffic_source": TRAFFIC_FILE,
        "algorithmic_bytes_per_layer": layer_bytes,
        "kernel_only": {"achieved": achieved, "frac": achieved / peak, "algorithmic_bytes_per_launch": ffn_bytes,
                        "us": ffn_ms * 1e3, "note": "events between the kernels serialise them"},
        "kernel_us": {n: v * 1e3 for n, v in kt.items()},
        # share of the event-bracketed kernel time spent choosing experts (router, shortlist, re-routing,
        # gather); the paper quotes 2-3 % of whole-model generation time for its selection step
        "selection_share_of_layer": (sum(v for n, v in kt.items() if n != "ffn") / sum(kt.values())),
    }

    sweep = []
    if not args.no_sweep:
        for Bs in synth.SWEEPS[WORKLOAD]["B"]:
            ms_b = time_steps(layers, hiddens, outs, k, Bs, max(20, args.steps // 4), 5, barrier)
            act = sum(L.get_stats()["n_active"] for L in layers) / len(layers)
            us_b = ms_b * 1e3 / max(20, args.steps // 4)
            by = algorithmic_bytes(cfg, M, act, 4)
            sweep.append({"M": M, "B": Bs, "us": us_b, "n_active": act, "GBs": by / (us_b * 1e-6) / 1e9,
                          "frac": by / (us_b * 1e-6) / 1e9 / peak})

    # raw (non-renormalised) mixing weights, the other architecture choice of Section 2.1: same kernels
    raw_line = None
    if not args.no_sweep:
        from paper_2602_16052_b200 import moespec as _m
        raw_layers = []
        for L0 in layers:
            rw, rb, wg, wu, wd = L0._keep
            raw_layers.append(_m.Layer(rw, rb, wg, wu, wd, max_M=M, max_k=cfg.k, policy=_m.SUBSTITUTION,
                                       shortlist=_m.FROM_ALL, renormalize=False, out_dtype=out_dtype))
        n_raw = max(20, args.steps // 4)
        ms_raw = time_steps(raw_layers, hiddens, outs, k, B, n_raw, 5, barrier)
        raw_line = {"M": M, "B": B, "us": ms_raw * 1e3 / n_raw, "renormalize": False}
        for RL in raw_layers:
            RL.destroy()

    # time against kept experts: slope = FFN stream per expert, intercept = routing chain + FFN ramp and tail
    fit = None
    if len(sweep) >= 3:
        xs = np.array([p_["n_active"] for p_ in sweep]); ys = np.array([p_["us"] for p_ in sweep])
        slope, icpt = np.polyfit(xs, ys, 1)
        fit = {"us_per_expert": float(slope), "intercept_us": float(icpt),
               "marginal_GBs": cfg.expert_weight_bytes() / (float(slope) * 1e-6) / 1e9 if slope > 0 else None}

    # read-only stream rate of this GPU (a library reduction over 2 GiB), context for the copy-based peak
    big = torch.empty(1 << 30, dtype=torch.bfloat16, device=device).fill_(1)
    for _ in range(2):
        big.sum()
    torch.cuda.synchronize()
    r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    r0.record()
    for _ in range(5):
        big.sum()
    r1.record()
    torch.cuda.synchronize()
    read_stream_gbs = 5 * big.numel() * 2 / (r0.elapsed_time(r1) * 1e-3) / 1e9
    del big

    # static ranking (Eq. 4) on the same workload: fixed ordering from 512 calibration tokens per copy
    static_line = None
    if not args.no_sweep:
        from paper_2602_16052_b200 import moespec
        st_layers = []
        for c, L0 in enumerate(layers):
            rw, rb, wg, wu, wd = L0._keep
            SL = moespec.Layer(rw, rb, wg, wu, wd, max_M=128, max_k=cfg.k, policy=moespec.SUBSTITUTION,
                               shortlist=moespec.STATIC, renormalize=True, out_dtype=out_dtype)
            for j in range(4):
                SL.calibrate(synth.gen_hidden(cfg, 128, seed=5000 + 10 * c + j, device=device), cfg.k)
            SL.set_static_ranking()
            st_layers.append(SL)
        n_st = max(20, args.steps // 4)
        ms_st = time_steps(st_layers, hiddens, outs, k, B, n_st, 5, barrier)
        act = sum(L_.get_stats()["n_active"] for L_ in st_layers) / len(st_layers)
        cov = sum(L_.get_stats()["coverage"] for L_ in st_layers) / len(st_layers)
        static_line = {"M": M, "B": B, "us": ms_st * 1e3 / n_st, "n_active": act, "coverage": cov,
                       "calibration_tokens": 512}
        for SL in st_layers:
            SL.destroy()

    # expert-parallel shards of the same layers, each timed alone on this GPU: the compute part of an
    # expert-parallel step is the slowest shard (the all-reduce of out[M,d] is not in these numbers, and no
    # multi-GPU run is behind them)
    ep_line = None
    if not args.no_sweep and world == 1:
        from paper_2602_16052_b200 import ep as _ep, moespec as _m2
        ep_line = []
        for G in (2, 4, 8):
            per_rank = []
            for r_ in range(G):
                first, count = _ep.expert_range(r_, G, cfg.n_experts)
                sh = []
                for L0 in layers:
                    rw, rb, wg, wu, wd = L0._keep
                    sh.append(_m2.Layer(rw, rb, wg[first:first + count], wu[first:first + count], wd[first:first + count],
                                        max_M=M, max_k=cfg.k, policy=_m2.SUBSTITUTION, shortlist=_m2.FROM_ALL,
                                        renormalize=True, out_dtype=out_dtype, resident=(first, count)))
                n_sh = max(20, args.steps // 8)
                ms_sh = time_steps(sh, hiddens, outs, k, B, n_sh, 5, barrier)
                act = sum(L_.get_stats()["n_active"] for L_ in sh) / len(sh)
                per_rank.append({"rank": r_, "us": ms_sh * 1e3 / n_sh, "n_active": act})
                for L_ in sh:
                    L_.destroy()
            ep_line.append({"shards": G, "slowest_shard_us": max(p_["us"] for p_ in per_rank),
                            "fastest_shard_us": min(p_["us"] for p_ in per_rank),
                            "n_active_per_shard": [p_["n_active"] for p_ in per_rank]})

    # analysis mode on the same workload: reconstruction error of the three ranking strategies (Section 4.5)
    analysis_line = None
    if not args.no_sweep:
        analysis_line = run_analysis(cfg, layers[0], hiddens[0], M, device)

    # the 16-layer stack of the same shape: one graph launch per pass against layer-by-layer calls
    stack_line = None
    if not args.no_sweep:
        stack_line = time_stack(synth.CONFIGS["olmoe16"], M, B, device, max(3, args.steps // 64))

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        case = oracle_case(cfg, M, seed=1000)
        us, cores, reps = time_oracle(cfg, M, B, 10.0, 6, case)
        us1, _, reps1 = time_oracle(cfg, M, B, 5.0, 3, case, threads=1)
        cpu = {"value": us, "unit": "us", "cores": cores, "kind": "oracle",
               "sample": f"{reps} whole verify layers (M={M}, B={B}) of the same workload, median",
               "single_thread_us": us1, "single_thread_sample": f"{reps1} layers with the numerical library limited to one thread"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": us_per_layer, "unit": "us", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "median_us": median_us, "min_us": min_us,
            "distribution": {"batches": len(batch_us), "steps_per_batch": per_batch},
            "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": workload_name(cfg),
                       "l2": f"rotating over {args.copies} independently seeded layer copies "
                             f"({args.copies * cfg.n_experts * cfg.expert_weight_bytes() / 1e9:.1f} GB); each step streams "
                             f"{ffn_bytes / 1e6:.0f} MB > 126 MB L2",
                       "replicas": world, "n_active": mean_active, "n_union": stats["n_union"],
                       "coverage": stats["coverage"]},
            "clocks": clocks,
            "e2e": {"value": e2e_us, "unit": "us", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline,
            "cpu_baseline": cpu,
            "sweep": sweep,
            "static_ranking": static_line,
            "raw_gating": raw_line,
            "stack": stack_line,
            "analysis": analysis_line,
            "ep_shards_on_one_gpu": ep_line,
            "fit_time_vs_active_experts": fit,
            "read_stream_GBs_torch_sum": read_stream_gbs,
        }
        print(json.dumps(line), flush=True)
    for L in layers:
        L.destroy()
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
