#!/usr/bin/env python
"""bench.py -- one JSON line for the PRISM hot path on B200.

A step is one top-K selection request (prism_select: pack -> embed -> 28 layers with probe / route /
compact after the designated layers -> top-K) of the Qwen3-0.6B-shaped workload (configs[1]: 100
candidates, query 32 tokens, documents uniform 128-512 tokens, K = 10, cluster pruning with probes at
layers 8, 12, ..., 24).  `value` is candidate-tokens/s = submitted tokens of all requests / device
time with the inputs already in HBM; `e2e` is the same through prism_select_host with host buffers.
With --gpus N every rank serves its own stream of requests (no data-path collective; weak scaling).
At N = 1 the default run also measures the other four benchmark workloads (tiny fp32, 4B-shaped, 8B-shaped streamed
and chunked, 1000-candidate stress) and reports them in a `workloads` block of the same line; the headline keys stay
those of workload 1.  `cpu_baseline` times the CPU oracle on a length-stratified sample of request 0.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload 1]
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

METRIC = "candidate-tokens/s (p50/p99 top-K select latency in ms beside it)"
UNIT = "candidate-tokens/s"
KERNEL_CLASSES = ["pack", "embed", "rmsnorm", "gemm_qkv", "rope", "attention", "gemm_o", "gemm_gateup", "gemm_down",
                  "probe", "route", "compact", "dequant"]
GEMM_CLASSES = ("gemm_qkv", "gemm_o", "gemm_gateup", "gemm_down")
# dram__bytes_read.sum + dram__bytes_write.sum of one k_gemm_tc2 launch at M = 8192 with the cfg1 weight
# shapes, from the ncu captures summarised under profiles/gemm_tc2_*.md.
# Reads grow in proportion to M; writes are mostly absorbed by the 126 MB L2 inside the kernel's window.
NCU_TRAFFIC_M8192 = {"gemm_qkv": 42.6e6, "gemm_o": 72.5e6, "gemm_gateup": 36.8e6, "gemm_down": 94.5e6}
CFG1_NK = {"gemm_qkv": (4096, 1024), "gemm_o": (1024, 2048), "gemm_gateup": (6144, 1024), "gemm_down": (1024, 3072)}


# ----------------------------------------------------------------------------------------------- helpers
def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.samples, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        mhz, mx, reasons, power = [], None, set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for s in self.samples:
            f = [x.strip() for x in s.split(",")]
            if len(f) < 7:
                continue
            try:
                mhz.append(float(f[0]))
                mx = float(f[1])
                power.append(float(f[2]))
            except ValueError:
                continue
            for nm, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(mhz)) if mhz else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(mhz), "power_w_max": max(power) if power else None}


def shard_requests(rank: int, world: int, n_requests: int):
    """Request seeds served by `rank`: every rank gets its own n_requests seeds (weak scaling)."""
    return [rank * n_requests + i for i in range(n_requests)]


def max_over_ranks(value: float, world: int, device=None) -> float:
    """MAX all-reduce of a scalar over the process group (identity for world == 1)."""
    if world == 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, world: int, device=None) -> float:
    if world == 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


# ----------------------------------------------------------------------------------------------- oracle legs
def oracle_sample_ids(wl, req, budget_s: float = 25.0, max_cand: int = 2):
    """A bounded, length-stratified sample of the request for the CPU oracle: m candidates evenly spaced in
    length rank (the median first, then the extremes and the quantiles between them), with m the largest count
    up to max_cand whose estimated time stays within budget_s (2 * layer parameters flops per token at the
    ~4e11 flop/s the fp64 numpy forward sustains on 16 cores; 5e11 - 8e11 were measured); at least one."""
    cfg = wl.model
    p_layer = cfg.hidden * (cfg.n_q_heads + 2 * cfg.n_kv_heads) * cfg.head_dim + cfg.n_q_heads * cfg.head_dim * cfg.hidden \
        + 3 * cfg.hidden * cfg.ffn
    s_per_token = 2.0 * p_layer * cfg.n_layers / 4e11
    lens = np.diff(req["cand_offsets"]) + len(req["query"])
    order = np.argsort(lens, kind="stable")
    n = len(order)
    m = int(max(1, min(max_cand, n, budget_s / (float(np.mean(lens)) * s_per_token))))
    ranks = [n // 2] if m == 1 else sorted(set(int(round(j * (n - 1) / (m - 1))) for j in range(m)))
    if m == 1 and lens[order[n // 2]] * s_per_token > 1.5 * budget_s:
        ranks = [0]         # even the median candidate is far beyond the budget (8B shape): the shortest one
    return sorted(int(order[r]) for r in ranks)


def oracle_sample_rate(wl, weights_np, req, ids):
    """Times the CPU oracle, as it stands, on the candidates `ids` of the request through all layers
    (unpruned forward + scoring).  Returns (tokens/s, seconds, tokens)."""
    import oracle
    cfg = wl.model
    ids = list(ids)
    lens = np.diff(req["cand_offsets"])[ids] + len(req["query"])
    layers = sorted(set(list(wl.schedule.probe_layers) + [cfg.n_layers]))
    t0 = time.perf_counter()
    oracle.score_matrix(req["query"], req["cand_tokens"], req["cand_offsets"], weights_np, cfg, layers, candidates=ids)
    dt = time.perf_counter() - t0
    return float(lens.sum()) / dt, dt, int(lens.sum())


def run_reference(args):
    """--impl reference: the oracle on the host cores, each step a bounded sample of the workload."""
    import synth
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    wl = synth.workload(args.workload)
    w = synth.make_weights(wl.model, wl.weight_seed)
    n_cand = 3      # the shortest, the median and the longest candidate of each request (budget permitting)
    rates, times, toks = [], [], 0
    for step in range(args.warmup + args.steps):
        req = synth.make_request(wl, step)
        rate, dt, t = oracle_sample_rate(wl, w, req, oracle_sample_ids(wl, req, budget_s=20.0, max_cand=n_cand))
        if step >= args.warmup:
            rates.append(rate)
            times.append(dt)
            toks += t
    value = toks / sum(times)
    cores = os.cpu_count()
    sample = (f"up to {n_cand} of {wl.n_candidates} candidates per step, evenly spaced in length rank, all "
              f"{wl.model.n_layers} layers, unpruned fp64 numpy forward")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(times)), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))
    return 0


# ----------------------------------------------------------------------------------------------- side workloads
def _tensor_bytes(t, on_device):
    if isinstance(t, dict):
        return sum(_tensor_bytes(v, on_device) for v in t.values())
    if isinstance(t, (list, tuple)):
        return sum(_tensor_bytes(v, on_device) for v in t)
    return t.numel() * t.element_size() if (t.is_cuda == on_device) else 0


def profile_classes(P, model, step_fn, n_steps):
    """Per-kernel-class device time of n_steps requests (CUDA events the library records around every launch)."""
    import ctypes as C
    import torch

    class Stat(C.Structure):
        _fields_ = [("ms", C.c_double), ("work", C.c_double), ("launches", C.c_int64)]
    lib = P.lib()
    lib.prism_profile.argtypes = [C.c_void_p, C.c_int]
    lib.prism_profile_read.argtypes = [C.c_void_p, C.POINTER(Stat), C.c_int]
    stats = (Stat * len(KERNEL_CLASSES))()
    lib.prism_profile(model._h, 1)
    for i in range(n_steps):
        step_fn(i)
    torch.cuda.synchronize()
    lib.prism_profile_read(model._h, stats, 1)
    lib.prism_profile(model._h, 0)
    return {n: {"ms_per_step": stats[j].ms / n_steps, "launches_per_step": stats[j].launches / n_steps,
                "work_per_step": stats[j].work / n_steps} for j, n in enumerate(KERNEL_CLASSES)}


def measure_side_workload(P, index: int, steps: int, warmup: int, dev, local: int):
    """One of the other benchmark workloads, timed like the headline (device-resident inputs between CUDA events on
    the launching stream, then host buffers through prism_select_host, then pruning off), with per-class rates,
    clocks sampled during the timed region and the peak device memory.  No oracle leg."""
    import gc
    import torch
    import synth
    from synth.configs import MODE_NONE, Schedule

    wl = synth.workload(index)
    cfg = wl.model
    n_req = 10
    reqs = [synth.make_request(wl, s) for s in range(n_req)]
    lq = wl.query_len
    lens_all = [np.diff(r["cand_offsets"]) + lq for r in reqs]
    torch.cuda.synchronize()
    torch.cuda.reset_peak_memory_stats(dev)
    base_bytes = torch.cuda.memory_allocated(dev)
    w_np = synth.make_weights(cfg, wl.weight_seed)
    tw = P.upload_weights(w_np, cfg.dtype, device=str(dev), layers_pinned_host=bool(wl.stream_weights))
    del w_np
    gc.collect()
    model = P.PrismModel(cfg, tw, int(max(l.max() for l in lens_all)), wl.n_candidates, int(max(l.sum() for l in lens_all)),
                         activation_budget_bytes=wl.activation_budget_bytes, stream_weights=bool(wl.stream_weights))
    d = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).pin_memory().numpy()
    dreqs = [(d(r["query"]), d(r["cand_tokens"]), d(r["cand_offsets"])) for r in reqs]
    hreqs = [(pin(r["query"]), pin(r["cand_tokens"]), pin(r["cand_offsets"])) for r in reqs]
    hidx = torch.empty(wl.top_k, dtype=torch.int32).pin_memory().numpy()
    hsc = torch.empty(wl.top_k, dtype=torch.float32).pin_memory().numpy()
    stream = torch.cuda.current_stream()
    tr0 = model.select(*dreqs[0], wl.top_k, wl.schedule, want_trace=True)[2]

    def timed(fn, k, w):
        for i in range(w):
            fn(i)
        torch.cuda.synchronize()
        n0 = model.launch_count
        pairs = []
        for i in range(k):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn(w + i)
            b.record(stream)
            pairs.append((a, b))
        torch.cuda.synchronize()
        lat = [a.elapsed_time(b) for a, b in pairs]
        return pairs[0][0].elapsed_time(pairs[-1][1]), lat, model.launch_count - n0

    dev_step = lambda i, s=wl.schedule: model.select(*dreqs[i % n_req], wl.top_k, s, want_trace=False)
    host_step = lambda i: model.select_host(*hreqs[i % n_req], wl.top_k, wl.schedule, idx_out=hidx, sc_out=hsc)
    sampler = ClockSampler(local)
    sampler.start()
    total_ms, lat, launches = timed(dev_step, steps, warmup)
    clocks = sampler.stop()
    toks = sum(int(lens_all[(warmup + i) % n_req].sum()) for i in range(steps))
    e2e_steps = max(5, steps // 2)
    e2e_ms, e2e_lat, _ = timed(host_step, e2e_steps, 2)
    e2e_toks = sum(int(lens_all[(2 + i) % n_req].sum()) for i in range(e2e_steps))
    off_steps = max(3, steps // 6)
    off_ms, _, _ = timed(lambda i: dev_step(i, Schedule(MODE_NONE)), off_steps, 2)
    per = profile_classes(P, model, lambda i: dev_step(warmup + i), max(3, min(steps, 5)))
    peaks = measured_peaks()

    def rate(names, scale):
        ms = sum(per[n]["ms_per_step"] for n in names)
        return (sum(per[n]["work_per_step"] for n in names) / (ms * 1e-3) / scale) if ms > 0 else 0.0
    g_tf, a_tf = rate(GEMM_CLASSES, 1e12), rate(("attention",), 1e12)
    req_fl = sum(per[n]["work_per_step"] for n in GEMM_CLASSES + ("attention",))
    req_tf = req_fl / (total_ms / steps * 1e-3) / 1e12
    out = {"workload": wl.name, "steps": steps, "warmup": warmup, "requests_cycled": n_req,
           "tokens_per_request": int(np.mean([l.sum() for l in lens_all])), "candidates": wl.n_candidates, "top_k": wl.top_k,
           "dtype": "bf16" if cfg.dtype == 1 else "f32",
           "latency_ms": {"p50": float(np.percentile(lat, 50)), "p99": float(np.percentile(lat, 99))},
           "ms_per_step": total_ms / steps, "candidate_tokens_per_s": toks / (total_ms * 1e-3),
           "e2e": {"candidate_tokens_per_s": e2e_toks / (e2e_ms * 1e-3), "p50_ms": float(np.percentile(e2e_lat, 50)),
                   "steps": e2e_steps,
                   "h2d_bytes_per_step": int(np.mean([q.nbytes + c.nbytes + o.nbytes for q, c, o in hreqs])),
                   "d2h_bytes_per_step": int(hidx.nbytes + hsc.nbytes)},
           "pruning_off_ms_per_step": off_ms / off_steps, "pruning_speedup": (off_ms / off_steps) / (total_ms / steps),
           "gemm": {"tflops": g_tf, "frac_of_sustained_peak": g_tf / peaks["bf16_tflops_sustained"],
                    "frac_of_burst_peak": g_tf / peaks["bf16_tflops"], "frac_of_nominal_2250": g_tf / 2250.0},
           "attention": {"tflops": a_tf, "frac_of_sustained_peak": a_tf / peaks["bf16_tflops_sustained"],
                         "frac_of_burst_peak": a_tf / peaks["bf16_tflops"], "frac_of_nominal_2250": a_tf / 2250.0},
           "rmsnorm_gbs": rate(("rmsnorm",), 1e9), "compact_gbs": rate(("compact",), 1e9), "embed_gbs": rate(("embed",), 1e9),
           "route_us_per_launch": (1e3 * per["route"]["ms_per_step"] / per["route"]["launches_per_step"]
                                   if per["route"]["launches_per_step"] else None),
           "request_tflops": req_tf, "request_frac_of_sustained_peak": req_tf / peaks["bf16_tflops_sustained"],
           "gpu_launches": int(launches), "clocks": clocks,
           "handle_options": {"stream_weights": bool(wl.stream_weights), "activation_budget_bytes": wl.activation_budget_bytes,
                              "chunks_per_layer_max": tr0.n_chunks_max, "shared_query_prefix_rows": tr0.shared_prefix_rows},
           "device_bytes": {"handle": tr0.workspace_bytes, "weights_device": _tensor_bytes(tw, True),
                            "weights_pinned_host": _tensor_bytes(tw, False),
                            "torch_peak_allocated_above_start": int(torch.cuda.max_memory_allocated(dev) - base_bytes)}}
    model.close()
    return out


# ----------------------------------------------------------------------------------------------- CUDA arm
def run_prism(args):
    import torch
    import synth
    from synth.configs import MODE_NONE, Schedule
    import paper_2510_15620_b200 as P

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the PRISM path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    wl = synth.workload(args.workload)
    # memory options of the handle (Sec. 4.2 - 4.4) on top of what the workload prescribes
    from dataclasses import replace as _replace
    if args.stream_weights:
        wl = _replace(wl, stream_weights=1)
    if args.activation_budget_mb:
        wl = _replace(wl, activation_budget_bytes=int(args.activation_budget_mb) << 20)
    cfg = wl.model
    n_req = max(args.requests, 1)
    by_cand = args.shard == "candidates"
    seeds = list(range(n_req)) if by_cand else shard_requests(rank, world, n_req)
    reqs = [synth.make_request(wl, s) for s in seeds]
    lq = wl.query_len
    lens_all = [np.diff(r["cand_offsets"]) + lq for r in reqs]
    max_seq = int(max(l.max() for l in lens_all))
    max_tot = int(max(l.sum() for l in lens_all))
    # candidate sharding: every rank computes the same partition; this rank runs the candidates it owns
    owned = [(P.shard_candidates(l, world) == rank).astype(np.uint8) for l in lens_all] if by_cand else None
    if by_cand:
        max_tot = int(max(l[o != 0].sum() for l, o in zip(lens_all, owned))) or 1
    reduce = (lambda t: P.all_reduce_scores(t)) if (by_cand and world > 1) else (lambda t: None)
    w_np = synth.make_weights(cfg, wl.weight_seed)
    w4 = args.weight_format == "w4"
    if w4:  # Sec. 6.1's quantised arm: 4-bit codes + bf16 scale and 4-bit zero point per 128 input channels
        w_np = synth.quantize_weights(w_np, 128)
    tw = P.upload_weights(w_np, cfg.dtype, device=str(dev), layers_pinned_host=bool(wl.stream_weights),
                          embed_pinned_host=args.embed_cache_rows > 0)
    model = P.PrismModel(cfg, tw, max_seq, wl.n_candidates, max_tot, activation_budget_bytes=wl.activation_budget_bytes,
                         stream_weights=bool(wl.stream_weights), shared_prefix=args.shared_prefix == "on",
                         weight_format=P.PRISM_WFMT_W4 if w4 else P.PRISM_WFMT_PLAIN, quant_group=128 if w4 else 0,
                         embed_cache_rows=args.embed_cache_rows, hidden_offload=args.hidden_offload)
    d = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    dreqs = [(d(r["query"]), d(r["cand_tokens"]), d(r["cand_offsets"])) for r in reqs]
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).pin_memory().numpy()
    hreqs = [(pin(r["query"]), pin(r["cand_tokens"]), pin(r["cand_offsets"])) for r in reqs]
    hidx = torch.empty(wl.top_k, dtype=torch.int32).pin_memory().numpy()
    hsc = torch.empty(wl.top_k, dtype=torch.float32).pin_memory().numpy()
    sched = wl.schedule
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, warmup):
        """W untimed steps, then exactly K steps between events on the launching stream."""
        for i in range(warmup):
            fn(i)
        barrier()
        lat = []
        n0 = model.launch_count
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(stream)
        for i in range(steps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn(warmup + i)
            b.record(stream)
            lat.append((a, b))
        ev1.record(stream)
        barrier()
        total_ms = ev0.elapsed_time(ev1)
        return total_ms, [a.elapsed_time(b) for a, b in lat], model.launch_count - n0

    def dev_step(i, s=sched):
        q, c, o = dreqs[i % n_req]
        if by_cand:
            model.select_sharded(q, c, o, wl.top_k, s, owned[i % n_req], reduce, want_trace=False)
        else:
            model.select(q, c, o, wl.top_k, s, want_trace=False)

    prefix_rows, workspace_bytes = 0, None  # what the library reports for this workload (one untimed traced request)
    if not by_cand:
        tr0 = model.select(*dreqs[0], wl.top_k, sched, want_trace=True)[2]
        prefix_rows, workspace_bytes = tr0.shared_prefix_rows, tr0.workspace_bytes

    def tensor_bytes(t, on_device):
        if isinstance(t, dict):
            return sum(tensor_bytes(v, on_device) for v in t.values())
        if isinstance(t, (list, tuple)):
            return sum(tensor_bytes(v, on_device) for v in t)
        return t.numel() * t.element_size() if (t.is_cuda == on_device) else 0

    def host_step(i):
        q, c, o = hreqs[i % n_req]
        if by_cand:  # the sharded entry point takes device buffers: the copies are made here, inside the timed region
            tq, tc, to = (torch.from_numpy(a).to(dev, non_blocking=True) for a in (q, c, o))
            idx, sc, _ = model.select_sharded(tq, tc, to, wl.top_k, sched, owned[i % n_req], reduce, want_trace=False)
            hidx[: idx.numel()] = idx.cpu().numpy()
            hsc[: sc.numel()] = sc.cpu().numpy()
        else:
            model.select_host(q, c, o, wl.top_k, sched, idx_out=hidx, sc_out=hsc)

    tokens_of = lambda i: int(lens_all[i % n_req].sum())
    K, W = args.steps, args.warmup

    sampler = ClockSampler(local)
    sampler.start()
    total_ms, lat, launches = timed(dev_step, K, W)
    clocks = sampler.stop()
    total_ms = max_over_ranks(total_ms, world, dev)
    toks = sum(tokens_of(W + i) for i in range(K))
    toks_all = float(toks) if by_cand else sum_over_ranks(float(toks), world, dev)  # shared requests count once
    value = toks_all / (total_ms * 1e-3)

    e2e_ms, e2e_lat, _ = timed(host_step, K, W)
    e2e_ms = max_over_ranks(e2e_ms, world, dev)
    h2d = int(np.mean([q.nbytes + c.nbytes + o.nbytes for q, c, o in hreqs]))
    d2h = int(hidx.nbytes + hsc.nbytes)

    # document tokens only (the query is shared by all candidates of a request), beside the headline count
    doc_toks = sum(int(lens_all[(W + i) % n_req].sum()) - lq * len(lens_all[(W + i) % n_req]) for i in range(K))
    doc_toks_all = float(doc_toks) if by_cand else sum_over_ranks(float(doc_toks), world, dev)

    # streamed workloads: what crosses the host link per request, and the time that alone would take
    host_link = None
    if wl.stream_weights and rank == 0 and not by_cand:
        probe_host = torch.empty(1 << 30, dtype=torch.uint8).pin_memory()
        probe_dev = torch.empty(1 << 30, dtype=torch.uint8, device=dev)
        for _ in range(2):
            probe_dev.copy_(probe_host, non_blocking=True)
        ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ea.record()
        for _ in range(3):
            probe_dev.copy_(probe_host, non_blocking=True)
        eb.record()
        torch.cuda.synchronize()
        h2d_gbs = 3 * (1 << 30) / (ea.elapsed_time(eb) * 1e-3) / 1e9
        layer_bytes = tensor_bytes(tw["layers"], False) / cfg.n_layers
        runs = [model.select(*dreqs[i], wl.top_k, sched, want_trace=True)[2].layers_run for i in range(n_req)]
        per_req = float(np.mean(runs)) * layer_bytes
        host_link = {"pinned_h2d_gbs": h2d_gbs, "layer_bytes": int(layer_bytes), "layers_streamed_per_request": float(np.mean(runs)),
                     "bytes_per_request": int(per_req), "floor_ms": per_req / (h2d_gbs * 1e9) * 1e3,
                     "note": "streaming stops when the forward terminates; the floor is bytes / measured pinned copy rate"}
        del probe_host, probe_dev

    # the same kernels with pruning disabled -> what pruning buys on this workload
    off_ms, _, _ = timed(lambda i: dev_step(i, Schedule(MODE_NONE)), max(3, K // 4), 3)
    off_ms = max_over_ranks(off_ms / max(3, K // 4), world, dev)

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "strong" if by_cand else "weak", "vs_baseline": None,
            "dtype": "bf16" if cfg.dtype == 1 else "f32", "data": "synthetic",
            "config": {"workload": wl.name, "requests_cycled": n_req, "candidates": wl.n_candidates, "top_k": wl.top_k,
                       "tokens_per_request": int(np.mean([l.sum() for l in lens_all])),
                       # causal attention: the query's rows are computed once per request instead of once per
                       # candidate (same scores bit for bit); the metric keeps counting query + document per candidate
                       "weight_format": "w4a16 (round-to-nearest, group 128)" if w4 else "bf16" if cfg.dtype == 1 else "f32",
                       # what the request holds: the caller's weight tensors on the device and in pinned host memory
                       # (streamed layers), and everything the handle allocated on the device (activations, slots, scratch)
                       "handle_options": {"stream_weights": bool(wl.stream_weights), "activation_budget_bytes": wl.activation_budget_bytes,
                                          "embed_cache_rows": args.embed_cache_rows, "hidden_offload": bool(args.hidden_offload)},
                       "memory_bytes": {"weights_device": tensor_bytes(tw, True), "weights_pinned_host": tensor_bytes(tw, False),
                                        "handle_device": workspace_bytes},
                       "shared_query_prefix_rows": prefix_rows,
                       "rows_computed_first_layer": int(np.mean([l.sum() - (len(l) - 1) * prefix_rows for l in lens_all])),
                       "schedule": {"mode": sched.mode, "probe_layers": list(sched.probe_layers),
                                    "cv_threshold": sched.cv_threshold, "n_clusters": sched.n_clusters},
                       "l2": "no flush: each step streams 0.9 GB of weights and >1 GB of activations, far beyond the 126 MB L2",
                       "parallelism": (f"{world} ranks share each request's candidates, one score all-reduce per probe"
                                       if by_cand else f"dp{world} over requests")},
            "latency_ms": {"p50": float(np.percentile(lat, 50)), "p99": float(np.percentile(lat, 99))},
            "doc_tokens_per_s": doc_toks_all / (total_ms * 1e-3), "host_link": host_link,
            "pruning_off_ms_per_step": off_ms, "pruning_speedup": off_ms / (total_ms / K),
            "e2e": {"value": toks_all / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "p50_ms": float(np.percentile(e2e_lat, 50))},
            "gpu_launches": int(launches), "clocks": clocks}

    psteps = max(3, min(K, 10))
    if by_cand and world > 1 and rank != 0:
        for i in range(psteps):      # rank 0's profiled steps below contain all-reduces: take part in them
            dev_step(W + i)
        torch.cuda.synchronize()
    if rank == 0:
        # per-kernel device time, measured live with CUDA events around every launch of profiled steps
        lib = P.lib()
        import ctypes as C

        class Stat(C.Structure):
            _fields_ = [("ms", C.c_double), ("work", C.c_double), ("launches", C.c_int64)]
        lib.prism_profile.argtypes = [C.c_void_p, C.c_int]
        lib.prism_profile_read.argtypes = [C.c_void_p, C.POINTER(Stat), C.c_int]
        stats = (Stat * len(KERNEL_CLASSES))()
        lib.prism_profile(model._h, 1)
        for i in range(psteps):
            dev_step(W + i)
        torch.cuda.synchronize()
        lib.prism_profile_read(model._h, stats, 1)
        lib.prism_profile(model._h, 0)
        per = {n: {"ms_per_step": stats[j].ms / psteps, "launches_per_step": stats[j].launches / psteps,
                   "work_per_step": stats[j].work / psteps} for j, n in enumerate(KERNEL_CLASSES)}
        g_ms = sum(per[n]["ms_per_step"] for n in GEMM_CLASSES)
        g_fl = sum(per[n]["work_per_step"] for n in GEMM_CLASSES)
        g_n = sum(per[n]["launches_per_step"] for n in GEMM_CLASSES)
        peaks = measured_peaks()
        peak = peaks["bf16_tflops_sustained"]
        ach = g_fl / (g_ms * 1e-3) / 1e12 if g_ms > 0 else 0.0
        tot_ms = sum(v["ms_per_step"] for v in per.values())
        traffic = None
        if args.workload in (1, 4) and g_n:      # the captures are for the 0.6B weight shapes
            tb = 0.0
            for n in GEMM_CLASSES:
                nn, kk = CFG1_NK[n]
                rows_total = per[n]["work_per_step"] / (2.0 * nn * kk)          # sum of M over the class's launches
                tb += NCU_TRAFFIC_M8192[n] * rows_total / 8192.0
            traffic = tb / g_n
        gemm_names = "qkv, o, ffn1 + GELU, ffn2; all with bias" if getattr(cfg, "arch", 0) == 1 else "qkv, o, gate/up, down"
        line["roofline"] = {"kernel": f"k_gemm_tc2 (tcgen05 cta_group::2 projection GEMMs: {gemm_names})", "bound": "tensor",
                            "achieved": ach, "peak": peak, "unit": "TFLOP/s", "frac": ach / peak if peak else None,
                            "peak_source": f"bf16_tflops_sustained of {peaks['source']} (kernel timed inside a long step)",
                            "frac_of_burst_peak": ach / peaks["bf16_tflops"],
                            "frac_of_nominal_2250": ach / 2250.0,
                            "flops_per_launch": g_fl / g_n if g_n else 0, "avg_launch_ms": g_ms / g_n if g_n else 0,
                            "traffic": traffic,
                            "traffic_note": "bytes per launch: ncu dram read+write of each GEMM shape at M = 8192 "
                                            "(profiles/gemm_tc2_*.md) scaled by the rows each launch processed",
                            "share_of_kernel_time": g_ms / tot_ms if tot_ms else None}
        # the whole request against the tensor roofline: algorithmic flops of the live tokens (GEMMs and attention of
        # the profiled steps, pruning included) over the request time, against the measured and the nominal peak
        req_fl = g_fl + per["attention"]["work_per_step"]
        req_tf = req_fl / (total_ms / K * 1e-3) / 1e12
        line["request_roofline"] = {"flops_per_request": req_fl, "achieved_tflops": req_tf,
                                    "frac_of_sustained_peak": req_tf / peak if peak else None,
                                    "frac_of_burst_peak": req_tf / peaks["bf16_tflops"], "frac_of_nominal_2250": req_tf / 2250.0,
                                    "note": "sum over layers of live tokens x 2 x layer parameters, plus attention flops, "
                                            "divided by the request time (kernels of every kind, host round trips included)"}
        line["kernels"] = {n: {"ms_per_step": round(v["ms_per_step"], 4), "share": round(v["ms_per_step"] / tot_ms, 4),
                               "launches_per_step": v["launches_per_step"],
                               ("tflops" if n in GEMM_CLASSES or n == "attention" else "gbs"):
                                   (v["work_per_step"] / (v["ms_per_step"] * 1e-3) / (1e12 if n in GEMM_CLASSES or n == "attention" else 1e9)
                                    if v["ms_per_step"] > 0 else 0.0)}
                           for n, v in per.items()}
        if not args.no_cpu_baseline and not w4 and world == 1:   # the oracle leg (N = 1 only) times the unquantised model
            ids = oracle_sample_ids(wl, reqs[0], max_cand=20)
            n_c = len(ids)
            rate, dt, t = oracle_sample_rate(wl, w_np, reqs[0], ids)
            line["cpu_baseline"] = {"value": rate, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
                                    "sample": f"{n_c} of {wl.n_candidates} candidates of request 0, evenly spaced in length rank "
                                              f"(lengths {int(lens_all[0][ids].min())}..{int(lens_all[0][ids].max())} of "
                                              f"{int(lens_all[0].min())}..{int(lens_all[0].max())}, {t} tokens), all "
                                              f"{cfg.n_layers} layers, unpruned fp64 numpy forward, {dt:.1f} s"}
        plain = not (args.stream_weights or args.activation_budget_mb or args.embed_cache_rows or args.hidden_offload or w4)
        if args.side_workloads == "on" and world == 1 and args.workload == 1 and plain and not by_cand:
            # the other benchmark workloads (tiny fp32, 4B-, 8B-shaped, 1000-candidate stress) in the same run; the
            # headline above stays the 0.6B-shaped workload.  Its handle is closed first: one handle at a time.
            import gc
            model.close()
            line["workloads"] = {}
            for index, k in ((0, 100), (2, 20), (3, 20), (4, 100)):
                gc.collect()
                torch.cuda.empty_cache()            # the previous workload's weights go back to the driver
                line["workloads"][f"cfg{index}"] = measure_side_workload(P, index, k, 5, dev, local)
        print(json.dumps(line))
    model.close()
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="prism", choices=["prism", "reference"])
    ap.add_argument("--workload", type=int, default=1)
    ap.add_argument("--requests", type=int, default=10, help="distinct request seeds cycled through")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--shared-prefix", default="on", choices=["on", "off"],
                    help="on: the query's rows are stored and computed once per request where the path supports it "
                         "(causal attention; results are bit-identical); off: one query copy per candidate")
    ap.add_argument("--stream-weights", action="store_true", help="layer weights in pinned host memory, two device slots (Sec. 4.2)")
    ap.add_argument("--activation-budget-mb", type=int, default=0, help="chunked execution under this budget (Sec. 4.3)")
    ap.add_argument("--embed-cache-rows", type=int, default=0, help="embedding table in pinned host memory, LRU row cache (Sec. 4.4)")
    ap.add_argument("--hidden-offload", action="store_true", help="hidden states in pinned host memory, three device chunks (Sec. 4.3)")
    ap.add_argument("--weight-format", default="plain", choices=["plain", "w4"],
                    help="w4: the layer matrices are stored (and, for the streamed workload, copied) as 4-bit codes and "
                         "rebuilt as bf16 layer by layer on the device")
    ap.add_argument("--side-workloads", default="on", choices=["on", "off"],
                    help="on (1 GPU, workload 1, no memory options): the line also carries a `workloads` block with the "
                         "tiny fp32, 4B-shaped, 8B-shaped (streamed, chunked) and 1000-candidate workloads")
    ap.add_argument("--shard", default="requests", choices=["requests", "candidates"],
                    help="requests: every rank serves its own requests (weak scaling, the default); candidates: all "
                         "ranks share each request, one score all-reduce per probe (strong scaling)")
    args = ap.parse_args()
    if args.impl == "reference":
        args.steps = 5 if args.steps is None else args.steps
        args.warmup = 3 if args.warmup is None else args.warmup
        return run_reference(args)
    args.steps = 100 if args.steps is None else args.steps
    args.warmup = 5 if args.warmup is None else max(3, args.warmup)
    return run_prism(args)


if __name__ == "__main__":
    sys.exit(main())
