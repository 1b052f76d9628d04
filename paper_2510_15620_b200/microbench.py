"""Per-kernel microbenchmark through the C ABI (prism_op_*): CUDA-event timing of one kernel on
synthetic operands, one JSON line per run.  Also the small-case driver for profiler captures.

    python -m paper_2510_15620_b200.microbench --op gemm --m 35200 --n 4096 --k 1024 --epilogue 0
    python -m paper_2510_15620_b200.microbench --op attention --seqs 100 --len-lo 160 --len-hi 544
    python -m paper_2510_15620_b200.microbench --op rmsnorm|rope|compact --rows 35200 --d 1024
    python -m paper_2510_15620_b200.microbench --op gemm_bias --m 35200 --n 4096 --k 1024 --epilogue 2   (encoder stack)
    python -m paper_2510_15620_b200.microbench --op layernorm --rows 35200 --d 1024
    python -m paper_2510_15620_b200.microbench --op dequant --n 12288 --k 4096          (W4 -> bf16, group 128)
    python -m paper_2510_15620_b200.microbench --op probe|route --seqs 1000                (score probe; prune decision)
    python -m paper_2510_15620_b200.microbench --op attention --head-dim 64 --hq 16 --hkv 16 --causal 0
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import ops
from .binding import PRISM_BF16, PRISM_IMPL_AUTO


def _time(fn, iters, warmup, flush):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    ms = []
    for _ in range(iters):
        if flush is not None:
            flush.zero_()                      # > L2 bytes written between timed launches
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        torch.cuda.synchronize()
        ms.append(a.elapsed_time(b))
    return float(np.median(ms)), float(np.min(ms))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--op", required=True, choices=["gemm", "qkv_rope", "attention", "rmsnorm", "rope", "compact", "gemm_bias", "layernorm", "dequant", "probe", "route"])
    ap.add_argument("--head-dim", type=int, default=128)
    ap.add_argument("--m", type=int, default=35200)
    ap.add_argument("--n", type=int, default=4096)
    ap.add_argument("--k", type=int, default=1024)
    ap.add_argument("--epilogue", type=int, default=0)
    ap.add_argument("--impl", type=int, default=PRISM_IMPL_AUTO)
    ap.add_argument("--rows", type=int, default=35200)
    ap.add_argument("--d", type=int, default=1024)
    ap.add_argument("--seqs", type=int, default=100)
    ap.add_argument("--len-lo", type=int, default=160)
    ap.add_argument("--len-hi", type=int, default=544)
    ap.add_argument("--hq", type=int, default=16)
    ap.add_argument("--hkv", type=int, default=8)
    ap.add_argument("--causal", type=int, default=1)
    ap.add_argument("--qk-norm", type=int, default=1)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--no-flush", action="store_true")
    a = ap.parse_args()
    dev = "cuda"
    g = torch.Generator(device=dev).manual_seed(0)
    flush = None if a.no_flush else torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    rnd = lambda *s: torch.randn(*s, device=dev, generator=g)
    out = {"op": a.op}
    if a.op == "gemm":
        m, n, k = a.m, a.n, a.k
        A = rnd(m, k).to(torch.bfloat16)
        B = (rnd(n, k) * 0.05).to(torch.bfloat16)
        B2 = (rnd(n, k) * 0.05).to(torch.bfloat16)
        O = torch.empty(m, n, dtype=torch.bfloat16, device=dev)
        R = rnd(m, n)
        err = torch.zeros(1, dtype=torch.int32, device=dev)
        fn = lambda: ops.prism_op_gemm(A, B, B2, O, R, m, n, k, PRISM_BF16, a.epilogue, a.impl, err)
        med, best = _time(fn, a.iters, a.warmup, flush)
        fl = 2.0 * m * n * k * (2 if a.epilogue == 2 else 1)
        out.update(m=m, n=n, k=k, epilogue=a.epilogue, ms=med, ms_min=best, tflops=fl / med / 1e9, err=int(err.item()))
    elif a.op == "gemm_bias":
        m, n, k = a.m, a.n, a.k
        A = rnd(m, k).to(torch.bfloat16)
        B = (rnd(n, k) * 0.05).to(torch.bfloat16)
        bias = rnd(n)
        O = torch.empty(m, n, dtype=torch.bfloat16, device=dev)
        R = rnd(m, n)
        err = torch.zeros(1, dtype=torch.int32, device=dev)
        fn = lambda: ops.prism_op_gemm_bias(A, B, bias, O, R, m, n, k, PRISM_BF16, a.epilogue, a.impl, err)
        med, best = _time(fn, a.iters, a.warmup, flush)
        out.update(m=m, n=n, k=k, epilogue=a.epilogue, ms=med, ms_min=best, tflops=2.0 * m * n * k / med / 1e9, err=int(err.item()))
    elif a.op == "probe":
        rng = np.random.default_rng(0)
        lens = rng.integers(a.len_lo, a.len_hi + 1, size=a.seqs)
        cu = np.zeros(a.seqs + 1, np.int32)
        cu[1:] = np.cumsum(lens)
        x = rnd(int(cu[-1]), a.d)
        gain = torch.ones(a.d, dtype=torch.bfloat16, device=dev)
        head = (rnd(2, a.d) * 0.02).to(torch.bfloat16)
        sc = torch.empty(a.seqs, device=dev)
        cud = torch.from_numpy(cu).to(dev)
        fn = lambda: ops.prism_op_probe(x, cud, a.seqs, gain, head, PRISM_BF16, 1e-6, sc)
        med, best = _time(fn, a.iters, a.warmup, flush)
        out.update(seqs=a.seqs, d=a.d, ms=med, ms_min=best, gbs=a.seqs * a.d * 4.0 / med / 1e6,
                   note="the op wrapper also builds the head-difference vector, allocates and synchronises; the kernel alone is in the profile")
    elif a.op == "route":
        n = a.seqs
        rng = np.random.default_rng(0)
        lens = rng.integers(a.len_lo, a.len_hi + 1, size=n)
        cu = np.zeros(n + 1, np.int32)
        cu[1:] = np.cumsum(lens)
        t = lambda v: torch.from_numpy(v).to(dev)
        scores = t(rng.normal(size=n).astype(np.float32))
        cud, ids = t(cu), t(np.arange(n, dtype=np.int32))
        state0 = t(np.array([n, cu[-1], 10, 0, 0, 0, 0, 0], np.int32))
        state = state0.clone()
        cu_new, s2o, oon = (torch.empty(n + 1, dtype=torch.int32, device=dev) for _ in range(3))
        ridx, rsc = torch.empty(n + 1, dtype=torch.int32, device=dev), torch.empty(n + 1, device=dev)
        rec = torch.zeros(ops.RECORD_BYTES, dtype=torch.uint8, device=dev)

        def fn():
            state.copy_(state0)
            ops.prism_op_route(scores, cud, ids, n, 2, 0, 0.5, 3, 0, 1, 0, 8, cu_new, s2o, oon, state, ridx, rsc, rec)
        med, best = _time(fn, a.iters, a.warmup, flush)
        out.update(candidates=n, ms=med, ms_min=best,
                   note="includes the op wrapper's scratch allocation; the kernel alone is in the profile")
    elif a.op == "dequant":
        n, k, grp = a.n, a.k, 128
        ng = k // grp
        up16 = lambda v: (v + 15) // 16 * 16
        total = up16(up16(up16(n * k // 2) + 2 * n * ng) + n * ng)
        blob = torch.randint(0, 256, (total,), dtype=torch.uint8, device=dev, generator=g)
        off_s = up16(n * k // 2)
        blob[off_s: off_s + 2 * n * ng] = torch.tensor([0x00, 0x3C], dtype=torch.uint8, device=dev).repeat(n * ng)  # scales 2^-7
        o = torch.empty(n, k, dtype=torch.bfloat16, device=dev)
        fn = lambda: ops.prism_op_dequant_w4(blob, n, k, grp, o)
        med, best = _time(fn, a.iters, a.warmup, flush)
        out.update(n=n, k=k, group=grp, ms=med, ms_min=best, gbs=n * k * (2.5 + 3.0 / grp) / med / 1e6,
                   bytes_per_weight="0.5 code + 2 written + 3 / group for scale and zero point")
    elif a.op == "layernorm":
        x = rnd(a.rows, a.d)
        gain, shift = torch.ones(a.d, device=dev), torch.zeros(a.d, device=dev)
        o = torch.empty(a.rows, a.d, dtype=torch.bfloat16, device=dev)
        fn = lambda: ops.prism_op_layernorm(x, gain, shift, PRISM_BF16, 1e-5, o)
        med, best = _time(fn, a.iters, a.warmup, flush)
        out.update(rows=a.rows, d=a.d, ms=med, ms_min=best, gbs=a.rows * a.d * 10.0 / med / 1e6,
                   bytes_per_element="4 read + 4 written in place + 2 for the bf16 copy")
    elif a.op == "qkv_rope":
        m, k = a.m, a.k
        n = (a.hq + 2 * a.hkv) * 128
        A = rnd(m, k).to(torch.bfloat16)
        B = (rnd(n, k) * 0.05).to(torch.bfloat16)
        O = torch.empty(m, n, dtype=torch.bfloat16, device=dev)
        gq = torch.ones(128, dtype=torch.bfloat16, device=dev)
        pos = (torch.arange(m, dtype=torch.int32, device=dev) % 512).contiguous()
        err = torch.zeros(1, dtype=torch.int32, device=dev)
        fn = lambda: ops.prism_op_gemm_qkv_rope(A, B, O, m, k, a.hq, a.hkv, a.qk_norm, gq, gq, 1e-6, pos, 1e6, 512, err)
        med, best = _time(fn, a.iters, a.warmup, flush)
        out.update(m=m, n=n, k=k, qk_norm=a.qk_norm, ms=med, ms_min=best, tflops=2.0 * m * n * k / med / 1e9, err=int(err.item()))
    elif a.op == "attention":
        rng = np.random.default_rng(0)
        lens = rng.integers(a.len_lo, a.len_hi + 1, size=a.seqs)
        cu = np.zeros(a.seqs + 1, np.int32)
        cu[1:] = np.cumsum(lens)
        dh = a.head_dim
        qkv = rnd(int(cu[-1]), (a.hq + 2 * a.hkv) * dh).to(torch.bfloat16)
        o = torch.empty(int(cu[-1]), a.hq * dh, dtype=torch.bfloat16, device=dev)
        cud = torch.from_numpy(cu).to(dev)
        err = torch.zeros(1, dtype=torch.int32, device=dev)
        fn = lambda: ops.prism_op_attention(qkv, o, cud, a.seqs, int(lens.max()), a.hq, a.hkv, dh, a.causal, PRISM_BF16, a.impl, err)
        med, best = _time(fn, a.iters, a.warmup, flush)
        fl = float(np.sum((2.0 if a.causal else 4.0) * lens.astype(np.float64) ** 2 * a.hq * dh))
        # what the 128 x 128 (query block x key block) tiling executes: every block a sequence touches, whole
        nb = (lens + 127) // 128
        blocks = nb * (nb + 1) // 2 if a.causal else nb * nb
        fl_exec = float(np.sum(blocks)) * 4.0 * 128 * 128 * dh * a.hq
        out.update(seqs=a.seqs, tokens=int(cu[-1]), causal=a.causal, head_dim=dh, ms=med, ms_min=best, tflops=fl / med / 1e9,
                   executed_tile_tflops=fl_exec / med / 1e9, useful_fraction_of_executed_tiles=fl / fl_exec)
    elif a.op == "rmsnorm":
        x = rnd(a.rows, a.d)
        gain = torch.ones(a.d, dtype=torch.bfloat16, device=dev)
        o = torch.empty(a.rows, a.d, dtype=torch.bfloat16, device=dev)
        fn = lambda: ops.prism_op_rmsnorm(x, gain, PRISM_BF16, 1e-6, o)
        med, best = _time(fn, a.iters, a.warmup, flush)
        out.update(rows=a.rows, d=a.d, ms=med, ms_min=best, gbs=a.rows * a.d * 6.0 / med / 1e6)
    elif a.op == "rope":
        dh = 128
        qkv = rnd(a.rows, (a.hq + 2 * a.hkv) * dh).to(torch.bfloat16)
        pos = torch.randint(0, 512, (a.rows,), dtype=torch.int32, device=dev)
        gq = torch.ones(dh, dtype=torch.bfloat16, device=dev)
        fn = lambda: ops.prism_op_qknorm_rope(qkv, PRISM_BF16, pos, a.hq, a.hkv, dh, 1, gq, gq, 1e-6, 1e6, 512)
        med, best = _time(fn, a.iters, a.warmup, flush)
        out.update(rows=a.rows, ms=med, ms_min=best, gbs=a.rows * (a.hq + a.hkv) * dh * 4.0 / med / 1e6,
                   note="includes the op wrapper's table build and sync")
    else:
        n = a.seqs
        rng = np.random.default_rng(0)
        lens = rng.integers(a.len_lo, a.len_hi + 1, size=n)
        cu = np.zeros(n + 1, np.int32)
        cu[1:] = np.cumsum(lens)
        keep = np.sort(rng.choice(n, size=max(1, n // 3), replace=False)).astype(np.int32)
        cun = np.zeros(len(keep) + 1, np.int32)
        cun[1:] = np.cumsum(lens[keep])
        x = rnd(int(cu[-1]), a.d)
        y = torch.empty(int(cun[-1]), a.d, device=dev)
        t = lambda v: torch.from_numpy(v).to(dev)
        cu_d, cun_d, keep_d = t(cu), t(cun), t(keep)
        fn = lambda: ops.prism_op_compact(x, y, cu_d, cun_d, keep_d, len(keep), int(cun[-1]))
        med, best = _time(fn, a.iters, a.warmup, flush)
        out.update(rows_out=int(cun[-1]), d=a.d, ms=med, ms_min=best, gbs=int(cun[-1]) * a.d * 8.0 / med / 1e6)
    print(json.dumps(out))


if __name__ == "__main__":
    main()
