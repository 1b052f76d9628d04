"""Dispersion-threshold sweep (the synthetic analogue of the paper's threshold study, Sec. 6.2 "impact of
the dispersion threshold"): for each threshold, mean request latency and mean precision@K of the pruned
top-K against the unpruned one, on synthetic requests of one workload.  One JSON line per threshold.

    python -m paper_2510_15620_b200.sweep --workload 1 --requests 8 --thresholds 0.1,0.5,2,8,32,128
"""
from __future__ import annotations

import argparse
import json
import os
import sys
from dataclasses import replace

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import synth  # noqa: E402
from synth.configs import MODE_NONE, Schedule  # noqa: E402

from .binding import PrismModel, upload_weights  # noqa: E402


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", type=int, default=1)
    ap.add_argument("--requests", type=int, default=8)
    ap.add_argument("--thresholds", default="0.1,0.5,2,8,32,128")
    a = ap.parse_args()
    wl = synth.workload(a.workload)
    cfg = wl.model
    reqs = [synth.make_request(wl, r) for r in range(a.requests)]
    lens = [np.diff(r["cand_offsets"]) + wl.query_len for r in reqs]
    tw = upload_weights(synth.make_weights(cfg, wl.weight_seed), cfg.dtype, layers_pinned_host=bool(wl.stream_weights))
    model = PrismModel(cfg, tw, int(max(l.max() for l in lens)), wl.n_candidates, int(max(l.sum() for l in lens)),
                       activation_budget_bytes=wl.activation_budget_bytes, stream_weights=bool(wl.stream_weights))
    d = lambda x: torch.from_numpy(np.ascontiguousarray(x, dtype=np.int32)).cuda()
    dreqs = [(d(r["query"]), d(r["cand_tokens"]), d(r["cand_offsets"])) for r in reqs]

    def timed(sched):
        out, ms = [], []
        for q, c, o in dreqs:
            model.select(q, c, o, wl.top_k, sched, want_trace=False)          # warm
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            idx, _, tr = model.select(q, c, o, wl.top_k, sched, want_trace=True)
            e1.record()
            torch.cuda.synchronize()
            ms.append(e0.elapsed_time(e1))
            out.append((set(idx.cpu().numpy().tolist()), tr.layers_run))
        return out, float(np.mean(ms))

    truth, ms_off = timed(Schedule(MODE_NONE))
    print(json.dumps({"workload": wl.name, "threshold": None, "ms": ms_off, "precision_at_k": 1.0, "layers_run": cfg.n_layers}))
    for thr in [float(t) for t in a.thresholds.split(",")]:
        got, ms = timed(replace(wl.schedule, cv_threshold=thr))
        prec = float(np.mean([len(g & t) / max(1, len(t)) for (g, _), (t, _) in zip(got, truth)]))
        print(json.dumps({"workload": wl.name, "threshold": thr, "ms": ms, "precision_at_k": prec,
                          "layers_run": float(np.mean([l for _, l in got])), "speedup": ms_off / ms}))
    model.close()


if __name__ == "__main__":
    main()
