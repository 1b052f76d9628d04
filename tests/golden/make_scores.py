"""Writes tests/golden/<workload>_scores_r<r>.txt: the oracle's probe/final scores S[layer][i] of every
candidate of one synthetic request.  Calls only oracle/ and the seeded input generators.

    python tests/golden/make_scores.py 1 0          # workload index, request index
    python tests/golden/make_scores.py 4 0 --candidates 0:64   # a slice of the candidates

The file is plain text: a header with the recipe, then one line per scored layer."""
import argparse
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
import synth  # noqa: E402
from synth import weights as W  # noqa: E402


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("workload", type=int)
    ap.add_argument("request", type=int)
    ap.add_argument("--candidates", default=None, help="a:b slice of candidate indices")
    ap.add_argument("--out", default=None)
    ap.add_argument("--act", default="exact", choices=["exact", "bf16"],
                    help="bf16: round every stored activation to bfloat16 (the bf16 precision contract)")
    a = ap.parse_args()
    wl = synth.workload(a.workload)
    cfg = wl.model
    r = synth.make_request(wl, a.request)
    n = len(r["cand_offsets"]) - 1
    ids = list(range(n))
    if a.candidates:
        lo, hi = (int(x) for x in a.candidates.split(":"))
        ids = ids[lo:hi]
    layers = sorted(set(list(wl.schedule.probe_layers) + [cfg.n_layers]))
    weights = dict(W.make_globals(cfg, wl.weight_seed))
    weights["layers"] = W.iter_layers(cfg, wl.weight_seed)        # lazily, one layer at a time
    t0 = time.time()
    S = oracle.score_matrix(r["query"], r["cand_tokens"], r["cand_offsets"], weights, cfg, layers, candidates=ids, act=a.act)
    dt = time.time() - t0
    out = a.out or os.path.join(os.path.dirname(os.path.abspath(__file__)),
                                f"{wl.name}_scores_r{a.request}.txt")
    with open(out, "w") as f:
        f.write(f"# oracle scores (fp64 forward, bf16-rounded weights where the workload is bf16), activations: {a.act}\n")
        f.write(f"# workload {wl.name} request {a.request} weight_seed {wl.weight_seed} candidates {ids[0]}..{ids[-1]}\n")
        f.write(f"# written by tests/golden/make_scores.py in {dt:.0f} s; one line per layer: layer then scores\n")
        for l in layers:
            f.write(str(l) + " " + " ".join(repr(float(v)) for v in S[l]) + "\n")
    print(out, f"{dt:.1f}s")


if __name__ == "__main__":
    main()
