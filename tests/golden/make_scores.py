"""Writes tests/golden/<workload>_scores_r<r>.txt: the oracle's probe/final scores S[layer][i] of the
candidates of one synthetic request.  Calls only oracle/ and the seeded input generators.

    python tests/golden/make_scores.py 1 0                      # workload index, request index: every candidate
    python tests/golden/make_scores.py 4 0 --candidates 0:64    # a slice of the candidates
    python tests/golden/make_scores.py 3 0 --stratified 32      # 32 candidates evenly spaced in length rank
    python tests/golden/make_scores.py 3 0 --ids 4,17,63        # these candidates
    python tests/golden/make_scores.py 2 0 --merge a.txt b.txt  # join part files of one request into one file

Candidates whose documents are token-for-token equal (the stress workload's duplicates) have equal inputs,
so only one of each group is forwarded and its scores are written for all of them.

The file is plain text: a header with the recipe and an `# ids` line naming the candidates of the columns,
then one line per scored layer."""
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

HERE = os.path.dirname(os.path.abspath(__file__))


def read_scores(path):
    """(S, ids, header lines) of a file this script wrote: S[layer] is an array over the columns, ids[j] the
    candidate of column j.  Older files carry `candidates a..b` instead of an `# ids` line."""
    S, ids, head = {}, None, []
    for line in open(path):
        if line.startswith("#"):
            head.append(line.rstrip("\n"))
            if line.startswith("# ids"):
                ids = [int(x) for x in line.split()[2:]]
            elif ids is None and " candidates " in line and ".." in line:
                a, b = line.split(" candidates ")[1].split("..")
                ids = list(range(int(a), int(b) + 1))
            continue
        p = line.split()
        S[int(p[0])] = np.array([float(x) for x in p[1:]])
    return S, ids, head


def write_scores(path, wl, request, act, ids, layers, S, note):
    with open(path, "w") as f:
        f.write(f"# oracle scores (fp64 forward, bf16-rounded weights where the workload is bf16), activations: {act}\n")
        f.write(f"# workload {wl.name} request {request} weight_seed {wl.weight_seed} n_columns {len(ids)}\n")
        f.write(f"# written by tests/golden/make_scores.py {note}; one line per layer: layer then one score per column\n")
        f.write("# ids " + " ".join(str(int(i)) for i in ids) + "\n")
        for l in layers:
            f.write(str(l) + " " + " ".join(repr(float(v)) for v in S[l]) + "\n")


def stratified_ids(lengths, count):
    """`count` candidates evenly spaced in length rank (shortest and longest included)."""
    order = np.argsort(np.asarray(lengths), kind="stable")
    pos = np.unique(np.rint(np.linspace(0, len(order) - 1, count)).astype(np.int64))
    return sorted(int(order[p]) for p in pos)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("workload", type=int)
    ap.add_argument("request", type=int)
    ap.add_argument("--candidates", default=None, help="a:b slice of candidate indices")
    ap.add_argument("--ids", default=None, help="comma-separated candidate indices")
    ap.add_argument("--stratified", type=int, default=0, help="this many candidates evenly spaced in length rank")
    ap.add_argument("--part", default=None, help="i/n: of the chosen candidates, take the i-th of n contiguous parts")
    ap.add_argument("--merge", nargs="+", default=None, help="part files to join (columns sorted by candidate)")
    ap.add_argument("--out", default=None)
    ap.add_argument("--act", default="exact",
                    help="exact, bf16 (every stored activation rounded to bfloat16: the bf16 precision contract) or "
                         "a comma-separated subset of the oracle's rounding points")
    a = ap.parse_args()
    wl = synth.workload(a.workload)
    cfg = wl.model
    out = a.out or os.path.join(HERE, f"{wl.name}_scores_r{a.request}.txt")
    layers = sorted(set(list(wl.schedule.probe_layers) + [cfg.n_layers]))

    if a.merge:
        col = {}
        for path in a.merge:
            S, ids, head = read_scores(path)
            assert any(f"workload {wl.name} request {a.request} " in h for h in head), path
            assert any(h.endswith(f"activations: {a.act}") for h in head), path
            for j, i in enumerate(ids):
                col[i] = [S[l][j] for l in layers]
        ids = sorted(col)
        S = {l: np.array([col[i][k] for i in ids]) for k, l in enumerate(layers)}
        write_scores(out, wl, a.request, a.act, ids, layers, S, f"(joined from {len(a.merge)} part files)")
        print(out, len(ids), "columns")
        return

    r = synth.make_request(wl, a.request)
    off = r["cand_offsets"]
    n = len(off) - 1
    ids = list(range(n))
    if a.candidates:
        lo, hi = (int(x) for x in a.candidates.split(":"))
        ids = ids[lo:hi]
    if a.ids:
        ids = [int(x) for x in a.ids.split(",")]
    if a.stratified:
        ids = stratified_ids(np.diff(off), a.stratified)
    if a.part:
        i, m = (int(x) for x in a.part.split("/"))
        ids = ids[len(ids) * i // m: len(ids) * (i + 1) // m]
    # one representative per group of identical documents
    first, rep = {}, []
    for i in ids:
        key = r["cand_tokens"][off[i]:off[i + 1]].tobytes()
        rep.append(first.setdefault(key, i))
    uniq = sorted(set(rep))
    weights = dict(W.make_globals(cfg, wl.weight_seed))
    weights["layers"] = W.iter_layers(cfg, wl.weight_seed)        # lazily, one layer at a time
    t0 = time.time()
    Su = oracle.score_matrix(r["query"], r["cand_tokens"], off, weights, cfg, layers, candidates=uniq, act=a.act)
    dt = time.time() - t0
    at = {u: j for j, u in enumerate(uniq)}
    S = {l: np.array([Su[l][at[q]] for q in rep]) for l in layers}
    write_scores(out, wl, a.request, a.act, ids, layers, S, f"in {dt:.0f} s ({len(uniq)} distinct documents forwarded)")
    print(out, f"{dt:.1f}s")


if __name__ == "__main__":
    main()
