"""Helpers that compare a traced run of the CUDA path with the oracle (used by the -m gpu tests).

Three checks, from strict to tolerant:
  1. scores:  every probed score equals the oracle's S[layer][candidate] within the tolerance;
  2. replay:  the oracle's rule fed with the CUDA path's OWN traced scores reproduces every integer
              outcome (survivor sets and order, counts, cuts, K_rem, stop layer, top-K) exactly,
              and the CV bit for bit;
  3. end to end: the oracle's rule fed with the ORACLE's scores gives the same result, except where
              a candidate's oracle score lies within the tolerance of a cut."""
from __future__ import annotations

from typing import Dict, List, Sequence

import numpy as np

import oracle
from oracle.prune_rule import MODE_CLUSTER, MODE_FIXED_KEEP, MODE_NONE


def traced_score_fn(trace):
    table = {}
    for rec in trace.records:
        for i, s in zip(rec.active_ids, rec.scores):
            table[(rec.layer, int(i))] = np.float32(s)
    return lambda layer, ids: np.asarray([table[(layer, int(i))] for i in ids], np.float32)


def check_scores(trace, S: Dict[int, np.ndarray], tol: float, ids_known: Sequence[int] | None = None) -> float:
    worst = 0.0
    known = None if ids_known is None else {int(c): j for j, c in enumerate(ids_known)}
    for rec in trace.records:
        for i, s in zip(rec.active_ids, rec.scores):
            if known is not None:
                if int(i) not in known:
                    continue
                ref = S[rec.layer][known[int(i)]]
            else:
                ref = S[rec.layer][int(i)]
            err = abs(float(s) - float(ref))
            worst = max(worst, err)
            assert err <= tol, f"layer {rec.layer} candidate {i}: cuda {s} oracle {ref} |diff| {err} > {tol}"
    return worst


def check_replay(trace, topk_idx: Sequence[int], topk_scores: Sequence[float], n: int, k: int, n_layers: int, sched):
    ref = oracle.replay_select(traced_score_fn(trace), n, k, n_layers, sched)
    assert list(map(int, topk_idx)) == ref.topk_idx, (list(topk_idx), ref.topk_idx)
    assert [float(np.float32(x)) for x in topk_scores] == ref.topk_scores
    assert trace.layers_run == ref.layers_run
    probes = [r for r in trace.records if r.layer in set(sched.probe_layers) and sched.mode != MODE_NONE
              and r.layer != n_layers]
    assert len(probes) == len(ref.trace), (len(probes), len(ref.trace))
    for got, exp in zip(probes, ref.trace):
        assert got.layer == exp.layer
        assert got.active_ids == exp.active_ids
        assert got.n_active_before == exp.n_active_before
        assert (got.fired, got.n_selected, got.n_dropped, got.n_deferred, got.k_rem_after) == \
               (exp.fired, exp.n_selected, exp.n_dropped, exp.n_deferred, exp.k_rem_after), (got, exp)
        assert got.cuts == exp.cuts
        if sched.mode == MODE_CLUSTER:
            assert got.cv == exp.cv, (got.cv, exp.cv)           # same fp64 operations in the same order
    # live tokens per layer follow from the active sets
    return ref


def check_end_to_end(trace, topk_idx, S: Dict[int, np.ndarray], n: int, k: int, n_layers: int, sched, tol: float):
    """Oracle scores + oracle rule vs the CUDA result.  Differences must be explained by scores
    within `tol` of a cut: we walk the probes in lockstep on the CUDA path's active sets."""
    def fn(layer, ids):
        return np.asarray(S[layer], np.float64)[np.asarray(ids, np.int64)].astype(np.float32)
    ref = oracle.replay_select(fn, n, k, n_layers, sched)
    if ref.topk_idx == list(map(int, topk_idx)):
        return "identical"
    if set(ref.topk_idx) == set(map(int, topk_idx)):
        return "same set"
    # tolerance-band explanation on the final membership
    diff = set(ref.topk_idx) ^ set(map(int, topk_idx))
    last = {}
    for rec in trace.records:
        for i in rec.active_ids:
            last[int(i)] = rec.layer
    for i in diff:
        layer = last[i]
        sc = np.asarray(S[layer], np.float64)
        others = np.delete(sc, i)
        gap = np.min(np.abs(others - sc[i]))
        assert gap <= 2 * tol, f"candidate {i} differs but its oracle score at layer {layer} is {gap} from any other"
    return "within tolerance band"
