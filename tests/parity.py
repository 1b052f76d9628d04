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
    """Every traced score against the oracle's, within `tol` absolute."""
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


def _wss(sorted_scores: np.ndarray, cuts: List[int]) -> float:
    b = [0, *cuts, len(sorted_scores)]
    return float(sum(np.sum((sorted_scores[b[g]:b[g + 1]] - np.mean(sorted_scores[b[g]:b[g + 1]])) ** 2)
                     for g in range(len(b) - 1)))


def check_end_to_end(trace, topk_idx, S: Dict[int, np.ndarray], n: int, k: int, n_layers: int, sched, tol: float):
    """The oracle's rule on the ORACLE's scores vs the CUDA run.  Identical results pass outright.
    Otherwise the probes are walked in lockstep (the oracle is put on the CUDA path's active set, which
    is valid because a candidate's score does not depend on its batch mates) and every divergence must
    be one that scores within `tol` of the oracle's can cause:
      * the CV sits within reach of the threshold (the two CVs straddle it),
      * a different partition whose cost on the oracle's scores is within the perturbation bound
        4*tol*sum|z| + 2*n*tol^2 of the optimum,
      * membership differences only among candidates within 2*tol of the score at a cut,
      * final top-K differences only among candidates within 2*tol of the K-th score."""
    def fn(layer, ids):
        return np.asarray(S[layer], np.float64)[np.asarray(ids, np.int64)].astype(np.float32)
    ref = oracle.replay_select(fn, n, k, n_layers, sched)
    got_idx = list(map(int, topk_idx))
    if ref.topk_idx == got_idx:
        return "identical"
    verdict = "same set" if set(ref.topk_idx) == set(got_idx) else "within tolerance band"
    k_rem = min(k, n)
    n_sel_total = 0
    probes = set(sched.probe_layers) if sched.mode != MODE_NONE else set()
    for rec in trace.records:
        ids = np.asarray(rec.active_ids, np.int64)
        s = fn(rec.layer, ids)
        g = np.asarray(rec.scores, np.float32)
        assert np.max(np.abs(s.astype(np.float64) - g.astype(np.float64))) <= tol
        order_s = oracle.rank_order(s, ids)
        if rec.layer not in probes or rec.layer == n_layers or len(ids) <= k_rem:
            # final fill (or nothing left to decide): members may differ only near the K-th score
            take = min(k_rem, len(ids))
            exp = set(int(ids[p]) for p in order_s[:take])
            got = set(got_idx[n_sel_total:n_sel_total + take])
            if take < len(ids):
                kth = float(s[order_s[take - 1]])
                for c in exp ^ got:
                    assert abs(float(S[rec.layer][c]) - kth) <= 2 * tol, (rec.layer, c)
            break
        if sched.mode == MODE_FIXED_KEEP:
            m = sched.keep_counts[list(sched.probe_layers).index(rec.layer)]
            if m < len(ids):
                exp = set(int(ids[p]) for p in order_s[:m])
                order_g = oracle.rank_order(g, ids)
                got = set(int(ids[p]) for p in order_g[:m])
                mth = float(s[order_s[m - 1]])
                for c in exp ^ got:
                    assert abs(float(S[rec.layer][c]) - mth) <= 2 * tol, (rec.layer, c)
        else:
            cv_s = oracle.coefficient_of_variation(s, ids, sched.std_ddof)
            thr = sched.cv_threshold
            fired_s = cv_s > thr
            cuts_s = oracle.optimal_partition(s[order_s], sched.n_clusters) if fired_s else []
            if bool(rec.fired) != bool(cuts_s):
                assert (cv_s - thr) * (rec.cv - thr) <= 0, (rec.layer, cv_s, rec.cv, thr)   # CVs straddle the threshold
            elif rec.fired and rec.cuts != cuts_s:
                ss = s[order_s].astype(np.float64)
                z = ss - ss.mean()
                bound = 4 * tol * float(np.sum(np.abs(z))) + 2 * len(ss) * tol * tol
                assert _wss(ss, rec.cuts) - _wss(ss, cuts_s) <= bound, (rec.layer, rec.cuts, cuts_s)
            elif rec.fired:
                order_g = oracle.rank_order(g, ids)
                for cpos in rec.cuts:                                   # same cuts: only near-cut swaps
                    a = set(int(ids[p]) for p in order_s[:cpos])
                    b = set(int(ids[p]) for p in order_g[:cpos])
                    edge = float(s[order_s[cpos - 1]])
                    for c in a ^ b:
                        assert abs(float(S[rec.layer][c]) - edge) <= 2 * tol, (rec.layer, c)
        k_rem = rec.k_rem_after
        n_sel_total += rec.n_selected
    return verdict
