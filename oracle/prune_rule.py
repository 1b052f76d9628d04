"""Oracle of progressive cluster pruning (Sec. 4.1; working example Sec. 4.5).  Test infrastructure.

The rule is a heuristic, so this file follows the paper's steps in the paper's order:
  probe scores of the active candidates -> dispersion CV = |std/mean| -> if CV exceeds the
  dispersion threshold, cluster the scores (the paper runs K-Means) -> the boundary cluster is
  the one holding the K-th ranked candidate -> higher clusters are *selected* (enter the
  result, stop computing), lower clusters are *dropped*, the boundary cluster is *deferred*
  -> the forward stops when #deferred equals the remaining top-K slots.

Readings where the paper is silent (each also listed in the design notes):
  * K-Means is randomised and its k/init/iterations are not given; scores are 1-D, so we take
    the partition K-Means approximates: the contiguous split of the ranked scores into
    k_eff = min(n_clusters, #distinct scores) groups minimising the within-group sum of squares,
    cuts allowed only between strictly different scores.  Among equal-cost optima the one with
    the smallest last cut wins, then the smallest second-to-last cut, and so on.
  * std is the population std (ddof = 0) unless the schedule says otherwise; a zero mean with
    non-zero std gives CV = +inf; all-equal scores give CV = 0.
  * ranking is total: score descending, original index ascending.
  * after some candidates were selected, "K-th ranked" means rank K_rem = K - #selected among
    the still-active candidates; CV and clusters are computed over active candidates only.
Arithmetic is fp64 on fp32 scores in a fixed left-to-right order so that an implementation
following the same steps can be bit-identical.
parity: pinned (brute force over all partitions, two-class closed form, planted clusters,
closed-form CV, the paper's 20 -> 2/2/16 -> terminate count trace; tests/test_oracle_rule.py).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, Dict, List, Sequence, Tuple

import numpy as np

MODE_NONE = 0
MODE_FIXED_KEEP = 1
MODE_CLUSTER = 2


def rank_order(scores: np.ndarray, ids: np.ndarray) -> np.ndarray:
    """Permutation that orders candidates by (score descending, original id ascending)."""
    s = np.asarray(scores, dtype=np.float64)
    return np.lexsort((np.asarray(ids), -s))


def _centered_prefix_sums(sorted_scores: np.ndarray) -> Tuple[float, np.ndarray, np.ndarray]:
    """mu, P1, P2 with sequential (left-to-right) fp64 sums over the ranked scores:
    mu = (s_0 + s_1 + ...)/n, z_r = s_r - mu, P1[j] = sum_{r<j} z_r, P2[j] = sum_{r<j} z_r^2."""
    s = np.asarray(sorted_scores, dtype=np.float32).astype(np.float64)
    n = s.size
    mu = float(np.cumsum(s)[-1] / float(n))          # cumsum is a sequential accumulate
    z = s - mu
    p1 = np.concatenate([[0.0], np.cumsum(z)])
    p2 = np.concatenate([[0.0], np.cumsum(z * z)])
    return mu, p1, p2


def coefficient_of_variation(scores: np.ndarray, ids: np.ndarray | None = None, ddof: int = 0) -> float:
    """CV = |std(scores) / mean(scores)| (Sec. 4.1), sums taken over the ranked order."""
    s = np.asarray(scores, dtype=np.float32)
    ids = np.arange(s.size) if ids is None else np.asarray(ids)
    ss = s[rank_order(s, ids)]
    mu, _, p2 = _centered_prefix_sums(ss)
    denom = float(s.size - ddof)
    if denom <= 0.0:
        return 0.0
    sigma = float(np.sqrt(p2[-1] / denom))
    if sigma == 0.0:
        return 0.0
    if mu == 0.0:
        return float("inf")
    return sigma / abs(mu)


def optimal_partition(sorted_scores: np.ndarray, n_clusters: int) -> List[int]:
    """Cut positions (ascending, each in 1..n-1; a cut at p separates ranks p-1 and p) of the
    minimum within-group-sum-of-squares split of scores sorted descending into
    k_eff = min(n_clusters, #distinct) contiguous groups.  Returns [] when k_eff <= 1.

    Dynamic programme over the group index c and the group end j:
        D[1][j] = cost(0, j);   D[c][j] = min_i D[c-1][i] + cost(i, j)
        cost(i, j) = (P2[j]-P2[i]) - (P1[j]-P1[i])^2 / (j-i)      (sum of squared deviations)
    with i, j restricted to positions where the two neighbouring scores differ; the smallest
    minimising i is kept, and cuts are read back from j = n."""
    s32 = np.asarray(sorted_scores, dtype=np.float32)
    n = s32.size
    if n == 0:
        return []
    distinct = 1 + int(np.count_nonzero(s32[1:] != s32[:-1]))
    k = min(int(n_clusters), distinct)
    if k <= 1:
        return []
    _, p1, p2 = _centered_prefix_sums(s32)
    valid = np.zeros(n + 1, dtype=bool)          # valid[p]: a group may end right before rank p
    valid[1:n] = s32[1:] != s32[:-1]
    valid[n] = True
    inf = float("inf")

    def cost(i: np.ndarray, j: int) -> np.ndarray:
        s1 = p1[j] - p1[i]
        s2 = p2[j] - p2[i]
        return s2 - (s1 * s1) / (j - i).astype(np.float64)

    d_prev = np.full(n + 1, inf)
    for j in range(1, n + 1):
        if valid[j]:
            d_prev[j] = float(cost(np.array([0]), j)[0])
    arg = np.zeros((k + 1, n + 1), dtype=np.int64)
    for c in range(2, k + 1):
        d_cur = np.full(n + 1, inf)
        for j in range(c, n + 1):
            if not valid[j]:
                continue
            i = np.arange(c - 1, j)
            tot = d_prev[i] + cost(i, j)          # d_prev is +inf at invalid i
            b = int(np.argmin(tot))               # first (smallest i) among equal minima
            if tot[b] < inf:
                d_cur[j] = tot[b]
                arg[c, j] = i[b]
        d_prev = d_cur
    cuts: List[int] = []
    j = n
    for c in range(k, 1, -1):
        j = int(arg[c, j])
        cuts.append(j)
    return cuts[::-1]


def route_clusters(scores: np.ndarray, ids: np.ndarray, k_rem: int, n_clusters: int
                   ) -> Tuple[np.ndarray, np.ndarray, np.ndarray, List[int]]:
    """Three-way routing (Sec. 4.1): returns (selected, deferred, dropped) as arrays of positions
    into `scores` in ranked order, plus the cut positions.  The boundary cluster is the group
    that contains rank k_rem (1-based)."""
    order = rank_order(scores, ids)
    ss = np.asarray(scores, dtype=np.float32)[order]
    cuts = optimal_partition(ss, n_clusters)
    bounds = [0] + cuts + [len(order)]
    g = 0
    while not (bounds[g] < k_rem <= bounds[g + 1]):
        g += 1
    lo, hi = bounds[g], bounds[g + 1]
    return order[:lo], order[lo:hi], order[hi:], cuts


@dataclass
class ProbeRecord:
    layer: int
    n_active_before: int
    cv: float
    fired: int
    n_selected: int
    n_dropped: int
    n_deferred: int
    k_rem_after: int
    active_ids: List[int] = field(default_factory=list)     # ids scored at this probe, batch order
    scores: List[float] = field(default_factory=list)       # their fp32 scores
    cuts: List[int] = field(default_factory=list)


@dataclass
class SelectResult:
    topk_idx: List[int]
    topk_scores: List[float]
    trace: List[ProbeRecord]
    layers_run: int                       # number of layers after which the forward stopped
    active_per_layer: List[List[int]]     # ids forwarded through layer l (index l-1)


def replay_select(score_fn: Callable[[int, Sequence[int]], np.ndarray], n: int, k: int,
                  n_layers: int, sched) -> SelectResult:
    """Run the selection rule.  score_fn(layer, ids) returns the probe scores (after `layer`
    completed blocks) of the listed original candidate ids, as float32-representable values.

    sched has fields mode, probe_layers, keep_counts, cv_threshold, n_clusters, std_ddof,
    select_winners.  The active set keeps the candidates' original relative order (stable
    compaction).  Result order: candidates selected at earlier probes first (each probe's
    batch by score desc, id asc), then the final fill."""
    active = list(range(n))
    res_idx: List[int] = []
    res_sc: List[float] = []
    k_rem = min(int(k), int(n))
    trace: List[ProbeRecord] = []
    active_per_layer: List[List[int]] = []
    probes = list(sched.probe_layers) if sched.mode != MODE_NONE else []
    done_layer = None

    def take_sorted(ids: List[int], sc: np.ndarray, count: int) -> None:
        o = rank_order(sc, np.asarray(ids))[:count]
        for p in o:
            res_idx.append(int(ids[p]))
            res_sc.append(float(np.float32(sc[p])))

    for layer in range(1, n_layers + 1):
        if k_rem == 0 or not active:
            done_layer = layer - 1
            break
        active_per_layer.append(list(active))
        if layer == n_layers:
            sc = np.asarray(score_fn(layer, active), dtype=np.float32)
            take_sorted(active, sc, k_rem)
            done_layer = layer
            break
        if layer not in probes:
            continue
        j = probes.index(layer)
        sc = np.asarray(score_fn(layer, active), dtype=np.float32)
        ids = np.asarray(active)
        rec = ProbeRecord(layer, len(active), 0.0, 0, 0, 0, len(active), k_rem,
                          active_ids=list(active), scores=[float(x) for x in sc])
        trace.append(rec)
        if len(active) <= k_rem:                       # nothing left to decide
            take_sorted(active, sc, len(active))
            k_rem -= len(active)
            rec.k_rem_after = k_rem
            active = []
            done_layer = layer
            break
        if sched.mode == MODE_FIXED_KEEP:
            m = int(sched.keep_counts[j])
            if m < len(active):
                keep = set(int(p) for p in rank_order(sc, ids)[:m])
                rec.fired = 1
                rec.n_dropped = len(active) - m
                rec.n_deferred = m
                active = [a for p, a in enumerate(active) if p in keep]
                sc = np.asarray([s for p, s in enumerate(sc) if p in keep], dtype=np.float32)
        else:
            rec.cv = coefficient_of_variation(sc, ids, sched.std_ddof)
            if rec.cv > sched.cv_threshold:
                sel, dfr, drp, cuts = route_clusters(sc, ids, k_rem, sched.n_clusters)
                rec.cuts = cuts
                if cuts:
                    rec.fired = 1
                    rec.n_dropped = len(drp)
                    if sched.select_winners:
                        rec.n_selected = len(sel)
                        rec.n_deferred = len(dfr)
                        for p in sel:                   # already in ranked order
                            res_idx.append(int(ids[p]))
                            res_sc.append(float(sc[p]))
                        k_rem -= len(sel)
                        keep = set(int(p) for p in dfr)
                    else:                               # drop-only variant (Sec. 7)
                        rec.n_deferred = len(sel) + len(dfr)
                        keep = set(int(p) for p in sel) | set(int(p) for p in dfr)
                    active = [a for p, a in enumerate(active) if p in keep]
                    sc = np.asarray([s for p, s in enumerate(sc) if p in keep], dtype=np.float32)
        rec.k_rem_after = k_rem
        if len(active) == k_rem:                        # terminal condition (Sec. 4.1, 4.5)
            take_sorted(active, sc, k_rem)
            k_rem = 0
            rec.k_rem_after = 0
            active = []
            done_layer = layer
            break
    if done_layer is None:
        done_layer = n_layers
    return SelectResult(res_idx, res_sc, trace, done_layer, active_per_layer)
