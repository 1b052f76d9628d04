"""Pins for the oracle's pruning rule (Sec. 4.1, working example Sec. 4.5): closed-form CV,
brute force over every partition, the two-class closed form, planted clusters, the paper's
count trace, and the routing invariants."""
import itertools
import math

import numpy as np
import pytest

import oracle
from oracle.prune_rule import (MODE_CLUSTER, MODE_FIXED_KEEP, MODE_NONE, coefficient_of_variation,
                               optimal_partition, rank_order, replay_select, route_clusters)
from synth.configs import Schedule


# ---------------------------------------------------------------- CV (Sec. 4.1 formula)
def test_cv_closed_forms():
    assert coefficient_of_variation(np.full(7, 3.25, np.float32)) == 0.0
    n = 9
    s = np.arange(1, n + 1, dtype=np.float32)
    mean = (n + 1) / 2
    std_pop = math.sqrt((n * n - 1) / 12)
    assert abs(coefficient_of_variation(s) - std_pop / mean) < 1e-15
    std_smp = math.sqrt(n * (n + 1) / 12)
    assert abs(coefficient_of_variation(s, ddof=1) - std_smp / mean) < 1e-15
    assert coefficient_of_variation(-s) == coefficient_of_variation(s)        # |.| in the formula
    assert coefficient_of_variation(np.array([-1, 1], np.float32)) == float("inf")
    assert coefficient_of_variation(np.array([2.0], np.float32)) == 0.0
    # scale invariance, exact for powers of two
    assert coefficient_of_variation(4 * s) == coefficient_of_variation(s)


def test_rank_order_is_total():
    s = np.array([1.0, 3.0, 3.0, 2.0, 3.0], np.float32)
    ids = np.array([10, 7, 5, 1, 9])
    assert list(ids[rank_order(s, ids)]) == [5, 7, 9, 1, 10]


# ---------------------------------------------------------------- clustering
def _wss(groups):
    t = 0.0
    for g in groups:
        m = math.fsum(g) / len(g)
        t += math.fsum((x - m) ** 2 for x in g)
    return t


def _brute(sorted_scores, k):
    """Every contiguous split into k_eff groups with cuts only between different scores; cost
    from the definition sum (s - group mean)^2 (no prefix sums).  Returns (best cuts, margin to
    the runner-up cost)."""
    s = [float(x) for x in sorted_scores]
    n = len(s)
    pos = [p for p in range(1, n) if s[p] != s[p - 1]]
    k_eff = min(k, len(pos) + 1)
    if k_eff <= 1:
        return [], float("inf")
    res = []
    for cuts in itertools.combinations(pos, k_eff - 1):
        b = [0, *cuts, n]
        res.append((_wss([s[b[i]:b[i + 1]] for i in range(k_eff)]), tuple(reversed(cuts))))
    res.sort()
    margin = res[1][0] - res[0][0] if len(res) > 1 else float("inf")
    return list(reversed(res[0][1])), margin


@pytest.mark.parametrize("k", [2, 3, 4, 5])
def test_partition_equals_brute_force(k):
    rng = np.random.default_rng(100 + k)
    checked = 0
    for trial in range(120):
        n = int(rng.integers(2, 13))
        s = rng.normal(size=n).astype(np.float32)
        if trial % 3 == 0:                                  # duplicates
            s[rng.integers(0, n, size=n // 2)] = s[0]
        s = np.sort(s)[::-1]
        best, margin = _brute(s, k)
        if margin < 1e-9:
            continue                                        # exact ties have their own test
        assert optimal_partition(s, k) == best, (s, k)
        checked += 1
    assert checked > 80


def test_partition_tie_break_smallest_last_cut():
    # 0,1,2 with k = 2: cutting after rank 1 or after rank 2 both cost 0.5 -> the smaller cut
    assert optimal_partition(np.array([2, 1, 0], np.float32), 2) == [1]
    # symmetric five points, k = 2: {4,3 | 2,1,0} and {4,3,2 | 1,0} tie at 0.5 + 2 -> cut 2
    assert optimal_partition(np.array([4, 3, 2, 1, 0], np.float32), 2) == [2]
    # equal scores are never split; fewer distinct values than clusters shrinks k
    assert optimal_partition(np.array([1, 1, 1, 1], np.float32), 3) == []
    assert optimal_partition(np.array([5, 5, 1, 1, 1], np.float32), 3) == [2]
    assert optimal_partition(np.array([5, 5, 3, 1, 1], np.float32), 5) == [2, 3]


def test_two_clusters_is_max_between_class_variance():
    """k = 2 reduces to the textbook threshold rule: maximise n1*n2*(m1-m2)^2 / n."""
    rng = np.random.default_rng(7)
    for _ in range(50):
        n = int(rng.integers(3, 40))
        s = np.sort(rng.normal(size=n).astype(np.float32))[::-1]
        d = s.astype(np.float64)
        best = max(range(1, n), key=lambda p: p * (n - p) * (d[:p].mean() - d[p:].mean()) ** 2)
        assert optimal_partition(s, 2) == [best]


def test_planted_clusters_are_recovered():
    rng = np.random.default_rng(11)
    a = 10 + 0.1 * rng.normal(size=7)
    b = 0 + 0.1 * rng.normal(size=20)
    c = -10 + 0.1 * rng.normal(size=13)
    s = np.sort(np.concatenate([a, b, c]).astype(np.float32))[::-1]
    assert optimal_partition(s, 3) == [7, 27]
    # a large common offset must not change the partition (sums are centred first)
    assert optimal_partition((s + np.float32(4096)).astype(np.float32), 3) == [7, 27]


def test_cumsum_is_sequential():
    """The rule fixes a left-to-right summation order; numpy's accumulate must honour it."""
    x = np.random.default_rng(5).normal(size=1000)
    acc, ref = 0.0, []
    for v in x:
        acc = acc + float(v)
        ref.append(acc)
    assert np.array_equal(np.cumsum(x), np.array(ref))


# ---------------------------------------------------------------- routing + replay
def test_routing_definitions():
    s = np.array([9.0, 8.9, 5.0, 5.1, 4.9, 5.05, 0.0, 0.1, -0.1, 0.05], np.float32)
    ids = np.arange(10)
    sel, dfr, drp, cuts = route_clusters(s, ids, k_rem=4, n_clusters=3)
    assert cuts == [2, 6]
    assert sorted(sel) == [0, 1] and sorted(dfr) == [2, 3, 4, 5] and sorted(drp) == [6, 7, 8, 9]
    sel, dfr, drp, _ = route_clusters(s, ids, k_rem=2, n_clusters=3)      # K-th sits in the top cluster
    assert len(sel) == 0 and sorted(dfr) == [0, 1] and len(drp) == 8
    sel, dfr, drp, _ = route_clusters(s, ids, k_rem=7, n_clusters=3)      # K-th sits in the low cluster
    assert sorted(sel) == [0, 1, 2, 3, 4, 5] and sorted(dfr) == [6, 7, 8, 9] and len(drp) == 0


def _fn(table):
    return lambda layer, ids: np.asarray([table[layer][i] for i in ids], np.float32)


def test_working_example_count_trace():
    """Sec. 4.5: top-10 of 20.  First firing probe: 2 selected, 2 dropped, 16 deferred; next probe
    stays below the threshold; the following probe leaves deferred + selected == 10 and the
    forward stops there."""
    L = 12
    s9 = [20.0, 19.5] + [10 + 0.05 * i for i in range(16)] + [0.5, 0.0]
    s10 = list(s9)
    s10[2:18] = [10 + 0.01 * i for i in range(16)]                     # tight: CV small
    s11 = list(s9)
    s11[2:18] = [30 + 0.01 * i for i in range(8)] + [5 + 0.01 * i for i in range(8)]
    table = {9: s9, 10: s10, 11: s11, L: s11}
    sched = Schedule(MODE_CLUSTER, (9, 10, 11), cv_threshold=0.3, n_clusters=3)
    res = replay_select(_fn(table), 20, 10, L, sched)
    t = res.trace
    assert (t[0].layer, t[0].n_active_before, t[0].fired, t[0].n_selected, t[0].n_dropped, t[0].n_deferred,
            t[0].k_rem_after) == (9, 20, 1, 2, 2, 16, 8)
    assert (t[1].layer, t[1].n_active_before, t[1].fired, t[1].n_deferred) == (10, 16, 0, 16)
    assert t[1].cv <= 0.3
    assert t[2].layer == 11 and t[2].fired == 1 and t[2].n_deferred == 8 and t[2].k_rem_after == 0
    assert res.layers_run == 11 and len(res.topk_idx) == 10
    assert sorted(res.topk_idx) == [0, 1] + list(range(2, 10))
    assert res.topk_idx[:2] == [0, 1]                                 # earlier-selected first
    assert [len(a) for a in res.active_per_layer] == [20] * 9 + [16, 16]


def test_infinite_threshold_and_none_are_the_plain_sort():
    rng = np.random.default_rng(3)
    L, n, k = 6, 30, 7
    table = {l: rng.normal(size=n).astype(np.float32) for l in range(1, L + 1)}
    plain = sorted(range(n), key=lambda i: (-table[L][i], i))[:k]
    a = replay_select(_fn(table), n, k, L, Schedule(MODE_NONE))
    b = replay_select(_fn(table), n, k, L, Schedule(MODE_CLUSTER, (2, 4), cv_threshold=float("inf")))
    assert a.topk_idx == plain and b.topk_idx == plain
    assert a.layers_run == L and all(len(x) == n for x in b.active_per_layer)


def test_drop_only_keeps_final_scores_and_order():
    rng = np.random.default_rng(4)
    L, n, k = 8, 40, 5
    base = rng.normal(size=n)
    table = {l: (base * 3 + 0.05 * rng.normal(size=n)).astype(np.float32) for l in range(1, L + 1)}
    sched = Schedule(MODE_CLUSTER, (2, 4, 6), cv_threshold=0.1, n_clusters=3, select_winners=0)
    res = replay_select(_fn(table), n, k, L, sched)
    plain = sorted(range(n), key=lambda i: (-table[L][i], i))[:k]
    assert any(t.fired for t in res.trace)
    assert res.topk_idx == plain                                     # strongly correlated layers
    assert res.topk_scores == [float(table[L][i]) for i in plain]
    assert len(res.active_per_layer[-1]) < n


def test_n_not_larger_than_k_and_degenerate_inputs():
    table = {l: np.array([0.3, 0.9, 0.1], np.float32) for l in (1, 2, 3)}
    r = replay_select(_fn(table), 3, 5, 3, Schedule(MODE_CLUSTER, (1,), cv_threshold=0.0))
    assert r.topk_idx == [1, 0, 2] and r.layers_run == 1             # decided at the first scored layer
    r = replay_select(_fn(table), 3, 5, 3, Schedule(MODE_NONE))
    assert r.topk_idx == [1, 0, 2] and r.layers_run == 3
    same = {l: np.ones(6, np.float32) for l in (1, 2)}
    r = replay_select(_fn(same), 6, 2, 2, Schedule(MODE_CLUSTER, (1,), cv_threshold=0.0))
    assert r.trace[0].fired == 0 and r.topk_idx == [0, 1]            # all equal: nothing to cluster
    r = replay_select(_fn(table), 0, 2, 3, Schedule(MODE_NONE))
    assert r.topk_idx == []


@pytest.mark.parametrize("k_clusters", [2, 3, 4, 5])
@pytest.mark.parametrize("winners", [0, 1])
def test_routing_invariants_random(k_clusters, winners):
    rng = np.random.default_rng(17 * k_clusters + winners)
    for trial in range(40):
        n = int(rng.integers(1, 80))
        k = int(rng.integers(1, 12))
        L = 7
        base = rng.normal(size=n)
        table = {}
        for l in range(1, L + 1):
            s = (base + 0.3 * rng.normal(size=n)).astype(np.float32)
            if trial % 4 == 0 and n > 3:
                s[rng.integers(0, n, size=n // 3)] = s[0]            # ties at thresholds
            table[l] = s
        sched = Schedule(MODE_CLUSTER, (1, 3, 4, 6), cv_threshold=0.2, n_clusters=k_clusters,
                         select_winners=winners)
        res = replay_select(_fn(table), n, k, L, sched)
        assert len(res.topk_idx) == min(k, n) and len(set(res.topk_idx)) == len(res.topk_idx)
        assert res.layers_run <= L
        prev = list(range(n))
        for t in res.trace:
            assert t.active_ids == [i for i in prev if i in set(t.active_ids)]      # stable order
            assert t.n_selected + t.n_dropped + t.n_deferred == t.n_active_before or not t.fired
            if t.fired:
                sc = dict(zip(t.active_ids, t.scores))
                order = sorted(t.active_ids, key=lambda i: (-sc[i], i))
                b = [0, *t.cuts, len(order)]
                assert all(sc[order[p - 1]] > sc[order[p]] for p in t.cuts)         # never split ties
                if winners:
                    assert t.n_selected < t.n_active_before
                    assert t.n_deferred >= t.k_rem_after or t.k_rem_after == 0
            prev = t.active_ids
        if not winners:                                               # drop-only: final-layer scores
            if res.layers_run == L:
                assert res.topk_scores == sorted(res.topk_scores, reverse=True)


def test_fixed_keep():
    rng = np.random.default_rng(8)
    n, L = 16, 2
    table = {l: rng.normal(size=n).astype(np.float32) for l in (1, 2)}
    res = replay_select(_fn(table), n, 3, L, Schedule(MODE_FIXED_KEEP, (1,), (8,)))
    keep = sorted(sorted(range(n), key=lambda i: (-table[1][i], i))[:8])
    assert res.active_per_layer == [list(range(n)), keep]
    assert res.topk_idx == sorted(keep, key=lambda i: (-table[2][i], i))[:3]


# ---------------------------------------------------------------- threshold auto-calibration (Sec. 4.1)
def test_calibration_raises_below_target_and_lowers_otherwise():
    from oracle.calibrate import Calibrator, calibrated_step, precision_at_k
    assert precision_at_k([1, 2, 3, 4], [4, 3, 9, 8]) == 0.5 and precision_at_k([], []) == 1.0
    full = list(range(10))
    # scripted service: pruning at a threshold below 1.0 loses 3 of 10, at or above 1.0 loses none
    run = lambda thr: full if thr is None or thr >= 1.0 else full[:7] + [97, 98, 99]
    cal = Calibrator(threshold=0.25, target_precision=0.9, raise_factor=2.0, lower_factor=0.5, min_threshold=0.125,
                     max_threshold=8.0, sample_every=2, window=2)
    trail = []
    for _ in range(16):
        calibrated_step(cal, run)
        trail.append(cal.threshold)
    # every 2nd request is sampled, every 2 samples adjust: requests 1-4 at 0.25 (precision 0.7 -> x2), 5-8 at 0.5
    # (0.7 -> x2), 9-12 at 1.0 (precision 1.0 -> x0.5), 13-16 at 0.5 (0.7 -> x2)
    assert trail == [0.25, 0.25, 0.5, 0.5, 0.5, 0.5, 1.0, 1.0, 1.0, 1.0, 0.5, 0.5, 0.5, 0.5, 1.0, 1.0]
    assert cal.n_requests == 16 and cal.n_sampled == 8 and cal.n_adjustments == 4
    assert cal.last_window_precision == 0.7
    # clamping
    cal = Calibrator(threshold=0.2, target_precision=0.0, raise_factor=2.0, lower_factor=0.5, min_threshold=0.15,
                     max_threshold=8.0)
    calibrated_step(cal, run)
    assert cal.threshold == 0.15
