"""Oracle of the dispersion-threshold auto-calibration (Sec. 4.1, last paragraph).  Test infrastructure.

The paper's loop: sample requests at a frequency, log their top-K, re-run them without pruning for the
ground truth, compute the precision of the sampled requests, and raise the threshold if the precision is
below the target, otherwise lower it.  Readings (the paper gives no step size or window): the threshold is
multiplied by raise_factor (> 1) or lower_factor (< 1) after every `window` sampled requests, using the
mean precision of the window, and clamped to [min_threshold, max_threshold]; precision of one request is
|top-K with pruning  intersect  top-K without| / min(K, N).
parity: pinned (closed-form trajectories on scripted precisions; tests/test_oracle_rule.py)."""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable, List, Sequence


@dataclass
class Calibrator:
    threshold: float
    target_precision: float
    raise_factor: float = 1.5
    lower_factor: float = 0.8
    min_threshold: float = 1e-3
    max_threshold: float = 1e3
    sample_every: int = 1
    window: int = 1
    n_in_window: int = 0
    n_adjustments: int = 0
    n_requests: int = 0
    n_sampled: int = 0
    precision_sum: float = 0.0
    last_precision: float = 0.0
    last_window_precision: float = 0.0


def precision_at_k(pruned: Sequence[int], full: Sequence[int]) -> float:
    return len(set(pruned) & set(full)) / float(len(full)) if len(full) else 1.0


def calibrated_step(cal: Calibrator, run: Callable[[float | None], List[int]]) -> List[int]:
    """Serve one request.  run(threshold) returns the top-K indices with cluster pruning at that
    threshold; run(None) returns them without pruning."""
    result = run(cal.threshold)
    sample = (cal.n_requests % cal.sample_every) == 0
    cal.n_requests += 1
    if not sample or not result:
        return result
    p = precision_at_k(result, run(None))
    cal.last_precision = p
    cal.precision_sum += p
    cal.n_sampled += 1
    cal.n_in_window += 1
    if cal.n_in_window >= cal.window:
        mean = cal.precision_sum / cal.n_in_window
        cal.last_window_precision = mean
        t = cal.threshold * (cal.raise_factor if mean < cal.target_precision else cal.lower_factor)
        cal.threshold = min(cal.max_threshold, max(cal.min_threshold, t))
        cal.n_in_window = 0
        cal.precision_sum = 0.0
        cal.n_adjustments += 1
    return result
