"""Oracle end-to-end selection: per-candidate forward scores, then the rule (test infrastructure).

Because sequences never attend to each other, the monolithic layer-major run (Sec. 3.3) with
pruning equals: compute S[layer][i] for every candidate alone, then replay the rule over S.
With pruning disabled this is the plain definition: score every pair, sort, take K."""
from __future__ import annotations

from typing import Dict, Sequence

import numpy as np

from .prune_rule import MODE_NONE, SelectResult, replay_select
from .reranker import score_matrix


def oracle_select(query, cand_tokens, cand_offsets, k: int, weights: Dict[str, object], cfg, sched,
                  S: Dict[int, np.ndarray] | None = None) -> SelectResult:
    """If S is given ({layer: scores of ALL candidates}) it is used instead of forwarding."""
    n = len(cand_offsets) - 1
    layers = sorted(set(list(sched.probe_layers if sched.mode != MODE_NONE else ()) + [cfg.n_layers]))
    if S is None:
        S = score_matrix(query, cand_tokens, cand_offsets, weights, cfg, layers)

    def score_fn(layer: int, ids: Sequence[int]) -> np.ndarray:
        return np.asarray(S[layer], dtype=np.float64)[np.asarray(ids, dtype=np.int64)].astype(np.float32)

    return replay_select(score_fn, n, k, cfg.n_layers, sched)
