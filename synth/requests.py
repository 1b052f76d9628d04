"""Seeded request generator: one query, N candidate documents, packed token ids + offsets."""
from __future__ import annotations

from typing import Dict

import numpy as np

from .configs import Workload


def make_request(wl: Workload, r: int = 0, n_candidates: int | None = None) -> Dict[str, np.ndarray]:
    """Request r of workload wl.  Seed = 1000*cfg_index + r.

    Returns int32 arrays: query [Lq], cand_tokens [sum Ld], cand_offsets [N+1], and the python
    int top_k.  Token ids are uniform on [0, vocab).  With dup_fraction f, the last round(f*N)
    candidates (before a seeded shuffle) are exact copies of uniformly chosen originals."""
    rng = np.random.Generator(np.random.Philox(key=[1000 * wl.cfg_index + r, 0x5EED]))
    n = wl.n_candidates if n_candidates is None else n_candidates
    v = wl.model.vocab
    query = rng.integers(0, v, size=wl.query_len, dtype=np.int64).astype(np.int32)
    n_dup = int(round(wl.dup_fraction * n))
    n_orig = n - n_dup
    kind, a, b, lo, hi = wl.doc_len
    if kind == "uniform":
        lens = rng.integers(int(a), int(b) + 1, size=n_orig)
    elif kind == "lognormal":
        lens = np.rint(np.exp(rng.normal(np.log(a), b, size=n_orig))).astype(np.int64)
    else:
        raise ValueError(kind)
    lens = np.clip(lens, int(lo), int(hi)).astype(np.int64)
    docs = [rng.integers(0, v, size=int(l), dtype=np.int64).astype(np.int32) for l in lens]
    if n_dup:
        src = rng.integers(0, n_orig, size=n_dup)
        docs += [docs[int(s)].copy() for s in src]
        perm = rng.permutation(n)
        docs = [docs[int(p)] for p in perm]
    offs = np.zeros(n + 1, dtype=np.int32)
    offs[1:] = np.cumsum([len(d) for d in docs])
    toks = np.concatenate(docs).astype(np.int32) if docs else np.zeros(0, np.int32)
    return {"query": query, "cand_tokens": toks, "cand_offsets": offs, "top_k": wl.top_k}
