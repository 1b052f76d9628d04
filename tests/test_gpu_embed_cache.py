"""-m gpu: embedding table caching (Sec. 4.4): the table stays in pinned host memory, the device holds an LRU cache
of rows.  The cache must never change a result, and its counters must follow the LRU rule."""
import numpy as np
import pytest

import synth

from test_gpu_select import MID, MID_WL, make_model, run

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_2510_15620_b200 as pkg
    return pkg


def cached_model(P, cfg, w, req, rows, **kw):
    lens = np.diff(req["cand_offsets"]) + len(req["query"])
    tw = P.upload_weights(w, cfg.dtype, embed_pinned_host=True)
    return P.PrismModel(cfg, tw, int(lens.max()) + 64, len(lens), int(lens.sum()) + 4096, embed_cache_rows=rows, **kw)


def distinct(req):
    return len(set(req["query"].tolist()) | set(req["cand_tokens"].tolist()))


def same(a, b):
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1].view(np.uint32), b[1].view(np.uint32))
    for r1, r2 in zip(a[2].records, b[2].records):
        assert np.array_equal(r1.scores, r2.scores) and r1.active_ids == r2.active_ids


def test_cache_is_result_neutral_and_counts_hits(P):
    w = synth.make_weights(MID, seed=5)
    reqs = [synth.make_request(MID_WL, r) for r in range(3)]
    base = P.PrismModel(MID, P.upload_weights(w, MID.dtype), 512, MID_WL.n_candidates, 16384)
    ref = [run(P, base, r, MID_WL.top_k, MID_WL.schedule) for r in reqs]
    m = cached_model(P, MID, w, max(reqs, key=lambda r: r["cand_offsets"][-1]), rows=MID.vocab)   # everything fits
    assert m.embed_cache_stats() == (0, 0, 0)
    same(run(P, m, reqs[0], MID_WL.top_k, MID_WL.schedule), ref[0])
    d0 = distinct(reqs[0])
    assert m.embed_cache_stats() == (0, d0, 0)                       # cold: every distinct token is fetched once
    same(run(P, m, reqs[0], MID_WL.top_k, MID_WL.schedule), ref[0])
    assert m.embed_cache_stats() == (d0, d0, 0)                      # warm: all hits
    same(run(P, m, reqs[1], MID_WL.top_k, MID_WL.schedule), ref[1])
    h, mi, ev = m.embed_cache_stats()
    both = len((set(reqs[0]["query"].tolist()) | set(reqs[0]["cand_tokens"].tolist())) &
               (set(reqs[1]["query"].tolist()) | set(reqs[1]["cand_tokens"].tolist())))
    assert h == d0 + both and mi == d0 + distinct(reqs[1]) - both and ev == 0
    m.close()
    base.close()


def test_cache_evicts_least_recently_used_rows(P):
    """A cache barely larger than one request's distinct tokens: alternating requests evict each other's rows, the
    results stay those of the resident table, and a row used by the current request is never the victim."""
    w = synth.make_weights(MID, seed=5)
    reqs = [synth.make_request(MID_WL, r) for r in range(3)]
    base = P.PrismModel(MID, P.upload_weights(w, MID.dtype), 512, MID_WL.n_candidates, 16384)
    ref = [run(P, base, r, MID_WL.top_k, MID_WL.schedule) for r in reqs]
    rows = max(distinct(r) for r in reqs) + 8
    m = cached_model(P, MID, w, max(reqs, key=lambda r: r["cand_offsets"][-1]), rows=rows)
    for i in (0, 1, 2, 0, 2, 1, 0):
        same(run(P, m, reqs[i], MID_WL.top_k, MID_WL.schedule), ref[i])
    h, mi, ev = m.embed_cache_stats()
    assert ev > 0 and mi > max(distinct(r) for r in reqs) and h > 0
    # LRU, not FIFO: after request 0 then 1, re-running 0 keeps 0's rows fresh, so a following 1 misses only what 0's
    # second pass displaced -- fewer than a cold start of 1
    before = m.embed_cache_stats()[1]
    same(run(P, m, reqs[0], MID_WL.top_k, MID_WL.schedule), ref[0])
    assert m.embed_cache_stats()[1] == before                        # request 0 was the last one run: all hits
    m.close()
    base.close()


def test_cache_too_small_and_bad_table_location(P):
    w = synth.make_weights(MID, seed=5)
    req = synth.make_request(MID_WL, 0)
    m = cached_model(P, MID, w, req, rows=distinct(req) - 1)
    with pytest.raises(P.PrismError) as e:
        run(P, m, req, MID_WL.top_k, MID_WL.schedule)
    assert e.value.status == -2                                       # SHAPE_LIMIT
    m.close()
    lens = np.diff(req["cand_offsets"]) + len(req["query"])
    with pytest.raises(P.PrismError):                                 # a device table cannot be the host side of a cache
        P.PrismModel(MID, P.upload_weights(w, MID.dtype), int(lens.max()), len(lens), int(lens.sum()), embed_cache_rows=100)


def test_cache_with_fp32_path_and_streamed_layers(P):
    """cfg 0 (fp32 rows) and a bf16 model with streamed layer weights and chunked execution on top of the cache."""
    wl = synth.workload(0)
    w0 = synth.make_weights(wl.model)
    r0 = synth.make_request(wl, 0)
    base = make_model(P, wl.model, w0, r0)
    ref = run(P, base, r0, wl.top_k, wl.schedule)
    m = cached_model(P, wl.model, w0, r0, rows=distinct(r0) + 5)
    for _ in range(2):
        got = run(P, m, r0, wl.top_k, wl.schedule)
        assert np.array_equal(got[0], ref[0]) and np.array_equal(got[1].view(np.uint32), ref[1].view(np.uint32))
    m.close()
    base.close()

    w = synth.make_weights(MID, seed=5)
    req = synth.make_request(MID_WL, 0)
    lens = np.diff(req["cand_offsets"]) + len(req["query"])
    base = make_model(P, MID, w, req)
    ref = run(P, base, req, MID_WL.top_k, MID_WL.schedule)
    per_tok = (1024 + 4096 + 2048 + 3072) * 2
    budget = 2 * (int(lens.sum()) + 4096) * 1024 * 4 + per_tok * (int(lens.max()) + 100)
    tw = P.upload_weights(w, MID.dtype, layers_pinned_host=True, embed_pinned_host=True)
    m = P.PrismModel(MID, tw, int(lens.max()) + 64, len(lens), int(lens.sum()) + 4096, activation_budget_bytes=budget,
                     stream_weights=True, embed_cache_rows=distinct(req) + 16)
    for _ in range(2):
        same(run(P, m, req, MID_WL.top_k, MID_WL.schedule), ref)
    m.close()
    base.close()


def _request_of(tokens_per_doc, query):
    offs = np.zeros(len(tokens_per_doc) + 1, np.int32)
    offs[1:] = np.cumsum([len(t) for t in tokens_per_doc])
    return {"query": np.asarray(query, np.int32), "cand_tokens": np.concatenate(tokens_per_doc).astype(np.int32),
            "cand_offsets": offs}


def test_refused_request_leaves_the_eviction_order_alone(P):
    """Requests A then B fill a cache of 64 rows; a request that holds all of A's tokens and too many others is
    refused (SHAPE_LIMIT).  The refusal must not have refreshed A's rows: the next request's new tokens evict A's
    rows (used longest ago), so B afterwards still finds all of its rows."""
    wl = synth.workload(0)
    w = synth.make_weights(wl.model)
    q = [3, 4]
    A = _request_of([np.arange(100, 116), np.arange(116, 130)], q)             # 30 + 2 distinct tokens
    B = _request_of([np.arange(200, 216), np.arange(216, 230)], q)             # 30 new ones: 62 rows in use
    X = _request_of([np.arange(100, 130), np.arange(300, 340)], q)             # 72 distinct tokens > 64 rows
    C = _request_of([np.arange(400, 416), np.arange(416, 430)], q)             # 30 new ones: 28 evictions
    big = _request_of([np.arange(0, 64), np.arange(64, 128)], q)
    m = cached_model(P, wl.model, w, big, rows=64)
    sched = None
    run(P, m, A, 1, sched)
    run(P, m, B, 1, sched)
    assert m.embed_cache_stats() == (2, 62, 0)
    with pytest.raises(P.PrismError) as e:
        run(P, m, X, 1, sched)
    assert e.value.status == -2
    assert m.embed_cache_stats() == (2, 62, 0)
    run(P, m, C, 1, sched)
    h, mi, ev = m.embed_cache_stats()
    assert (h, mi, ev) == (4, 92, 28)
    run(P, m, B, 1, sched)                                                      # B's rows were younger than A's: all there
    assert m.embed_cache_stats() == (h + 32, mi, ev)
    run(P, m, A, 1, sched)                                                      # 28 of A's 30 rows went to C
    assert m.embed_cache_stats()[1] == mi + 28
    m.close()
