"""-m gpu: the shared query prefix.  Under causal attention the query's rows are the same in every sequence, so the
batch may hold them once; nothing a caller can see may change: indices, scores (bit for bit), every probe's score
vector and decision, and the token counts of the trace (which keep counting query + document per sequence)."""
from dataclasses import replace

import numpy as np
import pytest

import oracle
import synth
from synth.configs import MODE_CLUSTER, MODE_FIXED_KEEP, MODE_NONE, Schedule

from parity import check_scores
from test_gpu_select import MID, MID_WL, TOL_BF16, dev_i32, run

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_2510_15620_b200 as pkg
    return pkg


@pytest.fixture(scope="module")
def weights(P):
    w = synth.make_weights(MID, seed=5)
    return w, P.upload_weights(w, MID.dtype)


def request(lq, doc_lens, seed=0):
    rng = np.random.default_rng(seed)
    off = np.zeros(len(doc_lens) + 1, np.int32)
    off[1:] = np.cumsum(doc_lens)
    return {"query": rng.integers(0, MID.vocab, size=lq).astype(np.int32),
            "cand_tokens": rng.integers(0, MID.vocab, size=int(off[-1])).astype(np.int32), "cand_offsets": off}


def model(P, tw, req, **kw):
    lens = np.diff(req["cand_offsets"]) + len(req["query"])
    return P.PrismModel(MID, tw, int(lens.max()), len(lens), int(lens.sum()), **kw)


def both(P, tw, req, k, sched, **kw):
    a = run(P, model(P, tw, req, shared_prefix=True, **kw), req, k, sched)
    b = run(P, model(P, tw, req, shared_prefix=False, **kw), req, k, sched)
    return a, b


def same(a, b):
    assert np.array_equal(a[0], b[0])
    assert np.array_equal(a[1].view(np.uint32), b[1].view(np.uint32))
    ta, tb = a[2], b[2]
    assert ta.layers_run == tb.layers_run and ta.tokens_per_layer == tb.tokens_per_layer
    assert len(ta.records) == len(tb.records)
    for r1, r2 in zip(ta.records, tb.records):
        assert np.array_equal(r1.scores.view(np.uint32), r2.scores.view(np.uint32))
        assert r1.active_ids == r2.active_ids
        assert (r1.layer, r1.fired, r1.n_selected, r1.n_dropped, r1.n_deferred, r1.k_rem_after, r1.cuts, r1.tokens_before) == \
               (r2.layer, r2.fired, r2.n_selected, r2.n_dropped, r2.n_deferred, r2.k_rem_after, r2.cuts, r2.tokens_before)
        assert r1.cv == r2.cv


SCHEDS = [Schedule(MODE_NONE, ()), Schedule(MODE_CLUSTER, (2, 4), cv_threshold=0.3),
          Schedule(MODE_FIXED_KEEP, (1, 3, 5), (17, 9, 5))]


@pytest.mark.parametrize("lq", [8, 16, 64, 120])
@pytest.mark.parametrize("sched", SCHEDS, ids=["none", "cluster", "keep"])
def test_shared_prefix_changes_nothing(P, weights, lq, sched):
    """Document lengths chosen so that query + document ends before, on and after the 128-row block edges, spans
    up to four blocks, and one document is empty (its sequence is the query alone)."""
    _, tw = weights
    rng = np.random.default_rng(lq)
    docs = [0, 1, 128 - lq - 1, 128 - lq, 128 - lq + 1, 256 - lq, 257 - lq, 383, 300, 7] + rng.integers(1, 420, size=14).tolist()
    req = request(lq, docs, seed=lq)
    a, b = both(P, tw, req, 4, sched)
    assert a[2].shared_prefix_rows == lq and b[2].shared_prefix_rows == 0
    same(a, b)
    # what the trace calls tokens is query + document per live sequence
    assert a[2].tokens_per_layer[0] == sum(docs) + lq * len(docs)


def test_shared_prefix_against_the_oracle(P, weights):
    w, tw = weights
    req = synth.make_request(replace(MID_WL, query_len=32), 1)
    S = oracle.score_matrix(req["query"], req["cand_tokens"], req["cand_offsets"], w, MID, [2, 4, 6])
    m = model(P, tw, req)
    idx, sc, tr = run(P, m, req, 4, Schedule(MODE_FIXED_KEEP, (2, 4), (24, 24)))   # keeps everything: all layers scored
    assert tr.shared_prefix_rows == 32
    assert [r.layer for r in tr.records] == [2, 4, 6]
    check_scores(tr, S, TOL_BF16)


@pytest.mark.parametrize("lq,n", [(20, 6), (4, 6), (124, 6), (32, 1)])
def test_requests_the_prefix_path_does_not_take(P, weights, lq, n):
    """Query lengths off the 8-row grid or outside [8, 120], or a single candidate: one query copy per sequence,
    same results either way."""
    _, tw = weights
    req = request(lq, [50, 200, 131, 17, 260, 90][:n], seed=3)
    a, b = both(P, tw, req, 2, SCHEDS[1])
    assert a[2].shared_prefix_rows == 0
    same(a, b)


def test_shared_prefix_with_streamed_weights_and_chunked_execution(P):
    """Layer streaming and chunked execution keep the prefix: the first chunk of a layer holds the query's rows and
    saves their q/k/v for the attention of the later chunks."""
    w = synth.make_weights(MID, seed=5)
    tw = P.upload_weights(w, MID.dtype, layers_pinned_host=True)
    req = synth.make_request(replace(MID_WL, query_len=32), 2)
    a, b = both(P, tw, req, 4, SCHEDS[1], stream_weights=True)
    assert a[2].shared_prefix_rows == 32
    same(a, b)
    total = int(req["cand_offsets"][-1]) + 32 * MID_WL.n_candidates
    per_tok = 2 * (MID.hidden + (MID.n_q_heads + 2 * MID.n_kv_heads) * MID.head_dim + MID.n_q_heads * MID.head_dim + MID.ffn)
    budget = 2 * total * MID.hidden * 4 + (total // 3) * per_tok
    for sched in SCHEDS:
        ref = run(P, model(P, P.upload_weights(w, MID.dtype), req, shared_prefix=False), req, 4, sched)
        for div in (3, 7):
            budget = 2 * total * MID.hidden * 4 + (total // div) * per_tok
            c = run(P, model(P, P.upload_weights(w, MID.dtype), req, activation_budget_bytes=budget), req, 4, sched)
            assert c[2].n_chunks_max >= div and c[2].shared_prefix_rows == 32
            same(c, ref)


def test_repeated_requests_of_different_shape_on_one_handle(P, weights):
    """One handle serving prefix and non-prefix requests in turn."""
    _, tw = weights
    reqs = [request(32, [100, 37, 250, 400, 5], 1), request(20, [100, 37, 250], 2), request(64, [1, 2, 3, 500], 3),
            request(32, [100, 37, 250, 400, 5], 1)]
    lens = [np.diff(r["cand_offsets"]) + len(r["query"]) for r in reqs]
    m = P.PrismModel(MID, tw, max(int(l.max()) for l in lens), 8, max(int(l.sum()) for l in lens))
    ref = P.PrismModel(MID, tw, max(int(l.max()) for l in lens), 8, max(int(l.sum()) for l in lens), shared_prefix=False)
    outs = [run(P, m, r, 2, SCHEDS[1]) for r in reqs]
    for r, o in zip(reqs, outs):
        same(o, run(P, ref, r, 2, SCHEDS[1]))
    assert [o[2].shared_prefix_rows for o in outs] == [32, 0, 64, 32]
    assert np.array_equal(outs[0][1].view(np.uint32), outs[3][1].view(np.uint32))
