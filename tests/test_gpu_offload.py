"""-m gpu: dynamic offloading of the hidden states (Sec. 4.3): the hidden states of all sequences live in pinned host
memory and pass through three device chunk buffers.  Where the data lives must never change a result."""
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


def same(a, b):
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1].view(np.uint32), b[1].view(np.uint32))
    assert len(a[2].records) == len(b[2].records)
    for r1, r2 in zip(a[2].records, b[2].records):
        assert np.array_equal(r1.scores, r2.scores) and r1.active_ids == r2.active_ids


def budget_for(lens, chunk_rows, d=1024):
    per_tok = (1024 + 4096 + 2048 + 3072) * 2
    return (3 * d * 4 + per_tok) * chunk_rows


def test_offload_is_result_neutral(P):
    """Several chunk sizes (one long sequence per chunk ... everything in two chunks), with and without streamed
    layer weights, two requests in a row on one handle: bit-identical to the resident handle, fewer device bytes."""
    w = synth.make_weights(MID, seed=5)
    reqs = [synth.make_request(MID_WL, r) for r in range(2)]
    lens = [np.diff(r["cand_offsets"]) + len(r["query"]) for r in reqs]
    big = max(reqs, key=lambda r: r["cand_offsets"][-1])
    base = make_model(P, MID, w, big)
    ref = [run(P, base, r, MID_WL.top_k, MID_WL.schedule) for r in reqs]
    tot = int(max(l.sum() for l in lens))
    for chunk_rows, kw in ((int(max(l.max() for l in lens)) + 20, {}), (tot // 4, {}), (tot // 2 + 300, dict(stream_weights=True))):
        m = make_model(P, MID, w, big, activation_budget_bytes=budget_for(lens, chunk_rows), hidden_offload=True, **kw)
        for i in (0, 1, 0):
            got = run(P, m, reqs[i], MID_WL.top_k, MID_WL.schedule)
            same(got, ref[i])
        assert got[2].n_chunks_max >= 2
        assert got[2].shared_prefix_rows == len(reqs[0]["query"]) == ref[0][2].shared_prefix_rows   # the query rows stay shared
        if not kw:                                                      # (streaming adds its two layer slots)
            assert got[2].workspace_bytes < ref[0][2].workspace_bytes
        m.close()
    base.close()


def test_offload_with_fp32_path_unpruned_and_errors(P):
    wl = synth.workload(0)
    w0 = synth.make_weights(wl.model)
    r0 = synth.make_request(wl, 0)
    lens = np.diff(r0["cand_offsets"]) + len(r0["query"])
    base = make_model(P, wl.model, w0, r0)
    from synth.configs import MODE_NONE, Schedule
    c = wl.model
    per_tok = (c.hidden + (c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim + c.n_q_heads * c.head_dim + c.ffn) * 4
    budget = (3 * c.hidden * 4 + per_tok) * (int(lens.max()) + 8)
    m = make_model(P, wl.model, w0, r0, activation_budget_bytes=budget, hidden_offload=True)
    for sched in (wl.schedule, Schedule(MODE_NONE)):
        a, b = run(P, m, r0, wl.top_k, sched), run(P, base, r0, wl.top_k, sched)
        same(a, b)
    m.close()
    with pytest.raises(P.PrismError) as e:                             # offload without a budget
        make_model(P, wl.model, w0, r0, hidden_offload=True)
    assert e.value.status == -1
    with pytest.raises(P.PrismError) as e:                             # budget below three chunks of one sequence
        make_model(P, wl.model, w0, r0, activation_budget_bytes=(3 * c.hidden * 4 + per_tok) * 4, hidden_offload=True)
    assert e.value.status == -4
    base.close()
