"""-m gpu: prism_select end to end against the oracle (scores, replayed decisions, top-K)."""
import os
from dataclasses import replace

import numpy as np
import pytest

import oracle
import synth
from synth.configs import (MODE_CLUSTER, MODE_FIXED_KEEP, MODE_NONE, DTYPE_BF16, DTYPE_FP32, ModelCfg, Schedule,
                           Workload)

from parity import check_end_to_end, check_replay, check_scores

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL_FP32 = 1e-4      # stated tolerances: fp32 mode
TOL_BF16 = 3e-2      # bf16 mode
GOLD = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module")
def P():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_2510_15620_b200 as pkg
    return pkg


def dev_i32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()


def make_model(P, cfg, w, req, **kw):
    lq = len(req["query"])
    lens = np.diff(req["cand_offsets"]) + lq
    tw = P.upload_weights(w, cfg.dtype, layers_pinned_host=bool(kw.get("stream_weights", False)))
    return P.PrismModel(cfg, tw, max_seq_len=int(lens.max()), max_candidates=len(lens), max_total_tokens=int(lens.sum()), **kw)


def run(P, model, req, k, sched):
    idx, sc, tr = model.select(dev_i32(req["query"]), dev_i32(req["cand_tokens"]), dev_i32(req["cand_offsets"]), k, sched)
    return idx.cpu().numpy(), sc.cpu().numpy(), tr


def layers_scored(cfg, sched):
    return sorted(set(list(sched.probe_layers if sched.mode != MODE_NONE else ()) + [cfg.n_layers]))


# ------------------------------------------------------------------------------------------ cfg0: fp32, exact tolerances
@pytest.fixture(scope="module")
def tiny(P):
    wl = synth.workload(0)
    w = synth.make_weights(wl.model)
    req = synth.make_request(wl, 0)
    S = oracle.score_matrix(req["query"], req["cand_tokens"], req["cand_offsets"], w, wl.model, [1, 2])
    return wl, w, req, S


@pytest.mark.parametrize("sched", [
    None,
    Schedule(MODE_FIXED_KEEP, (1,), (8,)),
    Schedule(MODE_CLUSTER, (1,), cv_threshold=0.5, n_clusters=3),
    Schedule(MODE_CLUSTER, (1,), cv_threshold=0.5, n_clusters=3, select_winners=0),
    Schedule(MODE_CLUSTER, (1,), cv_threshold=1e30),
])
def test_cfg0_fp32_matches_oracle(P, tiny, sched):
    wl, w, req, S = tiny
    model = make_model(P, wl.model, w, req)
    s = sched or Schedule(MODE_NONE)
    idx, sc, tr = run(P, model, req, wl.top_k, sched)
    worst = check_scores(tr, S, TOL_FP32)
    check_replay(tr, idx, sc, wl.n_candidates, wl.top_k, wl.model.n_layers, s)
    verdict = check_end_to_end(tr, idx, S, wl.n_candidates, wl.top_k, wl.model.n_layers, s, TOL_FP32)
    assert verdict in ("identical", "same set", "within tolerance band")
    assert worst < TOL_FP32
    assert model.launch_count > 0
    model.close()


def test_cfg0_other_requests_and_k(P, tiny):
    wl, w, _, _ = tiny
    for r in (1, 2):
        req = synth.make_request(wl, r)
        S = oracle.score_matrix(req["query"], req["cand_tokens"], req["cand_offsets"], w, wl.model, [1, 2])
        model = make_model(P, wl.model, w, req)
        for k in (1, 3, 8, 16, 40):                                    # K > N is not an error
            sched = wl.schedule if k <= 8 else Schedule(MODE_CLUSTER, (1,), cv_threshold=0.2)
            idx, sc, tr = run(P, model, req, k, sched)
            assert len(idx) == min(k, wl.n_candidates)
            check_scores(tr, S, TOL_FP32)
            check_replay(tr, idx, sc, wl.n_candidates, k, wl.model.n_layers, sched)
        model.close()


def test_permutation_and_packing_invariance(P, tiny):
    """Scores follow the candidates when they are permuted, and a candidate scored alone (batch of one)
    gets the score it had inside the packed batch: sequences never see each other."""
    wl, w, req, S = tiny
    model = make_model(P, wl.model, w, req)
    _, _, tr = run(P, model, req, 3, None)
    base = dict(zip(tr.records[-1].active_ids, tr.records[-1].scores))
    perm = np.random.default_rng(1).permutation(wl.n_candidates)
    off = req["cand_offsets"]
    docs = [req["cand_tokens"][off[i]:off[i + 1]] for i in perm]
    req2 = dict(query=req["query"], cand_tokens=np.concatenate(docs),
                cand_offsets=np.concatenate([[0], np.cumsum([len(d) for d in docs])]).astype(np.int32))
    _, _, tr2 = run(P, model, req2, 3, None)
    got = dict(zip(tr2.records[-1].active_ids, tr2.records[-1].scores))
    for new, old in enumerate(perm):
        assert abs(got[new] - base[int(old)]) <= 2e-6
    i = 5
    req1 = dict(query=req["query"], cand_tokens=req["cand_tokens"][off[i]:off[i + 1]],
                cand_offsets=np.array([0, off[i + 1] - off[i]], np.int32))
    _, sc1, _ = run(P, model, req1, 1, None)
    assert abs(sc1[0] - base[i]) <= 2e-6
    model.close()


def test_argument_and_input_errors(P, tiny):
    wl, w, req, _ = tiny
    model = make_model(P, wl.model, w, req)
    q, c, o = dev_i32(req["query"]), dev_i32(req["cand_tokens"]), dev_i32(req["cand_offsets"])
    with pytest.raises(P.PrismError) as e:
        model.select(q, c, o, 0)                                       # K < 1
    assert e.value.status == -1
    with pytest.raises(P.PrismError) as e:
        model.select(q, c, o, 3, Schedule(MODE_CLUSTER, (2,)))         # probe at the last layer
    assert e.value.status == -1
    with pytest.raises(P.PrismError) as e:
        model.select(q, c, o, 3, Schedule(MODE_FIXED_KEEP, (1,), (2,)))  # keep < K
    assert e.value.status == -1
    bad = req["cand_tokens"].copy()
    bad[7] = wl.model.vocab + 5
    with pytest.raises(P.PrismError) as e:
        model.select(q, dev_i32(bad), o, 3)
    assert e.value.status == -3                                        # found on the device, no trap
    off = req["cand_offsets"].copy()
    off[3], off[4] = off[4], off[3]
    with pytest.raises(P.PrismError) as e:
        model.select(q, c, dev_i32(off), 3)
    assert e.value.status == -3
    big = np.concatenate([req["cand_tokens"], req["cand_tokens"]])
    off2 = req["cand_offsets"].copy()
    off2[-1] = len(big)
    with pytest.raises(P.PrismError) as e:
        model.select(q, dev_i32(big), dev_i32(off2), 3)
    assert e.value.status == -2                                        # beyond the handle's maxima
    idx, sc, tr = run(P, model, req, 3, wl.schedule)                   # the handle is still usable
    assert len(idx) == 3
    # N = 0 is an empty result, not an error
    idx, sc, _ = model.select(q, c, dev_i32(np.array([0])), 3)
    assert len(idx) == 0
    # a null cand_tokens with document tokens announced by the offsets: refused on the host, nothing launched
    before = model.launch_count
    out_i, out_s = dev_i32(np.zeros(3)), torch.zeros(3, device="cuda")
    with pytest.raises(P.PrismError) as e:
        model._call(P.lib().prism_select, q.data_ptr(), q.numel(), None, o.data_ptr(), len(req["cand_offsets"]) - 1, 3,
                    None, out_i.data_ptr(), out_s.data_ptr(), False, torch.cuda.current_stream().cuda_stream)
    assert e.value.status == -1 and model.launch_count == before
    # ... and allowed when every document is empty (each sequence is the query alone)
    idx, sc, _ = model._call(P.lib().prism_select, q.data_ptr(), q.numel(), None, dev_i32(np.zeros(5)).data_ptr(), 4, 3,
                             None, out_i.data_ptr(), out_s.data_ptr(), False, torch.cuda.current_stream().cuda_stream), None, None
    assert idx[0] == 3 and out_i.cpu().tolist() == [0, 1, 2]           # four equal sequences: ties go to the lower index
    model.close()


def test_select_host_equals_select(P, tiny):
    wl, w, req, _ = tiny
    model = make_model(P, wl.model, w, req)
    idx, sc, _ = run(P, model, req, 3, wl.schedule)
    hidx, hsc, _ = model.select_host(req["query"], req["cand_tokens"], req["cand_offsets"], 3, wl.schedule)
    assert np.array_equal(idx, hidx) and np.array_equal(sc, hsc)
    model.close()


def test_runs_are_bitwise_repeatable(P, tiny):
    wl, w, req, _ = tiny
    model = make_model(P, wl.model, w, req)
    a = run(P, model, req, 3, Schedule(MODE_CLUSTER, (1,), cv_threshold=0.1))
    b = run(P, model, req, 3, Schedule(MODE_CLUSTER, (1,), cv_threshold=0.1))
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    for r1, r2 in zip(a[2].records, b[2].records):
        assert np.array_equal(r1.scores, r2.scores)
    model.close()


def test_threshold_calibration_follows_the_oracle_loop(P, tiny):
    """Sec. 4.1 auto-calibration: the library's loop (pruned run, sampled unpruned re-run, precision,
    multiplicative adjustment) must walk the same threshold trajectory as the oracle's loop fed with the
    oracle's own scores, request after request."""
    import ctypes
    from oracle.calibrate import Calibrator as OCal, calibrated_step
    wl, w, _, _ = tiny
    cfg = wl.model
    sched = Schedule(MODE_CLUSTER, (1,), cv_threshold=0.0, n_clusters=3)
    reqs = [synth.make_request(wl, r) for r in range(10)]
    lens = [np.diff(r["cand_offsets"]) + wl.query_len for r in reqs]
    tw = P.upload_weights(w, cfg.dtype)
    model = P.PrismModel(cfg, tw, int(max(l.max() for l in lens)), wl.n_candidates, int(max(l.sum() for l in lens)))
    kw = dict(threshold=0.05, target_precision=0.99, raise_factor=2.0, lower_factor=0.75, min_threshold=0.01,
              max_threshold=64.0, sample_every=1, window=2)
    cal = P.Calibrator(**kw)
    ocal = OCal(**kw)
    k = 4
    for r in reqs:
        S = oracle.score_matrix(r["query"], r["cand_tokens"], r["cand_offsets"], w, cfg, [1, 2])

        def orun(thr, S=S, r=r):
            s = Schedule(MODE_NONE) if thr is None else Schedule(MODE_CLUSTER, (1,), cv_threshold=thr, n_clusters=3)
            return oracle.oracle_select(r["query"], r["cand_tokens"], r["cand_offsets"], k, w, cfg, s, S=S).topk_idx
        expect = calibrated_step(ocal, orun)
        idx, _ = model.select_calibrated(dev_i32(r["query"]), dev_i32(r["cand_tokens"]), dev_i32(r["cand_offsets"]), k, sched, cal)
        assert sorted(idx.cpu().numpy().tolist()) == sorted(expect)
        assert cal.threshold == ocal.threshold and cal.last_precision == ocal.last_precision
        assert (cal.n_requests, cal.n_sampled, cal.n_adjustments) == (ocal.n_requests, ocal.n_sampled, ocal.n_adjustments)
    assert ocal.n_adjustments == 5 and len({ocal.threshold, 0.05}) == 2      # the threshold really moved
    bad = P.Calibrator(**dict(kw, raise_factor=0.5))
    with pytest.raises(P.PrismError) as e:
        model.select_calibrated(dev_i32(reqs[0]["query"]), dev_i32(reqs[0]["cand_tokens"]), dev_i32(reqs[0]["cand_offsets"]), k, sched, bad)
    assert e.value.status == -1
    model.close()


# ------------------------------------------------------------------------------------------ bf16, mid-size (tensor-core path)
MID = ModelCfg(n_layers=6, hidden=1024, n_q_heads=16, n_kv_heads=8, head_dim=128, ffn=3072, vocab=4096,
               rope_theta=1e6, qk_norm=1, dtype=DTYPE_BF16, yes_id=3, no_id=4)
MID_WL = Workload("mid_bf16", MID, 24, 4, 16, ("uniform", 20, 260, 20, 260),
                  Schedule(MODE_CLUSTER, (2, 4), cv_threshold=0.3), cfg_index=7)


@pytest.fixture(scope="module")
def mid(P):
    w = synth.make_weights(MID, seed=5)
    req = synth.make_request(MID_WL, 0)
    S = oracle.score_matrix(req["query"], req["cand_tokens"], req["cand_offsets"], w, MID, [2, 4, 6])
    return w, req, S


@pytest.mark.parametrize("gemm_impl,attn_impl", [(1, 1), (0, 1), (1, 0), (0, 0), (3, 0)])
def test_bf16_paths_match_oracle(P, mid, gemm_impl, attn_impl):
    w, req, S = mid
    model = make_model(P, MID, w, req, gemm_impl=gemm_impl, attention_impl=attn_impl)
    for sched in (Schedule(MODE_NONE), MID_WL.schedule, replace(MID_WL.schedule, select_winners=0)):
        idx, sc, tr = run(P, model, req, MID_WL.top_k, sched)
        check_scores(tr, S, TOL_BF16)
        check_replay(tr, idx, sc, MID_WL.n_candidates, MID_WL.top_k, MID.n_layers, sched)
        check_end_to_end(tr, idx, S, MID_WL.n_candidates, MID_WL.top_k, MID.n_layers, sched, TOL_BF16)
    model.close()


def test_bidirectional_attention_end_to_end(P, mid):
    """causal = 0 (encoder-style attention) through every attention implementation against the oracle."""
    w, req, _ = mid
    cfg = replace(MID, causal=0, n_layers=3)
    wb = dict(w, layers=w["layers"][:3])
    S = oracle.score_matrix(req["query"], req["cand_tokens"], req["cand_offsets"], wb, cfg, [1, 2, 3])
    S_causal = oracle.score_matrix(req["query"], req["cand_tokens"], req["cand_offsets"], wb, replace(cfg, causal=1), [3],
                                   candidates=[0, 1])
    assert abs(S_causal[3][0] - S[3][0]) > 1e-3                       # the flag matters
    sched = Schedule(MODE_CLUSTER, (1, 2), cv_threshold=1e30)
    for attn_impl in (0, 1, 2):
        model = make_model(P, cfg, wb, req, attention_impl=attn_impl)
        idx, sc, tr = run(P, model, req, MID_WL.top_k, sched)
        check_scores(tr, S, TOL_BF16)
        check_replay(tr, idx, sc, MID_WL.n_candidates, MID_WL.top_k, cfg.n_layers, sched)
        model.close()


def test_chunked_and_streamed_are_result_neutral(P, mid):
    """Chunked execution (Sec. 4.3) and overlapped layer streaming (Sec. 4.2) change where data lives
    and when it moves, never the values."""
    w, req, S = mid
    base_model = make_model(P, MID, w, req)
    base = run(P, base_model, req, MID_WL.top_k, MID_WL.schedule)
    assert base[2].n_chunks_max == 1
    lq = len(req["query"])
    lens = np.diff(req["cand_offsets"]) + lq
    per_tok = (1024 + 4096 + 2048 + 3072) * 2
    budget = 2 * int(lens.sum()) * 1024 * 4 + per_tok * (int(lens.max()) + 50)     # about one long sequence per chunk
    for kw in (dict(activation_budget_bytes=budget), dict(stream_weights=True),
               dict(activation_budget_bytes=budget, stream_weights=True)):
        m = make_model(P, MID, w, req, **kw)
        for _ in range(2):                                             # a second request reuses the slots
            got = run(P, m, req, MID_WL.top_k, MID_WL.schedule)
            assert np.array_equal(got[0], base[0]) and np.array_equal(got[1], base[1])
            for r1, r2 in zip(got[2].records, base[2].records):
                assert np.array_equal(r1.scores, r2.scores) and r1.active_ids == r2.active_ids
        if "activation_budget_bytes" in kw:
            assert got[2].n_chunks_max > 3
        m.close()
    with pytest.raises(P.PrismError) as e:                             # budget below hidden + one sequence
        make_model(P, MID, w, req, activation_budget_bytes=2 * int(lens.sum()) * 1024 * 4 + 1000)
    assert e.value.status == -4
    base_model.close()


def test_duplicate_candidates_tie_exactly(P, mid):
    w, req, _ = mid
    off = req["cand_offsets"]
    docs = [req["cand_tokens"][off[i]:off[i + 1]] for i in range(8)]
    docs = docs + [docs[2], docs[5], docs[2]]
    req2 = dict(query=req["query"], cand_tokens=np.concatenate(docs),
                cand_offsets=np.concatenate([[0], np.cumsum([len(d) for d in docs])]).astype(np.int32))
    model = make_model(P, MID, w, req2)
    _, _, tr = run(P, model, req2, 3, Schedule(MODE_CLUSTER, (2, 4), cv_threshold=1e30))
    for rec in tr.records:
        s = dict(zip(rec.active_ids, rec.scores))
        assert s[2] == s[8] == s[10] and s[5] == s[9]                  # bit-identical, wherever they sit
    model.close()


# ------------------------------------------------------------------------------------------ full-size workload 1 (the bench configuration)
def _gold_scores(name, r):
    path = os.path.join(GOLD, f"{name}_scores_r{r}.txt")
    if not os.path.exists(path):
        return None
    S = {}
    for line in open(path):
        if line.startswith("#"):
            continue
        p = line.split()
        S[int(p[0])] = np.array([float(x) for x in p[1:]])
    return S


@pytest.mark.parametrize("r", [0, 1, 2])
def test_cfg1_full_size_in_bench_configuration(P, r):
    """Qwen3-0.6B-shaped, 100 candidates, the launch configuration bench.py times, request seeds 0, 1 and 2.  All
    candidates are checked against the stored oracle scores of the request (tests/golden/, written by
    make_scores.py); three sampled candidates are also forwarded by the oracle on the spot."""
    wl = synth.workload(1)
    cfg = wl.model
    w = synth.make_weights(cfg, wl.weight_seed)
    req = synth.make_request(wl, r)
    model = make_model(P, cfg, w, req)
    sched = wl.schedule
    # unpruned first: every candidate reaches the last layer
    idx0, sc0, tr0 = run(P, model, req, wl.top_k, Schedule(MODE_CLUSTER, sched.probe_layers, cv_threshold=1e30))
    idx, sc, tr = run(P, model, req, wl.top_k, sched)
    check_replay(tr0, idx0, sc0, wl.n_candidates, wl.top_k, cfg.n_layers, Schedule(MODE_CLUSTER, sched.probe_layers, cv_threshold=1e30))
    check_replay(tr, idx, sc, wl.n_candidates, wl.top_k, cfg.n_layers, sched)
    sample = [3, 41, 77]
    layers = layers_scored(cfg, sched)
    Ss = oracle.score_matrix(req["query"], req["cand_tokens"], req["cand_offsets"], w, cfg, layers, candidates=sample)
    worst = check_scores(tr0, Ss, TOL_BF16, ids_known=sample)
    check_scores(tr, Ss, TOL_BF16, ids_known=sample)
    S = _gold_scores(wl.name, r)
    assert S is not None, "stored oracle scores of this request are missing"
    if S is not None:
        for j, c in enumerate(sample):                                  # the stored file is what the oracle computes
            for l in layers:
                assert abs(S[l][c] - Ss[l][j]) < 1e-9
        worst = max(worst, check_scores(tr0, S, TOL_BF16))
        check_scores(tr, S, TOL_BF16)
        verdict = check_end_to_end(tr, idx, S, wl.n_candidates, wl.top_k, cfg.n_layers, sched, TOL_BF16)
        ref = oracle.replay_select(lambda layer, a: np.asarray(S[layer])[np.asarray(a, np.int64)].astype(np.float32),
                                   wl.n_candidates, wl.top_k, cfg.n_layers, sched)
        print(f"cfg1 request {r}: pruned run vs the oracle's own decisions: {verdict}, overlap@{wl.top_k} "
              f"{len(set(ref.topk_idx) & set(map(int, idx)))}/{len(idx)}")
        # tr0 was traced under the never-firing schedule: the walk has to be given that schedule (its probes), not NONE
        check_end_to_end(tr0, idx0, S, wl.n_candidates, wl.top_k, cfg.n_layers,
                         Schedule(MODE_CLUSTER, sched.probe_layers, cv_threshold=1e30), TOL_BF16)
    print(f"cfg1 request {r}: worst |score diff| vs oracle: {worst:.4g}; pruned run stopped after layer {tr.layers_run}; "
          f"tokens per layer {tr.tokens_per_layer}")
    assert any(rec.fired for rec in tr.records)
    model.close()


def test_maximum_candidate_count_end_to_end(P):
    """N = 4096 (PRISM_MAX_CANDIDATES) short candidates through a small bf16 model: every step that scales with N
    (packing, probe, ranking and partition on a cluster of blocks, compaction) against the oracle."""
    cfg = ModelCfg(n_layers=3, hidden=256, n_q_heads=2, n_kv_heads=1, head_dim=128, ffn=256, vocab=512, rope_theta=1e4,
                   qk_norm=1, dtype=DTYPE_BF16, yes_id=3, no_id=4)
    wl = Workload("max_n_bf16", cfg, 4096, 7, 8, ("uniform", 1, 40, 1, 40), Schedule(MODE_CLUSTER, (1, 2), cv_threshold=0.2),
                  cfg_index=13)
    w = synth.make_weights(cfg, seed=9)
    req = synth.make_request(wl, 0)
    S = oracle.score_matrix(req["query"], req["cand_tokens"], req["cand_offsets"], w, cfg, [1, 2, 3])
    model = make_model(P, cfg, w, req)
    for sched in (wl.schedule, Schedule(MODE_NONE)):
        idx, sc, tr = run(P, model, req, wl.top_k, sched)
        assert tr.records[0].n_active_before == 4096
        check_scores(tr, S, TOL_BF16)
        check_replay(tr, idx, sc, wl.n_candidates, wl.top_k, cfg.n_layers, sched)
        check_end_to_end(tr, idx, S, wl.n_candidates, wl.top_k, cfg.n_layers, sched, TOL_BF16)
    assert tr.shared_prefix_rows == 8
    model.close()
