"""-m gpu: the large workloads (4B-, 8B-shaped and the 1000-candidate stress case) at full size.

The oracle cannot forward these batches in test time, so its scores are stored under tests/golden/ (written by
tests/golden/make_scores.py, which calls only the oracle and the input generators): every candidate of the 4B-shaped
and the stress request, and the candidates named in the file's header for the 8B-shaped one.  Every integer outcome
is checked by replaying the oracle's rule on the traced scores (exact); every score of every stored candidate is
compared with the oracle's; and where all candidates are stored the oracle's rule on the oracle's scores is compared
with the CUDA result end to end."""
import gc
import os

import numpy as np
import pytest

import synth
from synth.configs import MODE_CLUSTER, Schedule

import oracle

from parity import check_end_to_end, check_replay, check_scores

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL_BF16 = 3e-2
GOLD = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module")
def P():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_2510_15620_b200 as pkg
    return pkg


def _gold(name):
    """(S, ids) of a stored oracle score file: S[layer] over the file's columns, ids[j] the candidate of column j."""
    path = os.path.join(GOLD, name)
    assert os.path.exists(path), f"{name} is missing: write it with tests/golden/make_scores.py"
    S, ids = {}, None
    for line in open(path):
        if line.startswith("#"):
            if line.startswith("# ids"):
                ids = [int(x) for x in line.split()[2:]]
            continue
        p = line.split()
        S[int(p[0])] = np.array([float(x) for x in p[1:]])
    assert ids is not None and all(len(v) == len(ids) for v in S.values())
    return S, ids


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()


def _bf16_storage_noise(exact_name, bf16_name):
    """RMS and maximum, over the candidates of the second file and all scored layers, of how far the ORACLE's own
    scores move when its stored activations are rounded to bfloat16 at the points where the bf16 precision contract
    stores them (same fp64 arithmetic otherwise): the deviation that any bf16 evaluation of this model carries."""
    a, ida = _gold(exact_name)
    b, idb = _gold(bf16_name)
    col = {c: j for j, c in enumerate(ida)}
    d = np.concatenate([b[l] - a[l][[col[c] for c in idb]] for l in sorted(b)])
    return float(np.sqrt(np.mean(d * d))), float(np.max(np.abs(d))), len(idb)


def _exact_file(index, r):
    return GOLD_FILES[index][0].replace("_r0.txt", f"_r{r}.txt")


def _tolerance(index):
    """The score tolerance of a workload.  3e-2 is the stated bf16 tolerance and holds for the 0.6B-shaped workloads.
    For the 36-layer 4B- and 8B-shaped models the oracle's own bf16-storage noise (measured on 32 length-stratified
    candidates, 8 scored layers each) has an RMS of 0.03 - 0.04, so no bf16 evaluation can stay within 3e-2 on every
    score.  There the deviation is treated as what it is, noise: no score may be further from the oracle than
    SIGMAS_MAX times the oracle's own noise RMS, and the RMS deviation of the CUDA path over all stored candidates may
    not exceed RMS_RATIO_MAX times it, nor their 99th percentile P99_SIGMAS_MAX times it (the per-score bound is loose
    by construction: the largest of 800 - 1600 heavy-tailed deviations, which moved between 3.7 and 5.5 sigma when a
    quarter of the attention kernel's exponentials changed from a cubic to ex2.approx; the RMS and percentile bounds
    are the ones that would catch an arithmetic fault)."""
    exact, bf16 = GOLD_FILES[index]
    sigma, worst, n = _bf16_storage_noise(exact, bf16)
    return max(TOL_BF16, SIGMAS_MAX * sigma), sigma, worst, n


SIGMAS_MAX = 6.0
RMS_RATIO_MAX = 1.5
P99_SIGMAS_MAX = 4.0
GOLD_FILES = {
    2: ("cfg2_qwen3_4b_scores_r0.txt", "cfg2_qwen3_4b_scores_bf16act_r0_s32.txt"),
    3: ("cfg3_qwen3_8b_streamed_scores_r0.txt", "cfg3_qwen3_8b_streamed_scores_bf16act_r0_s32.txt"),
    4: ("cfg4_stress_0p6b_scores_r0.txt", "cfg4_stress_0p6b_scores_bf16act_r0_s16.txt"),
}


def _score_stats(tr, S, ids):
    """RMS and maximum of (CUDA score - oracle score) over every traced score of a stored candidate."""
    col = {c: j for j, c in enumerate(ids)}
    d = [float(s) - float(S[rec.layer][col[int(i)]]) for rec in tr.records for i, s in zip(rec.active_ids, rec.scores)
         if int(i) in col]
    d = np.abs(np.asarray(d))
    return float(np.sqrt(np.mean(d * d))), float(np.max(d)), len(d), float(np.percentile(d, 99))


def _run_workload(P, index, budgets=(None,), r=0):
    """Runs request 0 of the workload at full size and checks it: decisions replayed exactly, every score of every
    stored candidate within the workload's tolerance, and -- where the oracle's scores of ALL candidates are stored --
    the oracle's rule on the oracle's scores against the CUDA result (identical, or different only where oracle
    scores lie within the tolerance of a cut)."""
    wl = synth.workload(index)
    cfg = wl.model
    req = synth.make_request(wl, r)
    lens = np.diff(req["cand_offsets"]) + wl.query_len
    w = synth.make_weights(cfg, wl.weight_seed)
    tw = P.upload_weights(w, cfg.dtype, layers_pinned_host=bool(wl.stream_weights))
    del w
    gc.collect()
    S, ids = _gold(_exact_file(index, r))
    tol, sigma, worst_oracle, n_noise = _tolerance(index)
    print(f"{wl.name} request {r}: oracle exact vs bf16-storage oracle on {n_noise} candidates of request 0: rms {sigma:.4f}, max {worst_oracle:.4f}; "
          f"tolerance {tol:.4f}; {len(ids)} of {wl.n_candidates} candidates stored")
    results = []
    for budget in budgets:
        b = wl.activation_budget_bytes if budget is None else budget
        model = P.PrismModel(cfg, tw, int(lens.max()), len(lens), int(lens.sum()), activation_budget_bytes=b,
                             stream_weights=bool(wl.stream_weights))
        q, c, o = _dev(req["query"]), _dev(req["cand_tokens"]), _dev(req["cand_offsets"])
        idx, sc, tr = model.select(q, c, o, wl.top_k, wl.schedule)
        idx, sc = idx.cpu().numpy(), sc.cpu().numpy()
        check_replay(tr, idx, sc, wl.n_candidates, wl.top_k, cfg.n_layers, wl.schedule)
        check_scores(tr, S, tol, ids_known=ids)
        verdict = "not run (scores of a sample only)"
        if len(ids) == wl.n_candidates:
            verdict = check_end_to_end(tr, idx, S, wl.n_candidates, wl.top_k, cfg.n_layers, wl.schedule, tol)
            assert verdict in ("identical", "same set", "within tolerance band")
            ref = oracle.replay_select(lambda layer, a: np.asarray(S[layer])[np.asarray(a, np.int64)].astype(np.float32),
                                       wl.n_candidates, wl.top_k, cfg.n_layers, wl.schedule)
            verdict += f", overlap@{wl.top_k} with the oracle's top-K {len(set(ref.topk_idx) & set(map(int, idx)))}/{len(idx)}"
        rms, worst, n_sc, _ = _score_stats(tr, S, ids)
        print(f"{wl.name}: budget {b}, chunks/layer <= {tr.n_chunks_max}, stopped after layer {tr.layers_run}, "
              f"active per probe {[r.n_active_before for r in tr.records]}, pruned run: {n_sc} scores of stored candidates, "
              f"rms {rms:.4f}, max {worst:.4f}; end to end: {verdict}; workspace {tr.workspace_bytes / 2**30:.2f} GiB")
        results.append((idx, sc, tr))
        if budget is None:
            # every stored candidate at every probe (the pruned run only scores survivors): the same schedule with a
            # threshold that never fires
            never = Schedule(MODE_CLUSTER, wl.schedule.probe_layers, cv_threshold=1e30)
            _, _, tr_all = model.select(q, c, o, wl.top_k, never)
            check_scores(tr_all, S, tol, ids_known=ids)
            rms, worst, n_sc, p99 = _score_stats(tr_all, S, ids)
            print(f"{wl.name}: all probes, nothing pruned: {n_sc} scores, rms {rms:.4f} (oracle's own bf16-storage noise "
                  f"{sigma:.4f}), 99th percentile {p99:.4f} = {p99 / sigma:.2f} sigma, max {worst:.4f} = {worst / sigma:.2f} sigma, "
                  f"max relative to the layer's score rms {max(_relative(tr_all, S, ids)):.4f}")
            if tol > TOL_BF16:
                assert rms <= RMS_RATIO_MAX * sigma, (rms, sigma)
                assert p99 <= P99_SIGMAS_MAX * sigma, (p99, sigma)
        model.close()
    return wl, req, results


def _relative(tr, S, ids):
    col = {c: j for j, c in enumerate(ids)}
    out = []
    for rec in tr.records:
        d = [abs(float(s) - float(S[rec.layer][col[int(i)]])) for i, s in zip(rec.active_ids, rec.scores) if int(i) in col]
        if d:
            out.append(max(d) / float(np.sqrt(np.mean(S[rec.layer] ** 2))))
    return out


def test_cfg4_stress_thousand_candidates_with_duplicates(P):
    wl, req, res = _run_workload(P, 4)
    idx, sc, tr = res[0]
    assert tr.records[0].n_active_before == 1000 and any(r.fired for r in tr.records)
    # exact duplicates (30 % of the candidates) must tie bit for bit at every probe, wherever they sit
    off = req["cand_offsets"]
    key = {}
    for i in range(wl.n_candidates):
        key.setdefault(req["cand_tokens"][off[i]:off[i + 1]].tobytes(), []).append(i)
    groups = [g for g in key.values() if len(g) > 1]
    assert len(groups) > 100
    for rec in tr.records:
        s = dict(zip(rec.active_ids, rec.scores))
        for g in groups:
            vals = {np.float32(s[i]).tobytes() for i in g if i in s}
            assert len(vals) <= 1
            present = [i in s for i in g]
            assert all(present) or not any(present)          # duplicates are always routed together


def test_cfg2_qwen3_4b_shaped(P):
    _, _, res = _run_workload(P, 2)
    assert any(r.fired for r in res[0][2].records)


def test_cfg3_qwen3_8b_streamed_and_chunked(P):
    """Weights stream layer by layer from pinned host memory; the 16 GB activation budget of the workload
    and a tighter one that forces several chunks per layer must give identical results."""
    wl = synth.workload(3)
    req = synth.make_request(wl, 0)
    total = int((np.diff(req["cand_offsets"]) + wl.query_len).sum())
    hidden = 2 * total * wl.model.hidden * 4
    per_tok = (4096 + 6144 + 4096 + 12288) * 2
    tight = hidden + per_tok * 30000
    _, _, res = _run_workload(P, 3, budgets=(None, tight))
    a, b = res
    assert b[2].n_chunks_max >= 4 and a[2].n_chunks_max < b[2].n_chunks_max
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    for r1, r2 in zip(a[2].records, b[2].records):
        assert np.array_equal(r1.scores, r2.scores) and r1.active_ids == r2.active_ids


@pytest.mark.parametrize("index", [2, 3, 4])
def test_second_request_of_the_large_workloads(P, index):
    """Request seed 1 of the same workloads against its own stored oracle scores (every candidate): scores, replayed
    decisions and the end-to-end check, as for request 0."""
    _, _, res = _run_workload(P, index, r=1)
    assert any(rec.fired for rec in res[0][2].records)
