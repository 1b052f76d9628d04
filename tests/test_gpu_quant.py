"""-m gpu: W4A16 weights (Sec. 6.1, the quantised arm).  The dequantisation kernel bit for bit against the oracle;
a W4 handle bit for bit against a plain handle that is given the dequantised matrices; the selection against the
oracle forward on those matrices; resident and streamed."""
from dataclasses import replace

import numpy as np
import pytest

import oracle
import synth
from synth.configs import MODE_CLUSTER, MODE_NONE, Schedule
from synth.weights import bf16_bits

from parity import check_end_to_end, check_replay, check_scores
from test_gpu_select import MID, MID_WL, TOL_BF16, run

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_2510_15620_b200 as pkg
    return pkg


@pytest.mark.parametrize("n,k,g", [(1, 32, 32), (24, 256, 64), (300, 1024, 128), (3072, 1024, 128), (1000, 3072, 32)])
def test_dequant_kernel_is_bit_exact(P, n, k, g):
    rng = np.random.default_rng(n + k + g)
    w = (rng.normal(size=(n, k)) * 0.02).astype(np.float32)
    w[0, :g] = 0.0                                     # an all-zero group (scale falls back to 1)
    blob = synth.pack_matrix(*synth.quantize_matrix(w, g), g)
    out = torch.zeros(n, k, dtype=torch.bfloat16, device="cuda")
    P.ops.prism_op_dequant_w4(torch.from_numpy(blob).cuda(), n, k, g, out)
    ref = oracle.dequantize_w4(blob, n, k, g)
    got = out.view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(got, bf16_bits(ref.astype(np.float32)))


@pytest.fixture(scope="module")
def quantised(P):
    w = synth.make_weights(MID, seed=5)
    wq = synth.quantize_weights(w, group=128)
    wd = oracle.dequantize_weights(wq, MID, 128)
    req = synth.make_request(MID_WL, 0)
    return w, wq, wd, req


def model(P, w, req, **kw):
    lens = np.diff(req["cand_offsets"]) + len(req["query"])
    tw = P.upload_weights(w, MID.dtype, layers_pinned_host=bool(kw.get("stream_weights", False)))
    return P.PrismModel(MID, tw, int(lens.max()), len(lens), int(lens.sum()), **kw)


def same(a, b):
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1].view(np.uint32), b[1].view(np.uint32))
    assert len(a[2].records) == len(b[2].records)
    for r1, r2 in zip(a[2].records, b[2].records):
        assert np.array_equal(r1.scores.view(np.uint32), r2.scores.view(np.uint32)) and r1.active_ids == r2.active_ids


@pytest.mark.parametrize("kw", [dict(), dict(stream_weights=True), dict(gemm_impl=1, attention_impl=1)],
                         ids=["resident", "streamed", "cuda-cores"])
def test_w4_handle_equals_plain_handle_on_the_dequantised_matrices(P, quantised, kw):
    _, wq, wd, req = quantised
    wd32 = {k: v for k, v in wd.items() if k != "layers"}
    wd32["layers"] = [{k: np.asarray(v, np.float32) for k, v in l.items()} for l in wd["layers"]]
    plain = model(P, wd32, req, **kw)
    q4 = model(P, wq, req, weight_format=P.PRISM_WFMT_W4, quant_group=128, **kw)
    for sched in (Schedule(MODE_NONE), MID_WL.schedule):
        same(run(P, q4, req, MID_WL.top_k, sched), run(P, plain, req, MID_WL.top_k, sched))
    # a second request on the same handle (the scratch is rebuilt layer by layer every time)
    req2 = synth.make_request(MID_WL, 1)
    lens2 = np.diff(req2["cand_offsets"]) + len(req2["query"])
    if int(lens2.sum()) <= int((np.diff(req["cand_offsets"]) + len(req["query"])).sum()) and int(lens2.max()) <= int((np.diff(req["cand_offsets"]) + len(req["query"])).max()):
        same(run(P, q4, req2, MID_WL.top_k, MID_WL.schedule), run(P, plain, req2, MID_WL.top_k, MID_WL.schedule))
    plain.close()
    q4.close()


def test_w4_selection_matches_the_oracle_on_the_dequantised_model(P, quantised):
    w, wq, wd, req = quantised
    S = oracle.score_matrix(req["query"], req["cand_tokens"], req["cand_offsets"], wd, MID, [2, 4, 6])
    S_plain = oracle.score_matrix(req["query"], req["cand_tokens"], req["cand_offsets"], w, MID, [6], candidates=[0, 1, 2])
    assert np.max(np.abs(S_plain[6] - S[6][:3])) > 1e-3          # quantisation changed the model
    m = model(P, wq, req, weight_format=P.PRISM_WFMT_W4, quant_group=128)
    for sched in (Schedule(MODE_NONE), MID_WL.schedule):
        idx, sc, tr = run(P, m, req, MID_WL.top_k, sched)
        check_scores(tr, S, TOL_BF16)
        check_replay(tr, idx, sc, MID_WL.n_candidates, MID_WL.top_k, MID.n_layers, sched)
        check_end_to_end(tr, idx, S, MID_WL.n_candidates, MID_WL.top_k, MID.n_layers, sched, TOL_BF16)
    m.close()


def test_w4_rejects_bad_configurations(P, quantised):
    _, wq, _, req = quantised
    with pytest.raises(P.PrismError) as e:
        model(P, wq, req, weight_format=P.PRISM_WFMT_W4, quant_group=48)
    assert e.value.status == -1


def test_w4_encoder_handle_equals_plain_handle_on_the_dequantised_matrices(P):
    from test_gpu_encoder import ENC_MID, ENC_MID_WL
    cfg, wl = ENC_MID, ENC_MID_WL
    w = synth.make_weights(cfg, seed=5)
    wq = synth.quantize_weights(w, group=64)
    wd = oracle.dequantize_weights(wq, cfg, 64)
    wd32 = {k: v for k, v in wd.items() if k != "layers"}
    wd32["layers"] = [{k: np.asarray(v, np.float32) for k, v in l.items()} for l in wd["layers"]]
    req = synth.make_request(wl, 0)
    lens = np.diff(req["cand_offsets"]) + len(req["query"])
    mk = lambda ww, **kw: P.PrismModel(cfg, P.upload_weights(ww, cfg.dtype, layers_pinned_host=bool(kw.get("stream_weights", False))),
                                       int(lens.max()), len(lens), int(lens.sum()), **kw)
    plain = mk(wd32)
    ref = run(P, plain, req, wl.top_k, wl.schedule)
    for kw in (dict(), dict(stream_weights=True)):
        q4 = mk(wq, weight_format=P.PRISM_WFMT_W4, quant_group=64, **kw)
        same(run(P, q4, req, wl.top_k, wl.schedule), ref)
        q4.close()
    S = oracle.score_matrix(req["query"], req["cand_tokens"], req["cand_offsets"], wd, cfg, [2, 4, 5])
    check_scores(ref[2], S, TOL_BF16)
    plain.close()
