"""-m gpu: the encoder-only reranker stack (Sec. 6.1, Table 1) through the C ABI against the encoder oracle: its
kernels one by one (embedding sum, LayerNorm, biased GEMM epilogues with the exact GELU, head_dim-64 tensor-core
attention, the first-token classifier probe) and prism_select end to end in fp32 (1e-4) and bf16 (3e-2)."""
from dataclasses import replace

import numpy as np
import pytest

import oracle
import synth
from synth.configs import (ARCH_ENCODER, DTYPE_BF16, DTYPE_FP32, MODE_CLUSTER, MODE_FIXED_KEEP, MODE_NONE, ModelCfg,
                           Schedule, Workload)
from synth.weights import round_to_bf16

from parity import check_end_to_end, check_replay, check_scores
from test_gpu_select import TOL_BF16, TOL_FP32, dev_i32, run

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu
FP32, BF16, AUTO, SIMT, SOLO = 0, 1, 0, 1, 3


@pytest.fixture(scope="module")
def P():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_2510_15620_b200 as pkg
    return pkg


def dev(a, dt=torch.float32):
    return torch.from_numpy(np.ascontiguousarray(a)).to("cuda").to(dt)


# ------------------------------------------------------------------------------------------ kernels
@pytest.mark.parametrize("dtype", [FP32, BF16])
@pytest.mark.parametrize("rows,d", [(1, 8), (37, 256), (300, 1024), (77, 2048), (19, 2560), (9, 8192)])
def test_layernorm(P, dtype, rows, d):
    """Warp-per-row (d <= 2048) and block-per-row kernels, in place plus the typed copy; rows with a large common
    offset check that the variance is taken about the mean."""
    rng = np.random.default_rng(rows + d)
    x = (rng.normal(size=(rows, d)) * 3 + 100.0 * rng.normal(size=(rows, 1))).astype(np.float32)
    g = (1 + 0.1 * rng.normal(size=d)).astype(np.float32)
    b = (0.1 * rng.normal(size=d)).astype(np.float32)
    tx = dev(x)
    out = torch.zeros(rows, d, dtype=torch.bfloat16 if dtype == BF16 else torch.float32, device="cuda")
    P.ops.prism_op_layernorm(tx, dev(g), dev(b), dtype, 1e-5, out)
    ref = oracle.layernorm(x.astype(np.float64), g.astype(np.float64), b.astype(np.float64), 1e-5)
    got = tx.cpu().numpy()
    assert np.max(np.abs(got - ref)) < 2e-4                      # fp32 sums over rows offset by ~100
    if dtype == BF16:
        assert np.array_equal(out.float().cpu().numpy(), round_to_bf16(got))      # the copy is the rounded in-place value
    else:
        assert np.array_equal(out.cpu().numpy(), got)


@pytest.mark.parametrize("dtype", [FP32, BF16])
def test_embed_encoder(P, dtype):
    rng = np.random.default_rng(3)
    v, mp, d, n = 50, 40, 64, 33
    tab, ptab, ty = (rng.normal(size=s).astype(np.float32) for s in ((v, d), (mp, d), (d,)))
    if dtype == BF16:
        tab, ptab = round_to_bf16(tab), round_to_bf16(ptab)
    tok = rng.integers(0, v, size=n).astype(np.int32)
    pos = rng.integers(0, mp - 2, size=n).astype(np.int32)
    tdt = torch.bfloat16 if dtype == BF16 else torch.float32
    x = torch.zeros(n, d, device="cuda")
    P.ops.prism_op_embed_encoder(dev(tab, tdt), dev(ptab, tdt), dev(ty), dtype, dev_i32(tok), dev_i32(pos), 2, x)
    ref = tab[tok].astype(np.float64) + ptab[pos + 2] + ty
    assert np.max(np.abs(x.cpu().numpy() - ref)) < 1e-6


def _gemm_bias_ref(a, b, bias, resid, epi):
    c = a.astype(np.float64) @ b.astype(np.float64).T + bias.astype(np.float64)
    return c if epi == 0 else resid.astype(np.float64) + c if epi == 1 else oracle.gelu(c)


@pytest.mark.parametrize("epi", [0, 1, 2])
@pytest.mark.parametrize("m,n,k", [(5, 64, 32), (130, 192, 100), (300, 512, 768)])
def test_gemm_bias_fp32_simt(P, m, n, k, epi):
    rng = np.random.default_rng(m + n + k + epi)
    a = rng.normal(size=(m, k)).astype(np.float32)
    b = (rng.normal(size=(n, k)) * 0.05).astype(np.float32)
    bias = rng.normal(size=n).astype(np.float32)
    resid = rng.normal(size=(m, n)).astype(np.float32)
    out, rs = torch.zeros(m, n, device="cuda"), dev(resid)
    P.ops.prism_op_gemm_bias(dev(a), dev(b), dev(bias), out, rs, m, n, k, FP32, epi, SIMT, None)
    ref = _gemm_bias_ref(a, b, bias, resid, epi)
    got = (rs if epi == 1 else out).cpu().numpy()
    assert np.max(np.abs(got - ref)) < 1e-5 * max(1.0, np.max(np.abs(ref)))


@pytest.mark.parametrize("impl", [AUTO, SIMT])
@pytest.mark.parametrize("epi", [0, 1, 2])
@pytest.mark.parametrize("m,n,k", [(1, 256, 64), (129, 256, 72), (300, 512, 320), (1000, 1024, 1024), (777, 384, 200),
                                   (4100, 3072, 512), (513, 4096, 1024)])
def test_gemm_bias_bf16(P, m, n, k, epi, impl):
    """The pair tcgen05 kernel's bias / bias + GELU / bias + residual epilogues (and the CUDA-core ones) against an
    fp64 matmul; a bias of order 1 makes a dropped or shifted bias fail by orders of magnitude."""
    rng = np.random.default_rng(m * 7 + n + k + epi)
    a = round_to_bf16(rng.normal(size=(m, k)).astype(np.float32))
    b = round_to_bf16((rng.normal(size=(n, k)) * 0.05).astype(np.float32))
    bias = rng.normal(size=n).astype(np.float32)
    resid = rng.normal(size=(m, n)).astype(np.float32)
    out = torch.zeros(m, n, dtype=torch.bfloat16, device="cuda")
    rs = dev(resid)
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    P.ops.prism_op_gemm_bias(dev(a, torch.bfloat16), dev(b, torch.bfloat16), dev(bias), out, rs, m, n, k, BF16, epi, impl, err)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    ref = _gemm_bias_ref(a, b, bias, resid, epi)
    got = (rs if epi == 1 else out.float()).cpu().numpy()
    scale = np.max(np.abs(ref))
    tol = (2.0 ** -8) * scale + 1e-3 if epi != 1 else 1e-4 * scale + 1e-4
    assert np.max(np.abs(got - ref)) < tol, np.max(np.abs(got - ref))


@pytest.mark.parametrize("causal", [0, 1])
@pytest.mark.parametrize("impl,hq,hkv", [(AUTO, 4, 4), (AUTO, 4, 2), (SOLO, 3, 1), (SIMT, 4, 4)])
def test_attention_head_dim_64(P, impl, hq, hkv, causal):
    from test_gpu_ops import _attn_ref
    rng = np.random.default_rng(64 + causal + hq)
    lens = np.array([1, 7, 64, 65, 130, 200, 63, 128, 129, 300, 513])
    cu = np.zeros(len(lens) + 1, np.int32)
    cu[1:] = np.cumsum(lens)
    qkv = round_to_bf16(rng.normal(size=(cu[-1], (hq + 2 * hkv) * 64)).astype(np.float32))
    out = torch.zeros(int(cu[-1]), hq * 64, dtype=torch.bfloat16, device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    P.ops.prism_op_attention(dev(qkv, torch.bfloat16), out, dev_i32(cu), len(lens), int(lens.max()), hq, hkv, 64, causal, BF16,
                             impl, err)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    ref = _attn_ref(qkv, cu, hq, hkv, 64, bool(causal))
    assert np.max(np.abs(out.float().cpu().numpy() - ref)) < 2e-2


@pytest.mark.parametrize("dtype", [FP32, BF16])
@pytest.mark.parametrize("d", [256, 768, 1024, 2048])
def test_probe_encoder(P, dtype, d):
    """Widths whose weight row sits in registers (768, 1024, 2048 in bf16; 1024 in fp32) and the generic path."""
    rng = np.random.default_rng(9)
    lens = np.array([5, 1, 40, 0, 17])
    cu = np.zeros(len(lens) + 1, np.int32)
    cu[1:] = np.cumsum(lens)
    x = rng.normal(size=(int(cu[-1]), d)).astype(np.float32)
    g, b = (1 + 0.1 * rng.normal(size=d)).astype(np.float32), (0.1 * rng.normal(size=d)).astype(np.float32)
    dw = (rng.normal(size=(d, d)) * (1.3 / np.sqrt(d))).astype(np.float32)
    if dtype == BF16:
        dw = round_to_bf16(dw)
    db, ow, ob = rng.normal(size=d).astype(np.float32) * 0.1, rng.normal(size=d).astype(np.float32) * 0.1, np.array([0.3], np.float32)
    sc = torch.zeros(len(lens), device="cuda")
    P.ops.prism_op_probe_encoder(dev(x), dev_i32(cu), len(lens), dev(g), dev(b), 1e-5, dev(dw, torch.bfloat16 if dtype == BF16 else torch.float32),
                                 dtype, dev(db), dev(ow), dev(ob), sc)
    w = {"head_dense_w": dw, "head_dense_b": db, "head_out_w": ow, "head_out_b": ob}
    ref = [oracle.head_score(oracle.layernorm(x[cu[i]].astype(np.float64), g.astype(np.float64), b.astype(np.float64), 1e-5), w)
           if lens[i] else 0.0 for i in range(len(lens))]
    assert np.max(np.abs(sc.cpu().numpy() - np.array(ref))) < 2e-5


# ------------------------------------------------------------------------------------------ end to end
ENC_TINY = ModelCfg(n_layers=3, hidden=128, n_q_heads=4, n_kv_heads=4, head_dim=32, ffn=256, vocab=997, rope_theta=1.0,
                    rms_eps=1e-5, causal=0, qk_norm=0, dtype=DTYPE_FP32, arch=ARCH_ENCODER, max_positions=130, pos_offset=2)
ENC_TINY_WL = Workload("enc_tiny_fp32", ENC_TINY, 16, 3, 8, ("uniform", 8, 100, 8, 100),
                       Schedule(MODE_FIXED_KEEP, (1, 2), (9, 5)), cfg_index=11)
ENC_MID = ModelCfg(n_layers=5, hidden=1024, n_q_heads=16, n_kv_heads=16, head_dim=64, ffn=4096, vocab=4096, rope_theta=1.0,
                   rms_eps=1e-5, causal=0, qk_norm=0, dtype=DTYPE_BF16, arch=ARCH_ENCODER, max_positions=514, pos_offset=2)
ENC_MID_WL = Workload("enc_mid_bf16", ENC_MID, 24, 4, 16, ("uniform", 20, 300, 20, 300),
                      Schedule(MODE_CLUSTER, (2, 4), cv_threshold=0.3), cfg_index=12)


def make_model(P, cfg, w, req, **kw):
    lens = np.diff(req["cand_offsets"]) + len(req["query"])
    tw = P.upload_weights(w, cfg.dtype, layers_pinned_host=bool(kw.get("stream_weights", False)))
    return P.PrismModel(cfg, tw, int(lens.max()), len(lens), int(lens.sum()), **kw)


def test_encoder_fp32_end_to_end(P):
    wl, cfg = ENC_TINY_WL, ENC_TINY
    w = synth.make_weights(cfg, seed=2)
    req = synth.make_request(wl, 0)
    S = oracle.score_matrix(req["query"], req["cand_tokens"], req["cand_offsets"], w, cfg, [1, 2, 3])
    m = make_model(P, cfg, w, req)
    for sched in (Schedule(MODE_NONE), wl.schedule, Schedule(MODE_CLUSTER, (1, 2), cv_threshold=0.05)):
        idx, sc, tr = run(P, m, req, wl.top_k, sched)
        assert check_scores(tr, S, TOL_FP32) < TOL_FP32
        check_replay(tr, idx, sc, wl.n_candidates, wl.top_k, cfg.n_layers, sched)
        check_end_to_end(tr, idx, S, wl.n_candidates, wl.top_k, cfg.n_layers, sched, TOL_FP32)
    # unpruned: the plain definition (score all, sort, take K)
    idx, sc, _ = run(P, m, req, wl.top_k, Schedule(MODE_NONE))
    ref = oracle.oracle_select(req["query"], req["cand_tokens"], req["cand_offsets"], wl.top_k, w, cfg, Schedule(MODE_NONE), S=S)
    assert list(idx) == ref.topk_idx
    m.close()


@pytest.mark.parametrize("gemm_impl,attn_impl", [(AUTO, AUTO), (SIMT, SIMT), (AUTO, SIMT), (SIMT, AUTO)])
def test_encoder_bf16_paths_match_oracle(P, gemm_impl, attn_impl):
    wl, cfg = ENC_MID_WL, ENC_MID
    w = synth.make_weights(cfg, seed=5)
    req = synth.make_request(wl, 0)
    S = oracle.score_matrix(req["query"], req["cand_tokens"], req["cand_offsets"], w, cfg, [2, 4, 5])
    m = make_model(P, cfg, w, req, gemm_impl=gemm_impl, attention_impl=attn_impl)
    for sched in (Schedule(MODE_NONE), wl.schedule, replace(wl.schedule, select_winners=0)):
        idx, sc, tr = run(P, m, req, wl.top_k, sched)
        check_scores(tr, S, TOL_BF16)
        check_replay(tr, idx, sc, wl.n_candidates, wl.top_k, cfg.n_layers, sched)
        check_end_to_end(tr, idx, S, wl.n_candidates, wl.top_k, cfg.n_layers, sched, TOL_BF16)
    assert tr.shared_prefix_rows == 0                      # bidirectional attention: the query rows depend on the document
    m.close()


def test_encoder_chunked_execution_is_result_neutral(P):
    wl, cfg = ENC_MID_WL, ENC_MID
    w = synth.make_weights(cfg, seed=5)
    req = synth.make_request(wl, 1)
    lens = np.diff(req["cand_offsets"]) + wl.query_len
    total = int(lens.sum())
    base = run(P, make_model(P, cfg, w, req), req, wl.top_k, wl.schedule)
    per_tok = 2 * (cfg.hidden + 3 * cfg.hidden + cfg.hidden + cfg.ffn)
    budget = 2 * total * cfg.hidden * 4 + (total // 4) * per_tok
    got = run(P, make_model(P, cfg, w, req, activation_budget_bytes=budget), req, wl.top_k, wl.schedule)
    assert got[2].n_chunks_max >= 3
    assert np.array_equal(base[0], got[0]) and np.array_equal(base[1].view(np.uint32), got[1].view(np.uint32))
    for r1, r2 in zip(base[2].records, got[2].records):
        assert np.array_equal(r1.scores.view(np.uint32), r2.scores.view(np.uint32)) and r1.active_ids == r2.active_ids


def test_encoder_rejects_what_it_does_not_support(P):
    cfg = ENC_TINY
    w = synth.make_weights(cfg, seed=2)
    req = synth.make_request(ENC_TINY_WL, 0)
    with pytest.raises(P.PrismError) as e:
        make_model(P, cfg, w, req, gemm_impl=3)                     # the single-CTA GEMM has no bias epilogues
    assert e.value.status == -8, e.value                     # PRISM_ERR_UNSUPPORTED
    with pytest.raises(P.PrismError) as e:
        make_model(P, replace(cfg, max_positions=20), w, req)       # positions would run past the table
    assert e.value.status == -1


def test_encoder_candidate_sharded_equals_unsharded(P):
    """The sharded entry point on an encoder handle: ranks as threads of this process (one GPU), host-side score sum."""
    from test_gpu_sharded import run_sharded
    wl, cfg = ENC_MID_WL, ENC_MID
    w = synth.make_weights(cfg, seed=5)
    req = synth.make_request(wl, 0)
    lens = np.diff(req["cand_offsets"]) + wl.query_len
    owner = P.shard_candidates(lens, 2)
    base = make_model(P, cfg, w, req)
    ref_idx, ref_sc, ref_tr = run(P, base, req, wl.top_k, wl.schedule)
    out, calls = run_sharded(P, cfg, w, req, wl.top_k, wl.schedule, owner, 2)
    assert calls == len(ref_tr.records)
    for idx, sc, tr in out:
        assert np.array_equal(idx, ref_idx) and np.array_equal(sc.view(np.uint32), ref_sc.view(np.uint32))
        for a, b in zip(tr.records, ref_tr.records):
            assert a.active_ids == b.active_ids
            assert np.array_equal(np.asarray(a.scores).view(np.uint32), np.asarray(b.scores).view(np.uint32))
    base.close()


def test_encoder_layer_streaming_is_result_neutral(P):
    """Overlapped layer streaming (Sec. 4.2) for the encoder stack: the four matrices of a block come from pinned
    host memory through two device slots; nothing a caller sees may change."""
    wl, cfg = ENC_MID_WL, ENC_MID
    w = synth.make_weights(cfg, seed=5)
    req = synth.make_request(wl, 2)
    for sched in (Schedule(MODE_NONE), wl.schedule):
        base = run(P, make_model(P, cfg, w, req), req, wl.top_k, sched)
        got = run(P, make_model(P, cfg, w, req, stream_weights=True), req, wl.top_k, sched)
        assert np.array_equal(base[0], got[0]) and np.array_equal(base[1].view(np.uint32), got[1].view(np.uint32))
        for r1, r2 in zip(base[2].records, got[2].records):
            assert np.array_equal(r1.scores.view(np.uint32), r2.scores.view(np.uint32)) and r1.active_ids == r2.active_ids


def test_encoder_hidden_state_offload_is_result_neutral(P):
    """Dynamic offloading of the hidden states (Sec. 4.3) for the encoder stack: host-resident hidden states through
    three device chunk buffers, alone and together with layer streaming."""
    wl, cfg = ENC_MID_WL, ENC_MID
    w = synth.make_weights(cfg, seed=5)
    req = synth.make_request(wl, 1)
    lens = np.diff(req["cand_offsets"]) + wl.query_len
    chunk_rows = int(lens.sum()) // 4
    per_tok = 2 * (cfg.hidden + 3 * cfg.hidden + cfg.hidden + cfg.ffn)
    budget = chunk_rows * (3 * cfg.hidden * 4 + per_tok)
    base = run(P, make_model(P, cfg, w, req), req, wl.top_k, wl.schedule)
    for kw in (dict(), dict(stream_weights=True)):
        got = run(P, make_model(P, cfg, w, req, hidden_offload=True, activation_budget_bytes=budget, **kw), req, wl.top_k, wl.schedule)
        assert got[2].n_chunks_max >= 3
        assert np.array_equal(base[0], got[0]) and np.array_equal(base[1].view(np.uint32), got[1].view(np.uint32))
        for r1, r2 in zip(base[2].records, got[2].records):
            assert np.array_equal(r1.scores.view(np.uint32), r2.scores.view(np.uint32)) and r1.active_ids == r2.active_ids


def test_encoder_embedding_row_cache_is_result_neutral(P):
    """Embedding table caching (Sec. 4.4) for the encoder stack: the token table stays in pinned host memory, the
    device holds an LRU cache of its rows."""
    wl, cfg = ENC_MID_WL, ENC_MID
    w = synth.make_weights(cfg, seed=5)
    reqs = [synth.make_request(wl, r) for r in range(2)]
    lens = [np.diff(r["cand_offsets"]) + wl.query_len for r in reqs]
    mx, tot = max(int(l.max()) for l in lens), max(int(l.sum()) for l in lens)
    base = P.PrismModel(cfg, P.upload_weights(w, cfg.dtype), mx, wl.n_candidates, tot)
    cached = P.PrismModel(cfg, P.upload_weights(w, cfg.dtype, embed_pinned_host=True), mx + 64, wl.n_candidates, tot + 4096,
                          embed_cache_rows=cfg.vocab)
    for r in reqs:
        a, b = run(P, base, r, wl.top_k, wl.schedule), run(P, cached, r, wl.top_k, wl.schedule)
        assert np.array_equal(a[0], b[0]) and np.array_equal(a[1].view(np.uint32), b[1].view(np.uint32))
    hits, misses, evictions = cached.embed_cache_stats()
    assert misses > 0 and hits > 0 and evictions == 0


@pytest.mark.parametrize("cfg,wl,tol", [(replace(ENC_TINY, causal=1), ENC_TINY_WL, TOL_FP32), (replace(ENC_MID, causal=1, n_layers=3), ENC_MID_WL, TOL_BF16)],
                         ids=["fp32", "bf16"])
def test_encoder_blocks_with_causal_attention(P, cfg, wl, tol):
    """The causal flag on the encoder blocks (a post-norm decoder with learned positions): not one of the paper's
    models, but the flag is honoured by every attention kernel and the oracle alike."""
    w = synth.make_weights(cfg, seed=3)
    if cfg.n_layers < len(w["layers"]):
        w = dict(w, layers=w["layers"][:cfg.n_layers])
    req = synth.make_request(wl, 3)
    layers = list(range(1, cfg.n_layers + 1))
    S = oracle.score_matrix(req["query"], req["cand_tokens"], req["cand_offsets"], w, cfg, layers)
    S_bi = oracle.score_matrix(req["query"], req["cand_tokens"], req["cand_offsets"], w, replace(cfg, causal=0), layers[-1:],
                               candidates=[0, 1])
    assert np.max(np.abs(S_bi[layers[-1]] - S[layers[-1]][:2])) > 1e-3              # the flag matters
    # under causal attention the first token sees only itself: every candidate of a request scores the same, which
    # makes this a test of exact ties as well (equal scores bit for bit, order by candidate index)
    assert np.ptp(S[layers[-1]]) < 1e-12
    m = make_model(P, cfg, w, req)
    sched = Schedule(MODE_FIXED_KEEP, tuple(layers[:-1]), tuple([wl.n_candidates] * (cfg.n_layers - 1)))
    idx, sc, tr = run(P, m, req, wl.top_k, sched)
    assert [r.layer for r in tr.records] == layers
    check_scores(tr, S, tol)
    check_replay(tr, idx, sc, wl.n_candidates, wl.top_k, cfg.n_layers, sched)
    assert tr.shared_prefix_rows == 0
    assert len(set(np.asarray(tr.records[-1].scores).view(np.uint32).tolist())) == 1 and list(idx) == list(range(wl.top_k))
    m.close()
