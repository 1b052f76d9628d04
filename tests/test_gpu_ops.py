"""-m gpu: every kernel of the hot path against the CPU oracle, through the C ABI (prism_op_*)."""
import numpy as np
import pytest

import oracle
from oracle.prune_rule import MODE_CLUSTER, MODE_FIXED_KEEP, replay_select
from synth.configs import Schedule
from synth.weights import round_to_bf16

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

FP32, BF16 = 0, 1
AUTO, SIMT, SOLO = 0, 1, 3


@pytest.fixture(scope="module")
def P():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_2510_15620_b200 as pkg
    return pkg


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def bf(a):
    return dev(np.asarray(a, np.float32), torch.bfloat16)


# ------------------------------------------------------------------------------------------ pack
@pytest.mark.parametrize("n,lq,lo,hi", [(1, 4, 0, 1), (16, 16, 16, 48), (257, 3, 0, 9), (1500, 32, 1, 40)])
def test_pack_bit_exact(P, n, lq, lo, hi):
    rng = np.random.default_rng(n)
    vocab = 1000
    lens = rng.integers(lo, hi + 1, size=n)
    off = np.zeros(n + 1, np.int32)
    off[1:] = np.cumsum(lens)
    cand = rng.integers(0, vocab, size=int(off[-1])).astype(np.int32)
    query = rng.integers(0, vocab, size=lq).astype(np.int32)
    total = int(off[-1]) + n * lq
    tokens = torch.empty(total, dtype=torch.int32, device="cuda")
    pos = torch.empty_like(tokens)
    cu = torch.empty(n + 1, dtype=torch.int32, device="cuda")
    s2o = torch.empty(n, dtype=torch.int32, device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    P.ops.prism_op_pack(dev(query), dev(cand) if cand.size else torch.zeros(1, dtype=torch.int32, device="cuda"),
                        dev(off), total, vocab, tokens, pos, cu, s2o, err)
    exp_cu = np.zeros(n + 1, np.int64)
    exp_cu[1:] = np.cumsum(lens + lq)
    exp_tok = np.concatenate([np.concatenate([query, cand[off[i]:off[i + 1]]]) for i in range(n)])
    exp_pos = np.concatenate([np.arange(lq + lens[i]) for i in range(n)])
    assert np.array_equal(cu.cpu().numpy(), exp_cu)
    assert np.array_equal(tokens.cpu().numpy(), exp_tok)
    assert np.array_equal(pos.cpu().numpy(), exp_pos)
    assert np.array_equal(s2o.cpu().numpy(), np.arange(n))
    assert int(err.item()) == 0


def test_pack_flags_bad_tokens_without_trapping(P):
    off = np.array([0, 3, 5], np.int32)
    cand = np.array([1, 2, 99, 4, -1], np.int32)
    query = np.array([0, 1], np.int32)
    total = 9
    tokens = torch.empty(total, dtype=torch.int32, device="cuda")
    pos = torch.empty_like(tokens)
    cu = torch.empty(3, dtype=torch.int32, device="cuda")
    s2o = torch.empty(2, dtype=torch.int32, device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    P.ops.prism_op_pack(dev(query), dev(cand), dev(off), total, 50, tokens, pos, cu, s2o, err)
    assert int(err.item()) & 1
    assert tokens.cpu().numpy().max() < 50 and tokens.cpu().numpy().min() >= 0


# ------------------------------------------------------------------------------------------ embed / norm / rope / probe
@pytest.mark.parametrize("dtype", [FP32, BF16])
def test_embed_rmsnorm_probe(P, dtype):
    rng = np.random.default_rng(5)
    v, d, t = 300, 1024 if dtype == BF16 else 256, 777
    table = (rng.normal(size=(v, d)) * 0.02).astype(np.float32)
    gain = (1 + 0.1 * rng.normal(size=d)).astype(np.float32)
    head = (rng.normal(size=(2, d)) * 0.02).astype(np.float32)
    if dtype == BF16:
        table, gain, head = round_to_bf16(table), round_to_bf16(gain), round_to_bf16(head)
    tdt = torch.bfloat16 if dtype == BF16 else torch.float32
    toks = rng.integers(0, v, size=t).astype(np.int32)
    x = torch.empty(t, d, dtype=torch.float32, device="cuda")
    P.ops.prism_op_embed(dev(table, tdt), dtype, dev(toks), x)
    assert np.array_equal(x.cpu().numpy(), table[toks])                     # a copy: exact
    xs = (rng.normal(size=(t, d)) * 3).astype(np.float32)
    out = torch.empty(t, d, dtype=tdt, device="cuda")
    P.ops.prism_op_rmsnorm(dev(xs), dev(gain, tdt), dtype, 1e-6, out)
    ref = oracle.rmsnorm(xs.astype(np.float64), gain.astype(np.float64), 1e-6)
    got = out.float().cpu().numpy()
    tol = 2.0 ** -8 if dtype == BF16 else 2e-6
    assert np.max(np.abs(got - ref) / (np.abs(ref) + 1e-3)) < tol
    lens = rng.integers(1, 40, size=30)
    cu = np.zeros(31, np.int32)
    cu[1:] = np.cumsum(lens)
    xs = xs[: cu[-1]]
    sc = torch.empty(30, dtype=torch.float32, device="cuda")
    P.ops.prism_op_probe(dev(xs), dev(cu), 30, dev(gain, tdt), dev(head, tdt), dtype, 1e-6, sc)
    ref = np.array([oracle.reranker.probe_score(xs[cu[i + 1] - 1], gain, head, 1e-6) for i in range(30)])
    assert np.max(np.abs(sc.cpu().numpy() - ref)) < 2e-5


@pytest.mark.parametrize("dtype,dh,qk_norm", [(FP32, 64, 0), (FP32, 64, 1), (BF16, 128, 1), (FP32, 20, 1)])
def test_qknorm_rope(P, dtype, dh, qk_norm):
    rng = np.random.default_rng(dh + qk_norm)
    hq, hkv, rows, theta = 4, 2, 333, 1e4
    qkv = rng.normal(size=(rows, (hq + 2 * hkv) * dh)).astype(np.float32)
    gq = (1 + 0.1 * rng.normal(size=dh)).astype(np.float32)
    gk = (1 + 0.1 * rng.normal(size=dh)).astype(np.float32)
    if dtype == BF16:
        qkv, gq, gk = round_to_bf16(qkv), round_to_bf16(gq), round_to_bf16(gk)
    pos = rng.integers(0, 600, size=rows).astype(np.int32)
    tdt = torch.bfloat16 if dtype == BF16 else torch.float32
    t = dev(qkv, tdt)
    P.ops.prism_op_qknorm_rope(t, dtype, dev(pos), hq, hkv, dh, qk_norm, dev(gq, tdt), dev(gk, tdt), 1e-6, theta, 600)
    got = t.float().cpu().numpy()
    q = qkv[:, : hq * dh].reshape(rows, hq, dh).astype(np.float64)
    k = qkv[:, hq * dh:(hq + hkv) * dh].reshape(rows, hkv, dh).astype(np.float64)
    if qk_norm:
        q, k = oracle.rmsnorm(q, gq.astype(np.float64), 1e-6), oracle.rmsnorm(k, gk.astype(np.float64), 1e-6)
    q, k = oracle.rope_rotate(q, pos, theta), oracle.rope_rotate(k, pos, theta)
    ref = np.concatenate([q.reshape(rows, -1), k.reshape(rows, -1), qkv[:, (hq + hkv) * dh:]], axis=1)
    tol = 2.0 ** -7 if dtype == BF16 else 3e-6
    assert np.max(np.abs(got - ref)) < tol * max(1.0, np.max(np.abs(ref)))
    assert np.array_equal(got[:, (hq + hkv) * dh:], qkv[:, (hq + hkv) * dh:])       # v untouched


# ------------------------------------------------------------------------------------------ GEMM
def _gemm_ref(a, b, b2, resid, epi):
    c = a.astype(np.float64) @ b.astype(np.float64).T
    if epi == 0:
        return c
    if epi == 1:
        return resid.astype(np.float64) + c
    u = a.astype(np.float64) @ b2.astype(np.float64).T
    return c / (1 + np.exp(-c)) * u


@pytest.mark.parametrize("m,n,k", [(5, 64, 32), (130, 192, 100), (300, 512, 768)])
@pytest.mark.parametrize("epi", [0, 1, 2])
def test_gemm_fp32_simt(P, m, n, k, epi):
    rng = np.random.default_rng(m + n + k + epi)
    a = rng.normal(size=(m, k)).astype(np.float32)
    b = (rng.normal(size=(n, k)) * 0.05).astype(np.float32)
    b2 = (rng.normal(size=(n, k)) * 0.05).astype(np.float32)
    resid = rng.normal(size=(m, n)).astype(np.float32)
    out = torch.zeros(m, n, device="cuda")
    rs = dev(resid)
    P.ops.prism_op_gemm(dev(a), dev(b), dev(b2), out, rs, m, n, k, FP32, epi, SIMT, None)
    got = (rs if epi == 1 else out).cpu().numpy()
    ref = _gemm_ref(a, b, b2, resid, epi)
    assert np.max(np.abs(got - ref)) < 1e-5 * max(1.0, np.max(np.abs(ref)))      # fp32 accumulation over k terms


@pytest.mark.parametrize("impl", [AUTO, SOLO, SIMT])
@pytest.mark.parametrize("epi", [0, 1, 2])
@pytest.mark.parametrize("m,n,k", [(1, 256, 64), (129, 256, 72), (300, 512, 320), (1000, 1024, 1024), (777, 384, 200),
                                   (4100, 2560, 512)])
def test_gemm_bf16(P, m, n, k, epi, impl):
    """tcgen05 kernels (AUTO: CTA pairs, 256x256 tiles; SOLO: single CTAs, 128x256) and the CUDA-core kernel on the
    same bf16 inputs vs an fp64 matmul.  Shapes span several tiles, ragged M/N/K tails (one where only the pair's
    first CTA has rows, one where the second has a single row) and more tiles than SMs."""
    rng = np.random.default_rng(m * 7 + n + k + epi)
    a = round_to_bf16(rng.normal(size=(m, k)).astype(np.float32))
    b = round_to_bf16((rng.normal(size=(n, k)) * 0.05).astype(np.float32))
    b2 = round_to_bf16((rng.normal(size=(n, k)) * 0.05).astype(np.float32))
    resid = rng.normal(size=(m, n)).astype(np.float32)
    out = torch.zeros(m, n, dtype=torch.bfloat16, device="cuda")
    rs = dev(resid)
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    P.ops.prism_op_gemm(bf(a), bf(b), bf(b2), out, rs, m, n, k, BF16, epi, impl, err)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    ref = _gemm_ref(a, b, b2, resid, epi)
    got = (rs if epi == 1 else out.float()).cpu().numpy()
    scale = np.max(np.abs(ref))
    tol = (2.0 ** -8) * scale + 1e-3 if epi != 1 else 1e-4 * scale + 1e-4    # bf16 store vs fp32 residual add
    assert np.max(np.abs(got - ref)) < tol, np.max(np.abs(got - ref))


@pytest.mark.parametrize("qk_norm", [1, 0])
@pytest.mark.parametrize("m,k,hq,hkv", [(300, 320, 2, 1), (1000, 1024, 16, 8), (4100, 256, 3, 1)])
def test_gemm_qkv_with_fused_qknorm_rope(P, m, k, hq, hkv, qk_norm):
    """QKV projection whose epilogue applies QK-norm and the rotary embedding, vs the oracle's
    rmsnorm/rope_rotate on an fp64 product."""
    rng = np.random.default_rng(m + k + qk_norm)
    dh, theta = 128, 1e6
    n = (hq + 2 * hkv) * dh
    a = round_to_bf16(rng.normal(size=(m, k)).astype(np.float32))
    w = round_to_bf16((rng.normal(size=(n, k)) * 0.05).astype(np.float32))
    gq = round_to_bf16((1 + 0.1 * rng.normal(size=dh)).astype(np.float32))
    gk = round_to_bf16((1 + 0.1 * rng.normal(size=dh)).astype(np.float32))
    pos = rng.integers(0, 700, size=m).astype(np.int32)
    out = torch.zeros(m, n, dtype=torch.bfloat16, device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    P.ops.prism_op_gemm_qkv_rope(bf(a), bf(w), out, m, k, hq, hkv, qk_norm, bf(gq), bf(gk), 1e-6, dev(pos), theta, 700, err)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    c = a.astype(np.float64) @ w.astype(np.float64).T
    q = c[:, : hq * dh].reshape(m, hq, dh)
    kk = c[:, hq * dh:(hq + hkv) * dh].reshape(m, hkv, dh)
    if qk_norm:
        q, kk = oracle.rmsnorm(q, gq.astype(np.float64), 1e-6), oracle.rmsnorm(kk, gk.astype(np.float64), 1e-6)
    q, kk = oracle.rope_rotate(q, pos, theta), oracle.rope_rotate(kk, pos, theta)
    ref = np.concatenate([q.reshape(m, -1), kk.reshape(m, -1), c[:, (hq + hkv) * dh:]], axis=1)
    got = out.float().cpu().numpy()
    assert np.max(np.abs(got - ref)) < (2.0 ** -8) * np.max(np.abs(ref)) + 1e-3


def test_gemm_tc_rows_do_not_depend_on_their_position(P):
    """Duplicate rows anywhere in the batch, and the same row in a smaller batch, give identical bits
    (exact score ties between duplicated candidates rely on this)."""
    rng = np.random.default_rng(0)
    m, n, k = 700, 512, 1024
    a = round_to_bf16(rng.normal(size=(m, k)).astype(np.float32))
    a[650] = a[3]
    a[129] = a[3]
    b = round_to_bf16((rng.normal(size=(n, k)) * 0.05).astype(np.float32))
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.zeros(m, n, dtype=torch.bfloat16, device="cuda")
    P.ops.prism_op_gemm(bf(a), bf(b), None, out, None, m, n, k, BF16, 0, AUTO, err)
    o = out.view(torch.int16).cpu().numpy()
    assert np.array_equal(o[3], o[650]) and np.array_equal(o[3], o[129])
    out2 = torch.zeros(5, n, dtype=torch.bfloat16, device="cuda")
    P.ops.prism_op_gemm(bf(a[:5]), bf(b), None, out2, None, 5, n, k, BF16, 0, AUTO, err)
    assert np.array_equal(out2.view(torch.int16).cpu().numpy()[3], o[3])
    assert int(err.item()) == 0


# ------------------------------------------------------------------------------------------ attention
def _attn_ref(qkv, cu, hq, hkv, dh, causal):
    out = np.zeros((qkv.shape[0], hq * dh))
    for s in range(len(cu) - 1):
        x = qkv[cu[s]:cu[s + 1]].astype(np.float64)
        L = x.shape[0]
        q = x[:, : hq * dh].reshape(L, hq, dh)
        k = x[:, hq * dh:(hq + hkv) * dh].reshape(L, hkv, dh)
        v = x[:, (hq + hkv) * dh:].reshape(L, hkv, dh)
        out[cu[s]:cu[s + 1]] = oracle.attention(q, k, v, causal).reshape(L, hq * dh)
    return out


@pytest.mark.parametrize("causal", [1, 0])
@pytest.mark.parametrize("dtype,impl,dh,hq,hkv", [(FP32, SIMT, 64, 4, 2), (BF16, SIMT, 128, 4, 2), (BF16, AUTO, 128, 4, 2),
                                                  (BF16, AUTO, 128, 8, 2), (BF16, AUTO, 128, 3, 1), (BF16, 2, 128, 4, 2),
                                                  (BF16, SOLO, 128, 4, 2), (BF16, AUTO, 64, 4, 2), (BF16, AUTO, 64, 4, 4),
                                                  (BF16, AUTO, 64, 3, 3), (BF16, SOLO, 64, 4, 4)])
def test_attention(P, dtype, impl, dh, hq, hkv, causal):
    """AUTO runs the two-heads-per-CTA tcgen05 kernel for even group sizes (2 and 4 here; at head_dim 64 also for an
    even number of heads with a K/V head each) and the one-head kernel otherwise (group 3, or three heads of 64);
    SOLO forces the one-head kernel; 2 is the mma.sync kernel."""
    rng = np.random.default_rng(dh + causal)
    lens = np.array([1, 7, 64, 65, 130, 200, 63, 128, 129, 300, 513])      # below, at and across the 64/128-row tiles
    cu = np.zeros(len(lens) + 1, np.int32)
    cu[1:] = np.cumsum(lens)
    qkv = rng.normal(size=(cu[-1], (hq + 2 * hkv) * dh)).astype(np.float32)
    if dtype == BF16:
        qkv = round_to_bf16(qkv)
    tdt = torch.bfloat16 if dtype == BF16 else torch.float32
    out = torch.zeros(int(cu[-1]), hq * dh, dtype=tdt, device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    P.ops.prism_op_attention(dev(qkv, tdt), out, dev(cu), len(lens), int(lens.max()), hq, hkv, dh, causal, dtype, impl, err)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    ref = _attn_ref(qkv, cu, hq, hkv, dh, bool(causal))
    got = out.float().cpu().numpy()
    tol = 2e-2 if dtype == BF16 else 2e-5
    assert np.max(np.abs(got - ref)) < tol, np.max(np.abs(got - ref))


def test_attention_tc_rescales_when_the_maximum_grows(P):
    """Scores that keep growing along the keys force the running reference maximum to move by far more
    than 2^8 between key blocks, so the in-TMEM rescale of O must run (and be right)."""
    rng = np.random.default_rng(4)
    hq, hkv, dh = 2, 1, 128
    lens = np.array([400, 150])
    cu = np.zeros(3, np.int32)
    cu[1:] = np.cumsum(lens)
    qkv = (rng.normal(size=(cu[-1], (hq + 2 * hkv) * dh)) * 0.5).astype(np.float32)
    ramp = np.concatenate([np.arange(l) for l in lens])[:, None] * 0.02           # key norm grows with position
    qkv[:, hq * dh:(hq + hkv) * dh] *= (1 + ramp * 3)
    qkv[:, : hq * dh] = np.abs(qkv[:, : hq * dh]) * 2
    qkv[:, hq * dh:(hq + hkv) * dh] = np.abs(qkv[:, hq * dh:(hq + hkv) * dh])
    qkv = round_to_bf16(qkv)
    out = torch.zeros(int(cu[-1]), hq * dh, dtype=torch.bfloat16, device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    for causal in (1, 0):
        P.ops.prism_op_attention(dev(qkv, torch.bfloat16), out, dev(cu), 2, 400, hq, hkv, dh, causal, BF16, AUTO, err)
        torch.cuda.synchronize()
        assert int(err.item()) == 0
        ref = _attn_ref(qkv, cu, hq, hkv, dh, bool(causal))
        assert np.max(np.abs(out.float().cpu().numpy() - ref)) < 2e-2 * max(1.0, np.max(np.abs(ref)))


def test_attention_tc_many_items_per_cta(P):
    """More work items than SMs x ring depth, mixed lengths from 1 to 6 key blocks, group size 4: the item ring of
    the two-head kernel wraps many times, items of different cost interleave, and the counters of one launch are
    rearmed for a later one.  Run twice on the same buffers: both runs must match the oracle and each other bit
    for bit (the dynamic hand-out changes which SM computes what, never the arithmetic of a row)."""
    rng = np.random.default_rng(21)
    hq, hkv, dh = 8, 2, 128
    lens = rng.integers(1, 700, size=96)
    lens[:4] = [1, 128, 129, 699]
    cu = np.zeros(len(lens) + 1, np.int32)
    cu[1:] = np.cumsum(lens)
    tot = int(cu[-1])
    qkv = round_to_bf16(rng.normal(size=(tot, (hq + 2 * hkv) * dh)).astype(np.float32))
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    dq, dcu = dev(qkv, torch.bfloat16), dev(cu)
    outs = []
    for _ in range(2):
        out = torch.zeros(tot, hq * dh, dtype=torch.bfloat16, device="cuda")
        P.ops.prism_op_attention(dq, out, dcu, len(lens), int(lens.max()), hq, hkv, dh, 1, BF16, AUTO, err)
        torch.cuda.synchronize()
        assert int(err.item()) == 0
        outs.append(out)
    assert torch.equal(outs[0], outs[1])
    ref = _attn_ref(qkv, cu, hq, hkv, dh, True)
    assert np.max(np.abs(outs[0].float().cpu().numpy() - ref)) < 2e-2


def test_attention_tc_work_counters_are_rearmed(P):
    """Each launch of the two-head kernel takes the next pair of device work counters from a table of 1024 and
    must leave it zeroed.  1100 small launches wrap the table; a counter left non-zero would make a later launch
    skip its work, so the last outputs are checked against the first."""
    rng = np.random.default_rng(5)
    hq, hkv, dh = 4, 2, 128
    lens = np.array([70, 130, 5])
    cu = np.zeros(len(lens) + 1, np.int32)
    cu[1:] = np.cumsum(lens)
    tot = int(cu[-1])
    qkv = dev(round_to_bf16(rng.normal(size=(tot, (hq + 2 * hkv) * dh)).astype(np.float32)), torch.bfloat16)
    dcu = dev(cu)
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    first = torch.zeros(tot, hq * dh, dtype=torch.bfloat16, device="cuda")
    P.ops.prism_op_attention(qkv, first, dcu, len(lens), 130, hq, hkv, dh, 1, BF16, AUTO, err)
    out = torch.zeros_like(first)
    for i in range(1100):
        if i >= 1096:
            out.zero_()
        P.ops.prism_op_attention(qkv, out, dcu, len(lens), 130, hq, hkv, dh, 1, BF16, AUTO, err)
        if i >= 1096:
            torch.cuda.synchronize()
            assert int(err.item()) == 0
            assert torch.equal(out, first), i


@pytest.mark.parametrize("impl", [AUTO, SOLO])
def test_attention_tc_scores_far_above_the_first_key(P, impl):
    """The two-head kernel exponentiates against the row's score on key 0 and moves that reference only when a
    row sum leaves fp32's comfortable range.  Here later keys score hundreds of powers of two above key 0
    (and, in other rows, far below it), inside one 32-key chunk, across chunks and across key blocks, so the
    reference must move (repeatedly) and O, l and the probabilities already written must follow exactly."""
    rng = np.random.default_rng(11)
    hq, hkv, dh = 4, 2, 128
    lens = np.array([300, 40, 129])
    cu = np.zeros(len(lens) + 1, np.int32)
    cu[1:] = np.cumsum(lens)
    tot = int(cu[-1])
    qkv = rng.normal(size=(tot, (hq + 2 * hkv) * dh)).astype(np.float32)
    pos = np.concatenate([np.arange(l) for l in lens])
    # key norm: a staircase over positions (x1 ... x40) with jumps inside chunks, between chunks and between blocks;
    # q . k / sqrt(dh) then spans roughly +-(4 * 40 * sqrt(128) / sqrt(128)) ~ +-500 in natural-log units
    stair = 1.0 + 39.0 * (((pos * 7) % 97) / 96.0) * (pos > 0) + 20.0 * (pos % 50 == 17)
    qkv[:, hq * dh:(hq + hkv) * dh] *= stair[:, None]
    qkv[:, : hq * dh] *= 2.0
    qkv = round_to_bf16(qkv)
    out = torch.zeros(tot, hq * dh, dtype=torch.bfloat16, device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    for causal in (1, 0):
        P.ops.prism_op_attention(dev(qkv, torch.bfloat16), out, dev(cu), len(lens), int(lens.max()), hq, hkv, dh, causal,
                                 BF16, impl, err)
        torch.cuda.synchronize()
        assert int(err.item()) == 0
        ref = _attn_ref(qkv, cu, hq, hkv, dh, bool(causal))
        got = out.float().cpu().numpy()
        assert np.isfinite(got).all()
        assert np.max(np.abs(got - ref)) < 2e-2 * max(1.0, np.max(np.abs(ref))), np.max(np.abs(got - ref))


def test_bounded_wait_gives_up_and_reports(P):
    """The wait every tensor-core kernel uses: on a barrier nothing arrives at it returns after its limit
    and sets the time-out bit; nothing hangs, the device keeps working."""
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    P.ops.prism_op_wait_selftest(20_000_000, err)              # about 10 ms
    t1.record()
    torch.cuda.synchronize()
    assert int(err.item()) == 4                                  # kErrTimeout and nothing else
    assert 2.0 < t0.elapsed_time(t1) < 500.0
    x = torch.arange(10, device="cuda").sum()                    # the context is intact
    assert int(x.item()) == 45
    with pytest.raises(P.PrismError):
        P.ops.prism_op_wait_selftest(0, err)


# ------------------------------------------------------------------------------------------ route / compact
def _run_route(P, scores, ids, lens, k_rem, n_result, sched_kw, is_final=0, layer=3):
    n = len(scores)
    cu = np.zeros(n + 1, np.int32)
    cu[1:] = np.cumsum(lens)
    state = np.array([n, cu[-1], k_rem, n_result, 0, 0, 0, 0], np.int32)
    d = dict(mode=MODE_CLUSTER, keep_count=0, cv_threshold=0.0, n_clusters=3, std_ddof=0, select_winners=1)
    d.update(sched_kw)
    cu_new = torch.full((n + 1,), -1, dtype=torch.int32, device="cuda")
    s2o_new = torch.full((max(n, 1),), -1, dtype=torch.int32, device="cuda")
    oon = torch.full((max(n, 1),), -1, dtype=torch.int32, device="cuda")
    st = dev(state)
    ridx = torch.full((n + n_result + 1,), -1, dtype=torch.int32, device="cuda")
    rsc = torch.zeros(n + n_result + 1, dtype=torch.float32, device="cuda")
    rec = torch.zeros(P.ops.RECORD_BYTES, dtype=torch.uint8, device="cuda")
    P.ops.prism_op_route(dev(np.asarray(scores, np.float32)), dev(cu), dev(np.asarray(ids, np.int32)), n, d["mode"],
                         d["keep_count"], d["cv_threshold"], d["n_clusters"], d["std_ddof"], d["select_winners"],
                         is_final, layer, cu_new, s2o_new, oon, st, ridx, rsc, rec)
    torch.cuda.synchronize()
    return (st.cpu().numpy(), cu_new.cpu().numpy(), s2o_new.cpu().numpy(), oon.cpu().numpy(), ridx.cpu().numpy(),
            rsc.cpu().numpy(), P.ops.decode_record(rec), cu)


@pytest.mark.parametrize("n_clusters", [2, 3, 5, 8])
@pytest.mark.parametrize("winners", [1, 0])
def test_route_matches_oracle_rule_bit_exact(P, n_clusters, winners):
    rng = np.random.default_rng(n_clusters * 2 + winners)
    for trial in range(25):
        n = int(rng.choice([1, 2, 3, 17, 100, 333, 1000, 1500]))
        k = int(rng.integers(1, 25))
        base = rng.normal(size=n) * (3 if trial % 2 else 0.3) + (0 if trial % 3 else 2.0)
        sc = base.astype(np.float32)
        if trial % 4 == 0 and n > 4:
            sc[rng.integers(0, n, size=n // 3)] = sc[0]                  # exact ties
        ids = np.sort(rng.choice(5000, size=n, replace=False)).astype(np.int32)
        lens = rng.integers(1, 50, size=n)
        thr = float(rng.choice([0.0, 0.3, 5.0]))
        st, cu_new, s2o_new, oon, ridx, rsc, rec, cu = _run_route(
            P, sc, ids, lens, min(k, n), 2, dict(cv_threshold=thr, n_clusters=n_clusters, select_winners=winners))
        # the oracle's rule on the same scores: a one-probe schedule over a two-layer "model"
        sched = Schedule(MODE_CLUSTER, (1,), cv_threshold=thr, n_clusters=n_clusters, select_winners=winners)
        table = {1: dict(zip(range(n), sc)), 2: dict(zip(range(n), sc))}
        ref = replay_select(lambda l, a: np.asarray([table[l][i] for i in a], np.float32), n, k, 2, sched)
        t = ref.trace[0]
        assert (rec.fired, rec.n_selected, rec.n_dropped, rec.n_deferred, rec.k_rem_after) == \
               (t.fired, t.n_selected, t.n_dropped, t.n_deferred, t.k_rem_after), (n, k, thr)
        assert [rec.cuts[i] for i in range(rec.n_cuts)] == t.cuts
        assert rec.cv == t.cv
        survivors = ref.active_per_layer[1] if len(ref.active_per_layer) > 1 else []
        n_new = int(st[0])
        assert n_new == len(survivors)
        assert list(oon[:n_new]) == survivors                          # positions in the old batch, order kept
        assert list(s2o_new[:n_new]) == [int(ids[p]) for p in survivors]
        exp_cu = np.concatenate([[0], np.cumsum(lens[survivors])]) if survivors else np.array([0])
        assert list(cu_new[: n_new + 1]) == list(exp_cu)
        assert int(st[1]) == int(exp_cu[-1]) and int(st[2]) == t.k_rem_after
        done = ref.layers_run == 1
        assert int(st[4]) == int(done)
        left = len(ref.topk_idx) if done else t.n_selected
        assert int(st[3]) == 2 + left
        assert list(ridx[2:2 + left]) == [int(ids[p]) for p in ref.topk_idx[:left]]
        assert list(rsc[2:2 + left]) == [np.float32(x) for x in ref.topk_scores[:left]]


def test_route_at_the_maximum_candidate_count(P):
    """n = PRISM_MAX_CANDIDATES (4096), with ties, against the oracle's rule."""
    rng = np.random.default_rng(77)
    n, k = 4096, 50
    sc = (rng.normal(size=n) * 2).astype(np.float32)
    sc[rng.integers(0, n, size=500)] = sc[7]
    ids = np.arange(n, dtype=np.int32)
    lens = rng.integers(1, 20, size=n)
    st, cu_new, s2o_new, oon, ridx, rsc, rec, cu = _run_route(P, sc, ids, lens, k, 0, dict(cv_threshold=0.1, n_clusters=4))
    sched = Schedule(MODE_CLUSTER, (1,), cv_threshold=0.1, n_clusters=4)
    ref = replay_select(lambda l, a: sc[np.asarray(a)], n, k, 2, sched)
    t = ref.trace[0]
    assert (rec.fired, rec.n_selected, rec.n_dropped, rec.n_deferred) == (t.fired, t.n_selected, t.n_dropped, t.n_deferred)
    assert [rec.cuts[i] for i in range(rec.n_cuts)] == t.cuts and rec.cv == t.cv
    survivors = ref.active_per_layer[1]
    assert list(oon[: int(st[0])]) == survivors
    assert list(cu_new[: len(survivors) + 1]) == list(np.concatenate([[0], np.cumsum(lens[survivors])]))


def test_route_fixed_keep_and_final(P):
    rng = np.random.default_rng(9)
    n = 40
    sc = rng.normal(size=n).astype(np.float32)
    sc[5] = sc[9]
    ids = np.arange(n, dtype=np.int32)
    lens = rng.integers(1, 9, size=n)
    st, cu_new, s2o_new, oon, ridx, rsc, rec, cu = _run_route(P, sc, ids, lens, 4, 0, dict(mode=MODE_FIXED_KEEP, keep_count=10))
    order = sorted(range(n), key=lambda i: (-sc[i], i))
    assert list(oon[:10]) == sorted(order[:10]) and int(st[0]) == 10 and rec.n_dropped == 30 and int(st[4]) == 0
    st, *_, ridx, rsc, rec, cu = _run_route(P, sc, ids, lens, 4, 0, dict(), is_final=1)
    assert int(st[4]) == 1 and list(ridx[:4]) == order[:4] and list(rsc[:4]) == [sc[i] for i in order[:4]]
    st, *_, ridx, rsc, rec, cu = _run_route(P, sc[:3], ids[:3], lens[:3], 5, 0, dict())          # n <= k_rem: all leave
    assert int(st[4]) == 1 and int(st[3]) == 3 and int(st[2]) == 2


def test_compact_rows_exact(P):
    rng = np.random.default_rng(3)
    n, d = 37, 1024
    lens = rng.integers(1, 30, size=n)
    cu = np.zeros(n + 1, np.int32)
    cu[1:] = np.cumsum(lens)
    x = rng.normal(size=(cu[-1], d)).astype(np.float32)
    keep = np.sort(rng.choice(n, size=11, replace=False)).astype(np.int32)
    cu_new = np.zeros(12, np.int32)
    cu_new[1:] = np.cumsum(lens[keep])
    out = torch.zeros(int(cu_new[-1]), d, device="cuda")
    P.ops.prism_op_compact(dev(x), out, dev(cu), dev(cu_new), dev(keep), 11, int(cu_new[-1]))
    exp = np.concatenate([x[cu[i]:cu[i + 1]] for i in keep])
    assert np.array_equal(out.cpu().numpy(), exp)
