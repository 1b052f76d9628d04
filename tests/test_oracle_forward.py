"""Pins for the oracle forward: hand-computed examples, an independent library model
(HuggingFace Qwen3), causality, permutation invariance, brute-force selection."""
import math
import os
from types import SimpleNamespace

import numpy as np
import pytest

import oracle
import synth
from synth.configs import MODE_FIXED_KEEP, MODE_NONE, ModelCfg, Schedule

GOLD = os.path.join(os.path.dirname(__file__), "golden", "hand_example_1layer.txt")


def _gold():
    out = {}
    for line in open(GOLD):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        out[k] = v
    return out


def _hand_cfg(theta=1e4):
    return ModelCfg(n_layers=1, hidden=4, n_q_heads=1, n_kv_heads=1, head_dim=4, ffn=4, vocab=2,
                    rope_theta=theta, rms_eps=0.0, causal=1, qk_norm=0, dtype=0)


def _hand_weights(wq, wk, wgate):
    I = np.eye(4)
    Z = np.zeros((4, 4))
    return {
        "embed": np.array([[3.0, 4, 0, 0], [0, 0, 6, 8]]),
        "g_final": np.ones(4),
        "score_head": np.array([[1.0, 0, 0, 0], [0, 0, 0, 1]]),
        "layers": [{
            "g_attn": np.ones(4), "g_ffn": np.ones(4),
            "w_qkv": np.concatenate([wq, wk, I]), "w_o": I,
            "w_gate": wgate, "w_up": I, "w_down": I,
        }],
    }


def test_hand_example_uniform_attention():
    g = _gold()
    w = _hand_weights(np.zeros((4, 4)), np.zeros((4, 4)), np.zeros((4, 4)))
    sc, hid = oracle.candidate_scores(np.array([0, 1]), w, _hand_cfg(), [1], return_hidden=True)
    np.testing.assert_allclose(hid[1][0], [float(x) for x in g["A_h0"]], rtol=0, atol=1e-14)
    np.testing.assert_allclose(hid[1][1], [float(x) for x in g["A_h1"]], rtol=0, atol=1e-14)
    assert abs(sc[1] - float(g["A_score"][0])) < 1e-14
    assert abs(sc[1] - (-8.2 / math.sqrt(30.5))) < 1e-14


def test_hand_example_rope_softmax():
    I = np.eye(4)
    w = _hand_weights(I, I, np.zeros((4, 4)))
    sc, hid = oracle.candidate_scores(np.array([0, 1]), w, _hand_cfg(1e4), [1], return_hidden=True)
    l0 = (-1.44 * math.sin(1.0) - 2.56 * math.sin(0.01)) / 2.0
    l1 = 2.0
    p0 = 1.0 / (1.0 + math.exp(l1 - l0))
    p1 = 1.0 - p0
    h1 = [1.2 * p0, 1.6 * p0, 6 + 1.2 * p1, 8 + 1.6 * p1]
    np.testing.assert_allclose(hid[1][1], h1, rtol=0, atol=1e-13)
    ms = sum(v * v for v in h1) / 4
    assert abs(sc[1] - (h1[0] - h1[3]) / math.sqrt(ms)) < 1e-13
    # a different theta must change the result (the second frequency is theta^-1/2)
    sc2 = oracle.candidate_scores(np.array([0, 1]), w, _hand_cfg(1e2), [1])
    l0b = (-1.44 * math.sin(1.0) - 2.56 * math.sin(0.1)) / 2.0
    p0b = 1.0 / (1.0 + math.exp(l1 - l0b))
    h1b = [1.2 * p0b, 1.6 * p0b, 6 + 1.2 * (1 - p0b), 8 + 1.6 * (1 - p0b)]
    assert abs(sc2[1] - (h1b[0] - h1b[3]) / math.sqrt(sum(v * v for v in h1b) / 4)) < 1e-13


def test_hand_example_swiglu():
    I = np.eye(4)
    w = _hand_weights(np.zeros((4, 4)), np.zeros((4, 4)), I)
    _, hid = oracle.candidate_scores(np.array([0, 1]), w, _hand_cfg(), [1], return_hidden=True)
    r = math.sqrt(30.5)
    h1 = [0.6, 0.8, 6.6, 8.8]
    exp = [h + (h / r) * (h / r) / (1 + math.exp(-h / r)) for h in h1]
    np.testing.assert_allclose(hid[1][1], exp, rtol=0, atol=1e-13)


def test_gain_and_eps_enter_rmsnorm():
    x = np.array([[3.0, 4.0, 0.0, 0.0]])
    y = oracle.rmsnorm(x, np.array([2.0, 1.0, 1.0, 1.0]), 0.0)
    np.testing.assert_allclose(y, [[2.4, 1.6, 0, 0]], atol=1e-15)
    y = oracle.rmsnorm(x, np.ones(4), 2.75)      # mean sq 6.25 + 2.75 = 9
    np.testing.assert_allclose(y, [[1.0, 4.0 / 3.0, 0, 0]], atol=1e-15)


@pytest.mark.parametrize("qk_norm", [0, 1])
def test_matches_huggingface_qwen3(qk_norm):
    """An independently written library model with the same architecture must give the same
    per-layer probe scores (pins GQA head mapping, RoPE convention, QK-norm placement, SwiGLU,
    pre-norm residual structure, final norm + head)."""
    torch = pytest.importorskip("torch")
    tr = pytest.importorskip("transformers")
    cfg = ModelCfg(n_layers=3, hidden=64, n_q_heads=4, n_kv_heads=2, head_dim=16, ffn=96, vocab=128,
                   rope_theta=1e4, rms_eps=1e-6, causal=1, qk_norm=1, dtype=0, yes_id=5, no_id=9)
    w = synth.make_weights(cfg, seed=3)
    if not qk_norm:  # HF Qwen3 always has QK-norm; gain sqrt-free check: all-ones gains + oracle flag on
        for l in w["layers"]:
            l["g_q"] = np.ones_like(l["g_q"])
            l["g_k"] = np.ones_like(l["g_k"])
    hc = tr.Qwen3Config(hidden_size=64, intermediate_size=96, num_hidden_layers=3, num_attention_heads=4,
                        num_key_value_heads=2, head_dim=16, vocab_size=128, rms_norm_eps=1e-6,
                        tie_word_embeddings=False, attention_bias=False, max_position_embeddings=512,
                        rope_parameters={"rope_type": "default", "rope_theta": 1e4},
                        attn_implementation="eager")
    m = tr.Qwen3ForCausalLM(hc).double().eval()
    sd = {}
    t = lambda a: torch.tensor(np.asarray(a, np.float64))
    sd["model.embed_tokens.weight"] = t(w["embed"])
    sd["model.norm.weight"] = t(w["g_final"])
    lm = np.zeros((128, 64))
    lm[5], lm[9] = w["score_head"][0], w["score_head"][1]
    sd["lm_head.weight"] = t(lm)
    hq, hkv, dh = 4, 2, 16
    for i, l in enumerate(w["layers"]):
        p = f"model.layers.{i}."
        sd[p + "self_attn.q_proj.weight"] = t(l["w_qkv"][: hq * dh])
        sd[p + "self_attn.k_proj.weight"] = t(l["w_qkv"][hq * dh:(hq + hkv) * dh])
        sd[p + "self_attn.v_proj.weight"] = t(l["w_qkv"][(hq + hkv) * dh:])
        sd[p + "self_attn.o_proj.weight"] = t(l["w_o"])
        sd[p + "self_attn.q_norm.weight"] = t(l["g_q"])
        sd[p + "self_attn.k_norm.weight"] = t(l["g_k"])
        sd[p + "mlp.gate_proj.weight"] = t(l["w_gate"])
        sd[p + "mlp.up_proj.weight"] = t(l["w_up"])
        sd[p + "mlp.down_proj.weight"] = t(l["w_down"])
        sd[p + "input_layernorm.weight"] = t(l["g_attn"])
        sd[p + "post_attention_layernorm.weight"] = t(l["g_ffn"])
    missing = m.load_state_dict(sd, strict=True)
    toks = np.random.default_rng(0).integers(0, 128, size=37)
    with torch.no_grad():
        out = m(torch.tensor(toks[None, :]), output_hidden_states=True)
        ours = oracle.candidate_scores(toks, w, cfg, [1, 2, 3])
        for layer in (1, 2, 3):
            h = out.hidden_states[layer][0, -1]
            if layer < 3:                       # HF applies the final norm only to the last entry
                h = m.model.norm(h)
            logits = m.lm_head(h)
            ref = float(logits[5] - logits[9])
            assert abs(ours[layer] - ref) < 1e-6, (layer, ours[layer], ref)   # HF builds its rotary table in fp32


def _tiny(causal=1):
    wl = synth.workload(0)
    from dataclasses import replace
    cfg = replace(wl.model, causal=causal)
    return wl, cfg, synth.make_weights(cfg)


def test_causality_and_bidirectional_flag():
    wl, cfg, w = _tiny(1)
    toks = np.random.default_rng(1).integers(0, cfg.vocab, size=24)
    toks2 = toks.copy()
    toks2[-1] = (toks2[-1] + 1) % cfg.vocab
    _, h1 = oracle.candidate_scores(toks, w, cfg, [2], return_hidden=True)
    _, h2 = oracle.candidate_scores(toks2, w, cfg, [2], return_hidden=True)
    assert np.array_equal(h1[2][:-1], h2[2][:-1])          # prefix untouched by a later token
    assert not np.allclose(h1[2][-1], h2[2][-1])
    _, cfgb, _ = _tiny(0)
    _, b1 = oracle.candidate_scores(toks, w, cfgb, [2], return_hidden=True)
    _, b2 = oracle.candidate_scores(toks2, w, cfgb, [2], return_hidden=True)
    assert not np.allclose(b1[2][0], b2[2][0])             # bidirectional: position 0 sees the change


def test_scores_permute_with_candidates_and_ignore_batch_mates():
    wl, cfg, w = _tiny()
    r = synth.make_request(wl)
    S = oracle.score_matrix(r["query"], r["cand_tokens"], r["cand_offsets"], w, cfg, [1, 2])
    perm = np.random.default_rng(2).permutation(wl.n_candidates)
    S2 = oracle.score_matrix(r["query"], r["cand_tokens"], r["cand_offsets"], w, cfg, [1, 2], candidates=perm)
    for l in (1, 2):
        assert np.array_equal(S[l][perm], S2[l])            # bitwise
    # one candidate alone through the candidate-major entry point
    i = 5
    seq = np.concatenate([r["query"], r["cand_tokens"][r["cand_offsets"][i]:r["cand_offsets"][i + 1]]])
    one = oracle.candidate_scores(seq, w, cfg, [1, 2])
    assert one[1] == S[1][i] and one[2] == S[2][i]


def test_unpruned_select_is_brute_force_sort():
    wl, cfg, w = _tiny()
    r = synth.make_request(wl)
    res = oracle.oracle_select(r["query"], r["cand_tokens"], r["cand_offsets"], 5, w, cfg, Schedule(MODE_NONE))
    final = []
    for i in range(wl.n_candidates):
        seq = np.concatenate([r["query"], r["cand_tokens"][r["cand_offsets"][i]:r["cand_offsets"][i + 1]]])
        final.append(np.float32(oracle.candidate_scores(seq, w, cfg, [cfg.n_layers])[cfg.n_layers]))
    order = sorted(range(wl.n_candidates), key=lambda i: (-final[i], i))[:5]
    assert res.topk_idx == order
    assert res.topk_scores == [float(final[i]) for i in order]
    assert res.layers_run == cfg.n_layers


def test_cfg0_fixed_keep_schedule():
    wl, cfg, w = _tiny()
    r = synth.make_request(wl)
    S = oracle.score_matrix(r["query"], r["cand_tokens"], r["cand_offsets"], w, cfg, [1, 2])
    res = oracle.oracle_select(r["query"], r["cand_tokens"], r["cand_offsets"], 3, w, cfg, wl.schedule, S=S)
    keep = sorted(sorted(range(16), key=lambda i: (-np.float32(S[1][i]), i))[:8])
    assert res.active_per_layer[1] == keep
    exp = sorted(keep, key=lambda i: (-np.float32(S[2][i]), i))[:3]
    assert res.topk_idx == exp


def test_float32_forward_agrees_with_float64():
    """The same forward evaluated by torch CPU ops in fp32 stays within 1e-5 of the fp64 oracle
    (bounds how much rounding order can matter at the tiny config)."""
    torch = pytest.importorskip("torch")
    import torch.nn.functional as F
    wl, cfg, w = _tiny()
    toks = np.random.default_rng(3).integers(0, cfg.vocab, size=40)
    ours = oracle.candidate_scores(toks, w, cfg, [1, 2])
    x = torch.tensor(w["embed"][toks])
    L = len(toks)
    hq, hkv, dh = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    pos = torch.arange(L, dtype=torch.float32)
    inv = cfg.rope_theta ** (-torch.arange(0, dh, 2, dtype=torch.float32) / dh)
    ang = pos[:, None] * inv[None, :]
    cos, sin = torch.cat([ang.cos(), ang.cos()], -1), torch.cat([ang.sin(), ang.sin()], -1)
    rot = lambda u: torch.cat([-u[..., dh // 2:], u[..., : dh // 2]], -1)
    got = {}
    for li, lw in enumerate(w["layers"], start=1):
        W = {k: torch.tensor(v) for k, v in lw.items()}
        a = F.rms_norm(x, (cfg.hidden,), W["g_attn"], cfg.rms_eps)
        qkv = a @ W["w_qkv"].T
        q = qkv[:, : hq * dh].view(L, hq, dh).transpose(0, 1)
        k = qkv[:, hq * dh:(hq + hkv) * dh].view(L, hkv, dh).transpose(0, 1)
        v = qkv[:, (hq + hkv) * dh:].view(L, hkv, dh).transpose(0, 1)
        q = q * cos + rot(q) * sin
        k = k * cos + rot(k) * sin
        o = F.scaled_dot_product_attention(q[None], k[None], v[None], is_causal=True, enable_gqa=True)[0]
        x = x + o.transpose(0, 1).reshape(L, hq * dh) @ W["w_o"].T
        b = F.rms_norm(x, (cfg.hidden,), W["g_ffn"], cfg.rms_eps)
        x = x + (F.silu(b @ W["w_gate"].T) * (b @ W["w_up"].T)) @ W["w_down"].T
        y = F.rms_norm(x[-1], (cfg.hidden,), torch.tensor(w["g_final"]), cfg.rms_eps)
        got[li] = float(y @ torch.tensor(w["score_head"][0] - w["score_head"][1]))
    for l in (1, 2):
        assert abs(got[l] - ours[l]) < 1e-5


def test_bf16_activation_mode_rounds_like_a_library_and_stays_close():
    """The optional bf16-activation mode of the oracle: its rounding equals torch's float32 -> bfloat16
    conversion bit for bit (ties to even included), rounding is idempotent, and on the tiny model the
    mode moves the scores only by rounding noise."""
    torch = pytest.importorskip("torch")
    from oracle.reranker import to_bf16
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.normal(size=5000) * 10.0 ** rng.integers(-6, 6, size=5000),
                        np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -(1.0 + 2.0 ** -8), 0.0, 65280.0])]).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy().astype(np.float64)
    got = to_bf16(x)
    assert np.array_equal(got, ref)
    assert np.array_equal(to_bf16(got), got)
    wl, cfg, w = _tiny()
    toks = np.random.default_rng(5).integers(0, cfg.vocab, size=40)
    exact = oracle.candidate_scores(toks, w, cfg, [1, 2])
    rounded = oracle.candidate_scores(toks, w, cfg, [1, 2], act="bf16")
    for l in (1, 2):
        assert 0 < abs(exact[l] - rounded[l]) < 5e-2


def test_rounding_points_of_the_bf16_mode_compose():
    """The rounded-activation mode takes a subset of its six storage points: all six named one by one are the full
    mode bit for bit, none is the exact forward, every single point moves the scores by less than all six together
    can at most (the sum of the single moves bounds nothing, but each is non-zero and small), and an unknown name is
    refused."""
    from oracle.reranker import ROUNDING_POINTS, rounding_points
    assert rounding_points("exact") == frozenset() and rounding_points("bf16") == frozenset(ROUNDING_POINTS)
    wl, cfg, w = _tiny()
    toks = np.random.default_rng(6).integers(0, cfg.vocab, size=48)
    exact = oracle.candidate_scores(toks, w, cfg, [1, 2])
    full = oracle.candidate_scores(toks, w, cfg, [1, 2], act="bf16")
    named = oracle.candidate_scores(toks, w, cfg, [1, 2], act=",".join(ROUNDING_POINTS))
    assert named == full
    for p in ROUNDING_POINTS:
        one = oracle.candidate_scores(toks, w, cfg, [1, 2], act=p)
        assert all(0 < abs(one[l] - exact[l]) < 5e-2 for l in (1, 2)), p
    with pytest.raises(ValueError):
        oracle.candidate_scores(toks, w, cfg, [1], act="norm,softmax")
