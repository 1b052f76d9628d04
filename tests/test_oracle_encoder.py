"""Pins for the encoder-stack oracle (CPU): library implementations of the same model (torch's post-norm
TransformerEncoderLayer, HuggingFace XLM-RoBERTa with a sequence-classification head), hand-computed values,
and the properties that tell a bidirectional encoder from the decoder stack."""
import math
from dataclasses import replace

import numpy as np
import pytest

import oracle
import synth
from synth.configs import ARCH_ENCODER, DTYPE_FP32, ModelCfg

torch = pytest.importorskip("torch")

ENC = ModelCfg(n_layers=2, hidden=32, n_q_heads=4, n_kv_heads=4, head_dim=8, ffn=64, vocab=97, rope_theta=1.0,
               rms_eps=1e-5, causal=0, qk_norm=0, dtype=DTYPE_FP32, arch=ARCH_ENCODER, max_positions=40, pos_offset=2)


def test_layernorm_hand_values():
    # mean 2.5, biased variance 1.25
    y = oracle.layernorm(np.array([1.0, 2.0, 3.0, 4.0]), np.array([1.0, 2.0, 3.0, 4.0]), np.array([0.5, 0.0, -0.5, 1.0]), 0.0)
    r = 1.0 / math.sqrt(1.25)
    np.testing.assert_allclose(y, [-1.5 * r + 0.5, -0.5 * r * 2, 0.5 * r * 3 - 0.5, 1.5 * r * 4 + 1.0], rtol=0, atol=1e-15)
    # eps enters under the root
    y2 = oracle.layernorm(np.array([0.0, 2.0]), np.ones(2), np.zeros(2), 3.0)
    np.testing.assert_allclose(y2, [-0.5, 0.5], rtol=0, atol=1e-15)


def test_gelu_is_x_times_the_normal_cdf():
    # Phi(1) = 0.8413447460685429 (tabulated), gelu(-x) = gelu(x) - x, gelu(0) = 0, gelu(x) -> x for large x
    assert abs(float(oracle.gelu(np.array(1.0))) - 0.8413447460685429) < 1e-15
    assert abs(float(oracle.gelu(np.array(-1.0))) + 0.15865525393145707) < 1e-15
    x = np.linspace(-6, 6, 41)
    np.testing.assert_allclose(oracle.gelu(x) - oracle.gelu(-x), x, rtol=0, atol=1e-14)
    assert float(oracle.gelu(np.array(0.0))) == 0.0 and abs(float(oracle.gelu(np.array(12.0))) - 12.0) < 1e-12
    # the tanh approximation differs from it by up to 5e-4: the exact form is what the model uses
    t = 0.5 * x * (1 + np.tanh(math.sqrt(2 / math.pi) * (x + 0.044715 * x ** 3)))
    assert 1e-4 < np.max(np.abs(t - oracle.gelu(x))) < 1e-3


def test_hand_example_uniform_attention_one_block():
    """D = 2, one head, W_q = W_k = 0 (uniform attention over both tokens), identity V and O, no FFN contribution
    (W_2 = 0): x_t = LN(e_t + mean(e) + b_o), worked by hand for e = [[1, 3], [5, 1]]."""
    cfg = replace(ENC, n_layers=1, hidden=2, n_q_heads=1, n_kv_heads=1, head_dim=2, ffn=2, vocab=2, rms_eps=0.0,
                  max_positions=4, pos_offset=0)
    I, Z = np.eye(2), np.zeros((2, 2))
    w = {"embed": np.array([[1.0, 3.0], [5.0, 1.0]]), "pos_embed": np.zeros((4, 2)), "type_embed": np.zeros(2),
         "emb_ln_g": np.ones(2), "emb_ln_b": np.zeros(2),
         "head_dense_w": I, "head_dense_b": np.zeros(2), "head_out_w": np.array([1.0, 0.0]), "head_out_b": np.array([0.25]),
         "layers": [{"w_qkv": np.concatenate([Z, Z, I]), "b_qkv": np.zeros(6), "w_o": I, "b_o": np.array([0.0, 1.0]),
                     "ln1_g": np.array([2.0, 1.0]), "ln1_b": np.zeros(2), "w_ffn1": I, "b_ffn1": np.zeros(2),
                     "w_ffn2": Z, "b_ffn2": np.zeros(2), "ln2_g": np.ones(2), "ln2_b": np.array([0.0, 0.5])}]}
    # embedding LayerNorm (eps 0): [1,3] -> [-1, 1], [5,1] -> [1, -1]; their mean is [0, 0]
    # attention output = mean of v = [0, 0]; + b_o: x + [0, 1] = [-1, 2] and [1, 0]
    # LN1 with gain [2, 1]: [-1, 2] -> [-1, 1] * [2, 1] = [-2, 1]; [1, 0] -> [1, -1] * [2, 1] = [2, -1]
    # FFN adds nothing; LN2 of [-2, 1] -> [-1, 1] + [0, .5] = [-1, 1.5]; of [2, -1] -> [1, -1] + [0, .5] = [1, -.5]
    sc, hid = oracle.encoder_candidate_scores(np.array([0, 1]), w, cfg, [1], return_hidden=True)
    np.testing.assert_allclose(hid[1], [[-1.0, 1.5], [1.0, -0.5]], rtol=0, atol=1e-14)
    assert abs(sc[1] - (math.tanh(-1.0) + 0.25)) < 1e-14          # first token, first unit of the head


def _torch_layer(w, cfg):
    layer = torch.nn.TransformerEncoderLayer(cfg.hidden, cfg.n_q_heads, cfg.ffn, dropout=0.0, activation="gelu",
                                             layer_norm_eps=cfg.rms_eps, batch_first=True, norm_first=False).double().eval()
    t = lambda k: torch.from_numpy(np.asarray(w[k], np.float64))
    with torch.no_grad():
        layer.self_attn.in_proj_weight.copy_(t("w_qkv")); layer.self_attn.in_proj_bias.copy_(t("b_qkv"))
        layer.self_attn.out_proj.weight.copy_(t("w_o")); layer.self_attn.out_proj.bias.copy_(t("b_o"))
        layer.norm1.weight.copy_(t("ln1_g")); layer.norm1.bias.copy_(t("ln1_b"))
        layer.linear1.weight.copy_(t("w_ffn1")); layer.linear1.bias.copy_(t("b_ffn1"))
        layer.linear2.weight.copy_(t("w_ffn2")); layer.linear2.bias.copy_(t("b_ffn2"))
        layer.norm2.weight.copy_(t("ln2_g")); layer.norm2.bias.copy_(t("ln2_b"))
    return layer


@pytest.mark.parametrize("causal", [0, 1])
def test_block_equals_torch_post_norm_encoder_layer(causal):
    cfg = replace(ENC, causal=causal)
    w = synth.make_weights(cfg, seed=3)["layers"][1]
    w = {k: np.asarray(v, np.float64) * (8.0 if k.startswith("w_") else 1.0) for k, v in w.items()}  # attention far from uniform
    rng = np.random.default_rng(0)
    x = rng.normal(size=(11, cfg.hidden))
    mask = torch.triu(torch.full((11, 11), float("-inf"), dtype=torch.float64), diagonal=1) if causal else None
    with torch.no_grad():
        ref = _torch_layer(w, cfg)(torch.from_numpy(x)[None], src_mask=mask)[0].numpy()
    np.testing.assert_allclose(oracle.encoder_layer_forward(x, w, cfg), ref, rtol=0, atol=1e-12)


def test_whole_stack_equals_huggingface_xlm_roberta():
    tf = pytest.importorskip("transformers")
    cfg = ENC
    w = synth.make_weights(cfg, seed=1)
    hc = tf.XLMRobertaConfig(vocab_size=cfg.vocab, hidden_size=cfg.hidden, num_hidden_layers=cfg.n_layers,
                             num_attention_heads=cfg.n_q_heads, intermediate_size=cfg.ffn, hidden_act="gelu",
                             hidden_dropout_prob=0.0, attention_probs_dropout_prob=0.0, classifier_dropout=0.0,
                             max_position_embeddings=cfg.max_positions, type_vocab_size=1, pad_token_id=1,
                             layer_norm_eps=cfg.rms_eps, num_labels=1)
    m = tf.XLMRobertaForSequenceClassification(hc).double().eval()
    sd = m.state_dict()
    t = lambda a: torch.from_numpy(np.asarray(a, np.float64))
    D, put = cfg.hidden, {}
    put["roberta.embeddings.word_embeddings.weight"] = t(w["embed"])
    put["roberta.embeddings.position_embeddings.weight"] = t(w["pos_embed"])
    put["roberta.embeddings.token_type_embeddings.weight"] = t(w["type_embed"])[None]
    put["roberta.embeddings.LayerNorm.weight"] = t(w["emb_ln_g"])
    put["roberta.embeddings.LayerNorm.bias"] = t(w["emb_ln_b"])
    for l, lw in enumerate(w["layers"]):
        p = f"roberta.encoder.layer.{l}."
        for j, nm in enumerate(("query", "key", "value")):
            put[p + f"attention.self.{nm}.weight"] = t(lw["w_qkv"][j * D:(j + 1) * D])
            put[p + f"attention.self.{nm}.bias"] = t(lw["b_qkv"][j * D:(j + 1) * D])
        put[p + "attention.output.dense.weight"] = t(lw["w_o"]); put[p + "attention.output.dense.bias"] = t(lw["b_o"])
        put[p + "attention.output.LayerNorm.weight"] = t(lw["ln1_g"]); put[p + "attention.output.LayerNorm.bias"] = t(lw["ln1_b"])
        put[p + "intermediate.dense.weight"] = t(lw["w_ffn1"]); put[p + "intermediate.dense.bias"] = t(lw["b_ffn1"])
        put[p + "output.dense.weight"] = t(lw["w_ffn2"]); put[p + "output.dense.bias"] = t(lw["b_ffn2"])
        put[p + "output.LayerNorm.weight"] = t(lw["ln2_g"]); put[p + "output.LayerNorm.bias"] = t(lw["ln2_b"])
    put["classifier.dense.weight"] = t(w["head_dense_w"]); put["classifier.dense.bias"] = t(w["head_dense_b"])
    put["classifier.out_proj.weight"] = t(w["head_out_w"])[None]; put["classifier.out_proj.bias"] = t(w["head_out_b"])
    for k, v in put.items():
        assert k in sd and tuple(sd[k].shape) == tuple(v.shape), k
    missing = [k for k in sd if k not in put and "position_ids" not in k and "token_type_ids" not in k]
    assert not missing, missing
    m.load_state_dict({**sd, **put})
    rng = np.random.default_rng(5)
    for L in (1, 7, 19):
        toks = rng.integers(2, cfg.vocab, size=L)                  # the pad id (1) never occurs inside a sequence
        with torch.no_grad():
            out = m(input_ids=torch.from_numpy(toks)[None], output_hidden_states=True)
        sc, hid = oracle.encoder_candidate_scores(toks, w, cfg, [1, 2], return_hidden=True)
        np.testing.assert_allclose(hid[1], out.hidden_states[1][0].numpy(), rtol=0, atol=1e-12)
        np.testing.assert_allclose(hid[2], out.hidden_states[2][0].numpy(), rtol=0, atol=1e-12)
        assert abs(sc[2] - float(out.logits[0, 0])) < 1e-12


def test_bidirectional_and_batch_independent():
    cfg = ENC
    w = synth.make_weights(cfg, seed=2)
    rng = np.random.default_rng(1)
    q = rng.integers(2, cfg.vocab, size=5)
    docs = [rng.integers(2, cfg.vocab, size=n) for n in (9, 3, 14)]
    off = np.concatenate([[0], np.cumsum([len(d) for d in docs])]).astype(np.int32)
    S = oracle.score_matrix(q, np.concatenate(docs), off, w, cfg, [1, 2])
    # a candidate's score is that of its own sequence alone, whatever else is in the request
    for i, d in enumerate(docs):
        alone = oracle.encoder_candidate_scores(np.concatenate([q, d]), w, cfg, [1, 2])
        assert alone[1] == S[1][i] and alone[2] == S[2][i]
    perm = [2, 0, 1]
    S2 = oracle.score_matrix(q, np.concatenate(docs), off, w, cfg, [2], candidates=perm)
    assert np.array_equal(S2[2], S[2][perm])
    # the score is read at the FIRST token and depends on the LAST one (bidirectional); with causal = 1 it cannot
    d2 = docs[0].copy()
    d2[-1] = (d2[-1] + 1 - 2) % (cfg.vocab - 2) + 2
    a = oracle.encoder_candidate_scores(np.concatenate([q, docs[0]]), w, cfg, [2])[2]
    b = oracle.encoder_candidate_scores(np.concatenate([q, d2]), w, cfg, [2])[2]
    assert abs(a - b) > 1e-6
    cc = replace(cfg, causal=1)
    assert oracle.encoder_candidate_scores(np.concatenate([q, docs[0]]), w, cc, [2])[2] == \
           oracle.encoder_candidate_scores(np.concatenate([q, d2]), w, cc, [2])[2]
    # positions matter: swapping two document tokens changes the score
    d3 = docs[0].copy()
    d3[[0, 1]] = d3[[1, 0]]
    assert abs(oracle.encoder_candidate_scores(np.concatenate([q, d3]), w, cfg, [2])[2] - a) > 1e-9


def test_selection_over_the_encoder_scores_is_the_plain_definition_when_unpruned():
    from synth.configs import MODE_NONE, Schedule
    cfg = ENC
    w = synth.make_weights(cfg, seed=4)
    rng = np.random.default_rng(2)
    q = rng.integers(2, cfg.vocab, size=4)
    docs = [rng.integers(2, cfg.vocab, size=int(n)) for n in rng.integers(2, 20, size=9)]
    off = np.concatenate([[0], np.cumsum([len(d) for d in docs])]).astype(np.int32)
    res = oracle.oracle_select(q, np.concatenate(docs), off, 3, w, cfg, Schedule(MODE_NONE))
    full = np.array([oracle.encoder_candidate_scores(np.concatenate([q, d]), w, cfg, [2])[2] for d in docs])
    order = sorted(range(9), key=lambda i: (-np.float32(full[i]), i))[:3]
    assert res.topk_idx == order
