"""Oracle forward pass of an encoder-only cross-encoder reranker (test infrastructure).

The paper evaluates its method on an encoder-only reranker as well (BGE-M3's reranker, Sec. 6.1, Table 1) and
states that monolithic forwarding and the probe apply to encoder and decoder models alike.  That model is an
XLM-RoBERTa stack; written here from the model definition, one candidate at a time, fp64:
  * input: token embedding + learned position embedding (position p of the sequence reads row p + pos_offset)
    + the token-type-0 embedding, then LayerNorm;
  * block (post-norm): x = LN1(x + O(attention(QKV(x)))), x = LN2(x + W2 gelu(W1 x + b1) + b2); every linear map
    has a bias, attention is bidirectional (cfg.causal = 0) with softmax(q k^T / sqrt(dh)), GELU is the exact
    x Phi(x);
  * classifier ("the model's original classifier" of the probe, Sec. 3.1, 4.1): on the FIRST token's hidden
    state, dense + tanh, then a single-logit projection; the logit is the score.
Readings where the paper is silent: the probe after block l applies the classifier to block l's output (which
is already normalised by LN2); sequence = query tokens followed by document tokens as the caller gives them
(separator tokens included by the caller), positions restart at 0 per sequence.
parity: pinned (torch.nn.TransformerEncoderLayer, HuggingFace XLM-RoBERTa, hand-computed values; see
tests/test_oracle_encoder.py).
"""
from __future__ import annotations

from typing import Dict, Iterable, List, Sequence

import numpy as np
from scipy.special import erf

from .reranker import attention


def layernorm(x: np.ndarray, g: np.ndarray, b: np.ndarray, eps: float) -> np.ndarray:
    """y = (x - mean) / sqrt(var + eps) * g + b over the last axis (biased variance)."""
    mu = np.mean(x, axis=-1, keepdims=True)
    var = np.mean((x - mu) ** 2, axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + eps) * g + b


def gelu(x: np.ndarray) -> np.ndarray:
    """x * Phi(x), Phi the standard normal distribution function."""
    return 0.5 * x * (1.0 + erf(x / np.sqrt(2.0)))


def embed_tokens(tokens: np.ndarray, weights: Dict[str, object], cfg) -> np.ndarray:
    """Sum of the three embeddings followed by the embedding LayerNorm.  tokens: [L] -> [L, D]."""
    t = np.asarray(tokens, dtype=np.int64)
    pos = np.arange(len(t)) + int(cfg.pos_offset)
    e = (np.asarray(weights["embed"][t], np.float64) + np.asarray(weights["pos_embed"][pos], np.float64)
         + np.asarray(weights["type_embed"], np.float64))
    return layernorm(e, np.asarray(weights["emb_ln_g"], np.float64), np.asarray(weights["emb_ln_b"], np.float64),
                     cfg.rms_eps)


def encoder_layer_forward(x: np.ndarray, w: Dict[str, np.ndarray], cfg) -> np.ndarray:
    """One post-norm encoder block on one sequence.  x: [L, D] fp64 -> [L, D]."""
    L = x.shape[0]
    hq, hkv, dh = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    W = {k: np.asarray(t, dtype=np.float64) for k, t in w.items()}
    qkv = x @ W["w_qkv"].T + W["b_qkv"]
    q = qkv[:, : hq * dh].reshape(L, hq, dh)
    k = qkv[:, hq * dh: (hq + hkv) * dh].reshape(L, hkv, dh)
    v = qkv[:, (hq + hkv) * dh:].reshape(L, hkv, dh)
    o = attention(q, k, v, bool(cfg.causal)).reshape(L, hq * dh)
    x = layernorm(x + o @ W["w_o"].T + W["b_o"], W["ln1_g"], W["ln1_b"], cfg.rms_eps)
    h = gelu(x @ W["w_ffn1"].T + W["b_ffn1"])
    return layernorm(x + h @ W["w_ffn2"].T + W["b_ffn2"], W["ln2_g"], W["ln2_b"], cfg.rms_eps)


def head_score(x_first: np.ndarray, weights: Dict[str, object]) -> float:
    """Classifier on the first token's hidden state: out_w . tanh(dense_w x + dense_b) + out_b."""
    x = np.asarray(x_first, np.float64)
    y = np.tanh(np.asarray(weights["head_dense_w"], np.float64) @ x + np.asarray(weights["head_dense_b"], np.float64))
    return float(np.asarray(weights["head_out_w"], np.float64) @ y + np.asarray(weights["head_out_b"], np.float64)[0])


def encoder_candidate_scores(tokens: np.ndarray, weights: Dict[str, object], cfg, score_layers: Iterable[int],
                             return_hidden: bool = False):
    """Forward one sequence (query||doc token ids) and return {layer: score} for every layer count in
    score_layers (1-based: after that many blocks)."""
    want = sorted(set(int(l) for l in score_layers))
    x = embed_tokens(tokens, weights, cfg)
    out: Dict[int, float] = {}
    hidden: Dict[int, np.ndarray] = {}
    last = want[-1] if want else 0
    for l, w in enumerate(weights["layers"], start=1):
        if l > last:
            break
        x = encoder_layer_forward(x, w, cfg)
        if l in want:
            out[l] = head_score(x[0], weights)
            if return_hidden:
                hidden[l] = x.copy()
    return (out, hidden) if return_hidden else out


def encoder_score_matrix(query: np.ndarray, cand_tokens: np.ndarray, cand_offsets: np.ndarray,
                         weights: Dict[str, object], cfg, score_layers: Sequence[int],
                         candidates: Sequence[int] | None = None) -> Dict[int, np.ndarray]:
    """S[layer][i] for the requested candidates (default all): each candidate is forwarded alone as
    query||doc_i (sequences never attend to each other, so batching changes the schedule, not the values;
    Sec. 3.3).  Layer-major over the weights so that each layer is widened to fp64 once."""
    n = len(cand_offsets) - 1
    ids = list(range(n)) if candidates is None else [int(c) for c in candidates]
    want = sorted(set(int(l) for l in score_layers))
    xs: List[np.ndarray] = []
    for i in ids:
        doc = cand_tokens[int(cand_offsets[i]): int(cand_offsets[i + 1])]
        xs.append(embed_tokens(np.concatenate([np.asarray(query), np.asarray(doc)]), weights, cfg))
    S = {l: np.zeros(len(ids), dtype=np.float64) for l in want}
    last = want[-1] if want else 0
    for l, w in enumerate(weights["layers"], start=1):
        if l > last:
            break
        w = {k: np.asarray(t, dtype=np.float64) for k, t in w.items()}
        for c in range(len(ids)):
            xs[c] = encoder_layer_forward(xs[c], w, cfg)
        if l in S:
            for c in range(len(ids)):
                S[l][c] = head_score(xs[c][0], weights)
    return S
