"""Oracle forward pass of a decoder cross-encoder reranker (test infrastructure).

One candidate at a time, fp64, written from the model definition the paper relies on
(its rerankers are the Qwen3 family: pre-norm decoder blocks with RMSNorm, grouped-query
attention with per-head QK-norm and rotary embeddings, SwiGLU FFN; Sec. 6.1, Table 1) and
the paper's probe: "the model's original classifier" applied to an intermediate hidden
state (Sec. 3.1, Sec. 4.1).  Readings taken where the paper is silent:
  * the classifier is everything after the last block: final RMSNorm, then the score head;
  * score = logit("yes") - logit("no") at the last token of query||doc;
  * sequence = query tokens followed by doc tokens, positions restart at 0 per sequence;
  * RoPE pairs element j with j + dh/2; QK-norm (if on) is applied before RoPE; no biases.
Sequences never attend to each other, so a candidate's scores do not depend on which other
candidates share its batch; monolithic forwarding (Sec. 3.3) changes the schedule, not the
values.  parity: pinned (hand-computed examples, HF Qwen3 cross-check, causality,
permutation invariance; see tests/test_oracle_forward.py).
"""
from __future__ import annotations

from typing import Dict, Iterable, List, Sequence

import numpy as np


def to_bf16(x: np.ndarray) -> np.ndarray:
    """Round to the nearest bfloat16 (ties to even), returned as float64.  Used only by the optional
    "bf16 activations" mode below, which places one rounding wherever the precision contract of the
    bf16 path stores an activation as bfloat16."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (b + (np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1)))) & np.uint32(0xFFFF0000)
    return r.view(np.float32).astype(np.float64)


def rmsnorm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    """y = x / sqrt(mean(x^2) + eps) * g over the last axis."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * g


def rope_rotate(u: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotary embedding, half-split pairing.  u: [L, H, dh], pos: [L].

    For j < dh/2 and angle phi = pos * theta^(-2j/dh):
      out[j]        = u[j] cos(phi) - u[j+dh/2] sin(phi)
      out[j+dh/2]   = u[j+dh/2] cos(phi) + u[j] sin(phi)"""
    dh = u.shape[-1]
    half = dh // 2
    j = np.arange(half, dtype=np.float64)
    inv_freq = theta ** (-2.0 * j / dh)
    phi = pos.astype(np.float64)[:, None] * inv_freq[None, :]          # [L, half]
    c, s = np.cos(phi)[:, None, :], np.sin(phi)[:, None, :]
    a, b = u[..., :half], u[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, causal: bool, round_p=None) -> np.ndarray:
    """q: [L, Hq, dh], k/v: [L, Hkv, dh] -> [L, Hq, dh].  Query head h reads kv head
    h // (Hq/Hkv).  softmax(q k^T / sqrt(dh)) over keys u <= t (causal) or all keys.
    round_p (optional) rounds the unnormalised probabilities that multiply v; the normaliser is
    the sum of the unrounded ones."""
    L, hq, dh = q.shape
    hkv = k.shape[1]
    grp = hq // hkv
    out = np.empty_like(q)
    mask = np.tril(np.ones((L, L), dtype=bool)) if causal else np.ones((L, L), dtype=bool)
    for h in range(hq):
        kh = h // grp
        s = (q[:, h, :] @ k[:, kh, :].T) / np.sqrt(float(dh))
        s = np.where(mask, s, -np.inf)
        s = s - s.max(axis=-1, keepdims=True)
        p = np.exp(s)
        den = p.sum(axis=-1, keepdims=True)
        if round_p is not None:
            p = round_p(p)
        out[:, h, :] = (p @ v[:, kh, :]) / den
    return out


ROUNDING_POINTS = ("norm", "qk", "v", "p", "attn", "swiglu")


def rounding_points(act: str):
    """The set of stored tensors the mode `act` rounds to bfloat16."""
    if act == "exact":
        return frozenset()
    if act == "bf16":
        return frozenset(ROUNDING_POINTS)
    on = frozenset(p for p in act.split(",") if p)
    if not on <= set(ROUNDING_POINTS):
        raise ValueError(f"unknown rounding point in {act!r}")
    return on


def layer_forward(x: np.ndarray, w: Dict[str, np.ndarray], cfg, act: str = "exact") -> np.ndarray:
    """One pre-norm decoder block on one sequence.  x: [L, D] fp64 -> [L, D].

    act = "exact": no rounding anywhere (the definition).  act = "bf16": the same steps with every
    stored activation rounded to bfloat16 where the bf16 precision contract stores it (normed inputs,
    q/k after the rotary embedding, v, attention probabilities, attention output, SwiGLU output); the
    residual stream, norms, softmax and all sums stay exact.  A comma-separated subset of
    ROUNDING_POINTS rounds at those points only (used to tell which stored tensor carries the noise)."""
    on = rounding_points(act)
    rnd = {p: (to_bf16 if p in on else (lambda t: t)) for p in ROUNDING_POINTS}
    L = x.shape[0]
    hq, hkv, dh = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    W = {k: np.asarray(t, dtype=np.float64) for k, t in w.items()}
    a = rnd["norm"](rmsnorm(x, W["g_attn"], cfg.rms_eps))
    qkv = a @ W["w_qkv"].T
    q = qkv[:, : hq * dh].reshape(L, hq, dh)
    k = qkv[:, hq * dh: (hq + hkv) * dh].reshape(L, hkv, dh)
    v = qkv[:, (hq + hkv) * dh:].reshape(L, hkv, dh)
    if cfg.qk_norm:
        q = rmsnorm(q, W["g_q"], cfg.rms_eps)
        k = rmsnorm(k, W["g_k"], cfg.rms_eps)
    pos = np.arange(L)
    q = rnd["qk"](rope_rotate(q, pos, cfg.rope_theta))
    k = rnd["qk"](rope_rotate(k, pos, cfg.rope_theta))
    v = rnd["v"](v)
    o = rnd["attn"](attention(q, k, v, bool(cfg.causal), round_p=to_bf16 if "p" in on else None)).reshape(L, hq * dh)
    x = x + o @ W["w_o"].T
    b = rnd["norm"](rmsnorm(x, W["g_ffn"], cfg.rms_eps))
    gate = b @ W["w_gate"].T
    up = b @ W["w_up"].T
    h = rnd["swiglu"](gate / (1.0 + np.exp(-gate)) * up)     # silu(gate) * up
    return x + h @ W["w_down"].T


def probe_score(x_last: np.ndarray, g_final: np.ndarray, score_head: np.ndarray, eps: float) -> float:
    """Score of one candidate from its last-token hidden state: final RMSNorm, then
    logit(row 0, "yes") - logit(row 1, "no")."""
    y = rmsnorm(np.asarray(x_last, np.float64), np.asarray(g_final, np.float64), eps)
    sh = np.asarray(score_head, np.float64)
    return float(y @ sh[0] - y @ sh[1])


def candidate_scores(tokens: np.ndarray, weights: Dict[str, object], cfg,
                     score_layers: Iterable[int], return_hidden: bool = False, act: str = "exact"):
    """Forward one sequence (query||doc token ids) through all layers needed and return
    {layer: score} for every layer count in score_layers (1-based: after that many blocks).
    `weights['layers']` may be a list or any iterable yielding per-layer dicts in order."""
    want = sorted(set(int(l) for l in score_layers))
    emb = weights["embed"]
    x = np.asarray(emb[np.asarray(tokens, dtype=np.int64)], dtype=np.float64)
    out: Dict[int, float] = {}
    hidden: Dict[int, np.ndarray] = {}
    last = want[-1] if want else 0
    for l, w in enumerate(weights["layers"], start=1):
        if l > last:
            break
        x = layer_forward(x, w, cfg, act)
        if l in want:
            out[l] = probe_score(x[-1], weights["g_final"], weights["score_head"], cfg.rms_eps)
            if return_hidden:
                hidden[l] = x.copy()
    return (out, hidden) if return_hidden else out


def score_matrix(query: np.ndarray, cand_tokens: np.ndarray, cand_offsets: np.ndarray,
                 weights: Dict[str, object], cfg, score_layers: Sequence[int],
                 candidates: Sequence[int] | None = None, act: str = "exact") -> Dict[int, np.ndarray]:
    """S[layer][i] for the requested candidates (default all): each candidate is forwarded
    alone as query||doc_i.  Returns {layer: float64 array indexed like `candidates`}.

    Layer-major over the weights (each layer's weights are materialised once, then applied to
    every requested candidate separately) so that 4B/8B-shaped weights need not be resident
    all at once; the values are those of the candidate-major loop."""
    if getattr(cfg, "arch", 0) == 1:   # encoder-only stack: same contract, other model definition
        from .encoder import encoder_score_matrix
        if act != "exact":
            raise ValueError("the encoder oracle has no rounded-activation mode")
        return encoder_score_matrix(query, cand_tokens, cand_offsets, weights, cfg, score_layers, candidates)
    n = len(cand_offsets) - 1
    ids = list(range(n)) if candidates is None else [int(c) for c in candidates]
    want = sorted(set(int(l) for l in score_layers))
    emb = weights["embed"]
    xs: List[np.ndarray] = []
    for i in ids:
        doc = cand_tokens[int(cand_offsets[i]): int(cand_offsets[i + 1])]
        seq = np.concatenate([np.asarray(query), np.asarray(doc)]).astype(np.int64)
        xs.append(np.asarray(emb[seq], dtype=np.float64))
    S = {l: np.zeros(len(ids), dtype=np.float64) for l in want}
    last = want[-1] if want else 0
    for l, w in enumerate(weights["layers"], start=1):
        if l > last:
            break
        w = {k: np.asarray(t, dtype=np.float64) for k, t in w.items()}   # widen once per layer
        for c in range(len(ids)):
            xs[c] = layer_forward(xs[c], w, cfg, act)
        if l in S:
            for c in range(len(ids)):
                S[l][c] = probe_score(xs[c][-1], weights["g_final"], weights["score_head"], cfg.rms_eps)
    return S
