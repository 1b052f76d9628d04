"""Counter-based weight generator: every tensor is a pure function of (seed, tensor name).

Values are i.i.d. N(0, 0.02^2) for matrices and 1 + 0.1*N(0,1) for norm gains (gains are
jittered away from exactly 1 so that a kernel that forgot the gain multiply fails parity).
In bf16 mode every value is rounded once to bf16 (round-to-nearest-even) and both the
oracle and the CUDA path consume the rounded values.
"""
from __future__ import annotations

import os
import zlib
from concurrent.futures import ThreadPoolExecutor
from typing import Dict, Iterator, Tuple

import numpy as np

from .configs import ARCH_ENCODER, DTYPE_BF16, ModelCfg

W_STD = 0.02
GAIN_JITTER = 0.1


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """fp32 array -> fp32 array whose values are exactly representable in bf16 (RNE)."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (b + (np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1)))) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bf16_bits(x_rounded: np.ndarray) -> np.ndarray:
    """fp32 array of bf16-representable values -> uint16 bf16 bit patterns."""
    b = np.ascontiguousarray(x_rounded, dtype=np.float32).view(np.uint32)
    return (b >> np.uint32(16)).astype(np.uint16)


CHUNK = 1 << 20   # elements per independently keyed Philox stream (part of the definition)
_POOL = ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1))


def _fill_chunk(args) -> None:
    out, seed, name_key, c, gain, to_bf16 = args
    g = np.random.Generator(np.random.Philox(key=[seed & 0xFFFFFFFFFFFFFFFF, name_key | (c << 32)]))
    lo = c * CHUNK
    hi = min(out.size, lo + CHUNK)
    x = g.standard_normal(hi - lo, dtype=np.float32)
    if gain:
        x = np.float32(1.0) + np.float32(GAIN_JITTER) * x
    else:
        x *= np.float32(W_STD)
    out[lo:hi] = round_to_bf16(x) if to_bf16 else x


def tensor(seed: int, name: str, shape: Tuple[int, ...], cfg: ModelCfg, gain: bool = False) -> np.ndarray:
    """Element e of the tensor is draw (e mod CHUNK) of the Philox stream keyed by
    (seed, crc32(name) + 2^32 * (e div CHUNK)); chunks are filled by a thread pool."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.float32)
    key = zlib.crc32(name.encode())
    jobs = [(out, seed, key, c, gain, cfg.dtype == DTYPE_BF16) for c in range((n + CHUNK - 1) // CHUNK)]
    list(_POOL.map(_fill_chunk, jobs))
    return out.reshape(shape)


def layer_tensor_shapes(cfg: ModelCfg) -> Dict[str, Tuple[Tuple[int, ...], bool]]:
    d, dh = cfg.hidden, cfg.head_dim
    if cfg.arch == ARCH_ENCODER:
        # biases and LayerNorm shifts are drawn like matrix entries (non-zero, so that a dropped bias fails parity)
        return {
            "w_qkv": ((cfg.qkv_rows, d), False), "b_qkv": ((cfg.qkv_rows,), False),
            "w_o": ((d, cfg.n_q_heads * dh), False), "b_o": ((d,), False),
            "ln1_g": ((d,), True), "ln1_b": ((d,), False),
            "w_ffn1": ((cfg.ffn, d), False), "b_ffn1": ((cfg.ffn,), False),
            "w_ffn2": ((d, cfg.ffn), False), "b_ffn2": ((d,), False),
            "ln2_g": ((d,), True), "ln2_b": ((d,), False),
        }
    out = {
        "g_attn": ((d,), True),
        "w_qkv": ((cfg.qkv_rows, d), False),   # rows: all q heads, then k heads, then v heads
        "w_o": ((d, cfg.n_q_heads * dh), False),
        "g_ffn": ((d,), True),
        "w_gate": ((cfg.ffn, d), False),
        "w_up": ((cfg.ffn, d), False),
        "w_down": ((d, cfg.ffn), False),
    }
    if cfg.qk_norm:
        out["g_q"] = ((dh,), True)
        out["g_k"] = ((dh,), True)
    return out


def make_layer(cfg: ModelCfg, layer: int, seed: int = 0) -> Dict[str, np.ndarray]:
    return {k: tensor(seed, f"layers.{layer}.{k}", shp, cfg, gain)
            for k, (shp, gain) in layer_tensor_shapes(cfg).items()}


def make_globals(cfg: ModelCfg, seed: int = 0, embed_rows: np.ndarray | None = None) -> Dict[str, np.ndarray]:
    """embed [V, D], g_final [D], score_head [2, D] (row 0 = "yes", row 1 = "no").

    The score head is a separate two-row matrix, not tied to the embedding table.
    ARCH_ENCODER: embed, pos_embed [max_positions, D], type_embed [D], the embedding LayerNorm, and the
    classification head: dense [D, D] + bias, tanh, out_proj [D] + bias [1]."""
    if cfg.arch == ARCH_ENCODER:
        d = cfg.hidden
        shapes = {"embed": ((cfg.vocab, d), False), "pos_embed": ((cfg.max_positions, d), False),
                  "type_embed": ((d,), False), "emb_ln_g": ((d,), True), "emb_ln_b": ((d,), False),
                  "head_dense_w": ((d, d), False), "head_dense_b": ((d,), False),
                  "head_out_w": ((d,), False), "head_out_b": ((1,), False)}
        return {k: tensor(seed, k, shp, cfg, gain) for k, (shp, gain) in shapes.items()}
    out = {
        "embed": tensor(seed, "embed", (cfg.vocab, cfg.hidden), cfg),
        "g_final": tensor(seed, "g_final", (cfg.hidden,), cfg, gain=True),
        "score_head": tensor(seed, "score_head", (2, cfg.hidden), cfg),
    }
    return out


def iter_layers(cfg: ModelCfg, seed: int = 0) -> Iterator[Dict[str, np.ndarray]]:
    for l in range(cfg.n_layers):
        yield make_layer(cfg, l, seed)


def make_weights(cfg: ModelCfg, seed: int = 0) -> Dict[str, object]:
    """All weights in host memory: {'embed', 'g_final', 'score_head', 'layers': [dict, ...]}."""
    w: Dict[str, object] = dict(make_globals(cfg, seed))
    w["layers"] = list(iter_layers(cfg, seed))
    return w
