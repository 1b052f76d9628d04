"""Oracle for 4-bit weight-only quantised weights (W4A16; test infrastructure).

The paper's quantised arm (Sec. 6.1) stores the weights as 4-bit codes with per-group scale and zero point and
computes with 16-bit activations: the forward pass is the unquantised one on the DEQUANTISED matrices.  This
module reads the packed format and rebuilds those matrices; the forward itself is reranker.py's.

Packed [N, K] matrix, group size G: N*K/2 code bytes (low nibble = even k, high nibble = odd k), then N*K/G bf16
scales, then N*K/G zero-point bytes, each section starting on a 16-byte boundary.
    value(n, k) = bf16( float32(scale[n, k // G]) * (code(n, k) - zero[n, k // G]) )
The product of a bf16 scale and an integer in [-15, 15] is exact in float32, so the only rounding is the final
one to bfloat16 (the type the GEMMs consume).
parity: pinned (hand-packed bytes with hand-computed values, nibble order, grid membership, fixed point of
re-quantisation; tests/test_oracle_quant.py).
"""
from __future__ import annotations

from typing import Dict

import numpy as np

from .reranker import to_bf16

MATRIX_SHAPES = {  # name -> (rows, cols) from the model configuration
    "w_qkv": lambda c: ((c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim, c.hidden),
    "w_o": lambda c: (c.hidden, c.n_q_heads * c.head_dim),
    "w_gate": lambda c: (c.ffn, c.hidden),
    "w_up": lambda c: (c.ffn, c.hidden),
    "w_down": lambda c: (c.hidden, c.ffn),
    "w_ffn1": lambda c: (c.ffn, c.hidden),   # encoder stack
    "w_ffn2": lambda c: (c.hidden, c.ffn),
}


def unpack_w4(blob: np.ndarray, n: int, k: int, group: int):
    """(codes [N, K] int, scales [N, K/G] float64, zeros [N, K/G] int) of a packed matrix."""
    b = np.asarray(blob, np.uint8)
    ng = k // group
    up16 = lambda v: (v + 15) // 16 * 16
    off_s = up16(n * k // 2)
    off_z = up16(off_s + 2 * n * ng)
    by = b[: n * k // 2].reshape(n, k // 2).astype(np.int64)
    codes = np.empty((n, k), np.int64)
    codes[:, 0::2] = by & 15
    codes[:, 1::2] = by >> 4
    bits = b[off_s: off_s + 2 * n * ng].reshape(n * ng, 2).astype(np.uint32)
    pattern = (bits[:, 0] | (bits[:, 1] << 8)) << 16          # bf16 pattern in the high half of a float32
    scales = pattern.astype(np.uint32).view(np.float32).astype(np.float64).reshape(n, ng)
    zeros = b[off_z: off_z + n * ng].reshape(n, ng).astype(np.int64)
    return codes, scales, zeros


def dequantize_w4(blob: np.ndarray, n: int, k: int, group: int) -> np.ndarray:
    """The [N, K] matrix a packed blob stands for, as float64 holding bf16-representable values."""
    codes, scales, zeros = unpack_w4(blob, n, k, group)
    g = np.arange(k) // group
    return to_bf16((scales[:, g] * (codes - zeros[:, g])).astype(np.float32))


def dequantize_weights(wq: Dict[str, object], cfg, group: int) -> Dict[str, object]:
    """Model weights with every packed layer matrix replaced by the matrix it stands for."""
    out = {k: v for k, v in wq.items() if k != "layers"}
    out["layers"] = [{name: (dequantize_w4(t, *MATRIX_SHAPES[name](cfg), group) if name in MATRIX_SHAPES else t)
                      for name, t in layer.items()} for layer in wq["layers"]]
    return out
