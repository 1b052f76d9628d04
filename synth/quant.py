"""Seeded stand-in for the W4A16 weights of the paper's quantised arm (Sec. 6.1: the method composed with 4-bit
weight-only quantisation).  GPTQ's calibrated rounding needs trained weights and calibration data; here every
matrix of the synthetic model is quantised round-to-nearest with one asymmetric 4-bit grid per group of `group`
consecutive input channels, which yields the same storage format: 4-bit codes, one bf16 scale and one 4-bit zero
point per group.  This module only PRODUCES the packed inputs; reading them back (dequantisation) is the path's
arithmetic and is implemented separately by the oracle and by the CUDA kernels.

Packed layout of one [N, K] matrix (a single byte blob; every section starts on a 16-byte boundary):
    codes   N * K / 2 bytes   row-major; byte (n, k // 2) holds code(n, k) in its low nibble for even k and
                              code(n, k) in its high nibble for odd k
    scales  N * K / group bf16 values (little-endian 16-bit patterns), row-major [N, K / group]
    zeros   N * K / group bytes, row-major, values 0..15
value(n, k) = bf16( float32(scale[n, k // group]) * (code(n, k) - zero[n, k // group]) )
"""
from __future__ import annotations

from typing import Dict

import numpy as np

from .weights import bf16_bits, round_to_bf16

MATRICES = ("w_qkv", "w_o", "w_gate", "w_up", "w_down", "w_ffn1", "w_ffn2")   # decoder and encoder layer matrices


def _align16(v: int) -> int:
    return (v + 15) // 16 * 16


def packed_sections(n: int, k: int, group: int):
    """(offset of scales, offset of zeros, total bytes) of the blob of an [n, k] matrix."""
    off_s = _align16(n * k // 2)
    off_z = _align16(off_s + 2 * n * (k // group))
    return off_s, off_z, _align16(off_z + n * (k // group))


def quantize_matrix(w: np.ndarray, group: int):
    """Round-to-nearest asymmetric 4-bit quantisation per group.  Returns (codes uint8 [N, K], scales float32
    [N, K/group] holding bf16-representable values, zeros uint8 [N, K/group])."""
    n, k = w.shape
    assert k % group == 0 and group % 2 == 0
    g = np.asarray(w, np.float32).reshape(n, k // group, group)
    lo = np.minimum(g.min(axis=2), 0.0)
    hi = np.maximum(g.max(axis=2), 0.0)
    scale = round_to_bf16(((hi - lo) / np.float32(15.0)).astype(np.float32))
    scale = np.where(scale > 0, scale, np.float32(1.0)).astype(np.float32)
    zero = np.clip(np.rint(-lo / scale), 0, 15).astype(np.uint8)
    codes = np.clip(np.rint(g / scale[..., None]) + zero[..., None], 0, 15).astype(np.uint8)
    return codes.reshape(n, k), scale, zero


def pack_matrix(codes: np.ndarray, scales: np.ndarray, zeros: np.ndarray, group: int) -> np.ndarray:
    n, k = codes.shape
    off_s, off_z, total = packed_sections(n, k, group)
    blob = np.zeros(total, np.uint8)
    blob[: n * k // 2] = (codes[:, 0::2] | (codes[:, 1::2] << 4)).reshape(-1)
    blob[off_s: off_s + 2 * n * (k // group)] = bf16_bits(scales).astype("<u2").view(np.uint8).reshape(-1)
    blob[off_z: off_z + n * (k // group)] = zeros.reshape(-1)
    return blob


def quantize_layer(layer: Dict[str, np.ndarray], group: int) -> Dict[str, np.ndarray]:
    """A layer dict whose matrices are replaced by packed uint8 blobs (vectors are kept)."""
    out = {}
    for name, t in layer.items():
        out[name] = pack_matrix(*quantize_matrix(t, group), group) if name in MATRICES else t
    return out


def quantize_weights(w: Dict[str, object], group: int = 128) -> Dict[str, object]:
    """The model with every layer matrix packed as W4; embedding, norms and score head unchanged."""
    out = {k: v for k, v in w.items() if k != "layers"}
    out["layers"] = [quantize_layer(l, group) for l in w["layers"]]
    return out
