"""Pins for the W4A16 dequantisation oracle (CPU): bytes packed by hand with values computed by hand, the nibble
order, membership of every value in its group's grid, and re-quantisation as a fixed point."""
import numpy as np

import oracle
import synth
from synth.configs import DTYPE_BF16, ModelCfg


def test_hand_packed_matrix():
    """N = 1, K = 4, G = 2.  Codes 3, 12, 0, 15; scales 0.5 and 2.0 (bf16 patterns 0x3F00, 0x4000); zero points 4, 7.
    Values: 0.5 * (3 - 4) = -0.5, 0.5 * (12 - 4) = 4, 2 * (0 - 7) = -14, 2 * (15 - 7) = 16."""
    blob = np.zeros(48, np.uint8)
    blob[0] = 3 | (12 << 4)          # k = 0 in the low nibble, k = 1 in the high nibble
    blob[1] = 0 | (15 << 4)
    blob[16:20] = [0x00, 0x3F, 0x00, 0x40]   # little-endian bf16: 0.5, 2.0 (section starts at byte 16)
    blob[32:34] = [4, 7]                     # zero points (section starts at byte 32)
    codes, scales, zeros = oracle.unpack_w4(blob, 1, 4, 2)
    assert codes.tolist() == [[3, 12, 0, 15]] and scales.tolist() == [[0.5, 2.0]] and zeros.tolist() == [[4, 7]]
    assert oracle.dequantize_w4(blob, 1, 4, 2).tolist() == [[-0.5, 4.0, -14.0, 16.0]]


def test_value_is_rounded_to_bfloat16_once():
    """scale 0.00170135498046875 (bf16 0x3ADF) times 13 = 0.02211761474609375 is not a bf16 value; the nearest is
    0.0220947265625 (0x3CB5)."""
    blob = np.zeros(48, np.uint8)
    blob[0] = 15 | (2 << 4)
    blob[16:18] = [0xDF, 0x3A]
    blob[32] = 2
    v = oracle.dequantize_w4(blob, 1, 2, 2)
    assert v.tolist() == [[0.0220947265625, 0.0]]


def test_values_lie_on_the_group_grid_and_requantise_to_themselves():
    rng = np.random.default_rng(0)
    n, k, g = 24, 256, 64
    w = (rng.normal(size=(n, k)) * 0.02).astype(np.float32)
    codes, scales, zeros = synth.quantize_matrix(w, g)
    blob = synth.pack_matrix(codes, scales, zeros, g)
    assert blob.size == synth.packed_sections(n, k, g)[2]
    c2, s2, z2 = oracle.unpack_w4(blob, n, k, g)
    assert np.array_equal(c2, codes) and np.array_equal(s2, scales.astype(np.float64)) and np.array_equal(z2, zeros)
    d = oracle.dequantize_w4(blob, n, k, g)
    grp = np.arange(k) // g
    exact = scales.astype(np.float64)[:, grp] * (codes.astype(np.int64) - zeros.astype(np.int64)[:, grp])
    assert np.max(np.abs(d - exact)) <= np.max(np.abs(exact)) * 2.0 ** -8            # one bf16 rounding
    assert np.max(np.abs(d - w)) <= 0.5 * scales.max() * 1.01 + np.max(np.abs(exact)) * 2.0 ** -8   # round to nearest code
    # 16 levels per group at most
    for r in range(n):
        for j in range(k // g):
            assert len(np.unique(d[r, j * g:(j + 1) * g])) <= 16
    # quantising the dequantised matrix with the same grid gives the same codes
    again = np.clip(np.rint(exact / scales.astype(np.float64)[:, grp]) + zeros.astype(np.int64)[:, grp], 0, 15)
    assert np.array_equal(again, codes)


def test_quantised_model_forward_uses_the_dequantised_matrices():
    cfg = ModelCfg(n_layers=2, hidden=64, n_q_heads=2, n_kv_heads=1, head_dim=32, ffn=128, vocab=50, rope_theta=1e4,
                   dtype=DTYPE_BF16)
    w = synth.make_weights(cfg, seed=1)
    wq = synth.quantize_weights(w, group=32)
    wd = oracle.dequantize_weights(wq, cfg, 32)
    assert wd["layers"][0]["w_qkv"].shape == (128, 64) and wd["layers"][1]["w_down"].shape == (64, 128)
    assert np.array_equal(wd["layers"][0]["g_attn"], w["layers"][0]["g_attn"])       # vectors untouched
    toks = np.arange(9) % 50
    a = oracle.candidate_scores(toks, wd, cfg, [2])[2]
    b = oracle.candidate_scores(toks, w, cfg, [2])[2]
    assert a != b and abs(a - b) < 0.25                   # a different model, close to the unquantised one
