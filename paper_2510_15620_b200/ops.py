"""Same-name Python bindings of include/prism_ops.h (argument marshalling only; device tensors in,
device tensors out; work is enqueued on torch's current stream)."""
from __future__ import annotations

import ctypes as C

import torch

from .binding import PrismError, lib, _ProbeRecord

_proto_done = False


def _L():
    global _proto_done
    L = lib()
    if not _proto_done:
        vp, i32, f32, f64 = C.c_void_p, C.c_int32, C.c_float, C.c_double
        L.prism_op_pack.argtypes = [vp, i32, vp, vp, i32, i32, i32, vp, vp, vp, vp, vp, vp]
        L.prism_op_embed.argtypes = [vp, i32, vp, i32, i32, vp, vp]
        L.prism_op_rmsnorm.argtypes = [vp, vp, i32, i32, i32, f32, vp, vp]
        L.prism_op_qknorm_rope.argtypes = [vp, i32, vp, i32, i32, i32, i32, i32, vp, vp, f32, f32, i32, vp]
        L.prism_op_gemm.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, vp, vp]
        L.prism_op_gemm_qkv_rope.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, vp, vp, f32, vp, f32, i32, vp, vp]
        L.prism_op_gemm_qkv_rope.restype = C.c_int
        L.prism_op_attention.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, i32, i32, vp, vp]
        L.prism_op_probe.argtypes = [vp, vp, i32, i32, vp, vp, i32, f32, vp, vp]
        L.prism_op_route.argtypes = [vp, vp, vp, i32, i32, i32, f64, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]
        L.prism_op_route_static.argtypes = L.prism_op_route.argtypes
        L.prism_op_route_static.restype = C.c_int
        L.prism_op_wait_selftest.argtypes = [C.c_uint64, vp, vp]
        L.prism_op_wait_selftest.restype = C.c_int
        L.prism_op_compact.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, vp]
        L.prism_op_gemm_bias.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, vp, vp]
        L.prism_op_layernorm.argtypes = [vp, vp, vp, i32, i32, i32, f32, vp, vp]
        L.prism_op_embed_encoder.argtypes = [vp, vp, vp, i32, vp, vp, i32, i32, i32, vp, vp]
        L.prism_op_probe_encoder.argtypes = [vp, vp, i32, i32, vp, vp, f32, vp, i32, vp, vp, vp, vp, vp]
        L.prism_op_dequant_w4.argtypes = [vp, i32, i32, i32, vp, vp]
        for n in ("gemm_bias", "layernorm", "embed_encoder", "probe_encoder", "dequant_w4"):
            getattr(L, "prism_op_" + n).restype = C.c_int
        for n in ("pack", "embed", "rmsnorm", "qknorm_rope", "gemm", "attention", "probe", "route", "compact"):
            getattr(L, "prism_op_" + n).restype = C.c_int
        _proto_done = True
    return L


def _p(t):
    return None if t is None else t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def _check(rc, what):
    if rc != 0:
        raise PrismError(rc, what)


def prism_op_pack(query, cand_tokens, cand_offsets, total, vocab, tokens, pos, cu, seq2orig, err_word):
    _check(_L().prism_op_pack(_p(query), query.numel(), _p(cand_tokens), _p(cand_offsets), cand_offsets.numel() - 1,
                              total, vocab, _p(tokens), _p(pos), _p(cu), _p(seq2orig), _p(err_word), _stream()), "pack")


def prism_op_embed(table, dtype, tokens, x):
    _check(_L().prism_op_embed(_p(table), dtype, _p(tokens), tokens.numel(), x.shape[1], _p(x), _stream()), "embed")


def prism_op_rmsnorm(x, gain, dtype, eps, out):
    _check(_L().prism_op_rmsnorm(_p(x), _p(gain), dtype, x.shape[0], x.shape[1], eps, _p(out), _stream()), "rmsnorm")


def prism_op_qknorm_rope(qkv, dtype, pos, n_q_heads, n_kv_heads, head_dim, qk_norm, g_q, g_k, eps, theta, max_pos):
    _check(_L().prism_op_qknorm_rope(_p(qkv), dtype, _p(pos), qkv.shape[0], n_q_heads, n_kv_heads, head_dim, qk_norm,
                                     _p(g_q), _p(g_k), eps, theta, max_pos, _stream()), "qknorm_rope")


def prism_op_gemm(a, b, b2, out, resid, m, n, k, dtype, epilogue, impl, err_word):
    _check(_L().prism_op_gemm(_p(a), _p(b), _p(b2), _p(out), _p(resid), m, n, k, dtype, epilogue, impl, _p(err_word),
                              _stream()), "gemm")


def prism_op_dequant_w4(blob, n, k, group, out):
    _check(_L().prism_op_dequant_w4(_p(blob), n, k, group, _p(out), _stream()), "dequant_w4")


def prism_op_gemm_bias(a, b, bias, out, resid, m, n, k, dtype, epilogue, impl, err_word):
    _check(_L().prism_op_gemm_bias(_p(a), _p(b), _p(bias), _p(out), _p(resid), m, n, k, dtype, epilogue, impl, _p(err_word),
                                   _stream()), "gemm_bias")


def prism_op_layernorm(x, gain, shift, dtype, eps, out):
    _check(_L().prism_op_layernorm(_p(x), _p(gain), _p(shift), dtype, x.shape[0], x.shape[1], eps, _p(out), _stream()),
           "layernorm")


def prism_op_embed_encoder(table, pos_table, type_row, dtype, tokens, pos, pos_offset, x):
    _check(_L().prism_op_embed_encoder(_p(table), _p(pos_table), _p(type_row), dtype, _p(tokens), _p(pos), pos_offset,
                                       tokens.numel(), x.shape[1], _p(x), _stream()), "embed_encoder")


def prism_op_probe_encoder(x, cu, n, gain, shift, eps, dense_w, dtype, dense_b, out_w, out_b, scores):
    _check(_L().prism_op_probe_encoder(_p(x), _p(cu), n, x.shape[1], _p(gain), _p(shift), eps, _p(dense_w), dtype, _p(dense_b),
                                       _p(out_w), _p(out_b), _p(scores), _stream()), "probe_encoder")


def prism_op_gemm_qkv_rope(a, w_qkv, out, m, k, n_q_heads, n_kv_heads, qk_norm, g_q, g_k, eps, pos, theta, max_pos, err_word):
    _check(_L().prism_op_gemm_qkv_rope(_p(a), _p(w_qkv), _p(out), m, k, n_q_heads, n_kv_heads, qk_norm, _p(g_q), _p(g_k),
                                       eps, _p(pos), theta, max_pos, _p(err_word), _stream()), "gemm_qkv_rope")


def prism_op_attention(qkv, out, cu, n_seq, max_len, n_q_heads, n_kv_heads, head_dim, causal, dtype, impl, err_word=None):
    _check(_L().prism_op_attention(_p(qkv), _p(out), _p(cu), n_seq, qkv.shape[0], max_len, n_q_heads, n_kv_heads, head_dim,
                                   causal, dtype, impl, _p(err_word), _stream()), "attention")


def prism_op_probe(x, cu, n, g_final, score_head, dtype, eps, scores):
    _check(_L().prism_op_probe(_p(x), _p(cu), n, x.shape[1], _p(g_final), _p(score_head), dtype, eps, _p(scores),
                               _stream()), "probe")


def prism_op_route(scores, cu_old, seq2orig_old, n, mode, keep_count, cv_threshold, n_clusters, std_ddof, select_winners,
                   is_final, layer, cu_new, seq2orig_new, old_of_new, state, res_idx, res_score, rec):
    _check(_L().prism_op_route(_p(scores), _p(cu_old), _p(seq2orig_old), n, mode, keep_count, cv_threshold, n_clusters,
                               std_ddof, select_winners, is_final, layer, _p(cu_new), _p(seq2orig_new), _p(old_of_new),
                               _p(state), _p(res_idx), _p(res_score), _p(rec), _stream()), "route")


def prism_op_route_static(scores, cu_old, seq2orig_old, n, mode, keep_count, cv_threshold, n_clusters, std_ddof,
                          select_winners, is_final, layer, cu_new, seq2orig_new, old_of_new, state, res_idx, res_score, rec):
    """prism_op_route without any device allocation (scratch built into the library; n <= 1024)."""
    _check(_L().prism_op_route_static(_p(scores), _p(cu_old), _p(seq2orig_old), n, mode, keep_count, cv_threshold,
                                      n_clusters, std_ddof, select_winners, is_final, layer, _p(cu_new), _p(seq2orig_new),
                                      _p(old_of_new), _p(state), _p(res_idx), _p(res_score), _p(rec), _stream()),
           "route_static")


def prism_op_compact(x_old, x_new, cu_old, cu_new, old_of_new, n_new, total_new):
    _check(_L().prism_op_compact(_p(x_old), _p(x_new), _p(cu_old), _p(cu_new), _p(old_of_new), n_new, total_new,
                                 x_old.shape[1], _stream()), "compact")


def prism_op_wait_selftest(limit_cycles, err_word):
    _check(_L().prism_op_wait_selftest(int(limit_cycles), _p(err_word), _stream()), "wait_selftest")


RECORD_BYTES = C.sizeof(_ProbeRecord)


def decode_record(buf: torch.Tensor) -> _ProbeRecord:
    """A uint8 tensor holding one prism_probe_record (copied from the device) -> ctypes struct."""
    raw = bytes(buf.cpu().numpy().tobytes())
    return _ProbeRecord.from_buffer_copy(raw)
