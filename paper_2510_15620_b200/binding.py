"""ctypes mirror of include/prism.h.  Argument marshalling only."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass, field
from typing import Callable, Dict, List, Optional, Sequence

import numpy as np
import torch

PRISM_FP32, PRISM_BF16 = 0, 1
PRISM_IMPL_AUTO, PRISM_IMPL_SIMT, PRISM_IMPL_MMA, PRISM_IMPL_SOLO = 0, 1, 2, 3
PRISM_ARCH_DECODER, PRISM_ARCH_ENCODER = 0, 1
PRISM_WFMT_PLAIN, PRISM_WFMT_W4 = 0, 1
PRISM_MAX_CLUSTERS = 8

# PRISM_LIBRARY overrides the in-tree library (e.g. an instrumented build of the same sources).
_LIB_PATH = os.environ.get("PRISM_LIBRARY") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "lib", "libprism.so")
_lib = None



EXCHANGE_FN = C.CFUNCTYPE(C.c_int, C.c_void_p, C.c_int32, C.c_void_p)


def shard_candidates(lengths: Sequence[int], world_size: int) -> np.ndarray:
    """Owner rank of every candidate: longest first, each to the rank with the fewest tokens so far (ties: lowest
    rank).  Deterministic, so every rank computes the same partition from the same lengths."""
    lengths = np.asarray(lengths, dtype=np.int64)
    owner = np.zeros(len(lengths), dtype=np.int32)
    load = np.zeros(max(world_size, 1), dtype=np.int64)
    for i in np.argsort(-lengths, kind="stable"):
        r = int(np.argmin(load))
        owner[i] = r
        load[r] += lengths[i]
    return owner


def all_reduce_scores(t: torch.Tensor, group=None) -> None:
    """The `reduce` argument of select_sharded for torch.distributed: a SUM all-reduce (NCCL on GPUs), enqueued
    on the current stream."""
    import torch.distributed as dist
    dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)


class PrismError(RuntimeError):
    def __init__(self, status: int, text: str = ""):
        self.status = status
        super().__init__(f"{status_str(status)} ({status}): {text}")


class _ModelCfg(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("hidden", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("ffn", C.c_int32), ("vocab", C.c_int32), ("rope_theta", C.c_float),
                ("rms_eps", C.c_float), ("causal", C.c_int32), ("qk_norm", C.c_int32), ("dtype", C.c_int32),
                ("max_seq_len", C.c_int32), ("max_candidates", C.c_int32), ("max_total_tokens", C.c_int32),
                ("activation_budget_bytes", C.c_int64), ("weight_residency", C.c_int32), ("gemm_impl", C.c_int32),
                ("attention_impl", C.c_int32), ("embed_cache_rows", C.c_int32), ("hidden_offload", C.c_int32),
                ("shared_prefix", C.c_int32), ("arch", C.c_int32), ("max_positions", C.c_int32),
                ("pos_offset", C.c_int32), ("weight_format", C.c_int32), ("quant_group", C.c_int32)]


class _LayerWeights(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in ("g_attn", "w_qkv", "g_q", "g_k", "w_o", "g_ffn", "w_gate", "w_up", "w_down")]


class _Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("g_final", C.c_void_p), ("score_head", C.c_void_p),
                ("layers", C.POINTER(_LayerWeights))]


_ENC_LAYER_KEYS = ("w_qkv", "b_qkv", "w_o", "b_o", "ln1_g", "ln1_b", "w_ffn1", "b_ffn1", "w_ffn2", "b_ffn2", "ln2_g", "ln2_b")
_ENC_GLOBAL_KEYS = ("embed", "pos_embed", "type_embed", "emb_ln_g", "emb_ln_b", "head_dense_w", "head_dense_b",
                    "head_out_w", "head_out_b")


class _EncLayerWeights(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in _ENC_LAYER_KEYS]


class _EncWeights(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in _ENC_GLOBAL_KEYS] + [("layers", C.POINTER(_EncLayerWeights))]


class _Schedule(C.Structure):
    _fields_ = [("mode", C.c_int32), ("n_probes", C.c_int32), ("probe_layers", C.POINTER(C.c_int32)),
                ("keep_counts", C.POINTER(C.c_int32)), ("cv_threshold", C.c_double), ("n_clusters", C.c_int32),
                ("std_ddof", C.c_int32), ("select_winners", C.c_int32)]


class _ProbeRecord(C.Structure):
    _fields_ = [("layer", C.c_int32), ("n_active_before", C.c_int32), ("fired", C.c_int32), ("n_selected", C.c_int32),
                ("n_dropped", C.c_int32), ("n_deferred", C.c_int32), ("k_rem_after", C.c_int32), ("n_cuts", C.c_int32),
                ("cuts", C.c_int32 * PRISM_MAX_CLUSTERS), ("tokens_before", C.c_int32), ("cv", C.c_double)]


class _Trace(C.Structure):
    _fields_ = [("capacity", C.c_int32), ("n_records", C.c_int32), ("records", C.POINTER(_ProbeRecord)),
                ("scores", C.POINTER(C.c_float)), ("ids", C.POINTER(C.c_int32)), ("layers_run", C.c_int32),
                ("tokens_per_layer", C.POINTER(C.c_int32)), ("n_chunks_max", C.c_int32),
                ("workspace_bytes", C.c_int64), ("shared_prefix_rows", C.c_int32), ("reserved", C.c_int32)]


class Calibrator(C.Structure):
    """Mirror of prism_calibrator; create with the `in` fields set, pass to PrismModel.select_calibrated."""
    _fields_ = [("threshold", C.c_double), ("target_precision", C.c_double), ("raise_factor", C.c_double),
                ("lower_factor", C.c_double), ("min_threshold", C.c_double), ("max_threshold", C.c_double),
                ("sample_every", C.c_int32), ("window", C.c_int32), ("n_in_window", C.c_int32),
                ("n_adjustments", C.c_int32), ("n_requests", C.c_int64), ("n_sampled", C.c_int64),
                ("precision_sum", C.c_double), ("last_precision", C.c_double), ("last_window_precision", C.c_double)]


def lib() -> C.CDLL:
    """The loaded C-ABI library.  Raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2510_15620_b200._build`")
        L = C.CDLL(_LIB_PATH)
        L.prism_status_str.restype = C.c_char_p
        L.prism_status_str.argtypes = [C.c_int]
        L.prism_last_error.restype = C.c_char_p
        L.prism_last_error.argtypes = [C.c_void_p]
        L.prism_launch_count.restype = C.c_int64
        L.prism_launch_count.argtypes = [C.c_void_p]
        L.prism_create.restype = C.c_int
        L.prism_create.argtypes = [C.POINTER(_ModelCfg), C.POINTER(_Weights), C.POINTER(C.c_void_p)]
        L.prism_create_encoder.restype = C.c_int
        L.prism_create_encoder.argtypes = [C.POINTER(_ModelCfg), C.POINTER(_EncWeights), C.POINTER(C.c_void_p)]
        L.prism_embed_cache_stats.restype = C.c_int
        L.prism_embed_cache_stats.argtypes = [C.c_void_p, C.POINTER(C.c_int64), C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
        L.prism_destroy.restype = None
        L.prism_destroy.argtypes = [C.c_void_p]
        sel = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.POINTER(_Schedule),
               C.c_void_p, C.c_void_p, C.POINTER(C.c_int32), C.POINTER(_Trace), C.c_void_p]
        for f in (L.prism_select, L.prism_select_host):
            f.restype = C.c_int
            f.argtypes = sel
        L.prism_select_calibrated.restype = C.c_int
        L.prism_select_calibrated.argtypes = sel[:8] + [C.POINTER(Calibrator)] + sel[8:]
        L.prism_select_sharded.restype = C.c_int
        L.prism_select_sharded.argtypes = sel[:8] + [C.c_void_p, C.c_void_p, EXCHANGE_FN, C.c_void_p] + sel[8:]
        _lib = L
    return _lib


def status_str(status: int) -> str:
    return lib().prism_status_str(int(status)).decode()


@dataclass
class ProbeRecord:
    layer: int
    n_active_before: int
    fired: int
    n_selected: int
    n_dropped: int
    n_deferred: int
    k_rem_after: int
    cuts: List[int]
    tokens_before: int
    cv: float
    active_ids: List[int] = field(default_factory=list)
    scores: np.ndarray = field(default_factory=lambda: np.zeros(0, np.float32))


@dataclass
class Trace:
    records: List[ProbeRecord]
    layers_run: int
    tokens_per_layer: List[int]
    n_chunks_max: int
    workspace_bytes: int
    shared_prefix_rows: int = 0


def upload_weights(w: Dict[str, object], dtype: int, device: str = "cuda", layers_pinned_host: bool = False,
                   embed_pinned_host: bool = False):
    """numpy weights (as produced by the synthetic generator: float32 values, already bf16-rounded in
    bf16 mode) -> torch tensors of the library's element type.  Layer tensors go to pinned host memory
    when they are to be streamed, the embedding table when it is to be cached row by row."""
    def conv(a: np.ndarray, pinned: bool) -> torch.Tensor:
        if a.dtype == np.uint8:             # a packed W4 matrix: bytes as they are
            t = torch.from_numpy(np.ascontiguousarray(a))
            return t.pin_memory() if pinned else t.to(device)
        t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
        if dtype == PRISM_BF16:
            t = t.to(torch.bfloat16)        # exact: the values are bf16-representable
        if pinned:
            return t.pin_memory()
        return t.to(device)
    out: Dict[str, object] = {k: conv(v, embed_pinned_host and k == "embed") for k, v in w.items() if k != "layers"}
    out["layers"] = [{k: conv(v, layers_pinned_host) for k, v in lw.items()} for lw in w["layers"]]
    return out


class PrismModel:
    """One prism_handle.  `cfg` is any object with the ModelCfg fields (n_layers, hidden, ...)."""

    def __init__(self, cfg, weights: Dict[str, object], max_seq_len: int, max_candidates: int, max_total_tokens: int,
                 activation_budget_bytes: int = 0, stream_weights: bool = False, gemm_impl: int = PRISM_IMPL_AUTO,
                 attention_impl: int = PRISM_IMPL_AUTO, embed_cache_rows: int = 0, hidden_offload: bool = False,
                 shared_prefix: bool = True, weight_format: int = 0, quant_group: int = 0):
        self._h = C.c_void_p()
        self.cfg = cfg
        self._weights = weights            # keep the tensors alive for the life of the handle
        c = _ModelCfg(cfg.n_layers, cfg.hidden, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.ffn, cfg.vocab,
                      cfg.rope_theta, cfg.rms_eps, cfg.causal, cfg.qk_norm, cfg.dtype, max_seq_len, max_candidates,
                      max_total_tokens, activation_budget_bytes, 1 if stream_weights else 0, gemm_impl, attention_impl,
                      embed_cache_rows, 1 if hidden_offload else 0, 0 if shared_prefix else 1,
                      getattr(cfg, "arch", 0), getattr(cfg, "max_positions", 0), getattr(cfg, "pos_offset", 0),
                      weight_format, quant_group)
        if getattr(cfg, "arch", 0) == PRISM_ARCH_ENCODER:
            elayers = (_EncLayerWeights * cfg.n_layers)()
            for i, lw in enumerate(weights["layers"]):
                for k in _ENC_LAYER_KEYS:
                    setattr(elayers[i], k, lw[k].data_ptr())
            ew = _EncWeights(*[weights[k].data_ptr() for k in _ENC_GLOBAL_KEYS], elayers)
            rc = lib().prism_create_encoder(C.byref(c), C.byref(ew), C.byref(self._h))
            if rc != 0:
                raise PrismError(rc, "prism_create_encoder")
            self.max_candidates = max_candidates
            return
        layers = (_LayerWeights * cfg.n_layers)()
        for i, lw in enumerate(weights["layers"]):
            for k, _ in _LayerWeights._fields_:
                setattr(layers[i], k, lw[k].data_ptr() if k in lw else None)
        w = _Weights(weights["embed"].data_ptr(), weights["g_final"].data_ptr(), weights["score_head"].data_ptr(), layers)
        rc = lib().prism_create(C.byref(c), C.byref(w), C.byref(self._h))
        if rc != 0:
            raise PrismError(rc, "prism_create")
        self.max_candidates = max_candidates

    def close(self) -> None:
        if self._h:
            lib().prism_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def embed_cache_stats(self):
        """(hits, misses, evictions) of the embedding-row cache since the handle was created."""
        h, m, e = C.c_int64(0), C.c_int64(0), C.c_int64(0)
        lib().prism_embed_cache_stats(self._h, C.byref(h), C.byref(m), C.byref(e))
        return int(h.value), int(m.value), int(e.value)

    @property
    def launch_count(self) -> int:
        return int(lib().prism_launch_count(self._h))

    def _schedule(self, sched) -> Optional[_Schedule]:
        if sched is None:
            return None
        pl = list(sched.probe_layers)
        kc = list(sched.keep_counts)
        self._pl = (C.c_int32 * max(1, len(pl)))(*pl)
        self._kc = (C.c_int32 * max(1, len(kc)))(*kc)
        return _Schedule(sched.mode, len(pl), self._pl, self._kc if kc else None, float(sched.cv_threshold),
                         sched.n_clusters, sched.std_ddof, sched.select_winners)

    def _call(self, fn, q_ptr, lq, c_ptr, o_ptr, n, k, sched, idx_ptr, sc_ptr, want_trace, stream):
        s = self._schedule(sched)
        n_out = C.c_int32(0)
        tr = None
        if want_trace:
            cap = self.cfg.n_layers
            recs = (_ProbeRecord * cap)()
            sc = np.zeros((cap, max(n, 1)), np.float32)
            ids = np.zeros((cap, max(n, 1)), np.int32)
            tpl = (C.c_int32 * self.cfg.n_layers)()
            tr = _Trace(cap, 0, recs, sc.ctypes.data_as(C.POINTER(C.c_float)), ids.ctypes.data_as(C.POINTER(C.c_int32)),
                        0, tpl, 0, 0, 0, 0)
        rc = fn(self._h, q_ptr, lq, c_ptr, o_ptr, n, k, C.byref(s) if s is not None else None, idx_ptr, sc_ptr,
                C.byref(n_out), C.byref(tr) if tr is not None else None, stream)
        if rc != 0:
            raise PrismError(rc, lib().prism_last_error(self._h).decode())
        trace = None
        if tr is not None:
            out = []
            for r in range(tr.n_records):
                x = recs[r]
                na = x.n_active_before
                out.append(ProbeRecord(x.layer, na, x.fired, x.n_selected, x.n_dropped, x.n_deferred, x.k_rem_after,
                                       [x.cuts[i] for i in range(x.n_cuts)], x.tokens_before, x.cv,
                                       [int(v) for v in ids[r, :na]], sc[r, :na].copy()))
            trace = Trace(out, tr.layers_run, [tpl[i] for i in range(tr.layers_run)], tr.n_chunks_max, tr.workspace_bytes,
                          tr.shared_prefix_rows)
        return int(n_out.value), trace

    def select(self, query: torch.Tensor, cand_tokens: torch.Tensor, cand_offsets: torch.Tensor, k: int, sched=None,
               want_trace: bool = True):
        """Device tensors (int32, cuda).  Returns (topk_idx, topk_scores, trace) with device outputs."""
        n = cand_offsets.numel() - 1
        idx = torch.empty(max(k, 1), dtype=torch.int32, device=query.device)
        sc = torch.empty(max(k, 1), dtype=torch.float32, device=query.device)
        stream = torch.cuda.current_stream().cuda_stream
        n_out, trace = self._call(lib().prism_select, query.data_ptr(), query.numel(), cand_tokens.data_ptr(),
                                  cand_offsets.data_ptr(), n, k, sched, idx.data_ptr(), sc.data_ptr(), want_trace, stream)
        return idx[:n_out], sc[:n_out], trace

    def select_sharded(self, query: torch.Tensor, cand_tokens: torch.Tensor, cand_offsets: torch.Tensor, k: int, sched,
                       owned: np.ndarray, reduce: Callable[[torch.Tensor], None], want_trace: bool = True):
        """prism_select_sharded: this rank runs the candidates with owned[i] != 0; `reduce(t)` must sum the float32
        device tensor t over all ranks in place, ordered on the current stream (see all_reduce_scores).  The
        outputs are the same on every rank."""
        n = cand_offsets.numel() - 1
        owned = np.ascontiguousarray(owned, dtype=np.uint8)
        if owned.shape != (n,):
            raise ValueError("owned must have one entry per candidate")
        idx = torch.empty(max(k, 1), dtype=torch.int32, device=query.device)
        sc = torch.empty(max(k, 1), dtype=torch.float32, device=query.device)
        exchange = torch.zeros(max(n, 1), dtype=torch.float32, device=query.device)
        failure = []

        def on_exchange(_ctx, n_active, _stream):
            try:
                reduce(exchange[:n_active])
                return 0
            except BaseException as e:  # must not propagate into the C caller
                failure.append(e)
                return 1

        cb = EXCHANGE_FN(on_exchange)
        stream = torch.cuda.current_stream().cuda_stream

        def fn(h, q, lq, c, o, n_, k_, s_, idx_, sc_, n_out_, tr_, st_):
            return lib().prism_select_sharded(h, q, lq, c, o, n_, k_, s_, owned.ctypes.data, exchange.data_ptr(), cb, None,
                                              idx_, sc_, n_out_, tr_, st_)

        try:
            n_out, trace = self._call(fn, query.data_ptr(), query.numel(), cand_tokens.data_ptr(), cand_offsets.data_ptr(),
                                      n, k, sched, idx.data_ptr(), sc.data_ptr(), want_trace, stream)
        except PrismError:
            if failure:
                raise failure[0]
            raise
        return idx[:n_out], sc[:n_out], trace

    def select_calibrated(self, query: torch.Tensor, cand_tokens: torch.Tensor, cand_offsets: torch.Tensor, k: int, sched,
                          cal: Calibrator):
        """prism_select_calibrated: the threshold comes from `cal`, which is updated in place."""
        n = cand_offsets.numel() - 1
        idx = torch.empty(max(k, 1), dtype=torch.int32, device=query.device)
        sc = torch.empty(max(k, 1), dtype=torch.float32, device=query.device)
        s = self._schedule(sched)
        n_out = C.c_int32(0)
        rc = lib().prism_select_calibrated(self._h, query.data_ptr(), query.numel(), cand_tokens.data_ptr(),
                                           cand_offsets.data_ptr(), n, k, C.byref(s), C.byref(cal), idx.data_ptr(),
                                           sc.data_ptr(), C.byref(n_out), None, torch.cuda.current_stream().cuda_stream)
        if rc != 0:
            raise PrismError(rc, lib().prism_last_error(self._h).decode())
        return idx[:n_out.value], sc[:n_out.value]

    def select_host(self, query: np.ndarray, cand_tokens: np.ndarray, cand_offsets: np.ndarray, k: int, sched=None,
                    want_trace: bool = False, idx_out: Optional[np.ndarray] = None, sc_out: Optional[np.ndarray] = None):
        """Host buffers in (int32 numpy, or pinned torch tensors via .numpy()), host results out."""
        n = len(cand_offsets) - 1
        idx = np.empty(max(k, 1), np.int32) if idx_out is None else idx_out
        sc = np.empty(max(k, 1), np.float32) if sc_out is None else sc_out
        stream = torch.cuda.current_stream().cuda_stream
        n_out, trace = self._call(lib().prism_select_host, query.ctypes.data, len(query), cand_tokens.ctypes.data,
                                  cand_offsets.ctypes.data, n, k, sched, idx.ctypes.data, sc.ctypes.data, want_trace, stream)
        return idx[:n_out], sc[:n_out], trace
