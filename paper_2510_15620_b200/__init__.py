"""PRISM hot path on B200: thin ctypes binding over the C-ABI library (include/prism.h).

Every step of the path runs in the CUDA kernels of lib/libprism.so; this package only marshals
arguments.  Importing it without a built library raises: there is no CPU fallback."""
from .binding import (PrismModel, PrismError, Calibrator, Trace, ProbeRecord, lib, upload_weights,  # noqa: F401
                      status_str, PRISM_FP32, PRISM_BF16, PRISM_IMPL_AUTO, PRISM_IMPL_SIMT, PRISM_IMPL_MMA, PRISM_IMPL_SOLO,
                      shard_candidates, all_reduce_scores, PRISM_ARCH_DECODER, PRISM_ARCH_ENCODER, PRISM_WFMT_PLAIN, PRISM_WFMT_W4)
from . import ops  # noqa: F401
