"""Seeded synthetic inputs (weights, requests, schedules) for the PRISM hot path.

This package only *draws inputs*: it contains none of the method's arithmetic
(no normalisation, attention, scoring, ranking or pruning).  Both the CPU
oracle's tests and the CUDA path's tests/bench take their inputs from here so
that the two sides see bit-identical weights and tokens without sharing any
compute code.
"""
from .configs import ModelCfg, Schedule, Workload, WORKLOADS, workload  # noqa: F401
from .weights import make_weights, round_to_bf16, bf16_bits  # noqa: F401
from .requests import make_request  # noqa: F401
from .quant import quantize_weights, quantize_matrix, pack_matrix, packed_sections  # noqa: F401
