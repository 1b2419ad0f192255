"""Seeded synthetic inputs shaped like the paper's workloads.

This package only *draws inputs* (images, tokens, weights).  It contains none of
the method's arithmetic and is the one module shared by the CPU oracle's tests
and the CUDA path's tests and benchmark, so both always see identical bytes.
"""
from .generate import (  # noqa: F401
    WORKLOADS,
    Workload,
    make_images,
    make_tokens,
    make_attention_weights,
    make_block_weights,
    make_peaked_attention_inputs,
    make_workload_inputs,
)
