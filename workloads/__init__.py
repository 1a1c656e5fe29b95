"""Seeded synthetic inputs for one WeDLM streaming-parallel-decoding step.

This module only *draws data*: window fill patterns, token ids, paged KV-cache
contents, block tables, window q/k/v and logits.  It contains none of the
method's arithmetic (no reordering, no RoPE, no attention, no softmax, no
commit logic), so both the CPU oracle's tests and the CUDA path's tests can
consume exactly the same arrays without sharing any computation.

bf16 tensors are produced in fp32 and rounded once (round-to-nearest-even) to
their 16-bit patterns; they are handed out as ``numpy.uint16`` arrays.  Every
consumer starts from those bit patterns.

The five named step configurations follow the workload shapes of the paper's
serving setting (a fixed W-slot window decoded on top of a paged prefix cache,
Algorithm 1) with Qwen3-8B attention geometry; the logits are synthetic
"boosted target" rows that emulate low/high entropy regimes.
"""
from .synth import (  # noqa: F401
    StepConfig,
    CONFIGS,
    get_config,
    make_step,
    bf16_bits,
    bf16_to_f32,
    BASE_SEED,
)
from .dual_stream import DualStreamConfig, DS_CONFIGS, make_dual_stream  # noqa: F401,E402
