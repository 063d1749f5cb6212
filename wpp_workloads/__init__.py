"""Seeded synthetic inputs for the chunked-prefill attention path.

This package only *describes and fills* inputs: request lengths, block
tables, physical page ids and bf16 values.  It holds none of the method's
arithmetic (no append, no gather, no softmax) and imports neither the CUDA
binding nor the oracle; both the GPU tests and the oracle tests draw their
inputs from here.
"""
from .generate import (  # noqa: F401
    Workload,
    counter_normal_bf16,
    make_workload,
    custom_workload,
    cfg1,
    cfg2,
    cfg3,
    cfg4,
    cfg5_cell,
    CONFIG_BUILDERS,
    KdaWorkload,
    kda_workload,
    kda_wave,
)
