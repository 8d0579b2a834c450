"""Seeded synthetic inputs shared by the CPU oracle tests and the CUDA path.

This package holds only input generation (random tensors, workload shapes,
probe-step coin flips).  None of the method's arithmetic lives here.
"""
from .synth import (  # noqa: F401
    CONFIGS,
    Workload,
    get_config,
    make_prefill,
    make_decode_step,
    decode_probe_flags,
    splitmix64_stream,
)
