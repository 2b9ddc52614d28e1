"""Seeded synthetic input generators (shared by the CPU oracle's tests and the CUDA path's tests)."""
from .generator import (  # noqa: F401
    PRESETS,
    Workload,
    bf16_bits_to_f32,
    custom,
    f32_to_bf16_bits,
    generate,
    generate_topk,
    get_workload,
    sweep_max,
    sweep_points,
    zipf_bias,
)
