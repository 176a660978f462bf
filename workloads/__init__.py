"""Seeded synthetic inputs for the batched LoRA-delta path.

This module only draws random numbers and lays them out; it holds none of the
method's arithmetic.  Both the CUDA path's tests/bench and the CPU oracle's
tests take their inputs from here, so the two sides always see the same bits.
"""
from .gen import (  # noqa: F401
    CONFIG_NAMES,
    PoolSpec,
    Workload,
    bf16_bits_to_f32,
    bf16_bits_to_f64,
    bounded_zipf_pmf,
    f32_to_bf16_bits,
    f32_to_fp16_bits,
    gen_adapter,
    gen_pool_device,
    gen_x,
    gen_y_in,
    make_workload,
)
