"""CPU oracle for the fused clip + block-wise 8-bit AdamW step.

TEST INFRASTRUCTURE, NOT PRODUCT: only the test suite, the smoke check and the benchmark's
cpu_baseline / reference legs may import this package. The CUDA library and its Python binding
never do, and this package never imports them.

`lt_oracle.cpp` holds the arithmetic (plain single-threaded C++, fp64 norm, fp32 element math
without fused multiply-add); this module only builds it with g++ and marshals numpy arrays to it.
"""
from .binding import (  # noqa: F401
    F32, BF16, HParams, OracleTensor, build, lib,
    code_table, nearest, nearest_brute, state_bytes, sqnorm, clip_factor, step_scalars,
    state_init, hybrid8_step, step_fp32state, dequant, bf16_bits_to_f32, f32_to_bf16_bits,
)
