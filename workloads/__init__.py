"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random numbers and shapes tensors.  It contains none of
the quantization method's arithmetic: no quantizer, no scale
reparameterization, no integer GEMM.  Where an input is defined through a
full-precision transformer forward (the calibration stand-in that yields
clipping bounds), that forward is made of PyTorch CPU library calls
(`layer_norm`, `linear`, `softmax`, `gelu`) used as black boxes.

Both the CPU oracle's tests and the CUDA path's tests/benchmarks draw their
inputs from here, so the two sides always see bit-identical arrays.
"""
from .block import BLOCK_CONFIGS, BlockInputs, make_block_inputs, block_config  # noqa: F401
from .kernels import (  # noqa: F401
    ln_inputs,
    ln_calibration_bounds,
    softmax_logits,
    gemm_codes,
    to_bf16_grid,
)
