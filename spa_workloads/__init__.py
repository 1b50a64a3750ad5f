"""Seeded synthetic workloads for one Select-and-Pack-Attention block.

This package only *draws inputs*: shapes, blob layouts, random tensors and their
rounding to the storage dtype.  It contains none of the block's arithmetic beyond
the input-validity check that keeps every gate logit away from the threshold, and
it is the one module that both the CPU oracle's tests and the CUDA path's tests
and benchmark may import.
"""
from .configs import CONFIGS, SpaConfig, get_config, scaled_config
from .generate import SpaInputs, make_inputs, bf16_round, to_bf16_bits, from_bf16_bits

__all__ = [
    "CONFIGS", "SpaConfig", "get_config", "scaled_config",
    "SpaInputs", "make_inputs", "bf16_round", "to_bf16_bits", "from_bf16_bits",
]
