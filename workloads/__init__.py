"""Seeded synthetic inputs for the RevFFN MoE coupling branch.

This package only draws random tensors of the shapes the benchmark
configurations fix.  It holds none of the method's arithmetic and is the one
module that both the CUDA path's callers and the CPU oracle's callers share.
"""
from .generate import (BlockConfig, CONFIGS, make_weights, make_streams,
                       zipf_router_bias, to_bf16_values, weight_shapes, make_weights_device)

__all__ = ["BlockConfig", "CONFIGS", "make_weights", "make_streams",
           "zipf_router_bias", "to_bf16_values", "weight_shapes", "make_weights_device"]
