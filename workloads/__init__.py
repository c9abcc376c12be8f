"""Seeded synthetic inputs shaped like the workloads of the RAD paper (App. A).

This package is the only code shared by the CPU oracle's tests and the CUDA
path's tests and benchmark.  It draws numbers and describes shapes; it holds
none of the method's arithmetic (no masks, no sampling, no gradients).
"""
from .configs import CONFIGS, MLPConfig, get_config
from .generate import (mlp_inputs, layer_inputs, to_bf16_grid, uniform_labels, irnn_inputs, cnn_inputs)

__all__ = ["CONFIGS", "MLPConfig", "get_config", "mlp_inputs", "layer_inputs",
           "to_bf16_grid", "uniform_labels", "irnn_inputs", "cnn_inputs"]
