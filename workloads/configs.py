"""Shapes of the feed-forward workloads.

The fully connected nets follow the MNIST multilayer perceptron of the paper's
App. A ("Architectures Used"): flattened 28x28 inputs in [0, 1), hidden width
300, ten classes, batch 150.  The wide net has no counterpart in the paper; it
exists to load the store and weight-gradient kernels at sizes where the HBM
and tensor-core rooflines are what bounds them.
"""
from dataclasses import dataclass, field
from typing import Tuple


@dataclass(frozen=True)
class MLPConfig:
    name: str
    dims: Tuple[int, ...]          # fan-in of layer 1, ..., fan-out of layer L
    batch: int
    dtype: str                     # "f32" or "bf16"
    act: str                       # "relu" or "gelu"
    x_dist: str                    # "uniform01" or "normal"
    variant: str                   # "different" or "same"
    p: float
    p_sweep: Tuple[float, ...] = field(default_factory=tuple)
    data_seed: int = 1234
    mask_seed: int = 0


CONFIGS = {
    # MNIST-shaped MLP, independent mask per minibatch element.
    "mlp_small_different": MLPConfig(
        "mlp_small_different", (784, 300, 300, 10), 150, "f32", "relu",
        "uniform01", "different", 0.1),
    # Same net, one mask per layer shared by the whole minibatch.
    "mlp_small_same": MLPConfig(
        "mlp_small_same", (784, 300, 300, 10), 150, "f32", "relu",
        "uniform01", "same", 0.1, (0.01, 0.05, 0.1, 0.2, 0.5, 1.0)),
    # Wide bf16 net for roofline measurement.
    "mlp_wide": MLPConfig(
        "mlp_wide", (8192, 8192, 8192, 8192, 8192, 1000), 65536, "bf16", "relu",
        "normal", "different", 0.1, (0.01, 0.05, 0.1, 0.5)),
    # A cut of the wide net the CPU oracle finishes in seconds (several tiles
    # in every dimension plus ragged tails).
    "mlp_wide_cut": MLPConfig(
        "mlp_wide_cut", (640, 520, 392, 200), 328, "bf16", "relu",
        "normal", "different", 0.1, (0.01, 0.05, 0.1, 0.5)),
}


def get_config(name: str) -> MLPConfig:
    return CONFIGS[name]
