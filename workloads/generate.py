"""Seeded generators for inputs, labels and weights (numpy PCG64 streams).

Every array is returned as float32 (labels as int32).  For bf16 workloads the
float32 values already lie on the bf16 grid, so converting them to bf16 on
either side of a comparison is exact.
"""
import numpy as np


def to_bf16_grid(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 value (ties to even), kept as float32."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32))
    return t.to(torch.bfloat16).to(torch.float32).numpy()


def uniform_labels(rng: np.random.Generator, batch: int, classes: int) -> np.ndarray:
    return rng.integers(0, classes, size=batch, dtype=np.int64).astype(np.int32)


def _draw(rng, shape, dist):
    if dist == "uniform01":
        return rng.random(shape, dtype=np.float32)
    if dist == "normal":
        return rng.standard_normal(shape, dtype=np.float32)
    raise ValueError(dist)


def mlp_inputs(dims, batch, dtype="f32", x_dist="uniform01", seed=1234, bias_zero=True):
    """Inputs of one training step of a fully connected net.

    X is batch x dims[0]; weight l is dims[l] x dims[l+1] (fan-in major, the
    paper's h = W^T x written row-wise as Z = A W), Kaiming-normal with
    std sqrt(2 / fan_in); biases are zero unless bias_zero is False, in which
    case they are small normals so bias paths are exercised.
    """
    rng = np.random.default_rng(seed)
    X = _draw(rng, (batch, dims[0]), x_dist)
    labels = uniform_labels(rng, batch, dims[-1])
    Ws, bs = [], []
    for l in range(len(dims) - 1):
        std = np.float32(np.sqrt(2.0 / dims[l]))
        Ws.append(rng.standard_normal((dims[l], dims[l + 1]), dtype=np.float32) * std)
        if bias_zero:
            bs.append(np.zeros(dims[l + 1], dtype=np.float32))
        else:
            bs.append(rng.standard_normal(dims[l + 1], dtype=np.float32) * np.float32(0.1))
    if dtype == "bf16":
        X = to_bf16_grid(X)
        Ws = [to_bf16_grid(W) for W in Ws]
    return X, labels, Ws, bs


def layer_inputs(B, D, H, dtype="f32", x_dist="normal", seed=1234, relu_like=False):
    """Inputs of the per-layer calls: activations A (B x D) and output gradient dZ (B x H).

    With relu_like=True about half of A is exactly zero and a few entries are
    -0.0, as after a ReLU, so the sign-bit cases of the 1-bit derivative store
    are covered.
    """
    rng = np.random.default_rng(seed)
    A = _draw(rng, (B, D), x_dist)
    if relu_like:
        A = np.maximum(A, np.float32(0))
        neg0 = rng.random((B, D)) < 0.01
        A = np.where(neg0 & (A == 0), np.float32(-0.0), A).astype(np.float32)
    dZ = rng.standard_normal((B, H), dtype=np.float32) * np.float32(1.0 / max(B, 1))
    if dtype == "bf16":
        A, dZ = to_bf16_grid(A), to_bf16_grid(dZ)
    return A, dZ


def irnn_inputs(batch, steps, hidden=100, classes=10, seed=1234, identity=True):
    """Inputs of the sequential-pixel IRNN (paper, App. A, "RNN training details"): x in [0, 1) fed
    one scalar per step, recurrent matrix initialised to the identity, input and output weights
    N(0, 0.001) (read as standard deviation 0.001), zero biases.  identity=False draws a random
    recurrent matrix of spectral norm about 0.9 and larger weights, so that tests exercise every term.
    """
    rng = np.random.default_rng(seed)
    x = rng.random((batch, steps), dtype=np.float32)
    labels = uniform_labels(rng, batch, classes)
    if identity:
        W_hh = np.eye(hidden, dtype=np.float32)
        W_ih = rng.standard_normal(hidden, dtype=np.float32) * np.float32(0.001)
        W_out = rng.standard_normal((hidden, classes), dtype=np.float32) * np.float32(0.001)
        b_ih = np.zeros(hidden, np.float32)
        b_hh = np.zeros(hidden, np.float32)
    else:
        W_hh = rng.standard_normal((hidden, hidden), dtype=np.float32) * np.float32(0.45 / np.sqrt(hidden))
        W_ih = rng.standard_normal(hidden, dtype=np.float32) * np.float32(0.5)
        W_out = rng.standard_normal((hidden, classes), dtype=np.float32) * np.float32(0.3)
        b_ih = rng.standard_normal(hidden, dtype=np.float32) * np.float32(0.1)
        b_hh = rng.standard_normal(hidden, dtype=np.float32) * np.float32(0.1)
    b_out = np.zeros(classes, np.float32)
    return x, labels, W_ih, b_ih, W_hh, b_hh, W_out, b_out


def cnn_inputs(batch, hw=32, cin=3, channels=(16, 32, 64), fc=(128, 10), dtype="bf16", seed=1234, bias_zero=True):
    """Inputs of the small convolutional net: N(0,1) images (NHWC), 3x3 filters and linear weights
    Kaiming-normal (std sqrt(2 / fan_in)), zero biases (or small normal ones for tests).  Filters are
    3 x 3 x Cin x Cout; each conv is followed by ReLU and 2x2 average pooling, so the first linear layer
    sees (hw / 2^n)^2 * channels[-1] features."""
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((batch, hw, hw, cin), dtype=np.float32)
    labels = uniform_labels(rng, batch, fc[-1])
    conv_Ws, conv_bs, c = [], [], cin
    for co in channels:
        conv_Ws.append(rng.standard_normal((3, 3, c, co), dtype=np.float32) * np.float32(np.sqrt(2.0 / (9 * c))))
        conv_bs.append(np.zeros(co, np.float32) if bias_zero else rng.standard_normal(co, dtype=np.float32) * np.float32(0.1))
        c = co
    feat = (hw >> len(channels)) ** 2 * c
    fc_Ws, fc_bs, d = [], [], feat
    for h in fc:
        fc_Ws.append(rng.standard_normal((d, h), dtype=np.float32) * np.float32(np.sqrt(2.0 / d)))
        fc_bs.append(np.zeros(h, np.float32) if bias_zero else rng.standard_normal(h, dtype=np.float32) * np.float32(0.1))
        d = h
    if dtype == "bf16":
        X = to_bf16_grid(X)
        conv_Ws = [to_bf16_grid(W) for W in conv_Ws]
        fc_Ws = [to_bf16_grid(W) for W in fc_Ws]
    return X, labels, conv_Ws, conv_bs, fc_Ws, fc_bs
