"""Small convolutional net with activation sampling on every conv / linear input: oracle (numpy,
float64).  TEST INFRASTRUCTURE ONLY.

Paper, Fig. "Convnet activation sampling" and Sec. 4.2: the input of each convolution is sampled at
spatial-element granularity (one keep decision per input entry, shared by all filter taps that read
it), the ReLU derivative of each conv output is kept at one bit per entry, average pooling and
biases need nothing stored, and the weight gradient is the convolution weight gradient evaluated on
the sparse input.  Everything else (forward, dX, bias gradients) is exact.

Layout: NHWC.  A 3x3 convolution with zero padding 1 is
    Z[b, y, x, :] = sum_{ky, kx} Xpad[b, y + ky, x + kx, :] @ W[ky, kx]         W: 3 x 3 x Cin x Cout
followed by ReLU and 2x2 average pooling; the flattened (y, x, c) output of the last pool feeds a
stack of linear layers handled exactly like oracle.rad.mlp_step.  Layers are numbered conv first,
then linear, for the Philox counter.  Device-resident tensors (activations, pooled maps, dZ, dP) are
rounded to the working type (bf16 or float32) where the device holds them; sums are float64.
"""
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

from . import rad


def conv3x3(X, W):
    """Zero-padded 3x3 convolution, NHWC, stride 1."""
    B, H, Wd, _ = X.shape
    Xp = np.pad(X, ((0, 0), (1, 1), (1, 1), (0, 0)))
    Z = np.zeros((B, H, Wd, W.shape[3]))
    for ky in range(3):
        for kx in range(3):
            Z += Xp[:, ky:ky + H, kx:kx + Wd, :] @ W[ky, kx]
    return Z


def conv3x3_weight_grad(X, dZ):
    """dW[ky, kx, ci, co] = sum_{b, y, x} Xpad[b, y + ky, x + kx, ci] dZ[b, y, x, co]."""
    B, H, Wd, Cin = X.shape
    Xp = np.pad(X, ((0, 0), (1, 1), (1, 1), (0, 0)))
    dW = np.zeros((3, 3, Cin, dZ.shape[3]))
    flat = dZ.reshape(-1, dZ.shape[3])
    for ky in range(3):
        for kx in range(3):
            dW[ky, kx] = Xp[:, ky:ky + H, kx:kx + Wd, :].reshape(-1, Cin).T @ flat
    return dW


def conv3x3_input_grad(dZ, W):
    """dX[b, yi, xi, ci] = sum_{ky, kx, co} dZ[b, yi - ky + 1, xi - kx + 1, co] W[ky, kx, ci, co]."""
    B, H, Wd, _ = dZ.shape
    dZp = np.pad(dZ, ((0, 0), (1, 1), (1, 1), (0, 0)))
    dX = np.zeros((B, H, Wd, W.shape[2]))
    for ky in range(3):
        for kx in range(3):
            dX += dZp[:, 2 - ky:2 - ky + H, 2 - kx:2 - kx + Wd, :] @ W[ky, kx].T
    return dX


def avgpool2(A):
    B, H, W, C = A.shape
    return A.reshape(B, H // 2, 2, W // 2, 2, C).mean(axis=(2, 4))


def avgpool2_backward(dP):
    return 0.25 * np.repeat(np.repeat(dP, 2, axis=1), 2, axis=2)


@dataclass
class CnnResult:
    loss: float
    dW_conv: List[np.ndarray]
    db_conv: List[np.ndarray]
    dW_fc: List[np.ndarray]
    db_fc: List[np.ndarray]
    nnz: List[int] = field(default_factory=list)


def cnn_step(X, labels, conv_Ws, conv_bs, fc_Ws, fc_bs, dtype="bf16", variant=None, p=1.0, seed=0, step=0) -> CnnResult:
    """Forward, loss, backward.  variant None = exact backprop; "f64" dtype = no rounding at all."""
    if dtype == "bf16":
        rnd = lambda v: rad.round_bf16(np.asarray(v, np.float32)).astype(np.float64)
    elif dtype == "f32":
        rnd = lambda v: np.asarray(v, np.float32).astype(np.float64)
    elif dtype == "f64" and variant is None:
        rnd = lambda v: np.asarray(v, np.float64)
    else:
        raise ValueError(dtype)
    nc, nf = len(conv_Ws), len(fc_Ws)
    B = X.shape[0]
    A = np.asarray(X, np.float64)
    conv_in, relu_out, stores = [], [], []
    layer = 0
    for l in range(nc):
        conv_in.append(A)
        if variant is not None:
            stores.append(rad.forward_store(A.reshape(B, -1).astype(np.float32), dtype, variant, p, seed, layer, step,
                                            with_relu_bits=False))
        Z = conv3x3(A, np.asarray(conv_Ws[l], np.float64)) + np.asarray(conv_bs[l], np.float64)
        R = rnd(np.maximum(Z, 0.0))
        relu_out.append(R)
        A = rnd(avgpool2(R))
        layer += 1
    pooled_shape = A.shape
    F = [A.reshape(B, -1)]
    Zf = []
    for l in range(nf):
        if variant is not None:
            stores.append(rad.forward_store(F[l].astype(np.float32), dtype, variant, p, seed, layer, step,
                                            with_relu_bits=False))
        z = F[l] @ np.asarray(fc_Ws[l], np.float64) + np.asarray(fc_bs[l], np.float64)
        Zf.append(z)
        if l < nf - 1:
            F.append(rnd(np.maximum(z, 0.0)))
        layer += 1
    loss, dz = rad.softmax_xent(Zf[-1], labels)
    dz = rnd(dz)
    dW_fc, db_fc = [None] * nf, [None] * nf
    for l in range(nf - 1, -1, -1):
        dW_fc[l] = F[l].T @ dz if variant is None else rad.weight_grad(stores[nc + l], dz)
        db_fc[l] = dz.sum(axis=0)
        dA = rnd(dz @ np.asarray(fc_Ws[l], np.float64).T)
        if l > 0:
            dA = dA * (F[l] > 0)                       # 1-bit ReLU derivative of the layer that made F[l]
        dz = dA
    dP = dz.reshape(pooled_shape)
    dW_conv, db_conv = [None] * nc, [None] * nc
    for l in range(nc - 1, -1, -1):
        dZ = rnd(avgpool2_backward(dP) * (relu_out[l] > 0))
        src = conv_in[l] if variant is None else rad.densify(stores[l]).reshape(conv_in[l].shape)
        dW_conv[l] = conv3x3_weight_grad(src, dZ)
        db_conv[l] = dZ.sum(axis=(0, 1, 2))
        if l > 0:
            dP = rnd(conv3x3_input_grad(dZ, np.asarray(conv_Ws[l], np.float64)))
    return CnnResult(loss, dW_conv, db_conv, dW_fc, db_fc, [s.nnz for s in stores])
