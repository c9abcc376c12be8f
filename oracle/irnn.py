"""IRNN with per-time-step activation sampling: oracle (numpy, float64).  TEST INFRASTRUCTURE ONLY.

Architecture (paper, App. A, "Architectures Used", item 3): one ReLU recurrent cell
h_t = relu(W_ih x_t + b_ih + W_hh h_{t-1} + b_hh) fed one scalar per step, and a linear output
layer on the last hidden state with softmax cross-entropy.  RAD (Sec. 4.3, "we sample different
activations at each time-step"; App. A memory calculation): the hidden state entering each step is
stored through a fresh mask (time index in the Philox counter), the scalar input is kept whole, the
last hidden state entering the output layer is sampled too, the softmax input is not.  Only
dW_hh and dW_out become random; dW_ih, the biases and the dh chain stay exact.

Conventions: row-wise, z_t = x_t * W_ih + b_ih + h_{t-1} @ W_hh + b_hh with W_hh (in, out);
h_0 = 0 (the paper does not say); tensors that live on the device in float32 (h_t, dh_t) are
rounded to float32 at those points, accumulations are float64.
"""
from dataclasses import dataclass
from typing import List, Optional

import numpy as np

from . import rad


@dataclass
class IrnnResult:
    loss: float
    h_last: np.ndarray
    dW_ih: np.ndarray
    db: np.ndarray              # gradient of b_ih, equal to that of b_hh
    dW_hh: np.ndarray
    dW_out: np.ndarray
    db_out: np.ndarray
    nnz_steps: Optional[np.ndarray] = None     # kept hidden entries per time step (all rows)
    nnz_out: int = 0


def _f32(v):
    return np.asarray(v, np.float32).astype(np.float64)


def irnn_step(x, labels, W_ih, b_ih, W_hh, b_hh, W_out, b_out, variant=None, p=1.0, seed=0, step0=0,
              exact_dtype="f32") -> IrnnResult:
    """Forward over T steps, loss, backward through time.  variant None = exact backprop.

    exact_dtype "f64" switches off every rounding (pins of the exact recurrence only).
    """
    x = np.asarray(x, np.float64)
    B, T = x.shape
    W_ih, b_ih, b_hh = (np.asarray(v, np.float64).reshape(-1) for v in (W_ih, b_ih, b_hh))
    W_hh, W_out, b_out = (np.asarray(v, np.float64) for v in (W_hh, W_out, b_out))
    Hd = W_hh.shape[0]
    rnd = _f32 if exact_dtype == "f32" else (lambda v: np.asarray(v, np.float64))
    h = [np.zeros((B, Hd))]
    stores: List[Optional[rad.Store]] = [None]
    for t in range(1, T + 1):
        if variant is not None:      # what step t keeps of its input h_{t-1}
            stores.append(rad.forward_store(h[t - 1].astype(np.float32), "f32", variant, p, seed, 0, step0 + t,
                                            with_relu_bits=False))
        z = x[:, t - 1:t] * W_ih[None, :] + b_ih + h[t - 1] @ W_hh + b_hh
        h.append(rnd(np.maximum(z, 0.0)))
    out_store = None
    if variant is not None:
        out_store = rad.forward_store(h[T].astype(np.float32), "f32", variant, p, seed, 1, step0,
                                      with_relu_bits=False)
    logits = h[T] @ W_out + b_out
    loss, dlogits = rad.softmax_xent(logits, labels)
    dlogits = rnd(dlogits)
    dW_out = h[T].T @ dlogits if variant is None else rad.weight_grad(out_store, dlogits)
    db_out = dlogits.sum(axis=0)
    dh = rnd(dlogits @ W_out.T)
    dW_hh = np.zeros((Hd, Hd))
    dW_ih = np.zeros(Hd)
    db = np.zeros(Hd)
    for t in range(T, 0, -1):
        dz = dh * (h[t] > 0)                         # 1-bit ReLU derivative of step t
        dW_hh += h[t - 1].T @ dz if variant is None else rad.weight_grad(stores[t], dz)
        dW_ih += x[:, t - 1] @ dz                    # the scalar input is stored whole: exact
        db += dz.sum(axis=0)
        dh = rnd(dz @ W_hh.T)
    nnz = None if variant is None else np.array([s.nnz for s in stores[1:]], dtype=np.int64)
    return IrnnResult(loss, h[T], dW_ih, db, dW_hh, dW_out, db_out, nnz,
                      0 if out_store is None else out_store.nnz)
