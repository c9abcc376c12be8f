"""Pins for the exact (never sampled) pieces of the oracle: forward, loss and backward (host only)."""
import numpy as np
import pytest
import torch

from oracle import rad
from workloads import mlp_inputs


def _torch_step(X, y, Ws, bs, act):
    Xt = torch.tensor(X, dtype=torch.float64)
    Wt = [torch.tensor(W, dtype=torch.float64, requires_grad=True) for W in Ws]
    bt = [torch.tensor(b, dtype=torch.float64, requires_grad=True) for b in bs]
    a = Xt
    for l, (W, b) in enumerate(zip(Wt, bt)):
        z = a @ W + b
        if l < len(Wt) - 1:
            a = torch.relu(z) if act == "relu" else torch.nn.functional.gelu(z)
    loss = torch.nn.functional.cross_entropy(z, torch.tensor(y, dtype=torch.long))
    loss.backward()
    return loss.item(), [W.grad.numpy() for W in Wt], [b.grad.numpy() for b in bt]


@pytest.mark.parametrize("act", ["relu", "gelu"])
def test_exact_step_matches_torch_autograd(act):
    X, y, Ws, bs = mlp_inputs((30, 24, 17, 7), 13, seed=5, bias_zero=False, x_dist="normal")
    loss, dWs, dbs = _torch_step(X, y, Ws, bs, act)
    r = rad.mlp_step(X, y, Ws, bs, act=act, dtype="f64")
    assert r.loss == pytest.approx(loss, rel=1e-12)
    for l in range(3):
        assert np.allclose(r.dW[l], dWs[l], rtol=1e-9, atol=1e-14)
        assert np.allclose(r.db[l], dbs[l], rtol=1e-9, atol=1e-14)


def test_finite_differences_tiny_net():
    X, y, Ws, bs = mlp_inputs((5, 4, 3), 3, seed=1, bias_zero=False, x_dist="normal")
    Ws = [W.astype(np.float64) for W in Ws]
    bs = [b.astype(np.float64) for b in bs]
    r = rad.mlp_step(X, y, Ws, bs, dtype="f64")
    eps = 1e-6
    for l in range(2):
        for idx in np.ndindex(Ws[l].shape):
            Wp = [w.copy() for w in Ws]
            Wm = [w.copy() for w in Ws]
            Wp[l][idx] += eps
            Wm[l][idx] -= eps
            fd = (rad.mlp_step(X, y, Wp, bs, dtype="f64").loss - rad.mlp_step(X, y, Wm, bs, dtype="f64").loss) / (2 * eps)
            assert fd == pytest.approx(r.dW[l][idx], rel=1e-5, abs=1e-9)
        for j in range(bs[l].size):
            bp = [b.copy() for b in bs]
            bm = [b.copy() for b in bs]
            bp[l][j] += eps
            bm[l][j] -= eps
            fd = (rad.mlp_step(X, y, Ws, bp, dtype="f64").loss - rad.mlp_step(X, y, Ws, bm, dtype="f64").loss) / (2 * eps)
            assert fd == pytest.approx(r.db[l][j], rel=1e-5, abs=1e-9)


def test_input_grad_uses_one_bit_relu_derivative():
    rng = np.random.default_rng(2)
    dZ = rng.standard_normal((6, 4))
    W = rng.standard_normal((9, 4))
    Aprev = np.maximum(rng.standard_normal((6, 9)), 0).astype(np.float32)
    dA, db = rad.input_grad(dZ, W, relubits_prev=rad.pack_bits(Aprev > 0))
    assert np.allclose(dA, (dZ @ W.T) * (Aprev > 0))
    assert np.allclose(db, dZ.sum(0))


def test_stored_bytes_counts():
    X, y, Ws, bs = mlp_inputs((784, 300, 300, 10), 150, seed=1234)
    r = rad.mlp_step(X, y, Ws, bs, variant="different", p=0.1, seed=0)
    sb = rad.stored_bytes(r.stores, r.Z[-1].shape, 4)
    assert sb["full_backprop_bytes"] == 150 * 1384 * 4 + 6000
    assert sb["index_bytes"] == 150 * (25 + 10 + 10) * 4
    assert sb["relu_bytes"] == 150 * 20 * 4
    assert sb["value_bytes"] == 4 * sum(st.nnz for st in r.stores)
    assert abs(sb["value_bytes"] / (150 * 1384 * 4) - rad.effective_p(0.1)) < 0.005
