"""Pins for the convolutional oracle (host only): exact step against torch conv2d / avg_pool2d
autograd in float64, p = 1 equals exact backprop, only weight gradients are random."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import cnn
from workloads import cnn_inputs


def _torch_step(X, y, cWs, cbs, fWs, fbs):
    t64 = lambda a: torch.tensor(np.asarray(a, np.float64), requires_grad=True)
    cW, cb, fW, fb = [t64(w) for w in cWs], [t64(b) for b in cbs], [t64(w) for w in fWs], [t64(b) for b in fbs]
    a = torch.tensor(np.asarray(X, np.float64)).permute(0, 3, 1, 2)          # NCHW
    for W, b in zip(cW, cb):
        a = F.avg_pool2d(torch.relu(F.conv2d(a, W.permute(3, 2, 0, 1), b, padding=1)), 2)
    a = a.permute(0, 2, 3, 1).reshape(a.shape[0], -1)                       # NHWC flatten
    for l, (W, b) in enumerate(zip(fW, fb)):
        a = a @ W + b
        if l < len(fW) - 1:
            a = torch.relu(a)
    loss = F.cross_entropy(a, torch.tensor(y, dtype=torch.long))
    loss.backward()
    g = lambda ts: [t.grad.numpy() for t in ts]
    return loss.item(), g(cW), g(cb), g(fW), g(fb)


def test_exact_step_matches_torch_autograd():
    args = cnn_inputs(3, hw=8, cin=3, channels=(4, 6), fc=(7, 5), dtype="f32", seed=2, bias_zero=False)
    loss, gcW, gcb, gfW, gfb = _torch_step(*args)
    r = cnn.cnn_step(*args, dtype="f64")
    assert r.loss == pytest.approx(loss, rel=1e-12)
    for got, want in zip(r.dW_conv + r.db_conv + r.dW_fc + r.db_fc, gcW + gcb + gfW + gfb):
        assert np.allclose(got, want, rtol=1e-9, atol=1e-14)


@pytest.mark.parametrize("variant", ["different", "same"])
def test_p_one_is_exact_and_only_weight_gradients_are_random(variant):
    args = cnn_inputs(4, hw=8, cin=3, channels=(8, 8), fc=(16, 5), dtype="bf16", seed=3, bias_zero=False)
    ex = cnn.cnn_step(*args)
    one = cnn.cnn_step(*args, variant=variant, p=1.0, seed=1)
    rd = cnn.cnn_step(*args, variant=variant, p=0.3, seed=1)
    for a, b in zip(one.dW_conv + one.dW_fc, ex.dW_conv + ex.dW_fc):
        assert np.array_equal(a, b)
    assert rd.loss == ex.loss
    for a, b in zip(rd.db_conv + rd.db_fc, ex.db_conv + ex.db_fc):
        assert np.array_equal(a, b)
    for a, b in zip(rd.dW_conv + rd.dW_fc, ex.dW_conv + ex.dW_fc):
        assert not np.array_equal(a, b)
    assert len(rd.nnz) == 4


def test_mean_over_seeds_is_unbiased_for_conv_weights():
    args = cnn_inputs(3, hw=8, cin=3, channels=(4,), fc=(5,), dtype="f32", seed=5)
    ex = cnn.cnn_step(*args, dtype="f32")
    S = 300
    acc = np.zeros_like(ex.dW_conv[0])
    for seed in range(S):
        acc += cnn.cnn_step(*args, dtype="f32", variant="different", p=0.5, seed=seed).dW_conv[0]
    one = np.linalg.norm(cnn.cnn_step(*args, dtype="f32", variant="different", p=0.5, seed=0).dW_conv[0] - ex.dW_conv[0])
    assert np.linalg.norm(acc / S - ex.dW_conv[0]) < 3.0 * one / np.sqrt(S)
