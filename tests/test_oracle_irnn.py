"""Pins for the recurrent oracle (host only): exact BPTT against torch autograd in float64, p = 1
equals exact backprop, only dW_hh and dW_out are random, unbiasedness over seeds."""
import numpy as np
import pytest
import torch

from oracle import irnn, rad
from workloads import irnn_inputs


def _torch_irnn(x, y, W_ih, b_ih, W_hh, b_hh, W_out, b_out):
    t64 = lambda a: torch.tensor(np.asarray(a, np.float64), requires_grad=True)
    W_ih, b_ih, W_hh, b_hh, W_out, b_out = map(t64, (W_ih, b_ih, W_hh, b_hh, W_out, b_out))
    xs = torch.tensor(np.asarray(x, np.float64))
    h = torch.zeros(x.shape[0], W_hh.shape[0], dtype=torch.float64)
    for t in range(x.shape[1]):
        h = torch.relu(xs[:, t:t + 1] * W_ih[None, :] + b_ih + h @ W_hh + b_hh)
    loss = torch.nn.functional.cross_entropy(h @ W_out + b_out, torch.tensor(y, dtype=torch.long))
    loss.backward()
    return loss.item(), [v.grad.numpy() for v in (W_ih, b_ih, W_hh, b_hh, W_out, b_out)]


def test_exact_bptt_matches_torch_autograd():
    args = irnn_inputs(5, 9, hidden=12, classes=4, seed=3, identity=False)
    loss, (gWih, gbih, gWhh, gbhh, gWout, gbout) = _torch_irnn(*args)
    r = irnn.irnn_step(*args, exact_dtype="f64")
    assert r.loss == pytest.approx(loss, rel=1e-12)
    for got, want in ((r.dW_ih, gWih), (r.db, gbih), (r.db, gbhh), (r.dW_hh, gWhh), (r.dW_out, gWout), (r.db_out, gbout)):
        assert np.allclose(got, want, rtol=1e-9, atol=1e-14)


@pytest.mark.parametrize("variant", ["different", "same"])
def test_p_one_is_exact_and_only_sampled_gradients_are_random(variant):
    args = irnn_inputs(6, 11, hidden=16, classes=3, seed=5, identity=False)
    ex = irnn.irnn_step(*args)
    one = irnn.irnn_step(*args, variant=variant, p=1.0, seed=4)
    rd = irnn.irnn_step(*args, variant=variant, p=0.3, seed=4)
    for a, b in ((one.dW_hh, ex.dW_hh), (one.dW_out, ex.dW_out)):
        assert np.array_equal(a, b)
    assert rd.loss == ex.loss
    assert np.array_equal(rd.dW_ih, ex.dW_ih) and np.array_equal(rd.db, ex.db) and np.array_equal(rd.db_out, ex.db_out)
    assert not np.array_equal(rd.dW_hh, ex.dW_hh) and not np.array_equal(rd.dW_out, ex.dW_out)
    # every step keeps about p * B * hidden entries of its input (h_0 = 0 included: the mask ignores data)
    assert rd.nnz_steps.shape == (11,) and abs(rd.nnz_steps.mean() - 0.3 * 6 * 16) < 12


def test_masks_differ_between_time_steps_and_mean_is_unbiased():
    args = irnn_inputs(8, 6, hidden=16, classes=3, seed=7, identity=False)
    ex = irnn.irnn_step(*args)
    m1 = rad.keep_mask("different", 8, 16, 0.5, 0, 0, 1)
    m2 = rad.keep_mask("different", 8, 16, 0.5, 0, 0, 2)
    assert not np.array_equal(m1, m2)
    S = 400
    acc = np.zeros_like(ex.dW_hh)
    for seed in range(S):
        acc += irnn.irnn_step(*args, variant="different", p=0.5, seed=seed).dW_hh
    err = np.linalg.norm(acc / S - ex.dW_hh) / np.linalg.norm(ex.dW_hh)
    one = np.linalg.norm(irnn.irnn_step(*args, variant="different", p=0.5, seed=0).dW_hh - ex.dW_hh) / np.linalg.norm(ex.dW_hh)
    assert err < 3.0 * one / np.sqrt(S)
