"""Pins for the oracle's estimator against what the paper and the mathematics fix (host only).

  * p = 1 is exact backprop (App. A: without replacement, fraction 1.0 equals the baseline);
  * only dW is random: loss, Z, dZ, db equal exact backprop for any p (Sec. 4.2);
  * E[P] = I (Sec. 3.2): expectation over ALL masks of a tiny layer equals A^T dZ, and the
    variance equals the closed forms q * sum_b a_b^2 (different) and q * dW^2 (same),
    q = (1 - p_eff) / p_eff, a_b = A[b,d] dZ[b,h];
  * same sample only touches kept rows of dW (Sec. 4.3);
  * structure of the compact form.
"""
import itertools

import numpy as np
import pytest

from oracle import rad
from workloads import layer_inputs, mlp_inputs


def exact_dW(A, dZ):
    return np.asarray(A, np.float64).T @ np.asarray(dZ, np.float64)


@pytest.mark.parametrize("variant", ["different", "same"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_p_one_is_exact_backprop(variant, dtype):
    A, dZ = layer_inputs(37, 70, 9, dtype=dtype, seed=3)
    st = rad.forward_store(A, dtype, variant, 1.0, seed=5, layer=2, step=1)
    assert st.T == 4096 and st.scale == np.float32(1.0)
    assert st.nnz == A.size
    assert np.array_equal(st.values.view(np.uint32), A.reshape(-1).view(np.uint32))
    assert np.array_equal(rad.weight_grad(st, dZ), exact_dW(A, dZ))


@pytest.mark.parametrize("variant", ["different", "same"])
def test_only_dW_is_random(variant):
    X, y, Ws, bs = mlp_inputs((20, 16, 12, 5), 9, seed=2, bias_zero=False)
    ex = rad.mlp_step(X, y, Ws, bs)
    rd = rad.mlp_step(X, y, Ws, bs, variant=variant, p=0.3, seed=9)
    assert rd.loss == ex.loss
    for l in range(3):
        assert np.array_equal(rd.Z[l], ex.Z[l])
        assert np.array_equal(rd.dZ[l], ex.dZ[l])
        assert np.array_equal(rd.db[l], ex.db[l])
        assert not np.array_equal(rd.dW[l], ex.dW[l])
    one = rad.mlp_step(X, y, Ws, bs, variant=variant, p=1.0, seed=9)
    for l in range(3):
        assert np.array_equal(one.dW[l], ex.dW[l])


def _all_masks(B, D, variant):
    if variant == "different":
        for bits in itertools.product([False, True], repeat=B * D):
            yield np.array(bits).reshape(B, D)
    else:
        for bits in itertools.product([False, True], repeat=D):
            yield np.broadcast_to(np.array(bits), (B, D))


@pytest.mark.parametrize("variant,B,D", [("different", 3, 4), ("different", 2, 6), ("same", 4, 7)])
@pytest.mark.parametrize("p", [0.1, 0.5, 0.8])
def test_exhaustive_mean_and_variance(variant, B, D, p):
    H = 3
    A, dZ = layer_inputs(B, D, H, seed=B * 100 + D)
    dZ = dZ * 5
    pe = rad.effective_p(p)
    s = float(rad.scale_factor(p))
    mean = np.zeros((D, H))
    second = np.zeros((D, H))
    total = 0.0
    for m in _all_masks(B, D, variant):
        k = int(m.sum()) if variant == "different" else int(m[0].sum())
        n = B * D if variant == "different" else D
        w = pe ** k * (1 - pe) ** (n - k)
        g = rad.weight_grad(rad.forward_store(A, "f32", variant, p, 0, 0, 0, mask=m), dZ)
        mean += w * g
        second += w * g * g
        total += w
    assert total == pytest.approx(1.0, abs=1e-12)
    dW = exact_dW(A, dZ)
    # stored values carry one float32 rounding of A*s and s carries one of 1/p_eff, so each
    # term a_b is off by at most ~2^-23 relative: bound the error by the sum of |a_b|
    bound = 2e-7 * (np.abs(np.asarray(A, np.float64)).T @ np.abs(np.asarray(dZ, np.float64)))
    assert (np.abs(mean - dW) <= bound + 1e-15).all()
    var = second - mean * mean
    q = (1 - pe) / pe
    a = np.asarray(A, np.float64)[:, :, None] * np.asarray(dZ, np.float64)[:, None, :]
    closed = q * (a * a).sum(axis=0) if variant == "different" else q * dW * dW
    assert np.allclose(var, closed, rtol=1e-5, atol=1e-14)
    # scaling by 1/p instead of 1/p_eff, or forgetting the scale, must fail the mean test
    assert abs(s * pe - 1.0) < 1e-7


def test_unbiased_over_philox_seeds():
    """Mean over Philox-driven masks approaches exact dW at the Monte-Carlo rate."""
    A, dZ = layer_inputs(24, 40, 6, seed=8)
    dW = exact_dW(A, dZ)
    a = np.asarray(A, np.float64)[:, :, None] * np.asarray(dZ, np.float64)[:, None, :]
    for variant in ("different", "same"):
        for p in (0.1, 0.5):
            pe = rad.effective_p(p)
            q = (1 - pe) / pe
            var_sum = (q * (a * a).sum(axis=0)).sum() if variant == "different" else (q * dW * dW).sum()
            S = 800
            acc = np.zeros_like(dW)
            sq = 0.0
            for seed in range(S):
                g = rad.weight_grad(rad.forward_store(A, "f32", variant, p, seed, 1, 0), dZ)
                acc += g
                sq += ((g - dW) ** 2).sum()
            err = ((acc / S - dW) ** 2).sum()
            assert err < 2.0 * var_sum / S            # E[err] = var_sum / S exactly
            assert sq / S == pytest.approx(var_sum, rel=0.15)


def test_same_sample_touches_only_kept_rows():
    A, dZ = layer_inputs(30, 64, 5, seed=4)
    st = rad.forward_store(A, "f32", "same", 0.2, seed=1, layer=0, step=0)
    g = rad.weight_grad(st, dZ)
    kept = np.zeros(64, bool)
    kept[st.idx] = True
    assert (g[~kept] == 0).all()
    dW = exact_dW(A, dZ)
    bound = 2e-7 * float(st.scale) * (np.abs(A.astype(np.float64)).T @ np.abs(dZ.astype(np.float64)))
    assert (np.abs(g - dW * float(st.scale))[kept] <= bound[kept]).all()
    assert 0 < st.idx.size < 64


def test_compact_form_structure():
    B, D = 50, 300
    A, _ = layer_inputs(B, D, 1, seed=6, relu_like=True)
    p = 0.1
    st = rad.forward_store(A, "f32", "different", p, seed=3, layer=1, step=0)
    m = rad.keep_mask("different", B, D, p, 3, 1, 0)
    assert st.keepbits.shape == (B, 10) and st.keepbits.dtype == np.uint32
    pop = sum(bin(int(w)).count("1") for w in st.keepbits.reshape(-1))
    assert pop == st.nnz == st.row_ptr[-1] == m.sum()
    assert (np.diff(st.row_ptr) == m.sum(axis=1)).all()
    # bit d%32 of word d//32, least significant bit first; no bits beyond column D
    for b, d in [(0, 0), (3, 31), (7, 32), (49, 299)]:
        assert bool((int(st.keepbits[b, d // 32]) >> (d % 32)) & 1) == bool(m[b, d])
    assert (st.keepbits[:, -1] >> np.uint32(300 - 288) == 0).all()
    # values are A*s in row-major, ascending-column order
    assert np.array_equal(st.values, (A * st.scale)[m])
    # keep fraction within a 5 sigma binomial band of p_eff
    pe = rad.effective_p(p)
    assert abs(m.mean() - pe) < 5 * np.sqrt(pe * (1 - pe) / m.size)
    # ReLU bits: (A > 0); zeros of either sign give 0
    r = rad.unpack_bits(st.relubits, D)
    assert np.array_equal(r, A > 0) and (A == 0).any() and np.signbit(A[A == 0]).any()


def test_mask_depends_on_key_fields_only():
    base = rad.keep_mask("different", 16, 80, 0.3, 1, 2, 3)
    assert not np.array_equal(base, rad.keep_mask("different", 16, 80, 0.3, 2, 2, 3))
    assert not np.array_equal(base, rad.keep_mask("different", 16, 80, 0.3, 1, 3, 3))
    assert not np.array_equal(base, rad.keep_mask("different", 16, 80, 0.3, 1, 2, 4))
    assert not np.array_equal(base, rad.keep_mask("different", 16, 80, 0.3, 1 << 32 | 1, 2, 3))
    # rows are keyed by their global index: any row partition gives the same mask
    assert np.array_equal(base[:5], rad.keep_mask("different", 5, 80, 0.3, 1, 2, 3))
    assert np.array_equal(base[:, :41], rad.keep_mask("different", 16, 41, 0.3, 1, 2, 3))
    # masks are nested in p (one lane, growing threshold)
    assert (rad.keep_mask("different", 16, 80, 0.5, 1, 2, 3) | ~base).all()
    same = rad.keep_mask("same", 16, 80, 0.3, 1, 2, 3)
    assert (same == same[0]).all() and not np.array_equal(same[0], base[0])


def test_threshold_table():
    for p, T in [(0.01, 41), (0.05, 205), (0.1, 410), (0.2, 819), (0.5, 2048), (1.0, 4096), (1e-9, 1),
                 (0.998, 4088), (0.99995, 4096), (1.0 / 4096, 1), (1.0 / 2048, 2), (1.0 / 512, 8)]:
        assert rad.keep_threshold(p) == T
    with pytest.raises(ValueError):
        rad.keep_threshold(0.0)
    with pytest.raises(ValueError):
        rad.keep_threshold(1.5)


def test_sampled_probability_is_the_requested_one():
    """The estimator is Bernoulli(p) rescaled by 1 / p (Sec. 3.2, E[P] = I): the probability really sampled
    stays within 0.1 % of the requested one for every value of the sweeps, the scale is its reciprocal, and
    small probabilities do not collapse onto one another."""
    for p in (0.01, 0.05, 0.1, 0.2, 0.3, 0.5, 0.8, 1.0):
        pe = rad.effective_p(p)
        assert abs(pe - p) / p <= 1e-3, (p, pe)
        assert rad.scale_factor(p) == np.float32(1.0 / pe)
    small = [rad.effective_p(2.0 ** -k) for k in range(1, 13)]
    assert small == [2.0 ** -k for k in range(1, 13)]
    # the frequency of kept entries follows p_eff (Binomial band of five standard deviations)
    for p in (0.01, 0.05):
        m = rad.keep_mask("different", 512, 1024, p, 3, 1, 0)
        n, pe = m.size, rad.effective_p(p)
        assert abs(m.sum() - n * pe) < 5 * np.sqrt(n * pe * (1 - pe))


def test_bf16_rounding_matches_torch():
    import torch
    rng = np.random.default_rng(0)
    x = rng.standard_normal(100000).astype(np.float32) * np.float32(10) ** rng.integers(-20, 20, 100000).astype(np.float32)
    ties = np.array([1.00390625, 1.01171875, -1.00390625, 3.0e38, 1e-40, 0.0, -0.0], np.float32)
    x = np.concatenate([x, ties])
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(rad.round_bf16(x).view(np.uint32), ref.view(np.uint32))
    assert np.array_equal(rad.bf16_bits(ref), torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))


def test_bf16_store_rounds_once_to_bf16():
    A, _ = layer_inputs(8, 64, 1, dtype="bf16", seed=1)
    st = rad.forward_store(A, "bf16", "different", 0.5, 0, 0, 0)
    m = rad.keep_mask("different", 8, 64, 0.5, 0, 0, 0)
    import torch
    ref = (torch.from_numpy(A) * 2.0).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(st.values, ref[m])
