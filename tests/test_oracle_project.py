"""Pins for the oracle's random-projection variant (host only).  Paper, Sec. 3.2 (after Eq. 5) and App. A
"Random Projections for RAD": P = R R^T, R a d x k matrix of independent Rademacher variables scaled by
1 / sqrt(k), E[P] = I.  Pinned: mean and variance of dW_hat over ALL sign matrices of a tiny layer, the
closed form Var = (1/k) sum_{d' != d} (A^T dZ)[d', h]^2, E[R' R'^T] / k = I, the bit-to-sign map against a
big-integer restatement, k = d with orthogonal signs reproduces the exact gradient, Monte-Carlo mean."""
import itertools

import numpy as np

from oracle import rad

from test_oracle_philox import bigint_philox, MASK


def _layer(B, D, H, seed):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((B, D)).astype(np.float32), rng.standard_normal((B, H)).astype(np.float32)


def test_mean_and_variance_over_all_sign_matrices():
    B, D, H, f = 3, 3, 2, 0.5
    k = rad.draws_per_row(f, D)
    assert k == 2
    A, dZ = _layer(B, D, H, 3)
    M = A.astype(np.float64).T @ dZ.astype(np.float64)
    grads = []
    for signs in itertools.product([1.0, -1.0], repeat=D * k):
        R = np.array(signs).reshape(D, k)
        grads.append(rad.weight_grad(rad.project_store(A, "f32", f, 0, 0, 0, R=R), dZ))
    grads = np.stack(grads)
    assert np.allclose(grads.mean(axis=0), M, rtol=1e-5, atol=1e-6)
    closed = ((M ** 2).sum(axis=0, keepdims=True) - M ** 2) / k
    assert np.allclose(grads.var(axis=0), closed, rtol=1e-4, atol=1e-6)
    # leaving out the 1 / k (R unscaled) must fail the mean test
    assert not np.allclose(grads.mean(axis=0) * k, M, rtol=1e-2, atol=1e-3)


def test_signs_against_big_integers_and_key_fields():
    D, k, seed, layer, step = 7, 300, 0x1122334455667788, 5, 2
    R = rad.rademacher(D, k, seed, layer, step)
    assert R.shape == (D, k) and set(np.unique(R)) == {-1.0, 1.0}
    for d in range(D):
        for j in (0, 1, 31, 32, 127, 128, 255, 299):
            out = bigint_philox([j // 128, d, layer | 6 << 24, step], [seed & MASK, seed >> 32])
            bit = (out[(j % 128) // 32] >> (j % 32)) & 1
            assert R[d, j] == (-1.0 if bit else 1.0)
    for other in [(seed + 1, layer, step), (seed, layer + 1, step), (seed, layer, step + 1)]:
        assert not np.array_equal(R, rad.rademacher(D, k, *other))
    assert np.array_equal(R[:, :100], rad.rademacher(D, 100, seed, layer, step))      # columns are keyed by index


def test_projection_is_identity_in_expectation():
    D, k, n = 12, 5, 4000
    acc = np.zeros((D, D))
    for seed in range(n):
        R = rad.rademacher(D, k, seed, 0, 0)
        acc += R @ R.T / k
    dev = acc / n - np.eye(D)
    # off-diagonal entries are means of k n independent signs divided by k; diagonal entries are exactly 1
    assert np.allclose(np.diag(dev), 0.0) and np.abs(dev).max() < 6 / np.sqrt(k * n)
    signs = R.reshape(-1)
    assert abs(signs.mean()) < 0.5


def test_orthogonal_signs_with_k_equal_d_give_the_exact_gradient():
    """With k = d and R' a Hadamard matrix, R R^T = I: the estimate is the exact gradient (up to rounding)."""
    H4 = np.array([[1, 1, 1, 1], [1, -1, 1, -1], [1, 1, -1, -1], [1, -1, -1, 1]], dtype=np.float64)
    A, dZ = _layer(6, 4, 3, 7)
    st = rad.project_store(A, "f32", 1.0, 0, 0, 0, R=H4)
    assert st.T == 4
    assert np.allclose(rad.weight_grad(st, dZ), A.astype(np.float64).T @ dZ.astype(np.float64), rtol=1e-5, atol=1e-6)


def test_unbiased_over_philox_seeds_and_bf16_store():
    B, D, H, f, n = 5, 16, 3, 0.25, 3000
    A, dZ = _layer(B, D, H, 10)
    M = A.astype(np.float64).T @ dZ.astype(np.float64)
    k = rad.draws_per_row(f, D)
    acc = np.zeros_like(M)
    for seed in range(n):
        acc += rad.weight_grad(rad.project_store(A, "f32", f, seed, 2, 1), dZ)
    var = ((M ** 2).sum(axis=0, keepdims=True) - M ** 2) / k
    assert (np.abs(acc / n - M) < 6 * np.sqrt(var / n) + 1e-6).all()
    st = rad.project_store(rad.round_bf16(A), "bf16", f, 1, 0, 0)
    S = st.values.reshape(B, k)
    assert np.array_equal(S, rad.round_bf16(S))                                        # stored on the bf16 grid
    assert np.allclose(S, rad.round_bf16(A).astype(np.float64) @ st.R, rtol=2 ** -8)
