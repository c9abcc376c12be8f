"""Pins for the oracle's fixed-count law: exactly k = ceil(fraction d) distinct coordinates per row,
weight d / k (host only).  Paper, App. A (caption of the fraction sweep): without replacement, a
fraction of 1.0 is the baseline.  Pinned: Floyd's subset sampling gives every subset equally often over
all draw sequences; expectation and variance of dW_hat over all subsets of a tiny layer; fraction 1.0
is exact backprop bit for bit; the draw map against a big-integer restatement; Monte-Carlo mean."""
import itertools

import numpy as np
import pytest

from oracle import rad

from test_oracle_philox import bigint_philox, MASK


def _layer(B, D, H, seed):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((B, D)).astype(np.float32), rng.standard_normal((B, H)).astype(np.float32)


def test_floyd_gives_every_subset_equally_often():
    D, k = 5, 3
    ranges = [range(D - k + i + 1) for i in range(k)]
    seqs = np.array(list(itertools.product(*ranges)))            # 3 * 4 * 5 = 60 equally likely sequences
    chosen = rad.floyd_subset(seqs, D)
    assert (chosen.sum(axis=1) == k).all()
    keys, counts = np.unique(chosen, axis=0, return_counts=True)
    assert len(keys) == 10 and (counts == 6).all()               # C(5, 3) subsets, 60 / 10 each
    with pytest.raises(ValueError):
        rad.floyd_subset(np.array([[3, 0, 0]]), D)               # first draw must lie in [0, D - k]


@pytest.mark.parametrize("variant", ["different", "same"])
def test_expectation_and_variance_over_all_subsets(variant):
    """D = 4, k = 2: six equally likely subsets per row.  Mean of dW_hat = A^T dZ; variance of an entry
    = (D - k) / k * sum_b (A[b,d] dZ[b,h])^2 (rows independent) or (D - k) / k * dW[d,h]^2 (shared subset)."""
    B, D, H, f = 2, 4, 2, 0.5
    k = rad.draws_per_row(f, D)
    A, dZ = _layer(B, D, H, 6)
    exact = A.astype(np.float64).T @ dZ.astype(np.float64)
    subsets = [np.isin(np.arange(D), c).astype(np.int64) for c in itertools.combinations(range(D), k)]
    combos = list(itertools.product(subsets, repeat=B)) if variant == "different" else [(s,) * B for s in subsets]
    grads = np.stack([rad.weight_grad(rad.forward_store(A, "f32", variant, f, 0, 0, 0, law="fixed",
                                                        counts=np.stack(c)), dZ) for c in combos])
    assert np.allclose(grads.mean(axis=0), exact, rtol=1e-6, atol=1e-6)
    terms = A.astype(np.float64)[:, :, None] * dZ.astype(np.float64)[:, None, :]
    q = (D - k) / k
    closed = q * (terms ** 2).sum(axis=0) if variant == "different" else q * exact ** 2
    assert np.allclose(grads.var(axis=0), closed, rtol=1e-5, atol=1e-6)


@pytest.mark.parametrize("variant", ["different", "same"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_fraction_one_is_exact_backprop(variant, dtype):
    A, dZ = _layer(9, 33, 4, 1)
    if dtype == "bf16":
        A, dZ = rad.round_bf16(A), rad.round_bf16(dZ)
    st = rad.forward_store(A, dtype, variant, 1.0, 3, 1, 2, law="fixed")
    assert st.T == 33 and st.scale == np.float32(1.0) and st.nnz == A.size
    assert np.array_equal(rad.weight_grad(st, dZ), A.astype(np.float64).T @ dZ.astype(np.float64))


@pytest.mark.parametrize("variant", ["different", "same"])
def test_subset_structure_and_draw_map(variant):
    B, D, f, seed, layer, step = 5, 41, 0.3, 0xFEDCBA9876543210, 3, 8
    k = rad.draws_per_row(f, D)
    c = rad.fixed_subset(variant, B, D, f, seed, layer, step)
    assert c.shape == (B, D) and (c.sum(axis=1) == k).all() and set(np.unique(c)) <= {0, 1}
    if variant == "same":
        assert (c == c[0]).all()
    stream = 4 if variant == "different" else 5
    for b in range(B):
        chosen = set()
        for i in range(k):
            out = bigint_philox([i // 4, b if variant == "different" else 0, layer | stream << 24, step],
                                [seed & MASK, seed >> 32])
            j = D - k + i
            t = (out[i % 4] * (j + 1)) >> 32
            chosen.add(j if t in chosen else t)
        assert set(np.flatnonzero(c[b])) == chosen
    for other in [(seed + 1, layer, step), (seed, layer + 1, step), (seed, layer, step + 1)]:
        assert not np.array_equal(c, rad.fixed_subset(variant, B, D, f, *other))
    assert not np.array_equal(c, rad.multiplicity(variant, B, D, f, seed, layer, step) > 0)


def test_columns_are_kept_uniformly():
    D, B, f = 48, 3000, 0.25
    c = rad.fixed_subset("different", B, D, f, 5, 0, 0)
    k = rad.draws_per_row(f, D)
    hits = c.sum(axis=0).astype(np.float64)
    expected = B * k / D
    # a column's count is Binomial(B, k/D); the columns are negatively correlated, which only tightens the sum
    z = (hits - expected) / np.sqrt(expected * (1 - k / D))
    assert np.abs(z).max() < 5.0


@pytest.mark.parametrize("variant", ["different", "same"])
def test_unbiased_over_philox_seeds(variant):
    B, D, H, f, n = 4, 24, 3, 0.25, 3000
    A, dZ = _layer(B, D, H, 9)
    exact = A.astype(np.float64).T @ dZ.astype(np.float64)
    acc = np.zeros_like(exact)
    for seed in range(n):
        acc += rad.weight_grad(rad.forward_store(A, "f32", variant, f, seed, 1, 0, law="fixed"), dZ)
    k = rad.draws_per_row(f, D)
    terms = A.astype(np.float64)[:, :, None] * dZ.astype(np.float64)[:, None, :]
    var = (D - k) / k * ((terms ** 2).sum(axis=0) if variant == "different" else exact ** 2)
    assert (np.abs(acc / n - exact) < 6 * np.sqrt(var / n) + 1e-6).all()
