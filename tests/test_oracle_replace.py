"""Pins for the oracle's with-replacement sampling law (host only).

Paper, Sec. 3.2: P = (d / k) sum_{s=1..k} P_s with P_s drawn uniformly from {e_i e_i^T}, E[P] = I;
App. A: k = fraction * d activations sampled with replacement, and a fraction of 1.0 is therefore not
the exact gradient.  Pinned here: expectation and variance over ALL draw sequences of a tiny layer,
the closed forms, the count of distinct coordinates, the draw-to-column map against a big-integer
restatement, and the mean over Philox seeds.
"""
import itertools

import numpy as np
import pytest

from oracle import rad

from test_oracle_philox import bigint_philox, MASK


def _layer(B, D, H, seed):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((B, D)).astype(np.float32), rng.standard_normal((B, H)).astype(np.float32)


def _counts_of(seq, D):
    return np.bincount(np.asarray(seq), minlength=D)


def test_draw_count_is_ceil_of_fraction_times_d():
    for f, D, k in [(0.1, 784, 79), (0.1, 300, 30), (0.1, 10, 1), (0.5, 3, 2), (1.0, 7, 7), (0.05, 8192, 410),
                    (0.1, 8192, 820), (1e-9, 50, 1)]:
        assert rad.draws_per_row(f, D) == k
    # App. A counts 79 of the 784 inputs at fraction 0.1
    assert rad.draws_per_row(0.1, 784) == 79
    with pytest.raises(ValueError):
        rad.draws_per_row(0.0, 5)


@pytest.mark.parametrize("variant", ["different", "same"])
def test_expectation_and_variance_over_all_draw_sequences(variant):
    """D = 3, k = 2: nine equally likely sequences per row.  Mean of dW_hat = A^T dZ; variance of an entry
    = (D - 1) / k * sum_b (A[b,d] dZ[b,h])^2 when rows draw independently, (D - 1) / k * dW[d,h]^2 when
    they share the draws (Var of a Binomial(k, 1/D) count times (D/k)^2)."""
    B, D, H, f = 2, 3, 2, 0.5
    k = rad.draws_per_row(f, D)
    assert k == 2
    A, dZ = _layer(B, D, H, 5)
    exact = A.astype(np.float64).T @ dZ.astype(np.float64)
    seqs = list(itertools.product(range(D), repeat=k))
    if variant == "different":
        combos = list(itertools.product(seqs, repeat=B))
    else:
        combos = [(sq,) * B for sq in seqs]
    grads = []
    for combo in combos:
        c = np.stack([_counts_of(sq, D) for sq in combo])
        st = rad.forward_store(A, "f32", variant, f, 0, 0, 0, law="replace", counts=c)
        assert st.T == k and st.scale == np.float32(1.5)
        grads.append(rad.weight_grad(st, dZ))
    grads = np.stack(grads)
    mean, var = grads.mean(axis=0), grads.var(axis=0)
    assert np.allclose(mean, exact, rtol=1e-6, atol=1e-6)
    terms = A.astype(np.float64)[:, :, None] * dZ.astype(np.float64)[:, None, :]      # B x D x H
    q = (D - 1) / k
    closed = q * (terms ** 2).sum(axis=0) if variant == "different" else q * exact ** 2
    assert np.allclose(var, closed, rtol=1e-5, atol=1e-6)
    # a wrong weight (d/k counted once per distinct coordinate instead of once per draw) must fail
    wrong = []
    for combo in combos:
        c = np.stack([_counts_of(sq, D) for sq in combo])
        wrong.append(rad.weight_grad(rad.forward_store(A, "f32", variant, f, 0, 0, 0, law="replace",
                                                       counts=np.minimum(c, 1)), dZ))
    assert not np.allclose(np.stack(wrong).mean(axis=0), exact, rtol=1e-3, atol=1e-3)


@pytest.mark.parametrize("variant", ["different", "same"])
def test_multiplicities_structure(variant):
    B, D, f = 9, 203, 0.3
    c = rad.multiplicity(variant, B, D, f, 11, 2, 5)
    k = rad.draws_per_row(f, D)
    assert c.shape == (B, D) and (c.sum(axis=1) == k).all() and (c >= 0).all()
    if variant == "same":
        assert (c == c[0]).all()
    else:
        assert not (c == c[0]).all()
        assert np.array_equal(c[:4], rad.multiplicity(variant, 4, D, f, 11, 2, 5))      # rows keyed globally
    for other in [(12, 2, 5), (11, 3, 5), (11, 2, 6), (11 | 1 << 32, 2, 5)]:
        assert not np.array_equal(c, rad.multiplicity(variant, B, D, f, *other))
    # not the Bernoulli stream, and the two with-replacement streams differ
    assert not np.array_equal(rad.multiplicity("same", B, D, f, 11, 2, 5)[0],
                              rad.multiplicity("different", B, D, f, 11, 2, 5)[0])


@pytest.mark.parametrize("variant", ["different", "same"])
def test_draw_to_column_map_against_big_integers(variant):
    """Draw j reads word j % 4 of the output for counter j // 4 and picks floor(word * D / 2^32)."""
    B, D, f, seed, layer, step = 3, 37, 0.4, 0x0123456789ABCDEF, 4, 9
    k = rad.draws_per_row(f, D)
    c = rad.multiplicity(variant, B, D, f, seed, layer, step)
    stream = 2 if variant == "different" else 3
    for b in range(B):
        want = [0] * D
        for j in range(k):
            out = bigint_philox([j // 4, b if variant == "different" else 0, layer | stream << 24, step],
                                [seed & MASK, seed >> 32])
            want[(out[j % 4] * D) >> 32] += 1
        assert list(c[b]) == want


def test_distinct_fraction_and_fraction_one_is_not_exact():
    """E[distinct coordinates] = D (1 - (1 - 1/D)^k); at fraction 1.0 about 1 - 1/e of the coordinates
    are kept, so the estimate is not the exact gradient (App. A, caption of the fraction sweep)."""
    B, D = 400, 256
    for f in (0.1, 0.5, 1.0):
        k = rad.draws_per_row(f, D)
        c = rad.multiplicity("different", B, D, f, 3, 0, 0)
        distinct = (c > 0).sum(axis=1)
        expect = D * (1.0 - (1.0 - 1.0 / D) ** k)
        # Var of the distinct count is below its mean; 6 sigma of the mean over B rows
        assert abs(distinct.mean() - expect) < 6 * np.sqrt(expect / B)
    A, dZ = _layer(8, 64, 3, 2)
    st = rad.forward_store(A, "f32", "different", 1.0, 0, 0, 0, law="replace")
    assert st.nnz < A.size
    assert not np.allclose(rad.weight_grad(st, dZ), A.astype(np.float64).T @ dZ.astype(np.float64), rtol=1e-3)


def test_columns_are_hit_uniformly():
    D, B, f = 64, 2000, 0.5
    c = rad.multiplicity("different", B, D, f, 9, 1, 1)
    hits = c.sum(axis=0).astype(np.float64)
    expected = B * rad.draws_per_row(f, D) / D
    chi2 = ((hits - expected) ** 2 / expected).sum()
    assert abs(chi2 - (D - 1)) < 6 * np.sqrt(2 * (D - 1))


@pytest.mark.parametrize("variant", ["different", "same"])
def test_unbiased_over_philox_seeds(variant):
    B, D, H, f, n = 4, 24, 3, 0.25, 3000
    A, dZ = _layer(B, D, H, 8)
    exact = A.astype(np.float64).T @ dZ.astype(np.float64)
    acc = np.zeros_like(exact)
    for seed in range(n):
        acc += rad.weight_grad(rad.forward_store(A, "f32", variant, f, seed, 1, 0, law="replace"), dZ)
    k = rad.draws_per_row(f, D)
    terms = A.astype(np.float64)[:, :, None] * dZ.astype(np.float64)[:, None, :]
    var = (D - 1) / k * ((terms ** 2).sum(axis=0) if variant == "different" else exact ** 2)
    assert (np.abs(acc / n - exact) < 6 * np.sqrt(var / n) + 1e-6).all()


def test_store_structure_and_rounding():
    B, D, f = 20, 100, 0.2
    A, _ = _layer(B, D, 1, 4)
    c = rad.multiplicity("different", B, D, f, 1, 0, 2)
    st = rad.forward_store(A, "bf16", "different", f, 1, 0, 2, law="replace")
    assert np.array_equal(rad.unpack_bits(st.keepbits, D), c > 0)
    s = np.float32(D) / np.float32(rad.draws_per_row(f, D))
    want = rad.round_bf16(A * (c.astype(np.float32) * s))[c > 0]
    assert np.array_equal(st.values.view(np.uint32), want.view(np.uint32))
    assert (c > 1).any()            # the case has repeated draws, so the multiplicity weight is exercised
    same = rad.forward_store(A, "f32", "same", f, 1, 0, 2, law="replace")
    c1 = rad.multiplicity("same", B, D, f, 1, 0, 2)[0]
    assert np.array_equal(same.idx, np.flatnonzero(c1))
    assert np.array_equal(same.values.reshape(B, -1), (A * (c1.astype(np.float32) * s))[:, c1 > 0])


def test_rows_argument_is_the_full_matrix_restricted_to_those_rows():
    B, D, f = 40, 150, 0.2
    rows = np.array([0, 7, 39, 12, 12])
    assert np.array_equal(rad.multiplicity("different", B, D, f, 3, 1, 2, rows=rows),
                          rad.multiplicity("different", B, D, f, 3, 1, 2)[rows])
    assert np.array_equal(rad.fixed_subset("different", B, D, f, 3, 1, 2, rows=rows),
                          rad.fixed_subset("different", B, D, f, 3, 1, 2)[rows])
