"""Pins for the oracle's Philox-4x32-10 (host only).

Pinned: the generator's published known-answer vectors (tests/golden), agreement with an
independent restatement in Python big integers, invertibility of each round
(multiplication by an odd constant is a bijection mod 2^32), sensitivity to
every counter/key word, and lane uniformity.
"""
import os
import numpy as np
import pytest

from oracle import philox as ph
from oracle import rad as orc

M0, M1, W0, W1 = 0xD2511F53, 0xCD9E8D57, 0x9E3779B9, 0xBB67AE85
MASK = (1 << 32) - 1


def bigint_philox(ctr, key, rounds=10):
    c = list(ctr)
    k = list(key)
    for r in range(rounds):
        if r:
            k = [(k[0] + W0) & MASK, (k[1] + W1) & MASK]
        p0, p1 = M0 * c[0], M1 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k[0], p1 & MASK, (p0 >> 32) ^ c[3] ^ k[1], p0 & MASK]
    return c


def inverse_round(c, k):
    """Undo one round: word 1 and 3 are the low product halves, so the inputs follow by modular inverse."""
    inv0, inv1 = pow(M0, -1, 1 << 32), pow(M1, -1, 1 << 32)
    c0 = (c[3] * inv0) & MASK
    c2 = (c[1] * inv1) & MASK
    c1 = c[0] ^ ((M1 * c2) >> 32) ^ k[0]
    c3 = c[2] ^ ((M0 * c0) >> 32) ^ k[1]
    return [c0, c1, c2, c3]


def test_published_known_answer_vectors():
    path = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_known_answers.txt")
    rows = [[int(t, 16) for t in line.split()] for line in open(path) if line.strip() and not line.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        ctr, key, want = r[:4], r[4:6], r[6:]
        got = ph.philox4x32_10(*(np.uint64(v) for v in ctr), *(np.uint64(v) for v in key))
        assert [int(v) for v in got] == want
        assert bigint_philox(ctr, key) == want


def test_matches_bigint_restatement():
    rng = np.random.default_rng(7)
    n = 20000
    ctr = rng.integers(0, 1 << 32, size=(n, 4), dtype=np.uint64)
    key = rng.integers(0, 1 << 32, size=(n, 2), dtype=np.uint64)
    # include the corners where carries and masks matter
    ctr[:4] = [[0, 0, 0, 0], [MASK] * 4, [1, 0, 0, 0], [0, 0, MASK, 1]]
    key[:4] = [[0, 0], [MASK, MASK], [0, 1], [MASK, 0]]
    out = ph.philox4x32_10(ctr[:, 0], ctr[:, 1], ctr[:, 2], ctr[:, 3], key[:, 0], key[:, 1])
    out = np.stack(out, axis=1)
    for i in range(0, n, 7):
        assert list(out[i]) == bigint_philox([int(v) for v in ctr[i]], [int(v) for v in key[i]])
    for i in range(4):
        assert list(out[i]) == bigint_philox([int(v) for v in ctr[i]], [int(v) for v in key[i]])


def test_round_is_invertible():
    rng = np.random.default_rng(11)
    for _ in range(200):
        c = [int(v) for v in rng.integers(0, 1 << 32, size=4, dtype=np.uint64)]
        k = [int(v) for v in rng.integers(0, 1 << 32, size=2, dtype=np.uint64)]
        out = ph.philox4x32_round(*(np.uint64(v) for v in c), *(np.uint64(v) for v in k))
        assert inverse_round([int(v) for v in out], k) == c


def test_every_input_word_matters():
    base = [3, 5, 7, 11, 13, 17]
    ref = np.stack(ph.philox4x32_10(*[np.uint64(v) for v in base]))
    for i in range(6):
        alt = list(base)
        alt[i] ^= 1
        out = np.stack(ph.philox4x32_10(*[np.uint64(v) for v in alt]))
        assert (out != ref).all()


def test_lane_uniformity_chi_square():
    n = 1 << 16
    words = ph.philox4x32_10(np.arange(n, dtype=np.uint64), 9, 2, 0, 42, 0)
    lanes = np.concatenate([(w >> np.uint32(8 * k)) & np.uint32(0xFF) for w in words for k in range(4)])
    hist = np.bincount(lanes, minlength=256).astype(np.float64)
    expected = lanes.size / 256.0
    chi2 = ((hist - expected) ** 2 / expected).sum()
    # 255 degrees of freedom: mean 255, sd ~22.6; 6 sigma band
    assert abs(chi2 - 255.0) < 6 * 22.6


@pytest.mark.parametrize("variant", ["different", "same"])
def test_keep_mask_at_agrees_with_the_full_mask(variant):
    """The block-wise form is the full mask restricted to the rows and columns asked for."""
    B, D, p, seed, layer, step = 37, 203, 0.3, 0x1234567890, 5, 9
    full = orc.keep_mask(variant, B, D, p, seed, layer, step)
    rows = np.array([0, 3, 36, 17, 17])
    cols = np.array([202, 0, 7, 8, 9, 100, 64])
    got = orc.keep_mask_at(variant, rows, cols, p, seed, layer, step)
    assert np.array_equal(got, full[np.ix_(rows, cols)])
    assert np.array_equal(orc.keep_mask_at(variant, np.arange(B), np.arange(D), p, seed, layer, step), full)


@pytest.mark.parametrize("variant", ["different", "same"])
def test_number_of_a_column_is_laid_across_the_twelve_words_of_three_outputs(variant):
    """Column d is decided by the 12-bit number whose bit 11 - i is the complement of bit d % 32 of word i
    of the three generator outputs for counters 3 (d // 32) + j, j = 0, 1, 2; restated here with Python
    integers, independent of the array code in the oracle."""
    B, D, p, seed, layer, step = 5, 77, 0.3, 0xABCDEF0123456789, 6, 11
    T = orc.keep_threshold(p)
    assert T == 1229          # rint(0.3 * 4096)
    full = orc.keep_mask(variant, B, D, p, seed, layer, step)
    stream = 0 if variant == "different" else 1
    for b in range(B):
        row = b if variant == "different" else 0
        for d in range(D):
            words = []
            for j in range(3):
                words += bigint_philox([3 * (d // 32) + j, row, layer | stream << 24, step], [seed & MASK, seed >> 32])
            u = sum((1 - ((w >> (d % 32)) & 1)) << (11 - i) for i, w in enumerate(words))
            assert bool(full[b, d]) == (u < T)


def test_decision_numbers_are_uniform():
    u = orc._decision_numbers(np.arange(128, dtype=np.uint64)[None, :], np.arange(128, dtype=np.uint64)[:, None], 0, 42, 2, 0)
    assert u.max() < 4096
    hist = np.bincount(u.reshape(-1), minlength=4096).astype(np.float64)
    expected = u.size / 4096.0
    chi2 = ((hist - expected) ** 2 / expected).sum()
    # 4095 degrees of freedom: mean 4095, sd ~90.5; 6 sigma band
    assert abs(chi2 - 4095.0) < 6 * 90.5
    # every bit plane on its own is balanced (a dropped or repeated plane would show here)
    for i in range(12):
        ones = int(((u >> i) & 1).sum())
        assert abs(ones - u.size / 2) < 6 * np.sqrt(u.size / 4)
