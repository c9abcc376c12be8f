"""Activation-sampling RAD for fully connected nets: oracle (numpy, float64).

TEST INFRASTRUCTURE ONLY; see the package docstring.

What is computed (paper, Sec. 4.2).  For a linear layer Z = A W + b with
A in R^{B x D} the weight gradient of exact backprop is dW = A^T dZ.  The only
Jacobian RAD samples is dh/dW, i.e. the layer input A: it is replaced by
A_hat = A P with a random P, E[P] = I (Sec. 3.2, the random matrix injection
S_P[J] = J P and its two required properties).  Everything else on the
backward path (the loss Jacobian, W, the ReLU derivative bits) is kept exact,
so only dW is random.

Reading of the sampling law used here.  The paper draws k of d coordinates
with replacement, P = (d/k) sum_s e_s e_s^T; it also notes that sampling
without replacement makes fraction 1.0 identical to exact backprop.  This
oracle uses independent Bernoulli keeps: P = diag(m) / p_eff with
m_i ~ Bernoulli(p_eff), which has E[P] = I and P = R R^T for
R = diag(sqrt(m / p_eff)) restricted to kept columns.  "different sample"
draws m per minibatch row, "same sample" draws one m per layer and step
(Sec. 4.3).

The keep decision for (row b, column d) compares a 12-bit number u with a
threshold T = round(p * 2^12) clipped to [1, 2^12]: kept iff u < T;
p_eff = T / 2^12 and stored values are scaled by fl32(2^12 / T), so the
estimator is exactly unbiased for the probability actually sampled.  The paper
leaves the source of randomness open.  The numbers of 32 consecutive columns
are laid across the twelve words of three Philox-4x32-10 outputs, one bit
plane per word: bit d % 32 of word i holds (complemented) bit 11 - i of the
number of column d.  A device then gets the 32 decisions of a keep-bit word
from twelve word-wide AND / OR steps along the binary digits of T instead of
32 compares.  Every keep probability of the sweeps (0.01 ... 0.5) is sampled
within 0.1 % of its value, and probabilities down to 2^-12 stay distinct.

Second sampling law, the paper's own (Sec. 3.2, App. A): k = ceil(fraction * d)
coordinates drawn uniformly WITH replacement, P = (d / k) sum_s e_s e_s^T, so a
coordinate hit c times is kept with weight c * d / k (`law="replace"`).

Third law (App. A, caption of the fraction sweep, which remarks that drawing
without replacement would make fraction 1.0 the exact gradient):
a uniformly random subset of exactly k = ceil(fraction * d) coordinates, each
kept with weight d / k (`law="fixed"`).

Random projection (Sec. 3.2 after Eq. 5; App. A "Random Projections for RAD"):
P = R R^T with R a d x k matrix of independent Rademacher signs scaled by
1 / sqrt(k).  The forward pass keeps S = A R' (B x k, R' the unscaled signs),
the backward pass forms dW_hat = R' ((S^T dZ) / k) (`variant="project"`).
"""
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np
from scipy.special import erf

from .philox import philox4x32_10

STREAM_DIFFERENT = 0     # counter stream of per-row masks
STREAM_SAME = 1          # counter stream of masks shared by the minibatch
STREAM_DIFFERENT_REPLACE = 2   # with-replacement draws, per row
STREAM_SAME_REPLACE = 3        # with-replacement draws, shared by the minibatch
STREAM_DIFFERENT_FIXED = 4     # k distinct columns, per row
STREAM_SAME_FIXED = 5          # k distinct columns, shared by the minibatch
STREAM_PROJECT = 6             # signs of the Rademacher projection
LANE_BITS = 12
OUTPUTS_PER_GROUP = LANE_BITS // 4   # generator outputs (four words each) behind one keep-bit word
COLUMNS_PER_GROUP = 32   # one keep-bit word: three generator outputs (384 bits), twelve bit planes of 32 columns
LANE_RANGE = 1 << LANE_BITS


# --------------------------------------------------------------------------
# mask (Sec. 3.2: E[P] = I; Sec. 4.3: "same sample" / "different sample")
# --------------------------------------------------------------------------
def keep_threshold(p) -> int:
    """T such that an entry whose 12-bit number is u is kept iff u < T."""
    p32 = float(np.float32(p))
    if not (0.0 < p32 <= 1.0):
        raise ValueError("p must be in (0, 1]")
    return int(min(max(np.rint(p32 * LANE_RANGE), 1.0), float(LANE_RANGE)))


def effective_p(p) -> float:
    return keep_threshold(p) / LANE_RANGE


def scale_factor(p) -> np.float32:
    """s = fl32(1 / p_eff), one correctly rounded float32 division."""
    return np.float32(LANE_RANGE) / np.float32(keep_threshold(p))


def _decision_numbers(group, rows, stream, seed, layer, step):
    """Numbers u of the 32 columns of each (row, group): shape rows x groups x 32, uint32 in [0, 4096).

    Outputs of the generator for counters (3 * group + j, row, layer | stream << 24, step), j = 0, 1, 2,
    key = (seed low word, seed high word), give words w_0 .. w_11 (first output first).  Column c of the
    group has u = sum_i (1 - bit c of w_i) << (11 - i).
    """
    c2 = np.uint64((layer & 0xFFFFFF) | (stream << 24))
    k0, k1 = np.uint64(seed & 0xFFFFFFFF), np.uint64((seed >> 32) & 0xFFFFFFFF)
    words = []
    for j in range(OUTPUTS_PER_GROUP):
        words.extend(philox4x32_10(np.uint64(OUTPUTS_PER_GROUP) * group + np.uint64(j), rows, c2,
                                   np.uint64(step & 0xFFFFFFFF), k0, k1))
    shape = np.broadcast(group, rows).shape
    u = np.zeros(shape + (COLUMNS_PER_GROUP,), dtype=np.uint32)
    cols = np.arange(COLUMNS_PER_GROUP, dtype=np.uint32)
    for i, w in enumerate(words):
        bits = (np.broadcast_to(w, shape)[..., None] >> cols) & np.uint32(1)
        u |= (np.uint32(1) - bits) << np.uint32(LANE_BITS - 1 - i)
    return u


def keep_mask(variant: str, B: int, D: int, p, seed: int, layer: int, step: int) -> np.ndarray:
    """Boolean B x D keep mask: column d of row b is kept iff its number (see _decision_numbers, group d // 32,
    column d % 32 of the group) is below T.  For "same" the row field of the counter is 0 and the single
    row of decisions is shared by every minibatch element."""
    T = keep_threshold(p)
    groups = (D + COLUMNS_PER_GROUP - 1) // COLUMNS_PER_GROUP
    if variant == "different":
        rows, stream = np.arange(B, dtype=np.uint64)[:, None], STREAM_DIFFERENT
    elif variant == "same":
        rows, stream = np.zeros((1, 1), dtype=np.uint64), STREAM_SAME
    else:
        raise ValueError(variant)
    u = _decision_numbers(np.arange(groups, dtype=np.uint64)[None, :], rows, stream, seed, layer, step)
    m = (u < T).reshape(u.shape[0], groups * COLUMNS_PER_GROUP)[:, :D]
    if variant == "same":
        m = np.broadcast_to(m, (B, D))
    return np.ascontiguousarray(m)


def keep_mask_at(variant: str, rows, cols, p, seed: int, layer: int, step: int) -> np.ndarray:
    """Keep decisions of the given rows x the given columns (len(rows) x len(cols), boolean): the same
    counter, key and threshold rule as keep_mask, evaluated only where asked, so that single tiles or
    single columns of a layer too large to expand in full can be checked."""
    T = keep_threshold(p)
    rows = np.asarray(rows, dtype=np.uint64).reshape(-1, 1)
    cols = np.asarray(cols, dtype=np.uint64).reshape(1, -1)
    if variant == "different":
        stream = STREAM_DIFFERENT
    elif variant == "same":
        rows, stream = np.zeros_like(rows), STREAM_SAME
    else:
        raise ValueError(variant)
    u = _decision_numbers(cols // np.uint64(COLUMNS_PER_GROUP) + np.zeros_like(rows), rows + np.zeros_like(cols), stream,
                        seed, layer, step)                                  # rows x cols x 32
    pick = (cols % np.uint64(COLUMNS_PER_GROUP)).astype(np.int64) + np.zeros(rows.shape, dtype=np.int64)
    return np.take_along_axis(u, pick[..., None], axis=-1)[..., 0] < T


# --------------------------------------------------------------------------
# the paper's own sampling law (Sec. 3.2, the example after Eq. 5: k of the d
# coordinates drawn with replacement; App. A: a fraction of the activations)
# --------------------------------------------------------------------------
def draws_per_row(fraction, D: int) -> int:
    """k = ceil(fraction * d), at least 1 and at most d.  The fraction arrives as a float32 (0.1 is then
    a little above one tenth), so the product is taken in float64 and shrunk by 2^-22 before the
    ceiling: 0.1 * 300 gives 30, not 31."""
    f32 = float(np.float32(fraction))
    if not (0.0 < f32 <= 1.0):
        raise ValueError("fraction must be in (0, 1]")
    return int(min(max(np.ceil(f32 * D * (1.0 - 2.0 ** -22)), 1.0), float(D)))


def replace_scale(fraction, D: int) -> np.float32:
    """d / k as one float32 division: the weight of a coordinate drawn once."""
    return np.float32(D) / np.float32(draws_per_row(fraction, D))


def multiplicity(variant: str, B: int, D: int, fraction, seed: int, layer: int, step: int, rows=None) -> np.ndarray:
    """c[b, d] = how many of the k draws of row b picked column d (B x D, int64).  `rows`: evaluate these
    minibatch rows only (len(rows) x D), for layers too large to expand in full.

    Draw j of a row reads 32-bit word j % 4 of the Philox output for counter
    (j // 4, row, layer | stream << 24, step) and picks column
    floor(word * D / 2^32).  "same": one set of draws (row field 0) for the whole
    minibatch.  Every row's multiplicities add up to k.
    """
    k = draws_per_row(fraction, D)
    if rows is not None:
        B = len(rows)
    if variant == "different":
        rows = np.arange(B, dtype=np.uint64) if rows is None else np.asarray(rows, dtype=np.uint64)
        rows, stream = rows[:, None], STREAM_DIFFERENT_REPLACE
    elif variant == "same":
        rows, stream = np.zeros((1, 1), dtype=np.uint64), STREAM_SAME_REPLACE
    else:
        raise ValueError(variant)
    calls = (k + 3) // 4
    c0 = np.arange(calls, dtype=np.uint64)[None, :]
    words = philox4x32_10(c0, rows, np.uint64((layer & 0xFFFFFF) | (stream << 24)), np.uint64(step & 0xFFFFFFFF),
                          np.uint64(seed & 0xFFFFFFFF), np.uint64((seed >> 32) & 0xFFFFFFFF))
    draws = np.stack([w.astype(np.uint64) for w in words], axis=-1).reshape(rows.shape[0], calls * 4)[:, :k]
    cols = (draws * np.uint64(D)) >> np.uint64(32)
    nrows = cols.shape[0]
    flat = (np.arange(nrows, dtype=np.uint64)[:, None] * np.uint64(D) + cols).reshape(-1).astype(np.int64)
    c = np.bincount(flat, minlength=nrows * D).reshape(nrows, D)
    if variant == "same":
        c = np.broadcast_to(c, (B, D))
    return np.ascontiguousarray(c.astype(np.int64))


# --------------------------------------------------------------------------
# exactly k distinct coordinates, without replacement (App. A, remark under the
# fraction sweep)
# --------------------------------------------------------------------------
def floyd_subset(ts, D: int) -> np.ndarray:
    """Floyd's subset sampling, vectorised over rows.  ts[:, i] is the i-th draw, an integer in
    [0, D - k + i]; step i adds ts[:, i] to the subset unless it is already in, in which case it adds
    D - k + i (never in before).  If every ts[:, i] is uniform on its range, every k-subset of
    {0, ..., D-1} is equally likely.  Returns the indicator (rows x D, bool)."""
    ts = np.asarray(ts, dtype=np.int64)
    rows, k = ts.shape
    chosen = np.zeros((rows, D), dtype=bool)
    r = np.arange(rows)
    for i in range(k):
        j = D - k + i
        t = ts[:, i]
        if (t < 0).any() or (t > j).any():
            raise ValueError("draw out of range")
        pick = np.where(chosen[r, t], j, t)
        chosen[r, pick] = True
    return chosen


def fixed_subset(variant: str, B: int, D: int, fraction, seed: int, layer: int, step: int, rows=None) -> np.ndarray:
    """Indicator (B x D, int64, k ones per row) of the k columns a row keeps.  `rows`: evaluate these
    minibatch rows only.

    Draw i of a row reads 32-bit word i % 4 of the Philox output for counter
    (i // 4, row, layer | stream << 24, step) and becomes floor(word * (D - k + i + 1) / 2^32), the i-th
    draw of floyd_subset.  "same": one subset (row field 0) for the whole minibatch.
    """
    k = draws_per_row(fraction, D)
    if rows is not None:
        B = len(rows)
    if variant == "different":
        rows = np.arange(B, dtype=np.uint64) if rows is None else np.asarray(rows, dtype=np.uint64)
        rows, stream = rows[:, None], STREAM_DIFFERENT_FIXED
    elif variant == "same":
        rows, stream = np.zeros((1, 1), dtype=np.uint64), STREAM_SAME_FIXED
    else:
        raise ValueError(variant)
    calls = (k + 3) // 4
    c0 = np.arange(calls, dtype=np.uint64)[None, :]
    words = philox4x32_10(c0, rows, np.uint64((layer & 0xFFFFFF) | (stream << 24)), np.uint64(step & 0xFFFFFFFF),
                          np.uint64(seed & 0xFFFFFFFF), np.uint64((seed >> 32) & 0xFFFFFFFF))
    draws = np.stack([w.astype(np.uint64) for w in words], axis=-1).reshape(rows.shape[0], calls * 4)[:, :k]
    span = (np.uint64(D - k + 1) + np.arange(k, dtype=np.uint64))[None, :]
    chosen = floyd_subset(((draws * span) >> np.uint64(32)).astype(np.int64), D).astype(np.int64)
    if variant == "same":
        chosen = np.broadcast_to(chosen, (B, D))
    return np.ascontiguousarray(chosen)


# --------------------------------------------------------------------------
# random projection (Sec. 3.2 after Eq. 5: R a matrix of independent Rademacher
# signs; App. A: scaled so that P = R R^T has E[P] = I)
# --------------------------------------------------------------------------
def rademacher(D: int, k: int, seed: int, layer: int, step: int) -> np.ndarray:
    """The unscaled sign matrix R' (D x k, entries +1 / -1, float64); R = R' / sqrt(k).

    Entry (d, j) reads bit j % 32 of word (j % 128) // 32 of the Philox output for counter
    (j // 128, d, layer | 6 << 24, step): set means -1.
    """
    calls = (k + 127) // 128
    c0 = np.arange(calls, dtype=np.uint64)[None, :]
    rows = np.arange(D, dtype=np.uint64)[:, None]
    words = philox4x32_10(c0, rows, np.uint64((layer & 0xFFFFFF) | (STREAM_PROJECT << 24)),
                          np.uint64(step & 0xFFFFFFFF), np.uint64(seed & 0xFFFFFFFF),
                          np.uint64((seed >> 32) & 0xFFFFFFFF))
    w = np.stack(words, axis=-1)                                   # D x calls x 4
    bits = (w[..., None] >> np.arange(32, dtype=np.uint32)) & np.uint32(1)     # D x calls x 4 x 32
    bits = bits.reshape(D, calls * 128)[:, :k]
    return 1.0 - 2.0 * bits.astype(np.float64)


def project_store(A, dtype: str, fraction, seed: int, layer: int, step: int, R=None) -> "Store":
    """What the forward pass keeps with the projection: S = round_dtype(A R') (B x k), k = ceil(fraction d).
    `R` replaces the Philox signs (test hook for exhaustive enumeration)."""
    A = np.ascontiguousarray(A, dtype=np.float32)
    B, D = A.shape
    k = draws_per_row(fraction, D)
    Rm = rademacher(D, k, seed, layer, step) if R is None else np.asarray(R, np.float64)
    S = (A.astype(np.float64) @ Rm).astype(np.float32)
    if dtype == "bf16":
        S = round_bf16(S)
    elif dtype != "f32":
        raise ValueError(dtype)
    return Store("project", dtype, B, D, k, np.float32(1.0) / np.float32(k), np.zeros((0, 0), np.uint32),
                 S.reshape(-1), R=Rm)


# --------------------------------------------------------------------------
# number formats
# --------------------------------------------------------------------------
def round_bf16(x) -> np.ndarray:
    """float32 -> nearest bf16 (ties to even), returned as float32.  Finite inputs."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    u = (u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))) >> np.uint64(16)
    return (u << np.uint64(16)).astype(np.uint32).view(np.float32).reshape(x.shape)


def bf16_bits(x) -> np.ndarray:
    """bf16 bit patterns (uint16) of float32 values that already lie on the bf16 grid."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> np.uint32(16)).astype(np.uint16).reshape(x.shape)


def pack_bits(m: np.ndarray) -> np.ndarray:
    """Boolean B x D -> uint32 B x ceil(D/32), bit (d % 32) of word d // 32, LSB first."""
    B, D = m.shape
    W = (D + 31) // 32
    padded = np.zeros((B, W * 32), dtype=np.uint64)
    padded[:, :D] = m
    weights = (np.uint64(1) << np.arange(32, dtype=np.uint64))
    return (padded.reshape(B, W, 32) * weights).sum(axis=2).astype(np.uint32)


def unpack_bits(words: np.ndarray, D: int) -> np.ndarray:
    B, W = words.shape
    bits = (words[:, :, None] >> np.arange(32, dtype=np.uint32)) & np.uint32(1)
    return bits.reshape(B, W * 32)[:, :D].astype(bool)


# --------------------------------------------------------------------------
# the compact store (Sec. 3.2, last paragraph: the layer input is what gets
# sparsified, not the Jacobian; App. A memory model)
# --------------------------------------------------------------------------
@dataclass
class Store:
    variant: str
    dtype: str
    B: int
    D: int
    T: int
    scale: np.float32
    keepbits: np.ndarray                 # uint32; different: B x ceil(D/32); same: 1 x ceil(D/32)
    values: np.ndarray                   # float32, canonical order (row-major, ascending column)
    row_ptr: Optional[np.ndarray] = None  # different: int64 B+1
    idx: Optional[np.ndarray] = None      # same: kept columns ascending
    R: Optional[np.ndarray] = None        # project: the D x k sign matrix (regenerated from the key on the device)
    relubits: Optional[np.ndarray] = None  # uint32 B x ceil(D/32): (A > 0)

    @property
    def nnz(self) -> int:
        return int(self.values.size)


def forward_store(A, dtype: str, variant: str, p, seed: int, layer: int, step: int,
                  mask: Optional[np.ndarray] = None, with_relu_bits: bool = True,
                  law: str = "bernoulli", counts: Optional[np.ndarray] = None) -> Store:
    """What the forward pass keeps of a layer input A (B x D).

    A_hat[b, d] = m[b, d] * round_dtype(fl32(A[b, d] * s)); only the kept
    entries are emitted.  `mask` replaces the Philox mask (test hook for
    exhaustive enumeration).  law="replace": the paper's k draws with
    replacement; `T` then holds k and `p` is the fraction.  The ReLU derivative of the layer that produced A
    is (A > 0), one bit per entry (Sec. 4.2; -0.0 and 0.0 give 0).
    """
    A = np.ascontiguousarray(A, dtype=np.float32)
    B, D = A.shape
    if law == "bernoulli":
        T = keep_threshold(p)
        s = scale_factor(p)
        m = keep_mask(variant, B, D, p, seed, layer, step) if mask is None else np.asarray(mask, bool)
        scaled = A * s                                   # float32 x float32, one rounding
    elif law == "replace":
        # `counts` replaces the Philox draws (test hook for exhaustive enumeration).  A coordinate drawn
        # c times weighs c * d / k: fl32(c * s) first, then one float32 product with the entry.
        T = draws_per_row(p, D)
        s = replace_scale(p, D)
        c = multiplicity(variant, B, D, p, seed, layer, step) if counts is None else np.asarray(counts, np.int64)
        m = c > 0
        scaled = A * (c.astype(np.float32) * s)
    elif law == "fixed":
        # exactly k distinct coordinates per row, weight d / k each; `counts` replaces the Philox subset
        T = draws_per_row(p, D)
        s = replace_scale(p, D)
        c = fixed_subset(variant, B, D, p, seed, layer, step) if counts is None else np.asarray(counts, np.int64)
        m = c > 0
        scaled = A * (c.astype(np.float32) * s)
    else:
        raise ValueError(law)
    if dtype == "bf16":
        scaled = round_bf16(scaled)
    elif dtype != "f32":
        raise ValueError(dtype)
    relubits = pack_bits(A > 0) if with_relu_bits else None
    if variant == "different":
        counts = m.sum(axis=1)
        row_ptr = np.concatenate([[0], np.cumsum(counts)]).astype(np.int64)
        return Store(variant, dtype, B, D, T, s, pack_bits(m), scaled[m], row_ptr=row_ptr,
                     relubits=relubits)
    if not (m == m[0:1]).all():
        raise ValueError("same-sample mask must not depend on the row")
    idx = np.flatnonzero(m[0]).astype(np.int64)
    return Store(variant, dtype, B, D, T, s, pack_bits(m[0:1]),
                 np.ascontiguousarray(scaled[:, idx]).reshape(-1), idx=idx, relubits=relubits)


def densify(st: Store) -> np.ndarray:
    """A_hat (B x D, float64) rebuilt from the compact form alone."""
    Ah = np.zeros((st.B, st.D), dtype=np.float64)
    if st.variant == "different":
        m = unpack_bits(st.keepbits, st.D)
        for b in range(st.B):
            Ah[b, m[b]] = st.values[st.row_ptr[b]:st.row_ptr[b + 1]]
    else:
        Ah[:, st.idx] = st.values.reshape(st.B, st.idx.size)
    return Ah


def weight_grad(st: Store, dZ) -> np.ndarray:
    """dW_hat = A_hat^T dZ (D x H, float64), using nothing but the store and dZ.

    For "same" only the kept rows of dW_hat can be non-zero (Sec. 4.3: only
    part of the weight matrix is updated).
    """
    dZ = np.asarray(dZ, dtype=np.float64)
    if st.variant == "project":
        # dW_hat = R (R^T A^T dZ) with R = R' / sqrt(k): G = (S^T dZ) / k is a tensor of the working type
        # on the device (float32 product with fl32(1 / k), then one rounding), then R' G
        k = st.T
        G = (st.values.reshape(st.B, k).astype(np.float64).T @ dZ).astype(np.float32) * st.scale
        G = round_bf16(G) if st.dtype == "bf16" else G
        return st.R @ G.astype(np.float64)
    if st.variant == "same":
        dW = np.zeros((st.D, dZ.shape[1]), dtype=np.float64)
        Ac = st.values.reshape(st.B, st.idx.size).astype(np.float64)
        dW[st.idx, :] = Ac.T @ dZ
        return dW
    return densify(st).T @ dZ


# --------------------------------------------------------------------------
# exact pieces of the step (never sampled: Sec. 4.2)
# --------------------------------------------------------------------------
def act_forward(Z, act: str):
    if act == "relu":
        return np.maximum(Z, 0.0)
    if act == "gelu":
        return 0.5 * Z * (1.0 + erf(Z / np.sqrt(2.0)))
    if act == "none":
        return Z
    raise ValueError(act)


def gelu_grad(Z):
    return 0.5 * (1.0 + erf(Z / np.sqrt(2.0))) + Z * np.exp(-0.5 * Z * Z) / np.sqrt(2.0 * np.pi)


def softmax_xent(Z, labels):
    """Mean cross-entropy of softmax(Z) and its Jacobian dZ = (softmax - onehot) / B."""
    Z = np.asarray(Z, dtype=np.float64)
    B = Z.shape[0]
    zmax = Z.max(axis=1, keepdims=True)
    e = np.exp(Z - zmax)
    ssum = e.sum(axis=1, keepdims=True)
    logp = Z - zmax - np.log(ssum)
    loss = -logp[np.arange(B), labels].mean()
    dZ = e / ssum
    dZ[np.arange(B), labels] -= 1.0
    return loss, dZ / B


def input_grad(dZ, W, relubits_prev=None, Z_prev=None, act="relu", dtype="f32"):
    """Exact dA = dZ W^T, masked by the derivative of the activation that produced A; db = sum_b dZ."""
    dZ = np.asarray(dZ, dtype=np.float64)
    dA = dZ @ np.asarray(W, dtype=np.float64).T
    if act == "relu" and relubits_prev is not None:
        dA = dA * unpack_bits(relubits_prev, dA.shape[1])
    elif act == "gelu" and Z_prev is not None:
        dA = dA * gelu_grad(np.asarray(Z_prev, dtype=np.float64))
    if dtype == "bf16":
        dA = round_bf16(dA.astype(np.float32)).astype(np.float64)
    elif dtype == "f32":
        dA = dA.astype(np.float32).astype(np.float64)
    return dA, dZ.sum(axis=0)


@dataclass
class StepResult:
    loss: float
    Z: List[np.ndarray]
    A: List[np.ndarray]                 # A[0] = X, A[l] = act(Z[l-1])
    dZ: List[np.ndarray]
    dW: List[np.ndarray]
    db: List[np.ndarray]
    stores: List[Optional[Store]] = field(default_factory=list)


def mlp_step(X, labels, Ws, bs, act="relu", dtype="f32", variant=None, p=1.0, seed=0, step=0,
             masks=None, law="bernoulli") -> StepResult:
    """One forward + backward pass of a fully connected net with softmax cross-entropy.

    variant None: exact backprop (dW_l = A_{l-1}^T dZ_l).  Otherwise the input
    of every linear layer, the network input included, goes through
    forward_store and dW_l comes from the store; the softmax input is not
    sampled (App. A).  The tensors that live on the device in the working type
    (activations, stored pre-activations, dZ: float32 or bf16) are rounded to
    it at those points and nowhere else; accumulations stay in float64.
    """
    L = len(Ws)
    W64 = [np.asarray(W, dtype=np.float64) for W in Ws]
    b64 = [np.asarray(b, dtype=np.float64) for b in bs]
    if dtype == "bf16":
        rnd = lambda v: round_bf16(np.asarray(v, np.float32)).astype(np.float64)
    elif dtype == "f32":
        rnd = lambda v: np.asarray(v, np.float32).astype(np.float64)
    elif dtype == "f64" and variant is None:         # no rounding at all: for pins of the exact net
        rnd = lambda v: np.asarray(v, np.float64)
    else:
        raise ValueError(dtype)
    A = [np.asarray(X, dtype=np.float64)]
    Z, stores = [], []
    for l in range(L):
        if variant == "project":
            stores.append(project_store(A[l].astype(np.float32), dtype, p, seed, l, step))
        elif variant is not None:
            stores.append(forward_store(A[l].astype(np.float32), dtype, variant, p, seed, l, step,
                                        mask=None if masks is None else masks[l], law=law))
        else:
            stores.append(None)
        z = A[l] @ W64[l] + b64[l]
        if l < L - 1:
            Z.append(rnd(z) if act == "gelu" else z)   # a GELU net keeps Z (bf16) for the backward
            A.append(rnd(act_forward(z, act)))
        else:
            Z.append(z)
    loss, dz = softmax_xent(Z[-1], labels)
    dZ = [None] * L
    dW = [None] * L
    db = [None] * L
    dZ[L - 1] = rnd(dz)
    for l in range(L - 1, -1, -1):
        dW[l] = A[l].T @ dZ[l] if variant is None else weight_grad(stores[l], dZ[l])
        if l > 0:
            if act == "relu":
                dA, db[l] = input_grad(dZ[l], W64[l], relubits_prev=pack_bits(A[l] > 0), dtype=dtype)
            else:
                dA, db[l] = input_grad(dZ[l], W64[l], Z_prev=Z[l - 1], act=act, dtype=dtype)
            dZ[l - 1] = dA
        else:
            db[l] = dZ[l].sum(axis=0)
    return StepResult(loss, Z, A, dZ, dW, db, stores)


# --------------------------------------------------------------------------
# bytes held between forward and backward (App. A, "Calculation of memory saved")
# --------------------------------------------------------------------------
def stored_bytes(stores: List[Store], logits_shape, elem_bytes: int):
    """Bytes the compact stores really hold, split by kind, and the full-backprop figure."""
    value_bytes = sum(st.nnz * elem_bytes for st in stores)
    index_bytes = 0
    relu_bytes = 0
    full = 0
    for i, st in enumerate(stores):
        words = (st.D + 31) // 32
        index_bytes += 4 * words * (st.B if st.variant == "different" else 1)
        if i > 0:                                   # the network input is not a ReLU output
            relu_bytes += 4 * words * st.B
        full += st.B * st.D * elem_bytes
    unsampled = int(np.prod(logits_shape)) * 4
    return dict(value_bytes=value_bytes, index_bytes=index_bytes, relu_bytes=relu_bytes,
                unsampled_bytes=unsampled, full_backprop_bytes=full + unsampled)
