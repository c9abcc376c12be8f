"""Philox-4x32-10 counter-based generator (oracle side, numpy).

Definition followed: Salmon, Moraes, Dror, Shaw, "Parallel random numbers: as
easy as 1, 2, 3" (SC'11), Sec. 3.3 / Table 2 constants: a 4-word counter and a
2-word key; each round multiplies counter words 0 and 2 by fixed odd
constants, keeps both halves of the 64-bit products, and mixes the high halves
with the other two counter words and the key; the key is bumped by Weyl
constants between rounds; ten rounds.  The paper under test (Sec. 3.2) only
asks for *some* source of randomness; fixing a counter-based one is what makes
masks reproducible on both sides of the comparison.

Test infrastructure only; shares nothing with the CUDA implementation.
"""
import numpy as np

M0 = np.uint64(0xD2511F53)      # multiplier applied to counter word 0
M1 = np.uint64(0xCD9E8D57)      # multiplier applied to counter word 2
W0 = np.uint64(0x9E3779B9)      # Weyl increment of key word 0 (golden ratio)
W1 = np.uint64(0xBB67AE85)      # Weyl increment of key word 1 (sqrt 3 - 1)
MASK32 = np.uint64(0xFFFFFFFF)
SHIFT32 = np.uint64(32)


def _u64(x):
    return np.asarray(x, dtype=np.uint64) & MASK32


def philox4x32_round(c0, c1, c2, c3, k0, k1):
    """One round: (c0,c1,c2,c3) -> (hi(M1*c2)^c1^k0, lo(M1*c2), hi(M0*c0)^c3^k1, lo(M0*c0))."""
    p0 = M0 * c0
    p1 = M1 * c2
    return ((p1 >> SHIFT32) ^ c1 ^ k0, p1 & MASK32, (p0 >> SHIFT32) ^ c3 ^ k1, p0 & MASK32)


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Ten rounds over broadcastable arrays of 32-bit words; returns four uint32 arrays."""
    c0, c1, c2, c3, k0, k1 = np.broadcast_arrays(*(_u64(v) for v in (c0, c1, c2, c3, k0, k1)))
    for r in range(10):
        if r > 0:
            k0 = (k0 + W0) & MASK32
            k1 = (k1 + W1) & MASK32
        c0, c1, c2, c3 = philox4x32_round(c0, c1, c2, c3, k0, k1)
    return tuple(v.astype(np.uint32) for v in (c0, c1, c2, c3))
