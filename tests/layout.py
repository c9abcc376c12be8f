"""Host-side index shuffling between the oracle's canonical store and the device layout.

Pure reordering (no arithmetic of the method): the device keeps the kept values tile by tile
(64 rows x 128 columns), each tile padded with zeros to a multiple of 8 elements; the oracle
emits them row-major over the whole matrix.
"""
import numpy as np

from oracle import rad

TILE_ROWS, TILE_COLS, ALIGN = 64, 128, 8


def tile_major(st):
    """(keepbits words, padded values as float32, offsets) of an oracle different-sample store."""
    B, D = st.B, st.D
    mask = rad.unpack_bits(st.keepbits, D)
    dense = np.zeros((B, D), dtype=np.float32)
    dense[mask] = st.values
    nslab, ncb = -(-B // TILE_ROWS), -(-D // TILE_COLS)
    bits, vals, offs = [], [], [0]
    for s in range(nslab):
        for c in range(ncb):
            m = np.zeros((TILE_ROWS, TILE_COLS), dtype=bool)
            sub = mask[s * TILE_ROWS:(s + 1) * TILE_ROWS, c * TILE_COLS:(c + 1) * TILE_COLS]
            m[:sub.shape[0], :sub.shape[1]] = sub
            bits.append(rad.pack_bits(m).reshape(-1))
            rowoff = np.concatenate([[0], np.cumsum(m.sum(axis=1))[:-1]]).astype(np.uint16)
            bits.append(rowoff.view(np.uint32))
            v = dense[s * TILE_ROWS:(s + 1) * TILE_ROWS, c * TILE_COLS:(c + 1) * TILE_COLS][sub]
            pad = (-v.size) % ALIGN
            vals.append(np.concatenate([v, np.zeros(pad, np.float32)]))
            offs.append(offs[-1] + v.size + pad)
    return np.concatenate(bits), np.concatenate(vals), np.array(offs, dtype=np.uint32)


def bits_of(x_f32, dtype):
    """Bit patterns for exact comparison: float32 words, or bf16 halves of values on the bf16 grid."""
    x = np.ascontiguousarray(x_f32, dtype=np.float32)
    return x.view(np.uint32) if dtype == "f32" else rad.bf16_bits(x)
