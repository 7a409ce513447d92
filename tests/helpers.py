"""Test-side helpers, independent of both the oracle and the CUDA path."""
import numpy as np


def container_bits(bits):
    return {1: 1, 2: 2, 3: 4, 4: 4}.get(bits, 8)


def unpack_levels(codes, cols, bits):
    """Packed level indices -> int array [rows, cols] (element 0 in the low bits of a byte)."""
    cb = container_bits(bits)
    codes = np.asarray(codes, dtype=np.uint8)
    per = 8 // cb
    shifts = (np.arange(per) * cb).astype(np.uint8)
    vals = (codes[:, :, None] >> shifts[None, None, :]) & ((1 << cb) - 1)
    return vals.reshape(codes.shape[0], -1)[:, :cols].astype(np.int64)


def unpack_mask(mask, cols):
    return np.unpackbits(np.asarray(mask, np.uint8), axis=1, bitorder="little")[:, :cols].astype(bool)


def grid_values(levels, bits):
    return 2 * levels - (2 ** bits - 1)
