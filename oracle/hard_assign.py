"""Oracle of the hard quantiser q(w) = argmin_c ||w - c|| (Section 3.1: the map the soft quantiser r_tau tends to as
tau -> 0) and of the packed code format the library writes.  Test infrastructure: plain numpy in float64, written out
from the definition; nothing here is shared with the CUDA path.

Codes: weight i gets the index of its nearest centroid (lowest index on ties), stored in b bits, b the smallest of
1, 2, 4, 8 with 2^b >= k, at bit offset (i * b) mod 8 of byte (i * b) // 8 (little-endian within the byte).
"""
from __future__ import annotations

import numpy as np


def code_bits(k: int) -> int:
    for b in (1, 2, 4, 8):
        if (1 << b) >= k:
            return b
    raise ValueError("k must be at most 256")


def squared_distances(W, C) -> np.ndarray:
    """[m, k] float64 squared Euclidean distances."""
    W = np.asarray(W, dtype=np.float64)
    C = np.asarray(C, dtype=np.float64)
    diff = W[:, None, :] - C[None, :, :]
    return (diff * diff).sum(axis=2)


def hard_assign(W, C, chunk: int = 1 << 15) -> np.ndarray:
    """Index of the nearest centroid of every row of W (int64 [m]); ties go to the lowest index."""
    W = np.asarray(W, dtype=np.float64)
    out = np.empty(W.shape[0], dtype=np.int64)
    for a in range(0, W.shape[0], chunk):
        out[a:a + chunk] = np.argmin(squared_distances(W[a:a + chunk], C), axis=1)
    return out


def margins(W, C, chunk: int = 1 << 15) -> np.ndarray:
    """Gap between the smallest and the second smallest squared distance of every row (float64 [m]; inf for k = 1)."""
    W = np.asarray(W, dtype=np.float64)
    out = np.empty(W.shape[0], dtype=np.float64)
    for a in range(0, W.shape[0], chunk):
        d2 = squared_distances(W[a:a + chunk], C)
        if d2.shape[1] == 1:
            out[a:a + chunk] = np.inf
        else:
            part = np.partition(d2, 1, axis=1)
            out[a:a + chunk] = part[:, 1] - part[:, 0]
    return out


def dequantize(idx, C) -> np.ndarray:
    return np.asarray(C, dtype=np.float64)[np.asarray(idx)]


def pack_codes(idx, k: int) -> np.ndarray:
    b = code_bits(k)
    idx = np.asarray(idx, dtype=np.int64)
    m = idx.shape[0]
    out = np.zeros((m * b + 7) // 8, dtype=np.uint8)
    for i in range(m):            # plain loop: this is the definition of the format
        bit = i * b
        out[bit // 8] |= np.uint8((int(idx[i]) << (bit % 8)) & 0xFF)
    return out


def unpack_codes(codes, m: int, k: int) -> np.ndarray:
    b = code_bits(k)
    codes = np.asarray(codes, dtype=np.uint8)
    i = np.arange(m, dtype=np.int64)
    bit = i * b
    return ((codes[bit // 8].astype(np.int64) >> (bit % 8)) & ((1 << b) - 1)).astype(np.int64)
