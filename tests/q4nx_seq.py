"""A second, independent statement of the Q4NX byte layout, used only by tests.

Where the oracle and the library locate an element by an address formula, this
module walks the container in storage order and emits (or consumes) it byte by
byte: strip after strip, block after block, inside a block the code section
tile by tile and row by row, then the scale words, then the offset words.  A
mistake in either formulation shows up as a disagreement between the two.
"""
import numpy as np


def write_sequential(codes, scales, offsets):
    """codes[N,K] u8, scales/offsets[N,K/32] u16 -> packed bytes (python loops; small inputs only)."""
    N, K = codes.shape
    out = bytearray()
    for s in range(N // 32):
        rows = range(32 * s, 32 * s + 32)
        for k0 in range(0, K, 256):
            groups = range(k0 // 32, min(K, k0 + 256) // 32)
            for g in groups:                       # code section: one 32x32 tile per group
                for n in rows:
                    for p in range(16):
                        lo = int(codes[n, 32 * g + 2 * p])
                        hi = int(codes[n, 32 * g + 2 * p + 1])
                        out.append(lo | (hi << 4))
            for arr in (scales, offsets):          # then all scales, then all offsets
                for g in groups:
                    for n in rows:
                        v = int(arr[n, g])
                        out.append(v & 0xFF)
                        out.append(v >> 8)
    return np.frombuffer(bytes(out), np.uint8).copy()


def read_sequential(packed, K, N):
    """Inverse of write_sequential, also by walking the stream."""
    codes = np.zeros((N, K), np.uint8)
    scales = np.zeros((N, K // 32), np.uint16)
    offsets = np.zeros((N, K // 32), np.uint16)
    it = iter(bytes(packed))
    for s in range(N // 32):
        rows = range(32 * s, 32 * s + 32)
        for k0 in range(0, K, 256):
            groups = range(k0 // 32, min(K, k0 + 256) // 32)
            for g in groups:
                for n in rows:
                    for p in range(16):
                        b = next(it)
                        codes[n, 32 * g + 2 * p] = b & 15
                        codes[n, 32 * g + 2 * p + 1] = b >> 4
            for arr in (scales, offsets):
                for g in groups:
                    for n in rows:
                        lo = next(it)
                        arr[n, g] = lo | (next(it) << 8)
    assert next(it, None) is None
    return codes, scales, offsets
