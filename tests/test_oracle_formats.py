"""Pins of the oracle's format variants (group sizes 64 / 128, MXFP4) against what the formats' definitions fix:
bit-field definitions, exact rational arithmetic, the already-pinned group-32 routines, hand-located bytes, numpy."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
import synthgen

G64, G128, MX = oracle.FMT_G64, oracle.FMT_G128, oracle.FMT_MXFP4


def bf16_fraction(bits: int) -> Fraction:
    s, e, m = bits >> 15, (bits >> 7) & 0xFF, bits & 0x7F
    v = Fraction(m, 128) * Fraction(2) ** -126 if e == 0 else (1 + Fraction(m, 128)) * Fraction(2) ** (e - 127)
    return -v if s else v


def e2m1_from_bit_fields(q: int) -> Fraction:
    """OCP Microscaling FP4: 1 sign, 2 exponent (bias 1), 1 mantissa bit; exponent 0 is subnormal."""
    s, E, M = q >> 3, (q >> 1) & 3, q & 1
    v = Fraction(M, 2) if E == 0 else Fraction(2) ** (E - 1) * (1 + Fraction(M, 2))
    return -v if s else v


def test_byte_budgets():
    # 32 x 256 codes at 4 bits + per-group metadata: 2 x 2 bytes per (row, group) for Eq. 3, 1 byte for MXFP4
    assert oracle.fmt_packed_bytes(G64, 256, 32) == 4096 + 32 * 4 * 4 == 4608        # 4.5 bits per weight
    assert oracle.fmt_packed_bytes(G128, 256, 32) == 4096 + 32 * 2 * 4 == 4352       # 4.25
    assert oracle.fmt_packed_bytes(MX, 256, 32) == 4096 + 32 * 8 * 1 == 4352         # 4 + 8/32 bits
    assert oracle.fmt_packed_bytes(MX, 2560, 262144) * 8 == 2560 * 262144 * 17 // 4
    for fmt in (G64, G128, MX):
        assert oracle.fmt_packed_bytes(fmt, 288, 32) == 0      # whole blocks only
        assert oracle.fmt_packed_bytes(fmt, 256, 48) == 0
        assert oracle.fmt_packed_bytes(fmt, 512, 64) == 4 * oracle.fmt_packed_bytes(fmt, 256, 32)


def test_mxfp4_elements_and_scales_against_their_bit_field_definitions():
    # every code x every legal scale byte: the oracle's value is the exact rational, whenever that is an fp32 number
    codes = np.tile(np.arange(16, dtype=np.uint8), 16)[None, :].repeat(32, axis=0)      # [32, 256]
    for e in list(range(0, 255, 7)) + [1, 126, 127, 128, 254]:
        scales = np.full((32, 8), e, np.uint16)
        w32, w16 = oracle.fmt_dequant(MX, codes, scales)
        for q in range(16):
            exact = e2m1_from_bit_fields(q) * Fraction(2) ** (e - 127)
            if abs(exact) >= Fraction(2) ** 128:     # beyond fp32: the single rounding gives infinity
                assert np.isinf(w32[q, 0]) and (w32[q, 0] < 0) == (exact < 0)
                continue
            got = Fraction(float(w32[q, 0]))
            assert got == exact, (q, e)
            assert np.all(w32[q::16, :] == w32[q, 0])
    # the eight magnitudes named by the specification
    w32, _ = oracle.fmt_dequant(MX, codes, np.full((32, 8), 127, np.uint16))
    assert [float(v) for v in w32[:16, 0]] == [0, .5, 1, 1.5, 2, 3, 4, 6, -0.0, -.5, -1, -1.5, -2, -3, -4, -6]
    assert np.signbit(w32[8, 0])
    with pytest.raises(ValueError):
        oracle.fmt_dequant(MX, codes, np.full((32, 8), 255, np.uint16))   # E8M0 255 is NaN


@pytest.mark.parametrize("fmt,g", [(G64, 64), (G128, 128)])
def test_larger_groups_equal_group_32_with_repeated_scales(fmt, g):
    K, N, M = 512, 64, 3
    w = synthgen.weights_fmt(31 + g, K, N, fmt)
    x = synthgen.activations(77, M, K)
    rep = g // 32
    s32, o32 = np.repeat(w.scales, rep, axis=1), np.repeat(w.offsets, rep, axis=1)
    a32, a16 = oracle.fmt_dequant(fmt, w.codes, w.scales, w.offsets)
    b32, b16 = oracle.dequant(w.codes, s32, o32)
    assert np.array_equal(a32.view(np.uint32), b32.view(np.uint32)) and np.array_equal(a16, b16)
    ya, aa = oracle.fmt_project(fmt, x, w.codes, w.scales, w.offsets)
    yb, ab = oracle.project(x, w.codes, s32, o32)
    assert np.array_equal(ya, yb) and np.array_equal(aa, ab)
    # Eq. 3 per element, exactly, on a sample that includes both ends of a group
    for n, k in [(0, 0), (5, g - 1), (5, g), (63, K - 1), (17, 3 * g + 1)]:
        exact = bf16_fraction(int(w.scales[n, k // g])) * int(w.codes[n, k]) + bf16_fraction(int(w.offsets[n, k // g]))
        assert abs(Fraction(float(a32[k, n])) - exact) <= abs(exact) * Fraction(1, 2 ** 24)


def write_blocks(fmt, codes, scales, offsets):
    """A second, sequential statement of the variant layouts: walk strips, blocks, then sections in storage order."""
    N, K = codes.shape
    g = oracle.FMT_GROUP[fmt]
    out = bytearray()
    for s in range(N // 32):
        for b in range(K // 256):
            for t in range(8):                      # codes: group-of-32 column t, row r, 16 bytes of 32 nibbles
                for r in range(32):
                    c = codes[s * 32 + r, b * 256 + t * 32: b * 256 + t * 32 + 32]
                    out += bytes(int(c[2 * j]) | (int(c[2 * j + 1]) << 4) for j in range(16))
            for arr in ((scales,) if fmt == MX else (scales, offsets)):
                for t in range(256 // g):
                    for r in range(32):
                        v = int(arr[s * 32 + r, b * (256 // g) + t])
                        out += bytes([v]) if fmt == MX else bytes([v & 0xFF, v >> 8])
    return np.frombuffer(bytes(out), np.uint8)


@pytest.mark.parametrize("fmt", [G64, G128, MX])
def test_layout_against_sequential_writer_and_hand_located_bytes(fmt):
    K, N = 512, 64
    w = synthgen.weights_fmt(5 + fmt, K, N, fmt)
    packed = write_blocks(fmt, w.codes, w.scales, w.offsets)
    assert packed.size == oracle.fmt_packed_bytes(fmt, K, N)
    codes, scales, offsets = oracle.fmt_unpack(fmt, packed, K, N)
    assert np.array_equal(codes, w.codes) and np.array_equal(scales, w.scales)
    assert fmt == MX or np.array_equal(offsets, w.offsets)
    # element (n = 37, k = 270): strip 1, row 5, block 1, column 14 of the block -> low nibble of byte 7 of row 5, tile 0
    bb = {G64: 4608, G128: 4352, MX: 4352}[fmt]
    blk = (1 * (K // 256) + 1) * bb
    assert (packed[blk + 0 * 512 + 5 * 16 + 7] & 0x0F) == w.codes[37, 270]
    assert (packed[blk + 0 * 512 + 5 * 16 + 7] >> 4) == w.codes[37, 271]
    if fmt == MX:
        assert packed[blk + 4096 + 0 * 32 + 5] == w.scales[37, 270 // 32]
        # k = 300 of block 1 -> column 44 -> group 1 of the block
        assert packed[blk + 4096 + 1 * 32 + 5] == w.scales[37, (256 + 44) // 32]
    else:
        g = oracle.FMT_GROUP[fmt]
        sec = 64 * (256 // g)
        at = blk + 4096 + 2 * (0 * 32 + 5)
        assert int(packed[at]) | (int(packed[at + 1]) << 8) == w.scales[37, 270 // g]
        assert int(packed[at + sec]) | (int(packed[at + sec + 1]) << 8) == w.offsets[37, 270 // g]


@pytest.mark.parametrize("fmt", [G64, G128, MX])
def test_projection_against_numpy_and_invariants(fmt):
    K, N, M = 768, 96, 4
    w = synthgen.weights_fmt(11 * fmt, K, N, fmt)
    x = synthgen.activations(3, M, K)
    w32, _ = oracle.fmt_dequant(fmt, w.codes, w.scales, w.offsets)
    xf = synthgen.bf16_to_f32(x).astype(np.float64)
    y, a = oracle.fmt_project(fmt, x, w.codes, w.scales, w.offsets, nthreads=2)
    ref = xf @ w32.astype(np.float64)
    assert np.allclose(y, ref, rtol=0, atol=1e-12 * np.abs(xf).max() * K)
    assert np.allclose(a, np.abs(xf) @ np.abs(w32.astype(np.float64)), rtol=1e-12)
    # column ranges, one-hot read-out of a single weight, batched rows = single rows
    y2, _ = oracle.fmt_project(fmt, x, w.codes, w.scales, w.offsets, n0=32, n1=64)
    assert np.array_equal(y2, y[:, 32:64])
    onehot = np.zeros((1, K), np.float32)
    onehot[0, 300] = 1.0
    yo, _ = oracle.fmt_project(fmt, synthgen.bf16_bits(onehot), w.codes, w.scales, w.offsets)
    assert np.array_equal(yo[0], w32[300].astype(np.float64))
    y1, _ = oracle.fmt_project(fmt, x[2:3], w.codes, w.scales, w.offsets)
    assert np.array_equal(y1[0], y[2])
    if fmt == MX:
        # one more binade on every scale doubles the result exactly; negating every element negates it
        yd, _ = oracle.fmt_project(fmt, x, w.codes, w.scales + 1)
        assert np.array_equal(yd, 2.0 * y)
        yn, _ = oracle.fmt_project(fmt, x, w.codes ^ 8, w.scales)
        assert np.array_equal(yn, -y)
