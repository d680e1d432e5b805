"""Pins for the CPU oracle: what the paper and the mathematics fix, checked without a GPU.

Each test is chosen so that a plausible mistake in the oracle (a dropped term, a
wrong sign or index, a transposed operand, a wrong rounding) fails at least one.
Nothing here touches the CUDA library.
"""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
import synthgen
from q4nx_seq import read_sequential, write_sequential

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


# --------------------------------------------------------------------------- helpers

def bf16_fraction(bits: int) -> Fraction:
    """Exact value of a bf16 bit pattern (finite), by integer arithmetic only."""
    sign = -1 if bits & 0x8000 else 1
    e = (bits >> 7) & 0xFF
    man = bits & 0x7F
    if e == 0:
        return sign * Fraction(man, 1 << 7) * Fraction(1, 1 << 126)
    return sign * (1 + Fraction(man, 1 << 7)) * (Fraction(2) ** (e - 127))


def round_to_binary(v: Fraction, p: int, emin: int) -> Fraction:
    """Round v to nearest-even in a binary format with p significand bits and minimum
    normal exponent emin (subnormals kept), exactly."""
    if v == 0:
        return Fraction(0)
    s = -1 if v < 0 else 1
    a = abs(v)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    e = max(e, emin)
    ulp = Fraction(2) ** (e - (p - 1))
    q, r = divmod(a, ulp)
    if r * 2 > ulp or (r * 2 == ulp and q % 2 == 1):
        q += 1
    return s * q * ulp


def f32_bits_of(v: Fraction) -> int:
    return int(np.float32(float(v)).view(np.uint32))  # v is already fp32-exact: float() is exact


def structured(K, N, code_fn, d_fn, m_fn):
    n = np.arange(N)[:, None]
    k = np.arange(K)[None, :]
    g = np.arange(K // 32)[None, :]
    codes = (code_fn(n, k) % 16).astype(np.uint8)
    scales = synthgen.bf16_bits(d_fn(n, g).astype(np.float32) + np.zeros((N, K // 32), np.float32))
    offsets = synthgen.bf16_bits(m_fn(n, g).astype(np.float32) + np.zeros((N, K // 32), np.float32))
    return codes, scales, offsets


# --------------------------------------------------------------------------- container size

def test_block_byte_budget_from_paper():
    # Sec. "Dequantization Engine": a 32 x 256 block is 4096 + 512 + 512 = 5120 bytes (5 bits / weight).
    assert oracle.packed_bytes(256, 32) == 5120
    assert oracle.packed_bytes(1152, 6912) == 1152 * 6912 * 5 // 8 == 4976640
    assert oracle.packed_bytes(288, 32) == 5120 + 640
    for K, N in [(0, 32), (32, 0), (48, 32), (32, 48), (-32, 32)]:
        assert oracle.packed_bytes(K, N) == 0


# --------------------------------------------------------------------------- layout

def test_layout_hand_located_element():
    # K = 288 (one full block + a one-group tail), N = 32.  Element (n=5, k=270) sits in the tail
    # block: block offset 5120, tile 0, row 5, i = 14 -> code byte 5120 + 5*16 + 7 = 5207 (low nibble);
    # the tail has one group, so scales start at 5120 + 512 and offsets at 5120 + 576.
    K, N = 288, 32
    buf = np.zeros(oracle.packed_bytes(K, N), np.uint8)
    buf[5207] = 0x0B
    buf[5642], buf[5643] = 0x00, 0x3F      # scale (row 5, group 8) = 0.5
    buf[5706], buf[5707] = 0x80, 0xBF      # offset = -1
    codes, scales, offsets = oracle.unpack(buf, K, N)
    assert codes[5, 270] == 11 and codes.sum() == 11
    assert scales[5, 8] == 0x3F00 and np.count_nonzero(scales) == 1
    assert offsets[5, 8] == 0xBF80 and np.count_nonzero(offsets) == 1
    # high nibble of the same byte is the next k
    buf[5207] = 0xB0
    codes, _, _ = oracle.unpack(buf, K, N)
    assert codes[5, 271] == 11 and codes.sum() == 11
    # first block of the second strip would start at 20*K
    K, N = 288, 64
    buf = np.zeros(oracle.packed_bytes(K, N), np.uint8)
    buf[20 * K + 7 * 512 + 31 * 16 + 15] = 0xF0   # strip 1, block 0, tile 7, row 31, i = 31
    codes, _, _ = oracle.unpack(buf, K, N)
    assert codes[63, 255] == 15 and codes.sum() == 15


def test_layout_golden_dump():
    # tests/golden/q4nx_k32_n32.hex: the 640-byte container of the K = N = 32 matrix with
    # code[n][k] = (k + 3n) mod 16, every scale 0.5 (0x3F00), every offset -1 (0xBF80),
    # written out by hand rule: line r of the code section is row r, 16 bytes, low nibble first.
    with open(os.path.join(GOLDEN, "q4nx_k32_n32.hex")) as f:
        data = bytes.fromhex("".join(line.split("#")[0] for line in f))
    assert len(data) == 640
    codes, scales, offsets = oracle.unpack(np.frombuffer(data, np.uint8), 32, 32)
    n, k = np.arange(32)[:, None], np.arange(32)[None, :]
    assert np.array_equal(codes, (k + 3 * n) % 16)
    assert np.all(scales == 0x3F00) and np.all(offsets == 0xBF80)


@pytest.mark.parametrize("K,N", [(32, 32), (64, 64), (256, 32), (288, 32), (544, 96), (1152, 64)])
def test_layout_against_sequential_writer(K, N):
    w = synthgen.weights(100 + K + N, K, N)
    packed = write_sequential(w.codes, w.scales, w.offsets)
    assert packed.size == oracle.packed_bytes(K, N)
    codes, scales, offsets = oracle.unpack(packed, K, N)
    assert np.array_equal(codes, w.codes)
    assert np.array_equal(scales, w.scales)
    assert np.array_equal(offsets, w.offsets)
    c2, s2, o2 = read_sequential(packed, K, N)
    assert np.array_equal(c2, w.codes) and np.array_equal(s2, w.scales) and np.array_equal(o2, w.offsets)


# --------------------------------------------------------------------------- eq. 3

def _special_bf16():
    vals = [0x0000, 0x8000, 0x0001, 0x8001, 0x007F, 0x0080, 0x0081, 0x3F80, 0xBF80, 0x3F00, 0x3E80,
            0x7F7F, 0xFF7F, 0x7F00, 0x0100, 0x4B00, 0x3C23, 0xBC23, 0x3CA4, 0x5000, 0x2000]
    return vals


def test_dequant_exact_rational_all_codes():
    # Eq. 3 over all 16 codes for a sweep of (d, m) bf16 pairs, against exact rational arithmetic
    # rounded once to fp32 (and then to bf16) with integer arithmetic -- no floating point involved.
    rng = np.random.default_rng(7)
    special = _special_bf16()
    pairs = [(d, m) for d in special for m in special]
    rnd = rng.integers(0, 0x7F80, size=(3000, 2))                # finite magnitudes
    sgn = rng.integers(0, 2, size=(3000, 2)) << 15
    pairs += [tuple(int(v) for v in row) for row in (rnd | sgn)]
    near = rng.integers(0x3800, 0x4000, size=(3000, 2)) | (rng.integers(0, 2, size=(3000, 2)) << 15)
    pairs += [tuple(int(v) for v in row) for row in near]       # comparable magnitudes: real cancellation
    # lay the pairs out as a K = 32 * ceil(P/1) ... simpler: one group per (pair), N = 32 rows reuse
    P = len(pairs)
    G = (P + 31) // 32
    N, K = 32, 32 * G
    codes = np.tile(np.arange(32, dtype=np.uint8) % 16, (N, G))   # every code appears in each group
    scales = np.zeros((N, G), np.uint16)
    offsets = np.zeros((N, G), np.uint16)
    flat = pairs + [(0, 0)] * (N * G - P)
    for idx, (d, m) in enumerate(flat):
        scales[idx % N, idx // N] = d
        offsets[idx % N, idx // N] = m
    w32, w16 = oracle.dequant(codes, scales, offsets)
    w32b = w32.view(np.uint32)
    max_f32 = (2 - Fraction(1, 1 << 23)) * Fraction(2) ** 127
    checked = 0
    for idx, (d, m) in enumerate(pairs):
        n, g = idx % N, idx // N
        dv, mv = bf16_fraction(d), bf16_fraction(m)
        for q in range(16):
            exact = dv * q + mv
            r32 = round_to_binary(exact, 24, -126)
            if abs(r32) > max_f32:
                continue  # overflow to inf: outside the tested domain
            k = 32 * g + q
            got = int(w32b[k, n])
            want = f32_bits_of(r32)
            if r32 == 0:
                assert got & 0x7FFFFFFF == 0
            else:
                assert got == want, (hex(d), hex(m), q, hex(got), hex(want))
            r16 = round_to_binary(r32, 8, -126)
            if abs(r16) <= (2 - Fraction(1, 1 << 7)) * Fraction(2) ** 127 and r16 != 0:
                assert int(w16[k, n]) == f32_bits_of(r16) >> 16
            checked += 1
    assert checked > 90000


def test_dequant_special_cases():
    K, N = 32, 32
    codes = np.tile(np.arange(32, dtype=np.uint8) % 16, (N, 1))
    one, half, neg1 = 0x3F80, 0x3F00, 0xBF80
    # d = 0 -> offset only; m = 0 -> scale only; layout of the result is [K][N]
    w32, _ = oracle.dequant(codes, np.zeros((N, 1), np.uint16), np.full((N, 1), neg1, np.uint16))
    assert w32.shape == (K, N) and np.all(w32 == -1.0)
    w32, w16 = oracle.dequant(codes, np.full((N, 1), half, np.uint16), np.zeros((N, 1), np.uint16))
    assert np.array_equal(w32[:, 3], 0.5 * (np.arange(32) % 16))
    assert np.array_equal(synthgen.bf16_to_f32(w16), w32)
    # double rounding matters: 1 + 2^-8 + 2^-24-ish cases are covered by the rational sweep; here the
    # plain tie: w32 = 1 + 2^-8 exactly (d = 2^-8, q = 1, m = 1) -> bf16 tie rounds to even = 1.0
    w32, w16 = oracle.dequant(np.ones((N, K), np.uint8), np.full((N, 1), 0x3B80, np.uint16),
                              np.full((N, 1), one, np.uint16))
    assert np.all(w32 == np.float32(1 + 2.0 ** -8)) and np.all(w16 == 0x3F80)
    # 1 + 3*2^-8 is also a tie: rounds up to even mantissa 0x3F82
    w32, w16 = oracle.dequant(np.full((N, K), 3, np.uint8), np.full((N, 1), 0x3B80, np.uint16),
                              np.full((N, 1), one, np.uint16))
    assert np.all(w16 == 0x3F82)
    with pytest.raises(ValueError):
        oracle.dequant(np.full((N, K), 16, np.uint8), np.zeros((N, 1), np.uint16), np.zeros((N, 1), np.uint16))


# --------------------------------------------------------------------------- eq. 14 / 15: worked examples

def test_worked_example_E1_E2():
    # K = N = 32, code = (k + 3n) mod 16, d = 0.5, m = -1.
    # E1: x = 1 -> every row sees two full cycles 0..15: y = 0.5 * 240 - 32 = 88.
    # E2: x = one-hot at k = 5 -> y[n] = 0.5 * ((5 + 3n) mod 16) - 1 -> 1.5, 3, 4.5, 6, -0.5, 1, ...
    codes, scales, offsets = structured(32, 32, lambda n, k: k + 3 * n, lambda n, g: 0.5 + 0 * n, lambda n, g: -1.0 + 0 * n)
    x = synthgen.bf16_bits(np.ones((1, 32), np.float32))
    y, a = oracle.project(x, codes, scales, offsets)
    assert np.all(y == 88.0)
    x = synthgen.bf16_bits(np.eye(32, dtype=np.float32)[5:6])
    y, a = oracle.project(x, codes, scales, offsets)
    assert list(y[0, :6]) == [1.5, 3.0, 4.5, 6.0, -0.5, 1.0]
    assert np.array_equal(a, np.abs(y))


def _e3_inputs():
    K = N = 64
    codes, scales, offsets = structured(
        K, N, lambda n, k: 7 * k + 3 * n, lambda n, g: 2.0 ** -(1.0 + g) + 0 * n, lambda n, g: (n - 32) / 16.0 + g)
    m_idx, k_idx = np.arange(2)[:, None], np.arange(K)[None, :]
    xf = (((k_idx + m_idx) % 5) - 2).astype(np.float32)
    return K, N, codes, scales, offsets, xf


def test_worked_example_E3_closed_form():
    # K = N = 64, M = 2, code = (7k + 3n) mod 16, d[n][g] = 2^-(1+g), m[n][g] = (n-32)/16 + g,
    # x[m][k] = ((k + m) mod 5) - 2.  All values are small dyadics, so every sum is exact.
    K, N, codes, scales, offsets, xf = _e3_inputs()
    w32, _ = oracle.dequant(codes, scales, offsets)
    assert w32[33, 5] == 0.8125            # 0.25 * 6 + (-27/16 + 1)
    y, a = oracle.project(synthgen.bf16_bits(xf), codes, scales, offsets)
    expect = {(0, 0): 10.25, (0, 1): -1.625, (0, 31): -5.875, (0, 32): 6.25, (0, 63): -9.875,
              (1, 0): -9.5, (1, 17): -6.625, (1, 63): -6.375}
    for (m, n), v in expect.items():
        assert y[m, n] == v, (m, n, y[m, n], v)
    assert y[0].sum() == -532 and y[1].sum() == 308
    assert a[0, 0] == 137.25 and a[0, 63] == 402.75
    # the same numbers from the definition with exact rationals (independent of the oracle's code)
    for m in range(2):
        for n in (0, 1, 17, 31, 32, 63):
            acc = Fraction(0)
            for k in range(K):
                g = k // 32
                wq = (7 * k + 3 * n) % 16
                acc += Fraction(int(xf[m, k])) * (Fraction(1, 2 ** (1 + g)) * wq + Fraction(n - 32, 16) + g)
            assert Fraction(y[m, n]) == acc


# --------------------------------------------------------------------------- projection vs an independent fp64 matmul

@pytest.mark.parametrize("K,N,M", [(64, 32, 1), (288, 64, 3), (1152, 96, 2), (2560, 64, 8)])
def test_projection_against_numpy_matmul(K, N, M):
    w = synthgen.weights(200 + K, K, N)
    x = synthgen.activations(300 + K, M, K)
    packed = write_sequential(w.codes, w.scales, w.offsets) if K * N <= 300000 else None
    # independent dequantised matrix: numpy, fp64 (exact for these magnitudes up to one fp32 rounding)
    d = synthgen.bf16_to_f32(w.scales).astype(np.float64)
    m = synthgen.bf16_to_f32(w.offsets).astype(np.float64)
    W = (np.repeat(d, 32, axis=1) * w.codes + np.repeat(m, 32, axis=1)).astype(np.float32).astype(np.float64)  # [N, K]
    xd = synthgen.bf16_to_f32(x).astype(np.float64)
    y_np = xd @ W.T
    a_np = np.abs(xd) @ np.abs(W.T)
    y, a = oracle.project(x, w.codes, w.scales, w.offsets)
    assert y.shape == (M, N)
    assert np.allclose(a, a_np, rtol=1e-12, atol=0)
    assert np.all(np.abs(y - y_np) <= 1e-13 * a_np)
    w32, _ = oracle.dequant(w.codes, w.scales, w.offsets)
    assert np.array_equal(w32.astype(np.float64), W.T)
    if packed is not None:
        y2, a2 = oracle.project_packed(x, packed, K, N)
        assert np.array_equal(y2, y) and np.array_equal(a2, a)
    # column ranges and threads give the same bits
    y3, a3 = oracle.project(x, w.codes, w.scales, w.offsets, n0=32, n1=N, nthreads=4) if N > 32 else (y[:, 0:0], a[:, 0:0])
    assert np.array_equal(y3, y[:, 32:]) if N > 32 else True


# --------------------------------------------------------------------------- invariants

def test_invariants_zero_offsets_only_scales_only_onehot():
    K, N, M = 320, 64, 2
    w = synthgen.weights(5, K, N)
    x = synthgen.activations(6, M, K)
    xf = synthgen.bf16_to_f32(x).astype(np.float64)
    zc = np.zeros_like(w.codes)
    z16 = np.zeros_like(w.scales)
    # zero weights
    y, a = oracle.project(x, zc, w.scales, z16)
    assert np.all(y == 0) and np.all(a == 0)
    # offsets only: y[m][n] = sum_g m[n][g] * sum_{k in g} x[m][k]
    y, _ = oracle.project(x, zc, w.scales, w.offsets)
    X = xf.reshape(M, K // 32, 32)
    mo = synthgen.bf16_to_f32(w.offsets).astype(np.float64)
    want = np.einsum("mgk,ng->mn", X, mo)
    assert np.allclose(y, want, rtol=0, atol=1e-12)
    # scales only
    y, _ = oracle.project(x, w.codes, w.scales, z16)
    d = synthgen.bf16_to_f32(w.scales).astype(np.float64)
    want = np.einsum("mgk,ngk->mn", X, d[:, :, None] * w.codes.reshape(N, K // 32, 32))
    assert np.allclose(y, want, rtol=0, atol=1e-12)
    # one-hot x reads out a row of the dequantised matrix, exactly
    w32, w16 = oracle.dequant(w.codes, w.scales, w.offsets)
    for k in (0, 31, 32, 255, 256, 319):
        e = np.zeros((1, K), np.float32)
        e[0, k] = 1
        y, _ = oracle.project(synthgen.bf16_bits(e), w.codes, w.scales, w.offsets)
        assert np.array_equal(y[0], w32[k].astype(np.float64))
        y, _ = oracle.project(synthgen.bf16_bits(e), w.codes, w.scales, w.offsets, use_w16=True)
        assert np.array_equal(y[0], synthgen.bf16_to_f32(w16[k]).astype(np.float64))


def test_invariants_linearity_and_rows():
    K, N = 512, 32
    w = synthgen.weights(8, K, N)
    # small-integer activations: sums of them are bf16-exact and fp64 accumulation is exact enough
    r = synthgen.u64(9, 0, 2 * K).reshape(2, K)
    x1 = ((r[0] >> 60).astype(np.int64) - 8).astype(np.float32)[None]
    x2 = ((r[1] >> 60).astype(np.int64) - 8).astype(np.float32)[None]
    y1, _ = oracle.project(synthgen.bf16_bits(x1), w.codes, w.scales, w.offsets)
    y2, _ = oracle.project(synthgen.bf16_bits(x2), w.codes, w.scales, w.offsets)
    y12, a12 = oracle.project(synthgen.bf16_bits(x1 + x2), w.codes, w.scales, w.offsets)
    assert np.all(np.abs(y12 - (y1 + y2)) <= 1e-13 * (a12 + 1))
    ys, _ = oracle.project(synthgen.bf16_bits(2 * x1), w.codes, w.scales, w.offsets)
    assert np.array_equal(ys, 2 * y1)
    # each row of a batched call equals the single-row call; rows are not mixed up or transposed
    yb, _ = oracle.project(synthgen.bf16_bits(np.concatenate([x1, x2])), w.codes, w.scales, w.offsets)
    assert np.array_equal(yb[0], y1[0]) and np.array_equal(yb[1], y2[0])


# ---- gated GELU epilogue (next step beyond FusedDQP) ---------------------------------------------------------------

def test_gelu_tanh_against_the_error_function_form_and_limits():
    import math

    # the tanh form approximates x * Phi(x) (library erf) to within 1e-3 everywhere
    worst = 0.0
    for i in range(-1200, 1201):
        x = i / 200.0
        exact = 0.5 * x * (1.0 + math.erf(x / math.sqrt(2.0)))
        worst = max(worst, abs(oracle.gelu_tanh(x) - exact))
    assert worst < 1e-3
    assert worst > 1e-5                                  # ... and is not secretly the erf form
    assert oracle.gelu_tanh(0.0) == 0.0
    assert oracle.gelu_tanh(30.0) == 30.0                # tanh saturates: identity for large arguments
    assert abs(oracle.gelu_tanh(-30.0)) < 1e-300
    for x in (0.1, 0.7, 1.0, 2.5, 5.0):                  # gelu(x) - gelu(-x) = x for any odd inner function
        assert abs(oracle.gelu_tanh(x) - oracle.gelu_tanh(-x) - x) < 1e-15
    # widely tabulated values of the tanh form, four digits
    for x, v in ((1.0, 0.8412), (2.0, 1.9546), (-1.0, -0.1588), (3.0, 2.9964)):
        assert abs(oracle.gelu_tanh(x) - v) < 5e-5


def test_geglu_pairs_rows_r_and_r_plus_16_of_each_strip():
    # arguments >= 20 make the tanh exactly 1, so gelu(g) = g and every output is an exact integer product that
    # names the two rows it came from
    M, N = 2, 96
    y = np.array([[20.0 + n + 1000.0 * m for n in range(N)] for m in range(M)])
    out, out16 = oracle.geglu(y)
    assert out.shape == (M, N // 2)
    for m in range(M):
        for j in range(N // 32):
            for r in range(16):
                g, u = y[m, 32 * j + r], y[m, 32 * j + 16 + r]
                assert out[m, 16 * j + r] == g * u
    # bf16 output: round-to-nearest-even of the fp32 value, checked with integer arithmetic on the bits
    f32 = out.astype(np.float32).view(np.uint32).astype(np.uint64)
    expect = ((f32 + 0x7FFF + ((f32 >> 16) & 1)) >> 16).astype(np.uint16)
    assert np.array_equal(out16, expect)
    # a gate of zero silences its output whatever the up value is
    y[:, 0] = 0.0
    assert np.all(oracle.geglu(y)[0][:, 0] == 0.0)


# ---- RMS normalisation prologue (next step beyond FusedDQP) ---------------------------------------------------------

def _bf(vals):
    return synthgen.bf16_bits(np.asarray(vals, np.float32))


def test_rmsnorm_hand_case_invariances_and_unit_power():
    import math

    K = 32
    x = np.zeros((1, K), np.float32)
    x[0, 0], x[0, 1] = 3.0, 4.0                       # mean square = 25 / 32, r = sqrt(32) / 5
    zero = _bf(np.zeros(K))
    out = synthgen.bf16_to_f32(oracle.rmsnorm(_bf(x), zero, 0.0))
    r = math.sqrt(32.0) / 5.0
    assert abs(out[0, 0] - 3.0 * r) <= 2.0 ** -8 * 3.0 * r and abs(out[0, 1] - 4.0 * r) <= 2.0 ** -8 * 4.0 * r
    assert np.all(out[0, 2:] == 0.0)
    assert out[0, 0] == synthgen.bf16_to_f32(_bf([3.0 * r]))[0]          # exactly the nearest bf16
    # a constant row normalises to +-1 whatever its magnitude; with eps it is 1 / sqrt(1 + eps / c^2)
    for c in (0.5, -7.0, 1000.0):
        o = synthgen.bf16_to_f32(oracle.rmsnorm(_bf(np.full((1, K), c)), zero, 0.0))
        assert np.all(o == math.copysign(1.0, c))
    o = synthgen.bf16_to_f32(oracle.rmsnorm(_bf(np.full((1, K), 2.0)), zero, 12.0))   # 1 / sqrt(1 + 12/4) = 0.5
    assert np.all(o == 0.5)
    # power-of-two rescaling of the input changes nothing when eps = 0; gamma = 1 doubles every output exactly
    xs = synthgen.activations(3, 4, 256)
    a = oracle.rmsnorm(xs, _bf(np.zeros(256)), 0.0)
    x4 = _bf(synthgen.bf16_to_f32(xs) * 4.0)
    assert np.array_equal(oracle.rmsnorm(x4, _bf(np.zeros(256)), 0.0), a)
    b = oracle.rmsnorm(xs, _bf(np.ones(256)), 0.0)
    assert np.array_equal(synthgen.bf16_to_f32(b), 2.0 * synthgen.bf16_to_f32(a))
    # unit mean square of the output (gamma = 0, tiny eps) up to the bf16 rounding of each element
    o = synthgen.bf16_to_f32(oracle.rmsnorm(xs, _bf(np.zeros(256)), 1e-12)).astype(np.float64)
    assert np.all(np.abs((o * o).mean(axis=1) - 1.0) < 2.0 ** -7)
    # every row has its own r: rows normalised together equal rows normalised one by one
    for m in range(4):
        assert np.array_equal(oracle.rmsnorm(xs[m:m + 1], _bf(np.zeros(256)), 1e-6), oracle.rmsnorm(xs, _bf(np.zeros(256)), 1e-6)[m:m + 1])
    # gamma is indexed by k: a one-hot gamma touches exactly its own column
    g = np.zeros(256, np.float32)
    g[17] = 1.0
    c = synthgen.bf16_to_f32(oracle.rmsnorm(xs, _bf(g), 0.0))
    a32 = synthgen.bf16_to_f32(a)
    assert np.array_equal(np.delete(c, 17, axis=1), np.delete(a32, 17, axis=1)) and np.array_equal(c[:, 17], 2.0 * a32[:, 17])


# ---- decode attention over a KV cache (next step: the paper's second decode kernel) ---------------------------------

def test_decode_attention_closed_forms_and_invariances():
    import math

    d, G, H, pitch = 8, 2, 4, 16
    rng = np.random.default_rng(5)

    def bf(a):
        return synthgen.bf16_bits(np.asarray(a, np.float32))

    # two positions, scores 0 and ln 3 -> weights 1/4 and 3/4 (q = e0, k0 = 0, k1 = ln3 * e0 is not bf16-exact, so use
    # scale: q . k1 = 1 and scale = ln 3)
    q = np.zeros((H, d), np.float32)
    q[:, 0] = 1.0
    K = np.zeros((G, pitch, d), np.float32)
    V = np.zeros((G, pitch, d), np.float32)
    K[:, 1, 0] = 1.0
    V[0, 0], V[0, 1] = 4.0, 8.0
    V[1, 0], V[1, 1] = -4.0, 16.0
    out, absw = oracle.decode_attention(bf(q), bf(K), bf(V), L=2, scale=math.log(3.0))
    assert np.allclose(out[0], 0.25 * 4.0 + 0.75 * 8.0, rtol=0, atol=1e-14)
    assert np.allclose(out[2], 0.25 * -4.0 + 0.75 * 16.0, rtol=0, atol=1e-14)       # heads 2, 3 read KV head 1
    assert np.array_equal(out[0], out[1]) and np.array_equal(out[2], out[3])
    assert np.allclose(absw[2], 0.25 * 4.0 + 0.75 * 16.0, rtol=0, atol=1e-14)
    # equal keys -> uniform weights -> the mean of the values; a query of zero does the same
    L = 11
    K = np.tile(rng.standard_normal((G, 1, d)).astype(np.float32), (1, pitch, 1))
    V = rng.standard_normal((G, pitch, d)).astype(np.float32)
    q = rng.standard_normal((H, d)).astype(np.float32)
    Vb = synthgen.bf16_to_f32(bf(V)).astype(np.float64)
    out, _ = oracle.decode_attention(bf(q), bf(K), bf(V), L=L, scale=0.3)
    for h in range(H):
        assert np.allclose(out[h], Vb[h // 2, :L].mean(axis=0), rtol=0, atol=1e-13)
    K = rng.standard_normal((G, pitch, d)).astype(np.float32)
    out0, _ = oracle.decode_attention(bf(np.zeros((H, d))), bf(K), bf(V), L=L)
    assert np.allclose(out0[3], Vb[1, :L].mean(axis=0), rtol=0, atol=1e-13)
    # the window keeps the last `window` positions: same as attention over a cache that only holds those
    full, _ = oracle.decode_attention(bf(q), bf(K), bf(V), L=L, window=4, scale=0.5)
    cut, _ = oracle.decode_attention(bf(q), bf(K[:, L - 4:L]), bf(V[:, L - 4:L]), L=4, scale=0.5)
    assert np.array_equal(full, cut)
    same, _ = oracle.decode_attention(bf(q), bf(K), bf(V), L=L, window=L + 5, scale=0.5)
    allp, _ = oracle.decode_attention(bf(q), bf(K), bf(V), L=L, window=0, scale=0.5)
    assert np.array_equal(same, allp)
    # positions beyond L are never read
    K2, V2 = K.copy(), V.copy()
    K2[:, L:], V2[:, L:] = 1e30, -1e30
    assert np.array_equal(oracle.decode_attention(bf(q), bf(K2), bf(V2), L=L, scale=0.5)[0], allp)
    # a dominant score selects its value; an independent numpy softmax agrees everywhere
    Kb = synthgen.bf16_to_f32(bf(K)).astype(np.float64)
    qb = synthgen.bf16_to_f32(bf(q)).astype(np.float64)
    for h in range(H):
        s = 0.5 * Kb[h // 2, :L] @ qb[h]
        p = np.exp(s - s.max())
        p /= p.sum()
        assert np.allclose(allp[h], p @ Vb[h // 2, :L], rtol=1e-13, atol=1e-14)
    # one position -> its value, whatever the score; any permutation of the attended positions changes nothing
    one, _ = oracle.decode_attention(bf(q), bf(K), bf(V), L=1, scale=0.5)
    assert np.array_equal(one[1], Vb[0, 0]) and np.array_equal(one[2], Vb[1, 0])
    perm = rng.permutation(L)
    Kp, Vp = K.copy(), V.copy()
    Kp[:, :L], Vp[:, :L] = K[:, perm], V[:, perm]
    outp, _ = oracle.decode_attention(bf(q), bf(Kp), bf(Vp), L=L, scale=0.5)
    assert np.allclose(outp, allp, rtol=1e-13, atol=1e-14)
    big = np.zeros((H, d), np.float32)
    big[:, 1] = 64.0
    Kd = np.zeros((G, pitch, d), np.float32)
    Kd[:, 7, 1] = 8.0
    sel, _ = oracle.decode_attention(bf(big), bf(Kd), bf(V), L=L)
    assert np.allclose(sel[0], Vb[0, 7], rtol=0, atol=1e-12)


def test_add_residual_is_one_rounding_of_the_exact_sum():
    from fractions import Fraction

    def bf(a):
        return synthgen.bf16_bits(np.asarray(a, np.float32))

    def frac(bits):
        return Fraction(float(synthgen.bf16_to_f32(np.array([bits], np.uint16))[0]))

    # hand cases: below half an ulp, a tie to the even neighbour below, a tie to the even neighbour above, cancellation
    x = bf([[1.0, 1.0, 1.0078125, 3.0, -2.5, 0.0]])
    r = bf([[2.0 ** -9, 2.0 ** -8, 2.0 ** -8, -3.0, 2.5, 0.0]])
    h = synthgen.bf16_to_f32(oracle.add_residual(x, r))[0]
    assert list(h) == [1.0, 1.0, 1.015625, 0.0, 0.0, 0.0]
    # random pairs, wide exponent gaps and subnormals included: the nearest bf16 to the exact rational sum, found by
    # comparing the neighbours of a truncated estimate
    rng = np.random.default_rng(12)
    n = 4000
    xb = rng.integers(0, 1 << 16, n).astype(np.uint16)
    rb = rng.integers(0, 1 << 16, n).astype(np.uint16)
    expo = lambda b: (b >> 7) & 0xFF
    keep = (expo(xb) != 255) & (expo(rb) != 255)
    xb, rb = xb[keep], rb[keep]
    rb[::3] = (xb[::3] & 0x8000) | np.clip((xb[::3] & 0x7FFF).astype(np.int32) + rng.integers(-300, 300, xb[::3].size), 0, 0x7F7F).astype(np.uint16)
    got = oracle.add_residual(xb[None, :], rb[None, :])[0]
    for a, b, g in zip(xb.tolist(), rb.tolist(), got.tolist()):
        exact = frac(a) + frac(b)
        if exact == 0:
            assert g in (0, 0x8000)
            continue
        if abs(exact) >= Fraction(2) ** 128:      # beyond the largest finite value by more than half a step
            assert g == (0xFF80 if exact < 0 else 0x7F80)
            continue
        sign = 0x8000 if exact < 0 else 0
        mag = abs(exact)
        est = int(np.array([float(mag)], np.float32).view(np.uint32)[0] >> 16)
        best = None
        for c in range(max(est - 2, 0), min(est + 3, 0x7F81)):
            cv = frac(c) if c < 0x7F80 else Fraction(2) ** 128     # infinity stands in as the next step up
            d = abs(cv - mag)
            if best is None or d < best[0] or (d == best[0] and c % 2 == 0):
                best = (d, c)
        assert g == (sign | best[1]), (hex(a), hex(b), hex(g), hex(sign | best[1]))
    # identities: adding zero changes nothing, the sum commutes, x + (-x) = 0
    xs = synthgen.activations(5, 3, 64)
    zero = np.zeros_like(xs)
    assert np.array_equal(oracle.add_residual(xs, zero), xs)
    ys = synthgen.activations(6, 3, 64)
    assert np.array_equal(oracle.add_residual(xs, ys), oracle.add_residual(ys, xs))
    assert not np.any(oracle.add_residual(xs, xs ^ 0x8000) & 0x7FFF)
