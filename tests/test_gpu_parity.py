"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs -- element by element at sizes that span several tiles and ragged tails, bit-for-bit where
the arithmetic is exact, and on the full workload shapes."""
import numpy as np
import pytest
import torch

import oracle
import paper_2602_06063_b200 as fd
import synthgen
from gpu_common import (ABS_TOL, MAX_K, MAX_M, MAX_N, REL_TOL, Case, assert_close, dev_bytes, exact_regime_weights,
                        exact_regime_x)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    h = fd.fdqp_create(0, MAX_M, MAX_K, MAX_N)
    yield h
    torch.cuda.synchronize()
    fd.fdqp_destroy(h)


@pytest.fixture()
def fresh(ctx):
    """The shared context with every launch parameter back to automatic."""
    for key in ("path", "ctas_per_sm", "consumer_warps", "stages", "split_k", "l2_evict_first", "prep_inline", "strip_aligned", "blocks_per_warp", "prefill_pair", "prefill_split_k"):
        fd.fdqp_set_param(ctx, key, -1)
    fd.fdqp_set_param(ctx, "prefill_a_tmem", 1)
    yield ctx
    for key in ("path", "ctas_per_sm", "consumer_warps", "stages", "split_k", "l2_evict_first", "prep_inline", "strip_aligned", "blocks_per_warp", "prefill_pair", "prefill_split_k"):
        fd.fdqp_set_param(ctx, key, -1)
    fd.fdqp_set_param(ctx, "prefill_a_tmem", 1)


# ------------------------------------------------------------------ dequantisation engine: bit-exact

@pytest.mark.parametrize("K,N", [(32, 32), (288, 64), (1152, 96), (2560, 256)])
def test_dequant_bit_exact(fresh, K, N):
    case = Case(K, N, 1, seed=900 + K)
    w32, w16 = oracle.dequant(case.w.codes, case.w.scales, case.w.offsets)
    out32 = torch.empty((K, N), dtype=torch.float32, device="cuda")
    out16 = torch.empty((K, N), dtype=torch.bfloat16, device="cuda")
    fd.fdqp_dequant(fresh, case.W_dev, out32, False, K, N)
    fd.fdqp_dequant(fresh, case.W_dev, out16, True, K, N)
    torch.cuda.synchronize()
    assert np.array_equal(out32.cpu().numpy().view(np.uint32), w32.view(np.uint32))
    assert np.array_equal(out16.view(torch.int16).cpu().numpy().view(np.uint16), w16)


def test_dequant_bit_exact_extreme_scales(fresh):
    # scales and offsets over the whole finite bf16 range, subnormals included (nothing may flush to zero)
    K, N = 512, 64
    r = synthgen.u64(77, 0, 2 * N * (K // 32)).reshape(2, N, K // 32)
    bits = ((r >> np.uint64(48)) & np.uint64(0xFFFF)).astype(np.uint16)
    finite = (bits & 0x7F80) != 0x7F80
    bits = np.where(finite, bits, bits & 0x807F).astype(np.uint16)
    # keep exponents below 2^100 so that d*15 + m cannot overflow
    bits = np.where((bits & 0x7F80) > (227 << 7), bits & 0x80FF | (100 << 7), bits).astype(np.uint16)
    w = synthgen.weights(78, K, N)
    w.scales[:], w.offsets[:] = bits[0], bits[1]
    case = Case(K, N, 1, seed=78, weights=w)
    w32, w16 = oracle.dequant(w.codes, w.scales, w.offsets)
    out32 = torch.empty((K, N), dtype=torch.float32, device="cuda")
    out16 = torch.empty((K, N), dtype=torch.bfloat16, device="cuda")
    fd.fdqp_dequant(fresh, case.W_dev, out32, False, K, N)
    fd.fdqp_dequant(fresh, case.W_dev, out16, True, K, N)
    torch.cuda.synchronize()
    assert np.array_equal(out32.cpu().numpy().view(np.uint32), w32.view(np.uint32))
    assert np.array_equal(out16.view(torch.int16).cpu().numpy().view(np.uint16), w16)


# ------------------------------------------------------------------ projection: element by element

SMALL = [  # (K, N, M): tiny, tails (K % 256 != 0), several strips, several blocks, every M of the GEMV family, M >= 9
    (32, 32, 1), (64, 64, 2), (288, 32, 1), (544, 96, 3), (1152, 6912, 1), (2560, 1024, 1), (2560, 2048, 8),
    (2048, 2560, 5), (4096, 4736, 4), (10240, 2560, 1), (3840, 1280, 7), (1024, 512, 9), (1056, 320, 20),
]


@pytest.mark.parametrize("K,N,M", SMALL)
@pytest.mark.parametrize("path", [0, 1])
def test_projection_matches_oracle(fresh, K, N, M, path):
    fd.fdqp_set_param(fresh, "path", path)
    case = Case(K, N, M, seed=1000 + K + N + M)
    y = case.run(fresh)
    y_ref, a_ref = case.reference()
    assert_close(y, y_ref, a_ref, f"K={K} N={N} M={M} path={path}")


@pytest.mark.parametrize("K,N,M", [(64, 64, 2), (1152, 96, 1), (4096, 1024, 8), (2560, 4736, 3), (21504, 64, 1)])
def test_exact_arithmetic_regime_is_bit_exact(fresh, K, N, M):
    # d = 2^-3, m in {-1,0,1}, x in {-2..2}: every partial sum is a multiple of 2^-3 far below 2^24, so any
    # summation order is exact in fp32 and the result must equal the oracle bit for bit.
    case = Case(K, N, M, seed=0, weights=exact_regime_weights(31 + K, K, N), x=exact_regime_x(32 + K, M, K))
    y_ref, _ = case.reference()
    for path in (0, 1):
        fd.fdqp_set_param(fresh, "path", path)
        y = case.run(fresh)
        assert np.array_equal(y.astype(np.float64), y_ref), f"path {path}"


PREFILL = [(64, 32, 9), (1024, 512, 9), (1056, 320, 20), (2560, 1024, 100), (512, 288, 300), (4096, 768, 512),
           (1056, 320, 257), (544, 1056, 511), (512, 512, 272), (512, 512, 400)]


@pytest.mark.parametrize("K,N,M", PREFILL)
def test_prefill_tensor_path_matches_oracle(fresh, K, N, M):
    # M >= 9: dequantise-into-shared-memory + tcgen05 path.  Ragged token tiles, a K that is not a multiple of
    # the 64-wide pipeline step, N that is not a multiple of the 256-row tile, more than one token tile.
    case = Case(K, N, M, seed=2000 + K + N + M)
    fd.fdqp_set_param(fresh, "path", 3)
    assert ("fdqp_prefill_pair_kernel" if M > 256 else "fdqp_prefill_kernel") in fd.fdqp_describe(fresh, M, K, N)
    y = case.run(fresh)
    y_ref, a_ref = case.reference()
    assert_close(y, y_ref, a_ref, f"prefill K={K} N={N} M={M}")
    # the other tensor-core kernel (two-SM 256 x 512 tile <-> one-SM 256 x 256 tile) on the same inputs
    fd.fdqp_set_param(fresh, "prefill_pair", 0 if M > 256 else 1)
    assert ("fdqp_prefill_kernel" if M > 256 else "fdqp_prefill_pair_kernel") in fd.fdqp_describe(fresh, M, K, N)
    assert_close(case.run(fresh), y_ref, a_ref, f"prefill (other tile) K={K} N={N} M={M}")
    fd.fdqp_set_param(fresh, "prefill_pair", -1)
    if M <= 128:
        # up to 128 token rows the converted weights live in tensor memory by default; in shared memory: the same bits
        assert "weights in TMEM" in fd.fdqp_describe(fresh, M, K, N)
        fd.fdqp_set_param(fresh, "prefill_a_tmem", 0)
        assert "weights in TMEM" not in fd.fdqp_describe(fresh, M, K, N)
        assert np.array_equal(case.run(fresh), y)
        fd.fdqp_set_param(fresh, "prefill_a_tmem", 1)
    # the same rows through the GEMV kernel, eight at a time: both are within the bound of the oracle
    fd.fdqp_set_param(fresh, "path", 2)
    assert "fdqp_gemv_kernel" in fd.fdqp_describe(fresh, M, K, N)
    assert_close(case.run(fresh), y_ref, a_ref, f"gemv-chunked K={K} N={N} M={M}")


@pytest.mark.parametrize("K,N,M,Z", [(64, 32, 9, 1), (1056, 320, 20, 1), (2560, 1024, 64, 1), (544, 1056, 33, 1), (2048, 256, 64, 4),
                                     (1024, 32, 40, 2), (2592, 160, 16, 3)])
def test_prefill_three_ctas_per_sm_same_bits(fresh, K, N, M, Z):
    # up to 64 token rows: the form with 64 accumulator columns, two weight stages and a four-deep weight prefetch that
    # fits three CTAs per SM (chosen by itself for calls with that many CTAs; forced here) -- within the bound of the
    # oracle and bit for bit what the two-CTA form computes
    case = Case(K, N, M, seed=2500 + K + N + M)
    fd.fdqp_set_param(fresh, "path", 3)
    if Z > 1:
        fd.fdqp_set_param(fresh, "prefill_split_k", Z)
    fd.fdqp_set_param(fresh, "prefill_a_tmem", 2)
    assert "three CTAs per SM" in fd.fdqp_describe(fresh, M, K, N)
    y3 = case.run(fresh)
    fd.fdqp_set_param(fresh, "prefill_a_tmem", 1)
    assert "two CTAs per SM" in fd.fdqp_describe(fresh, M, K, N)
    y2 = case.run(fresh)
    y_ref, a_ref = case.reference()
    assert_close(y3, y_ref, a_ref, f"three CTAs K={K} N={N} M={M} Z={Z}")
    assert np.array_equal(y3, y2)


@pytest.mark.parametrize("K,N,M,Z", [(2048, 256, 64, 4), (2112, 544, 300, 3), (4096, 288, 512, 8), (1024, 32, 40, 2)])
def test_prefill_k_slices(fresh, K, N, M, Z):
    # few output tiles: K is cut into slices whose partial results a second kernel adds in slice order
    case = Case(K, N, M, seed=3000 + K + N + M)
    fd.fdqp_set_param(fresh, "path", 3)
    y_ref, a_ref = case.reference()
    auto = fd.fdqp_describe(fresh, M, K, N)
    if K >= 2048:                                               # long reductions over few tiles are split without being
        assert "split_k=" in auto and "split_k=1" not in auto  # asked (a short one is not worth the second kernel)
    y_auto = case.run(fresh)
    assert_close(y_auto, y_ref, a_ref, f"prefill auto split K={K} N={N} M={M}")
    fd.fdqp_set_param(fresh, "prefill_split_k", Z)
    assert f"split_k={Z}" in fd.fdqp_describe(fresh, M, K, N)
    y_z = case.run(fresh)
    assert_close(y_z, y_ref, a_ref, f"prefill split_k={Z} K={K} N={N} M={M}")
    assert np.array_equal(y_z, case.run(fresh))                 # fixed summation order: reruns are bit-identical
    fd.fdqp_set_param(fresh, "prefill_split_k", 1)
    assert_close(case.run(fresh), y_ref, a_ref, f"prefill unsplit K={K} N={N} M={M}")


def test_prefill_exact_cases(fresh):
    # (i) exact-arithmetic regime: weights are bf16-exact, every fp32 sum is exact -> bit-equal to the oracle
    K, N, M = 1152, 288, 40
    fd.fdqp_set_param(fresh, "path", 3)
    case = Case(K, N, M, seed=0, weights=exact_regime_weights(71, K, N), x=exact_regime_x(72, M, K))
    y_ref, _ = case.reference()
    assert np.array_equal(case.run(fresh).astype(np.float64), y_ref)
    # (ii) one-hot activations read out rows of the bf16-rounded dequantised matrix, bit for bit
    K, N, M = 544, 96, 16
    c2 = Case(K, N, M, seed=73)
    _, w16 = oracle.dequant(c2.w.codes, c2.w.scales, c2.w.offsets)
    ks = [0, 31, 32, 63, 64, 255, 256, 300, 511, 512, 543, 7, 100, 200, 400, 500]
    x = np.zeros((M, K), np.float32)
    for i, kk in enumerate(ks):
        x[i, kk] = 1.0
    y = Case(K, N, M, 0, weights=c2.w, x=synthgen.bf16_bits(x)).run(fresh)
    assert np.array_equal(y.view(np.uint32) >> 16, w16[ks].astype(np.uint32))
    assert np.all((y.view(np.uint32) & 0xFFFF) == 0)


def test_worked_examples_on_gpu(fresh):
    # E1/E2: K = N = 32, code = (k + 3n) mod 16, d = 0.5, m = -1; x = 1 -> 88; x = e_5 -> 0.5*((5+3n)%16) - 1
    n, k = np.arange(32)[:, None], np.arange(32)[None, :]
    w = synthgen.Q4NXWeights(((k + 3 * n) % 16).astype(np.uint8), np.full((32, 1), 0x3F00, np.uint16),
                             np.full((32, 1), 0xBF80, np.uint16))
    ones = synthgen.bf16_bits(np.ones((1, 32), np.float32))
    assert np.all(Case(32, 32, 1, 0, weights=w, x=ones).run(fresh) == 88.0)
    e5 = synthgen.bf16_bits(np.eye(32, dtype=np.float32)[5:6])
    y = Case(32, 32, 1, 0, weights=w, x=e5).run(fresh)
    assert list(y[0, :6]) == [1.5, 3.0, 4.5, 6.0, -0.5, 1.0]
    # E3: K = N = 64, M = 2 (and the same rows padded to M = 9), all values dyadic
    K = N = 64
    n, k, g = np.arange(N)[:, None], np.arange(K)[None, :], np.arange(2)[None, :]
    w = synthgen.Q4NXWeights(((7 * k + 3 * n) % 16).astype(np.uint8),
                             synthgen.bf16_bits((2.0 ** -(1.0 + g) + 0 * n).astype(np.float32)),
                             synthgen.bf16_bits(((n - 32) / 16.0 + g).astype(np.float32)))
    m_idx = np.arange(9)[:, None]
    xf = (((k + m_idx) % 5) - 2).astype(np.float32)
    for M, path in ((2, 0), (9, 2), (9, 3)):
        fd.fdqp_set_param(fresh, "path", path)
        y = Case(K, N, M, 0, weights=w, x=synthgen.bf16_bits(xf[:M])).run(fresh)
        assert y[0, 0] == 10.25 and y[0, 1] == -1.625 and y[0, 31] == -5.875 and y[0, 32] == 6.25
        assert y[0, 63] == -9.875 and y[1, 0] == -9.5 and y[1, 17] == -6.625 and y[1, 63] == -6.375
        assert y[0].sum() == -532 and y[1].sum() == 308


def test_one_hot_reads_out_dequantised_rows(fresh):
    K, N = 544, 64
    case = Case(K, N, 8, seed=55)
    w32, _ = oracle.dequant(case.w.codes, case.w.scales, case.w.offsets)
    ks = [0, 31, 32, 255, 256, 300, 511, 543]
    x = np.zeros((8, K), np.float32)
    for i, kk in enumerate(ks):
        x[i, kk] = 1.0
    y = Case(K, N, 8, 0, weights=case.w, x=synthgen.bf16_bits(x)).run(fresh)
    want = w32[ks].astype(np.float64)
    assert np.all(np.abs(y - want) <= REL_TOL * np.abs(want) + ABS_TOL)
    # (the GEMV forms d * 2^e * (integer sum) + m * (sum of x) with two roundings, so this read-out is close, not
    # necessarily bit-equal; the bit-exact statement of Eq. 3 is fdqp_dequant's)


def test_zero_and_offsets_only(fresh):
    K, N, M = 1152, 64, 4
    case = Case(K, N, M, seed=66)
    zero = synthgen.Q4NXWeights(np.zeros_like(case.w.codes), case.w.scales, np.zeros_like(case.w.offsets))
    # codes 0 and offsets 0 (scales left non-zero): every w_hat is 0 and so is every output, exactly
    assert np.all(Case(K, N, M, 0, weights=zero, x=case.x).run(fresh) == 0)
    off = synthgen.Q4NXWeights(np.zeros_like(case.w.codes), case.w.scales, case.w.offsets)
    c = Case(K, N, M, 0, weights=off, x=case.x)
    y_ref, a_ref = c.reference()
    assert_close(c.run(fresh), y_ref, a_ref, "offsets only")


def test_reruns_are_bit_identical_and_scaling_by_two_commutes(fresh):
    for K, N, M in [(21504, 5376, 4), (2560, 10240, 1)]:
        case = Case(K, N, M, seed=70 + M, amp=K ** -0.5)
        y1 = case.run(fresh)
        y2 = case.run(fresh)
        assert np.array_equal(y1.view(np.uint32), y2.view(np.uint32))
        x2 = synthgen.bf16_bits(2 * synthgen.bf16_to_f32(case.x))
        y3 = Case(K, N, M, 0, weights=case.w, x=x2).run(fresh)
        assert np.array_equal(y3, 2 * y1)


def test_batched_rows_match_single_row_calls(fresh):
    K, N, M = 3840, 2048, 8
    case = Case(K, N, M, seed=81)
    y = case.run(fresh)
    y_ref, a_ref = case.reference()
    for m in (0, 3, 7):
        xm = dev_bytes(case.x[m:m + 1])
        y1 = case.run(fresh, M=1, x_dev=xm)
        assert_close(y1, y_ref[m:m + 1], a_ref[m:m + 1], f"row {m}")
        assert np.all(np.abs(y1[0] - y[m]) <= 2 * (REL_TOL * a_ref[m] + ABS_TOL))


@pytest.mark.parametrize("key,values", [("split_k", [1, 2, 4, 8]), ("consumer_warps", [8, 16]), ("ctas_per_sm", [1, 2]),
                                        ("stages", [2, 3, 7]), ("l2_evict_first", [0, 1]), ("prep_inline", [0, 1]), ("strip_aligned", [0, 1]), ("blocks_per_warp", [2, 4])])
def test_launch_parameters_do_not_change_results(fresh, key, values):
    K, N, M = 4352, 2080, 3   # 17 blocks per strip, 65 strips: ragged against every split and grid
    case = Case(K, N, M, seed=90)
    y_ref, a_ref = case.reference()
    exact = Case(K, N, M, 0, weights=exact_regime_weights(91, K, N), x=exact_regime_x(92, M, K))
    e_ref, _ = exact.reference()
    for v in values:
        fd.fdqp_set_param(fresh, key, v)
        assert_close(case.run(fresh), y_ref, a_ref, f"{key}={v}")
        assert np.array_equal(exact.run(fresh).astype(np.float64), e_ref), f"{key}={v}"


def test_output_is_fully_overwritten_and_nothing_else(fresh):
    K, N, M = 2560, 1024, 3
    case = Case(K, N, M, seed=95)
    buf = torch.full((M * N + 512,), 12345.0, dtype=torch.float32, device="cuda")
    y = buf[256:256 + M * N]
    fd.fdqp_run(fresh, case.x_dev, case.W_dev, y, M, K, N)
    torch.cuda.synchronize()
    host = buf.cpu().numpy()
    assert np.all(host[:256] == 12345.0) and np.all(host[256 + M * N:] == 12345.0)
    y_ref, a_ref = case.reference()
    assert_close(host[256:256 + M * N].reshape(M, N), y_ref, a_ref, "guarded output")


def test_argument_errors_launch_nothing(fresh):
    K, N, M = 256, 64, 1
    case = Case(K, N, M, seed=96)
    y = torch.zeros((M, N), dtype=torch.float32, device="cuda")
    lib = fd.load_library()
    before = fd.fdqp_launch_count(fresh)
    s = torch.cuda.current_stream().cuda_stream
    xp, wp, yp = case.x_dev.data_ptr(), case.W_dev.data_ptr(), y.data_ptr()
    assert lib.fdqp_run(fresh, None, wp, yp, M, K, N, s) == 1
    assert lib.fdqp_run(fresh, xp, wp, yp, 0, K, N, s) == 2
    assert lib.fdqp_run(fresh, xp, wp, yp, M, K + 16, N, s) == 2
    assert lib.fdqp_run(fresh, xp, wp, yp, M, K, N + 16, s) == 2
    assert lib.fdqp_run(fresh, xp + 2, wp, yp, M, K, N, s) == 3
    assert lib.fdqp_run(fresh, xp, wp + 8, yp, M, K, N, s) == 3
    assert lib.fdqp_run(fresh, xp, wp, yp + 4, M, K, N, s) == 3
    assert lib.fdqp_run(fresh, xp, wp, yp, MAX_M + 1, K, N, s) == 4
    assert lib.fdqp_run(fresh, xp, wp, yp, M, MAX_K + 32, N, s) == 4
    assert lib.fdqp_dequant(fresh, wp, yp, 2, K, N, s) == 1
    assert lib.fdqp_set_param(fresh, b"no_such_key", 1) == 1
    assert lib.fdqp_set_param(fresh, b"split_k", 3) == 1
    assert fd.fdqp_launch_count(fresh) == before
    assert "fdqp_gemv_kernel" in fd.fdqp_describe(fresh, 1, 2560, 10240)


def test_run_host_roundtrip(fresh):
    K, N, M = 2560, 2048, 2
    case = Case(K, N, M, seed=97)
    x_host = torch.from_numpy(case.x.view(np.int16)).pin_memory()
    y_host = torch.empty((M, N), dtype=torch.float32).pin_memory()
    fd.fdqp_run_host(fresh, x_host, case.W_dev, y_host, M, K, N)
    y_ref, a_ref = case.reference()
    assert_close(y_host.numpy(), y_ref, a_ref, "run_host")
    assert np.array_equal(y_host.numpy(), case.run(fresh))
    # the asynchronous form: two calls queued on one stream, results valid after the caller's synchronisation
    y2 = torch.zeros((M, N), dtype=torch.float32).pin_memory()
    y3 = torch.zeros((1, N), dtype=torch.float32).pin_memory()
    fd.fdqp_run_host_async(fresh, x_host, case.W_dev, y2, M, K, N)
    fd.fdqp_run_host_async(fresh, x_host[:1], case.W_dev, y3, 1, K, N)
    torch.cuda.synchronize()
    assert fd.fdqp_last_status(fresh) == 0
    assert np.array_equal(y2.numpy(), y_host.numpy())
    assert_close(y3.numpy(), y_ref[:1], a_ref[:1], "run_host_async M=1")


@pytest.mark.parametrize("K,N,M,params", [(2560, 2048, 1, {}), (21504, 320, 2, {}), (1056, 320, 20, {"path": 3}),
                                          (2560, 4096, 5, {}), (512, 288, 300, {"path": 3})])
def test_run_host_result_paths_agree(fresh, K, N, M, params):
    """Pinned (device-addressable) host buffers are used in place when small -- x read by the preparation kernel (up to
    eight token rows), y stored by the kernels themselves; pageable host memory and the staged route give the same bits,
    on every kernel family (whole strips, K slices with their sum kernel, the tensor-core kernels)."""
    case = Case(K, N, M, seed=980 + K + M, amp=1.0 / np.sqrt(K) if K > 20000 else 1.0)
    for k, v in params.items():
        fd.fdqp_set_param(fresh, k, v)
    ref = case.run(fresh)
    x_pin = torch.from_numpy(case.x.view(np.int16)).pin_memory()
    y_pin = torch.full((M, N), float("nan"), dtype=torch.float32).pin_memory()
    fd.fdqp_run_host(fresh, x_pin, case.W_dev, y_pin, M, K, N)
    assert np.array_equal(y_pin.numpy(), ref)
    y_page = torch.full((M, N), float("nan"), dtype=torch.float32)           # pageable: staged, then copied
    fd.fdqp_run_host(fresh, torch.from_numpy(case.x.view(np.int16)), case.W_dev, y_page, M, K, N)
    assert np.array_equal(y_page.numpy(), ref)
    fd.fdqp_set_param(fresh, "host_direct_y", 0)
    try:
        y_staged = torch.full((M, N), float("nan"), dtype=torch.float32).pin_memory()
        fd.fdqp_run_host(fresh, x_pin, case.W_dev, y_staged, M, K, N)
        assert np.array_equal(y_staged.numpy(), ref)
    finally:
        fd.fdqp_set_param(fresh, "host_direct_y", 1)


# ------------------------------------------------------------------ the give-up path of the bounded waits

def test_bounded_wait_gives_up_and_context_stays_usable():
    """A wait that nothing satisfies returns after its limit, records FDQP_ERR_TIMEOUT in the context's sticky status
    word and leaves the device usable: a second context on the same device computes a correct projection afterwards,
    and so does the first one (its status stays set, its results are still right)."""
    import time
    K, N, M = 512, 96, 1
    case = Case(K, N, M, seed=97)
    own = fd.fdqp_create(0, 8, K, N)
    other = fd.fdqp_create(0, 8, K, N)
    try:
        assert fd.fdqp_last_status(own) == 0
        t0 = time.perf_counter()
        fd.fdqp_selftest_bounded_wait(own, 500)      # microseconds
        torch.cuda.synchronize()
        assert time.perf_counter() - t0 < 5.0         # it returned by itself, well before the production limit
        assert fd.fdqp_last_status(own) == 8          # FDQP_ERR_TIMEOUT
        assert fd.fdqp_last_status(other) == 0
        ref, a_ref = case.reference()
        y = case.run(other)
        assert_close(y, ref, a_ref)
        yo = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        fd.fdqp_run(own, case.x_dev, case.W_dev, yo, M, K, N)
        torch.cuda.synchronize()
        assert fd.fdqp_last_status(own) == 8          # sticky
        assert_close(yo.cpu().numpy(), ref, a_ref)
        lib = fd.load_library()
        assert lib.fdqp_selftest_bounded_wait(own, 0, None) == 1
        assert lib.fdqp_selftest_bounded_wait(own, 100001, None) == 1
    finally:
        fd.fdqp_destroy(own)
        fd.fdqp_destroy(other)
