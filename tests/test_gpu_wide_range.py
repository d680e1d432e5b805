"""Activations with a wide dynamic range inside a 32-group, through the GEMV kernels (M = 1 .. 8).

At one and two token rows the kernels hold the activations of a quantisation group as 31-bit fixed point relative to
the group's largest exponent.  That is exact for values within 2^22 of the largest; a group with anything else -- a
tiny value next to an outlier channel, a subnormal next to a normal number, an infinity or a NaN -- is flagged by the
activation preparation and evaluated in fp32 straight from Eq. 3 inside the same kernel.  At three to eight rows the
activations enter the tensor cores as the bf16 numbers they are.  These tests go to both sides of that line and check
the stated acceptance bound against the fp64 oracle on inputs built to break a rounded fixed point: the outlier's own
weight is zero, so everything the output is made of comes from the small elements.
"""
import numpy as np
import pytest
import torch

import paper_2602_06063_b200 as fd
import synthgen
from gpu_common import Case, assert_close, exact_regime_weights, exact_regime_x

pytestmark = pytest.mark.gpu

PARAMS = ("path", "ctas_per_sm", "consumer_warps", "stages", "split_k", "l2_evict_first", "prep_inline", "strip_aligned",
          "blocks_per_warp")


@pytest.fixture(scope="module")
def ctx():
    h = fd.fdqp_create(0, 16, 8192, 4096)
    yield h
    torch.cuda.synchronize()
    fd.fdqp_destroy(h)


@pytest.fixture()
def fresh(ctx):
    for key in PARAMS:
        fd.fdqp_set_param(ctx, key, -1)
    yield ctx
    for key in PARAMS:
        fd.fdqp_set_param(ctx, key, -1)


def f32_of(bits):
    return synthgen.bf16_to_f32(bits)


def outlier_case(K, N, M, seed, log2_ratio, zero_weight, every=1, base=2.0 ** -9):
    """x: every `every`-th group holds one element 2^log2_ratio times larger than its 31 neighbours (which are
    `base` times N(0,1) draws); the other groups are all zero, so nothing else props the bound up.  With zero_weight the
    weight under the outlier is exactly 0 in every output row (code 0, offset 0 for that group)."""
    w = synthgen.weights(seed, K, N)
    codes, offsets = w.codes.copy(), w.offsets.copy()
    x = np.zeros((M, K), np.float32)
    small = f32_of(synthgen.activations(seed + 1, M, K)) * base
    for g in range(0, K // 32, every):
        pos = g * 32 + (7 * g + 3) % 32
        x[:, g * 32:(g + 1) * 32] = small[:, g * 32:(g + 1) * 32]
        x[:, pos] = np.sign(small[:, pos] + 1e-30) * base * 2.0 ** log2_ratio
        if zero_weight:
            codes[:, pos] = 0
            offsets[:, g] = 0
    return Case(K, N, M, 0, weights=synthgen.Q4NXWeights(codes, w.scales, offsets), x=synthgen.bf16_bits(x))


@pytest.mark.parametrize("M", [1, 2, 3, 8])
@pytest.mark.parametrize("log2_ratio", [10, 14, 15, 16, 24, 40])
@pytest.mark.parametrize("zero_weight", [True, False])
def test_outlier_groups_within_the_bound(fresh, M, log2_ratio, zero_weight):
    case = outlier_case(1024, 160, M, 300 + M, log2_ratio, zero_weight)
    y_ref, a_ref = case.reference()
    assert_close(case.run(fresh), y_ref, a_ref, f"M={M} ratio=2^{log2_ratio} zero_weight={zero_weight}")


@pytest.mark.parametrize("M", [1, 2, 8])
@pytest.mark.parametrize("prep_inline", [1, 0])
def test_outlier_groups_in_kernel_and_stand_alone_preparation(fresh, M, prep_inline):
    fd.fdqp_set_param(fresh, "prep_inline", prep_inline)
    # K = 2304 ends in a short block (one group): the fp32 path reads scales and offsets of a ragged block too
    case = outlier_case(2304, 96, M, 410 + M, 20, True, every=3)
    y_ref, a_ref = case.reference()
    assert_close(case.run(fresh), y_ref, a_ref, f"M={M} prep_inline={prep_inline}")


@pytest.mark.parametrize("M", [1, 2, 5])
def test_long_reduction_with_k_slices_and_outliers(fresh, M):
    fd.fdqp_set_param(fresh, "split_k", 2)
    case = outlier_case(8192, 64, M, 520 + M, 18, True, every=5)
    y_ref, a_ref = case.reference()
    assert_close(case.run(fresh), y_ref, a_ref, f"M={M} split_k=2")


@pytest.mark.parametrize("M", [1, 2, 4])
def test_exact_regime_with_a_huge_outlier_is_bit_equal(fresh, M):
    """d = 2^-3, m in {-1, 0, 1}, x small integers: every product and every partial sum is exact in fp32, on the
    tensor-core path and on the fp32 path alike.  One element of 2^30 per flagged group sits on a zero weight."""
    K, N = 768, 96
    w = exact_regime_weights(91, K, N)
    codes, offsets = w.codes.copy(), w.offsets.copy()
    x = f32_of(exact_regime_x(92 + M, M, K))
    for g in (0, 5, 11, 23):
        pos = g * 32 + 2 * g % 32
        x[:, pos] = 2.0 ** 30
        codes[:, pos] = 0
        offsets[:, g] = 0
    case = Case(K, N, M, 0, weights=synthgen.Q4NXWeights(codes, w.scales, offsets), x=synthgen.bf16_bits(x))
    y_ref, _ = case.reference()
    y = case.run(fresh)
    assert np.array_equal(y.astype(np.float64), y_ref)


@pytest.mark.parametrize("M", [1, 3])
def test_subnormal_activations(fresh, M):
    """bf16 subnormals (2^-133 .. 2^-126) alone and beside normal numbers: nothing is flushed to zero."""
    K, N = 512, 64
    w = synthgen.weights(700, K, N)
    scales = np.full_like(w.scales, synthgen.bf16_bits(np.float32(2.0 ** 60)))   # so that y is an ordinary fp32 number
    offsets = np.zeros_like(w.offsets)
    r = synthgen.u64(701, 0, M * K).reshape(M, K)
    bits = ((r >> np.uint64(57)) & np.uint64(0x7F)).astype(np.uint16) | ((r >> np.uint64(40)) & np.uint64(1)).astype(np.uint16) << 15
    bits[:, 256:] = 0
    bits[:, 40] = synthgen.bf16_bits(np.float32(2.0 ** -110))      # a normal number 2^16 .. 2^23 above its neighbours
    case = Case(K, N, M, 0, weights=synthgen.Q4NXWeights(w.codes, scales, offsets), x=bits.astype(np.uint16))
    y_ref, a_ref = case.reference()
    y = case.run(fresh)
    assert np.any(y != 0)
    err = np.abs(y.astype(np.float64) - y_ref)
    assert np.all(err <= 2e-3 * a_ref + 1e-30)      # the absolute term plays no part at this scale


@pytest.mark.parametrize("M", [1, 2, 8])
def test_non_finite_activations_propagate(fresh, M):
    """An infinity or a NaN in x makes the outputs of its token row non-finite (the flagged group goes through the fp32
    path, where it propagates as in any fp32 sum); the other token rows are unaffected."""
    K, N = 1024, 96
    case = Case(K, N, M, seed=800 + M)
    y_ref, a_ref = case.reference()
    for bad in (0x7F80, 0xFF80, 0x7FC0):     # +inf, -inf, NaN
        x = case.x.copy()
        x[M - 1, 333] = bad
        y = torch.empty((M, N), dtype=torch.float32, device="cuda")
        fd.fdqp_run(fresh, torch.from_numpy(x.view(np.int16)).cuda(), case.W_dev, y, M, K, N)
        torch.cuda.synchronize()
        got = y.cpu().numpy()
        assert not np.isfinite(got[M - 1]).any()
        if M > 1:
            assert_close(got[:M - 1], y_ref[:M - 1], a_ref[:M - 1], "rows beside the non-finite one")


@pytest.mark.parametrize("fmt", [fd.FMT_G64, fd.FMT_G128, fd.FMT_MXFP4])
@pytest.mark.parametrize("M", [1, 2, 6])
def test_format_variants_with_outlier_groups(fresh, fmt, M):
    import oracle
    K, N = 1024, 96
    w = synthgen.weights_fmt(930 + fmt, K, N, fmt)
    x = f32_of(synthgen.activations(931, M, K)) * 2.0 ** -9
    for g in range(0, K // 32, 2):
        x[:, g * 32 + g % 32] = 2.0 ** 12
    xb = synthgen.bf16_bits(x)
    packed = fd.q4nx_pack_fmt(fmt, w.codes, w.scales, w.offsets)
    y = torch.empty((M, N), dtype=torch.float32, device="cuda")
    fd.fdqp_run_fmt(fresh, fmt, torch.from_numpy(xb.view(np.int16)).cuda(), torch.from_numpy(packed).cuda(), y, M, K, N)
    torch.cuda.synchronize()
    assert fd.fdqp_last_status(fresh) == 0
    y_ref, a_ref = oracle.fmt_project(fmt, xb, w.codes, w.scales, w.offsets)
    assert_close(y.cpu().numpy(), y_ref, a_ref, f"fmt={fmt} M={M}")


@pytest.mark.parametrize("M", [1, 2, 3, 8])
def test_weights_that_cancel_to_zero_under_the_outlier(fresh, M):
    """The other side of the line: the weight under the outlier is zero through cancellation, d * code + m = 0 with
    m = -d * code, so d * (sum code x) and m * (sum x) both carry the outlier's magnitude and cancel.  What the library
    promises for EVERY finite input is |y - y_ref| <= 2^-17 * sum_k |x_k| (|d code_k| + |m|) + 1e-5 (the activations
    enter exactly; the factorised sums are combined in fp32); the acceptance bound follows from it unless almost all
    of that sum cancels, as it does here by construction."""
    K, N = 1024, 96
    w = synthgen.weights(990 + M, K, N)
    codes, scales, offsets = w.codes.copy(), w.scales.copy(), w.offsets.copy()
    x = f32_of(synthgen.activations(991 + M, M, K)) * 2.0 ** -9
    for g in range(0, K // 32, 4):
        pos = g * 32 + (3 * g + 2) % 32
        x[:, pos] = 2.0 ** 12
        codes[:, pos] = 8
        scales[:, g] = 0x3E00      # d = 2^-3
        offsets[:, g] = 0xBF80     # m = -1 = -d * 8
    case = Case(K, N, M, 0, weights=synthgen.Q4NXWeights(codes, scales, offsets), x=synthgen.bf16_bits(x))
    y_ref, _ = case.reference()
    y = case.run(fresh)
    d = f32_of(scales).astype(np.float64)
    m = f32_of(offsets).astype(np.float64)
    mag = np.abs(np.repeat(d, 32, axis=1) * codes) + np.abs(np.repeat(m, 32, axis=1))        # [N, K]
    big = np.abs(f32_of(case.x).astype(np.float64)) @ mag.T                                   # [M, N]
    assert np.all(np.isfinite(y))
    assert np.all(np.abs(y.astype(np.float64) - y_ref) <= 2.0 ** -17 * big + 1e-5)
