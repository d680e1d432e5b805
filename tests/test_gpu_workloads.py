"""GPU parity on the full workload shapes (the Gemma3 projections the benchmark times), in the launch
configuration the benchmark uses (automatic parameters).  Outputs the oracle can afford are compared in
full; the prefill-sized case is compared on sampled output columns."""
import numpy as np
import pytest
import torch

import oracle
import paper_2602_06063_b200 as fd
import synthgen
from gpu_common import MAX_K, MAX_M, MAX_N, Case, assert_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    h = fd.fdqp_create(0, MAX_M, MAX_K, MAX_N)
    yield h
    torch.cuda.synchronize()
    fd.fdqp_destroy(h)


def test_gemma3_1b_gate(ctx):
    _, K, N, seed = synthgen.GEMMA3_1B_GATE
    case = Case(K, N, 1, seed)
    y_ref, a_ref = case.reference()
    worst = assert_close(case.run(ctx), y_ref, a_ref, "1B gate")
    assert worst < 1e-4


@pytest.mark.parametrize("name,K,N,seed", synthgen.GEMMA3_4B_LAYER)
def test_gemma3_4b_layer_projection(ctx, name, K, N, seed):
    case = Case(K, N, 1, seed)
    y_ref, a_ref = case.reference()
    assert_close(case.run(ctx), y_ref, a_ref, name)


def test_gemma3_12b_gate_up(ctx):
    _, K, N, seed = synthgen.GEMMA3_12B_GATE_UP
    w = synthgen.weights(seed, K, N)
    x = synthgen.activations(seed, 8, K)
    base = Case(K, N, 8, seed, weights=w, x=x)
    y_ref, a_ref = base.reference()
    for M in (1, 2, 4, 8):
        y = base.run(ctx, M=M)
        assert_close(y, y_ref[:M], a_ref[:M], f"12B gate|up M={M}")


def test_gemma3_27b_down(ctx):
    _, K, N, seed = synthgen.GEMMA3_27B_DOWN
    w = synthgen.weights(seed, K, N)
    x = synthgen.activations(seed, 8, K, amp=K ** -0.5)
    base = Case(K, N, 8, seed, weights=w, x=x)
    y_ref, a_ref = base.reference()
    for M in (1, 4, 8):
        y = base.run(ctx, M=M)
        assert_close(y, y_ref[:M], a_ref[:M], f"27B down M={M}")


def test_gemma3_4b_lm_head_decode_and_prefill(ctx):
    _, K, N, seed = synthgen.GEMMA3_4B_LM_HEAD
    w = synthgen.weights(seed, K, N)
    x = synthgen.activations(seed, 512, K)
    base = Case(K, N, 512, seed, weights=w, x=x)
    # decode, M = 1: every output
    y = base.run(ctx, M=1)
    y_ref, a_ref = oracle.project(x[:1], w.codes, w.scales, w.offsets, nthreads=min(32, oracle.max_threads()))
    assert_close(y, y_ref, a_ref, "LM head M=1")
    # prefill chunk, M = 512: 64 strips spread over N (first and last included), all 512 rows
    y = base.run(ctx, M=512)
    strips = np.unique(np.linspace(0, N // 32 - 1, 64).astype(np.int64))
    for s in strips:
        n0 = int(s) * 32
        y_ref, a_ref = oracle.project(x, w.codes, w.scales, w.offsets, n0=n0, n1=n0 + 32,
                                      nthreads=min(32, oracle.max_threads()))
        assert_close(y[:, n0:n0 + 32], y_ref, a_ref, f"LM head M=512 strip {s}")
    assert np.all(np.isfinite(y))


@pytest.mark.parametrize("M,form", [(48, "three CTAs per SM"), (128, "two CTAs per SM")])
def test_gemma3_4b_lm_head_small_prefill_chunks(ctx, M, form):
    # the one-SM forms of the tensor-core kernel at full size, in the configuration the dispatch picks by itself:
    # 32 strips spread over N (first and last included), all M rows
    _, K, N, seed = synthgen.GEMMA3_4B_LM_HEAD
    w = synthgen.weights(seed, K, N)
    x = synthgen.activations(seed + 1, M, K)
    base = Case(K, N, M, seed, weights=w, x=x)
    assert form in fd.fdqp_describe(ctx, M, K, N)
    y = base.run(ctx)
    assert np.all(np.isfinite(y))
    for s in np.unique(np.linspace(0, N // 32 - 1, 32).astype(np.int64)):
        n0 = int(s) * 32
        y_ref, a_ref = oracle.project(x, w.codes, w.scales, w.offsets, n0=n0, n1=n0 + 32,
                                      nthreads=min(32, oracle.max_threads()))
        assert_close(y[:, n0:n0 + 32], y_ref, a_ref, f"LM head M={M} strip {s}")


def test_read_stream_reference_runs_and_reports_no_error():
    """The measurement aid reads whole 40 KB chunks of a buffer through the projection kernels' bulk-copy ring; sizes
    below a chunk read nothing; a misaligned buffer is refused."""
    ctx = fd.fdqp_create(0, 8, 256, 256)
    try:
        buf = torch.zeros(64 * 1024 * 1024 + 48, dtype=torch.uint8, device="cuda")
        for nbytes in (0, 16, 40960, 40960 * 3 + 16, 64 * 1024 * 1024):
            fd.fdqp_stream_read(ctx, buf, nbytes)
        torch.cuda.synchronize()
        assert fd.fdqp_last_status(ctx) == 0
        with pytest.raises(fd.FdqpError):
            fd.fdqp_stream_read(ctx, buf[8:], 40960)
    finally:
        torch.cuda.synchronize()
        fd.fdqp_destroy(ctx)
