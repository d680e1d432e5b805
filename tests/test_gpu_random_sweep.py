"""A seeded random sweep of shapes, token counts and launch parameters through every projection entry point, each case
checked against the CPU oracle under the acceptance bound (the hand-picked cases elsewhere cannot cover every way a
range of blocks can be cut)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2602_06063_b200 as fd
import synthgen
from gpu_common import ABS_TOL, REL_TOL, Case, assert_close, dev_bytes

pytestmark = pytest.mark.gpu

PARAMS = ("strip_aligned", "split_k", "blocks_per_warp", "path", "prefill_split_k", "prefill_pair")


@pytest.fixture(scope="module")
def ctx():
    h = fd.fdqp_create(0, 600, 8192, 16384)
    yield h
    torch.cuda.synchronize()
    fd.fdqp_destroy(h)


def one_case(ctx, rng):
    kind = rng.choice(["run", "fmt", "epi", "norm", "host"])
    M = int(rng.choice([1, 1, 2, 3, 4, 5, 7, 8, 9, 12, 17, 40, 130, 300]))
    K = int(rng.integers(1, 129)) * 32 if rng.random() < 0.7 else int(rng.integers(1, 25)) * 256
    N = int(rng.integers(1, 200)) * 32
    if kind == "fmt":
        K = max(256, (K // 256) * 256)
    params = {}
    if rng.random() < 0.3:
        params["strip_aligned"] = int(rng.integers(0, 2))
    if rng.random() < 0.2 and M <= 8:
        params["split_k"] = int(rng.choice([2, 4]))
    if rng.random() < 0.2:
        params["blocks_per_warp"] = int(rng.choice([2, 4]))
    if M >= 9 and K >= 256 and rng.random() < 0.5:
        params["path"] = int(rng.choice([2, 3]))
    if M >= 9 and rng.random() < 0.3:
        params["prefill_split_k"] = int(rng.integers(1, 5))
    if M >= 9 and rng.random() < 0.3:
        params["prefill_pair"] = int(rng.integers(0, 2))
    for k in PARAMS:
        fd.fdqp_set_param(ctx, k, params.get(k, -1))
    seed = int(rng.integers(1, 1 << 30))
    what = f"{kind} M={M} K={K} N={N} {params} seed={seed}"
    if kind == "fmt":
        fmt = int(rng.choice([1, 2, 3]))
        w = synthgen.weights_fmt(seed, K, N, fmt)
        x = synthgen.activations(seed + 1, M, K)
        W = dev_bytes(fd.q4nx_pack_fmt(fmt, w.codes, w.scales, w.offsets))
        y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        fd.fdqp_run_fmt(ctx, fmt, dev_bytes(x), W, y, M, K, N)
        torch.cuda.synchronize()
        y_ref, a_ref = oracle.fmt_project(fmt, x, w.codes, w.scales, w.offsets, nthreads=8)
        assert_close(y.cpu().numpy(), y_ref, a_ref, what)
        return
    c = Case(K, N, M, seed=seed)
    y_ref, a_ref = c.reference()
    if kind == "run":
        assert_close(c.run(ctx), y_ref, a_ref, what)
    elif kind == "host":
        xh = torch.from_numpy(c.x.view(np.int16)).pin_memory()
        yh = torch.full((M, N), float("nan"), dtype=torch.float32).pin_memory()
        fd.fdqp_run_host(ctx, xh, c.W_dev, yh, M, K, N)
        assert_close(yh.numpy(), y_ref, a_ref, what)
    elif kind == "epi":
        out = torch.zeros((M, N), dtype=torch.int16, device="cuda")
        fd.fdqp_run_epilogue(ctx, c.x_dev, c.W_dev, out, fd.EPI_BF16, M, K, N)
        torch.cuda.synchronize()
        got = synthgen.bf16_to_f32(out.cpu().numpy().view(np.uint16)).astype(np.float64)
        assert np.all(np.abs(got - y_ref) <= REL_TOL * a_ref + ABS_TOL + 2.0 ** -8 * np.abs(y_ref)), what
    else:
        gamma = synthgen.bf16_bits((0.25 * synthgen.bf16_to_f32(synthgen.activations(seed + 2, 1, K))[0]).astype(np.float32))
        res = synthgen.activations(seed + 3, M, K)
        h = torch.zeros((M, K), dtype=torch.int16, device="cuda")
        out = torch.zeros((M, N), dtype=torch.float32, device="cuda")
        fd.fdqp_run_add_rmsnorm_epilogue(ctx, c.x_dev, dev_bytes(res).view(torch.int16), h,
                                         torch.from_numpy(gamma.view(np.int16)).cuda(), 1e-6, c.W_dev, out, fd.EPI_NONE, M, K, N)
        torch.cuda.synchronize()
        h_ref = oracle.add_residual(c.x, res)
        assert np.array_equal(h.cpu().numpy().view(np.uint16), h_ref), what
        xn = oracle.rmsnorm(h_ref, gamma, 1e-6)
        yr, ar = oracle.project(xn, c.w.codes, c.w.scales, c.w.offsets, nthreads=8)
        assert_close(out.cpu().numpy(), yr, ar, what)
    assert fd.fdqp_last_status(ctx) == 0, what


@pytest.mark.parametrize("seed", [11, 12, 13, 14])
def test_random_sweep(ctx, seed):
    rng = np.random.default_rng(seed)
    try:
        for _ in range(25):
            one_case(ctx, rng)
    finally:
        for k in PARAMS:
            fd.fdqp_set_param(ctx, k, -1)
