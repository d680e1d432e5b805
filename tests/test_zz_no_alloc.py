"""The projection entry point for callers that cannot allocate device memory (fdqp_run_noalloc).

Some users of this library run where cudaMalloc is off limits once serving has started -- all device memory
belongs to their own pool, or an allocation's device-wide synchronisation would break a latency budget.  For
them the library offers the GEMV kernel with its scratch in a fixed array of the library image.  This test calls
that entry point through the C ABI, twice in a row on the same stream (the second call finds the scratch as the
first one left it), and checks each result against the ordinary fdqp_run within the tolerance the parity tests
use.  It lives in a file pytest collects last so that a failure here cannot hide other results.
"""
import numpy as np
import pytest
import torch

import paper_2602_06063_b200 as fd
from gpu_common import ABS_TOL, REL_TOL, Case

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("K,N,M", [(2560, 2080, 1), (4352, 1056, 3)])   # strips shared between CTAs in both
def test_noalloc_matches_run_twice_in_a_row(K, N, M):
    case = Case(K, N, M, seed=4242 + M)
    ctx = fd.fdqp_create(0, 8, K, N)
    try:
        want = case.run(ctx)
    finally:
        torch.cuda.synchronize()
        fd.fdqp_destroy(ctx)
    _, a_ref = case.reference()
    lib = fd.load_library()
    stream = torch.cuda.current_stream().cuda_stream
    outs = []
    for _ in range(2):
        y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        rc = lib.fdqp_run_noalloc(case.x_dev.data_ptr(), case.W_dev.data_ptr(), y.data_ptr(), M, K, N, stream)
        assert rc == 0, fd.fdqp_status_string(rc)
        outs.append(y)
    torch.cuda.synchronize()
    for y in outs:
        got = y.cpu().numpy()
        assert np.all(np.isfinite(got))
        assert np.all(np.abs(got.astype(np.float64) - want) <= REL_TOL * a_ref + ABS_TOL)
    assert np.array_equal(outs[0].cpu().numpy(), outs[1].cpu().numpy())


def test_noalloc_rejects_what_it_cannot_hold():
    lib = fd.load_library()
    case = Case(256, 64, 1, seed=7)
    y = torch.zeros((1, 64), dtype=torch.float32, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    xp, wp, yp = case.x_dev.data_ptr(), case.W_dev.data_ptr(), y.data_ptr()
    assert lib.fdqp_run_noalloc(xp, wp, yp, 9, 256, 64, s) == 4            # more than 8 token rows
    assert lib.fdqp_run_noalloc(xp, wp, yp, 1, 256, 262144 + 32, s) == 4   # more strips than arrival counters
    assert lib.fdqp_run_noalloc(xp, wp, yp, 8, 21504, 64, s) == 4          # activations would need a K split
    assert lib.fdqp_run_noalloc(xp, wp, yp, 1, 250, 64, s) == 2
    assert lib.fdqp_run_noalloc(None, wp, yp, 1, 256, 64, s) == 1
    assert lib.fdqp_run_noalloc(xp + 2, wp, yp, 1, 256, 64, s) == 3
    torch.cuda.synchronize()
