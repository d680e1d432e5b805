"""The projection entry point for callers that cannot allocate device memory (fdqp_run_noalloc).

Some users of this library run where cudaMalloc is off limits once serving has started -- all device memory
belongs to their own pool, or an allocation's device-wide synchronisation would break a latency budget.  For
them the library offers the GEMV kernel with its scratch in a fixed array of the library image.  This test calls
that entry point through the C ABI, twice in a row on the same stream (the second call finds the scratch as the
first one left it), and checks each result against the CPU oracle within the tolerance the parity tests use, and
against the ordinary fdqp_run; it also checks that the calls leave the device's free memory as they found it and
that the entry point's own status word stays clear.  It lives in a file pytest collects last so that a failure
here cannot hide other results.
"""
import numpy as np
import pytest
import torch

import paper_2602_06063_b200 as fd
from gpu_common import Case, assert_close

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("K,N,M", [
    (2560, 2080, 1), (4352, 1056, 3),      # strips shared between CTAs in both
    (2560, 20480, 1), (2560, 20480, 8),    # Gemma3-4B gate|up at full size
])
def test_noalloc_matches_oracle_twice_in_a_row(K, N, M):
    case = Case(K, N, M, seed=4242 + M)
    ctx = fd.fdqp_create(0, 8, K, N)
    try:
        want = case.run(ctx)
    finally:
        torch.cuda.synchronize()
        fd.fdqp_destroy(ctx)
    y_ref, a_ref = case.reference()
    lib = fd.load_library()
    stream = torch.cuda.current_stream().cuda_stream
    # every buffer exists before the calls; the first call on a device also does the entry point's set-up
    outs = [torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda") for _ in range(3)]
    rc = lib.fdqp_run_noalloc(case.x_dev.data_ptr(), case.W_dev.data_ptr(), outs[2].data_ptr(), M, K, N, stream)
    assert rc == 0, fd.fdqp_status_string(rc)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for y in outs[:2]:
        rc = lib.fdqp_run_noalloc(case.x_dev.data_ptr(), case.W_dev.data_ptr(), y.data_ptr(), M, K, N, stream)
        assert rc == 0, fd.fdqp_status_string(rc)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "fdqp_run_noalloc changed the device's free memory"
    assert fd.fdqp_noalloc_last_status() == 0
    for y in outs:
        got = y.cpu().numpy()
        assert_close(got, y_ref, a_ref, f"noalloc K={K} N={N} M={M}")
        assert np.array_equal(got, want)      # same kernel, same plan, same summation order as fdqp_run
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
    assert lib.fdqp_run_noalloc(xp, wp, yp, 1, (1 << 20) + 32, 64, s) == 4  # K beyond any shared-memory budget
    assert lib.fdqp_run_noalloc(xp, wp, yp, 1, 250, 64, s) == 2
    assert lib.fdqp_run_noalloc(None, wp, yp, 1, 256, 64, s) == 1
    assert lib.fdqp_run_noalloc(xp + 2, wp, yp, 1, 256, 64, s) == 3
    torch.cuda.synchronize()
    assert fd.fdqp_noalloc_last_status() == 0
