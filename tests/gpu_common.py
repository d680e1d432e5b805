"""Helpers for the GPU parity tests: move seeded inputs to the device, call the C ABI through the
binding, and compare with the CPU oracle under the acceptance bound."""
import numpy as np
import torch

import oracle
import paper_2602_06063_b200 as fd
import synthgen

REL_TOL = 2e-3   # |y - y_ref| <= REL_TOL * sum_k |x*w| + ABS_TOL, per element (the stated acceptance bound)
ABS_TOL = 1e-5

MAX_M, MAX_K, MAX_N = 512, 21504, 262144


def dev_bytes(a: np.ndarray) -> torch.Tensor:
    """numpy array -> device tensor of the same bytes."""
    return torch.from_numpy(np.ascontiguousarray(a).view(np.uint8).reshape(-1)).cuda()


class Case:
    """One projection: unpacked weights, packed bytes on host and device, activations."""

    def __init__(self, K, N, M, seed, amp=1.0, weights=None, x=None):
        self.K, self.N, self.M = K, N, M
        self.w = weights if weights is not None else synthgen.weights(seed, K, N)
        self.x = x if x is not None else synthgen.activations(seed, M, K, amp)
        self.packed = fd.q4nx_pack(self.w.codes, self.w.scales, self.w.offsets)
        self.W_dev = dev_bytes(self.packed)
        self.x_dev = dev_bytes(self.x)

    def run(self, ctx, M=None, x_dev=None):
        M = self.M if M is None else M
        y = torch.full((M, self.N), float("nan"), dtype=torch.float32, device="cuda")
        fd.fdqp_run(ctx, self.x_dev if x_dev is None else x_dev, self.W_dev, y, M, self.K, self.N)
        torch.cuda.synchronize()
        assert fd.fdqp_last_status(ctx) == 0
        return y.cpu().numpy()

    def reference(self, n0=0, n1=None, nthreads=None):
        nthreads = nthreads or min(16, oracle.max_threads())
        return oracle.project(self.x, self.w.codes, self.w.scales, self.w.offsets, n0=n0, n1=n1, nthreads=nthreads)


def assert_close(y, y_ref, a_ref, what=""):
    err = np.abs(y.astype(np.float64) - y_ref)
    bound = REL_TOL * a_ref + ABS_TOL
    bad = err > bound
    assert np.all(np.isfinite(y)), f"{what}: non-finite output"
    if bad.any():
        idx = np.argwhere(bad)[0]
        raise AssertionError(f"{what}: {bad.sum()} of {bad.size} outside the bound; first at {tuple(idx)}: "
                             f"got {y[tuple(idx)]!r} want {y_ref[tuple(idx)]!r} bound {bound[tuple(idx)]!r}")
    return float((err / (a_ref + 1e-30)).max())


def exact_regime_weights(seed, K, N):
    """Weights for which any fp32 summation order is exact: d = 2^-3, m in {-1, 0, 1}."""
    r = synthgen.u64(seed, 0, N * K).reshape(N, K)
    codes = (r >> np.uint64(60)).astype(np.uint8)
    rm = synthgen.u64(seed, 1, N * (K // 32)).reshape(N, K // 32)
    m = ((rm >> np.uint64(62)).astype(np.int64) % 3 - 1).astype(np.float32)
    return synthgen.Q4NXWeights(codes, np.full((N, K // 32), 0x3E00, np.uint16), synthgen.bf16_bits(m))


def exact_regime_x(seed, M, K):
    """Small-integer activations in {-2..2}."""
    r = synthgen.u64(seed, 2, M * K).reshape(M, K)
    return synthgen.bf16_bits(((r >> np.uint64(61)).astype(np.int64) % 5 - 2).astype(np.float32))
