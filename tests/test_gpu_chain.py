"""GPU parity of fdqp_run_chain -- several projections walked by one persistent launch -- against the CPU oracle.

Independent steps are checked one by one against the oracle's projection of the same inputs.  Dependent steps (the MLP
block of a decoder layer: residual addition + RMS normalisation -> gate|up with the gated-GELU epilogue -> down) are
checked stage by stage against the oracle chain add_residual -> rmsnorm -> project -> geglu -> project: the residual
stream bit for bit, the activation under the bound that follows from the projection's acceptance bound, and the final
projection against the oracle's projection of the activation the GPU really handed on."""
import numpy as np
import pytest
import torch

import oracle
import paper_2602_06063_b200 as fd
import synthgen
from gpu_common import ABS_TOL, REL_TOL, Case, assert_close, dev_bytes
from test_gpu_epilogue import geglu_bound

pytestmark = pytest.mark.gpu

PARAMS = ("stages", "l2_evict_first", "strip_aligned", "chain_launch", "chain_steps", "chain_wide", "chain_dependent", "blocks_per_warp")


@pytest.fixture(scope="module")
def ctx():
    h = fd.fdqp_create(0, 8, 21504, 32768)
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


def run_chain(ctx, steps, M):
    fd.fdqp_run_chain(ctx, steps, M)
    torch.cuda.synchronize()
    assert fd.fdqp_last_status(ctx) == 0


SMALL = [(1152, 288), (2560, 512), (2048, 640), (4352, 1056), (10240, 320), (32, 32), (544, 2080)]


@pytest.mark.parametrize("M", [1, 2, 3, 8])
def test_independent_steps_match_oracle_and_reruns_are_bit_identical(fresh, M):
    cases = [Case(K, N, M, seed=7000 + 10 * i + M) for i, (K, N) in enumerate(SMALL)]
    outs = [torch.full((M, c.N), float("nan"), dtype=torch.float32, device="cuda") for c in cases]
    steps = fd.make_chain([fd.chain_step(c.x_dev, c.W_dev, o, c.K, c.N) for c, o in zip(cases, outs)])
    before = fd.fdqp_launch_count(fresh)
    run_chain(fresh, steps, M)
    assert fd.fdqp_launch_count(fresh) - before == 1            # one launch for the whole chain
    first = [o.cpu().numpy().copy() for o in outs]
    for c, y in zip(cases, first):
        y_ref, a_ref = c.reference()
        assert_close(y, y_ref, a_ref, f"chain step K={c.K} N={c.N} M={M}")
    for o in outs:
        o.fill_(float("nan"))
    run_chain(fresh, steps, M)
    for y, o in zip(first, outs):
        assert np.array_equal(y, o.cpu().numpy())


@pytest.mark.parametrize("params", [{"strip_aligned": 0}, {"strip_aligned": 1}, {"stages": 2}, {"chain_launch": 0},
                                    {"chain_launch": 2}, {"chain_launch": 3}, {"chain_steps": 3}, {"l2_evict_first": 0}, {"chain_wide": 0}, {"blocks_per_warp": 2}, {"blocks_per_warp": 4}, {"blocks_per_warp": 4, "chain_wide": 0}])
def test_launch_parameters_do_not_change_the_result(fresh, params):
    M = 2
    cases = [Case(K, N, M, seed=7100 + i) for i, (K, N) in enumerate(SMALL[:5])]
    outs = [torch.zeros((M, c.N), dtype=torch.float32, device="cuda") for c in cases]
    steps = fd.make_chain([fd.chain_step(c.x_dev, c.W_dev, o, c.K, c.N) for c, o in zip(cases, outs)])
    for k, v in params.items():
        fd.fdqp_set_param(fresh, k, v)
    before = fd.fdqp_launch_count(fresh)
    run_chain(fresh, steps, M)
    assert fd.fdqp_launch_count(fresh) - before == (2 if "chain_steps" in params else 1)
    for c, o in zip(cases, outs):
        y_ref, a_ref = c.reference()
        assert_close(o.cpu().numpy(), y_ref, a_ref, f"{params} K={c.K} N={c.N}")


def test_decoder_layer_shapes_at_full_size(fresh):
    """The four calls of a Gemma3-4B decoder layer at M = 1 (q|k|v, o, gate|up, down) as one chain."""
    M = 1
    shapes = [(2560, 4096, 1), (2048, 2560, 4), (2560, 20480, 5), (10240, 2560, 7)]
    cases = [Case(K, N, M, seed) for K, N, seed in shapes]
    outs = [torch.full((M, c.N), float("nan"), dtype=torch.float32, device="cuda") for c in cases]
    run_chain(fresh, [fd.chain_step(c.x_dev, c.W_dev, o, c.K, c.N) for c, o in zip(cases, outs)], M)
    for c, o in zip(cases, outs):
        y_ref, a_ref = c.reference()
        assert_close(o.cpu().numpy(), y_ref, a_ref, f"layer call K={c.K} N={c.N}")


def interleave_gate_up(w_gate, w_up):
    """Rows of the fused gate|up matrix in the order the gated-GELU epilogue expects: sixteen gate rows, then the
    sixteen up rows of the same outputs."""
    n = w_gate.codes.shape[0]
    order = np.arange(2 * n).reshape(n // 16, 2, 16)
    order[:, 0, :] = np.arange(n).reshape(n // 16, 16)
    order[:, 1, :] = n + np.arange(n).reshape(n // 16, 16)
    order = order.reshape(-1)
    cat = lambda a, b: np.concatenate([a, b])[order]
    return synthgen.Q4NXWeights(cat(w_gate.codes, w_up.codes), cat(w_gate.scales, w_up.scales), cat(w_gate.offsets, w_up.offsets))


@pytest.mark.parametrize("in_kernel", [1, 0])
@pytest.mark.parametrize("D,inner,M", [(1024, 1536, 1), (1024, 1536, 2), (1024, 1536, 8), (1152, 512, 3),
                                       (2560, 10240, 1), (2560, 10240, 2), (2560, 10240, 8)])
def test_mlp_block_as_a_dependent_chain(fresh, D, inner, M, in_kernel):
    """normalise(x + residual) -> gate|up -> gated GELU -> down.  in_kernel = 1: both steps in ONE launch, the second
    waits on the first's completion counter; 0 (the library's default): the dependent step begins a new launch."""
    fd.fdqp_set_param(fresh, "chain_dependent", in_kernel)
    seed = 7300 + D + M
    w_gu = interleave_gate_up(synthgen.weights(seed, D, inner), synthgen.weights(seed + 1, D, inner))
    w_dn = synthgen.weights(seed + 2, inner, D, sigma_d=0.002, sigma_m=0.001)
    x = synthgen.activations(seed + 3, M, D, 2.0)
    res = synthgen.activations(seed + 4, M, D, 1.5)
    gamma = synthgen.bf16_bits((0.25 * synthgen.bf16_to_f32(synthgen.activations(seed + 5, 1, D))[0]).astype(np.float32))
    eps = 1e-6
    W_gu = dev_bytes(fd.q4nx_pack(w_gu.codes, w_gu.scales, w_gu.offsets))
    W_dn = dev_bytes(fd.q4nx_pack(w_dn.codes, w_dn.scales, w_dn.offsets))
    x_dev, res_dev, gamma_dev = dev_bytes(x), dev_bytes(res), dev_bytes(gamma)
    h_dev = torch.full((M, D), 0x7FC0, dtype=torch.int16, device="cuda")
    act_dev = torch.full((M, inner), 0x7FC0, dtype=torch.int16, device="cuda")
    y_dev = torch.full((M, D), float("nan"), dtype=torch.float32, device="cuda")
    steps = fd.make_chain([
        fd.chain_step(x_dev, W_gu, act_dev, D, 2 * inner, fd.EPI_GEGLU_BF16, False, gamma_dev, eps, res_dev, h_dev),
        fd.chain_step(act_dev, W_dn, y_dev, inner, D, fd.EPI_NONE, True),
    ])
    before = fd.fdqp_launch_count(fresh)
    run_chain(fresh, steps, M)
    launches = fd.fdqp_launch_count(fresh) - before
    assert launches == 1 if in_kernel else launches >= 2
    # the oracle chain
    h_ref = oracle.add_residual(x, res)
    assert np.array_equal(h_dev.cpu().numpy().view(np.uint16), h_ref)
    x_n = oracle.rmsnorm(h_ref, gamma, eps)
    g_ref, g_abs = oracle.project(x_n, w_gu.codes, w_gu.scales, w_gu.offsets, nthreads=8)
    act_ref, _ = oracle.geglu(g_ref)
    act_bits = act_dev.cpu().numpy().view(np.uint16)
    act = synthgen.bf16_to_f32(act_bits).astype(np.float64)
    assert np.all(np.isfinite(act))
    assert np.all(np.abs(act - act_ref) <= geglu_bound(g_ref, g_abs))
    y_ref, y_abs = oracle.project(act_bits, w_dn.codes, w_dn.scales, w_dn.offsets, nthreads=8)
    y = y_dev.cpu().numpy()
    assert_close(y, y_ref, y_abs, f"down projection of the chain D={D} M={M}")
    # the same chain again, and as separate calls of the library: bit-identical reruns, agreement within the bound
    y_dev.fill_(float("nan"))
    act_dev.fill_(0x7FC0)
    run_chain(fresh, steps, M)
    assert np.array_equal(y, y_dev.cpu().numpy())
    assert np.array_equal(act_bits, act_dev.cpu().numpy().view(np.uint16))


def test_dependent_chain_across_launches(fresh):
    """Six dependent projections with the bf16 epilogue, at most four steps per launch: the dependency inside a launch
    is the counter, across launches the stream order."""
    M, D = 2, 512
    fd.fdqp_set_param(fresh, "chain_steps", 4)
    fd.fdqp_set_param(fresh, "chain_dependent", 1)
    ws = [synthgen.weights(7500 + i, D, D, sigma_d=0.002, sigma_m=0.001) for i in range(6)]
    Ws = [dev_bytes(fd.q4nx_pack(w.codes, w.scales, w.offsets)) for w in ws]
    x0 = synthgen.activations(7510, M, D)
    bufs = [dev_bytes(x0)] + [torch.full((M, D), 0x7FC0, dtype=torch.int16, device="cuda") for _ in range(6)]
    steps = [fd.chain_step(bufs[i], Ws[i], bufs[i + 1], D, D, fd.EPI_BF16, i > 0) for i in range(6)]
    before = fd.fdqp_launch_count(fresh)
    run_chain(fresh, steps, M)
    assert fd.fdqp_launch_count(fresh) - before == 2
    prev = x0
    for i in range(6):
        got_bits = bufs[i + 1].cpu().numpy().view(np.uint16).reshape(M, D)
        y_ref, a_ref = oracle.project(prev, ws[i].codes, ws[i].scales, ws[i].offsets)
        got = synthgen.bf16_to_f32(got_bits).astype(np.float64)
        assert np.all(np.abs(got - y_ref) <= REL_TOL * a_ref + ABS_TOL + 2.0 ** -8 * np.abs(y_ref)), f"step {i}"
        prev = got_bits


def test_chain_with_flagged_groups(fresh):
    """Wide-range groups (an outlier over a zero weight beside tiny values) inside a chain: the fp32 path of flagged
    groups is part of the chained kernel too."""
    M, K, N = 1, 1024, 160
    w = synthgen.weights(7600, K, N)
    codes, offsets = w.codes.copy(), w.offsets.copy()
    x = synthgen.bf16_to_f32(synthgen.activations(7601, M, K)) * 2.0 ** -20
    for g in range(0, K // 32, 2):
        pos = g * 32 + (5 * g + 1) % 32
        x[:, pos] = 2.0 ** 12
        codes[:, pos] = 0
        offsets[:, g] = 0
    case = Case(K, N, M, 0, weights=synthgen.Q4NXWeights(codes, w.scales, offsets), x=synthgen.bf16_bits(x))
    plain = Case(2560, 512, M, seed=7602)
    o1 = torch.zeros((M, N), dtype=torch.float32, device="cuda")
    o2 = torch.zeros((M, plain.N), dtype=torch.float32, device="cuda")
    run_chain(fresh, [fd.chain_step(plain.x_dev, plain.W_dev, o2, plain.K, plain.N),
                      fd.chain_step(case.x_dev, case.W_dev, o1, K, N)], M)
    y_ref, a_ref = case.reference()
    assert_close(o1.cpu().numpy(), y_ref, a_ref, "flagged groups in a chain")
    y_ref, a_ref = plain.reference()
    assert_close(o2.cpu().numpy(), y_ref, a_ref, "the step beside it")


def test_chain_argument_errors(fresh):
    case = Case(256, 64, 1, seed=9)
    out = torch.zeros((1, 64), dtype=torch.float32, device="cuda")
    lib = fd.load_library()
    s = torch.cuda.current_stream().cuda_stream

    def call(steps, M=1):
        arr = fd.make_chain(steps)
        import ctypes
        return lib.fdqp_run_chain(fresh, ctypes.cast(arr, ctypes.c_void_p), len(arr), M, s)

    ok = fd.chain_step(case.x_dev, case.W_dev, out, 256, 64)
    assert call([ok]) == 0
    assert call([fd.chain_step(case.x_dev, case.W_dev, out, 256, 64, depends_on_previous=True)]) == 1   # nothing before it
    assert call([ok], M=9) == 4
    assert call([ok], M=0) == 2
    assert call([fd.chain_step(None, case.W_dev, out, 256, 64)]) == 1
    assert call([fd.chain_step(case.x_dev.data_ptr() + 2, case.W_dev, out, 256, 64)]) == 3
    assert call([fd.chain_step(case.x_dev, case.W_dev, out, 250, 64)]) == 2
    assert call([fd.chain_step(case.x_dev, case.W_dev, out, 256, 64, epilogue=7)]) == 1
    assert call([fd.chain_step(case.x_dev, case.W_dev, out, 256, 64, residual_bf16=case.x_dev)]) == 1  # residual without gamma
    assert lib.fdqp_run_chain(fresh, None, 1, 1, s) == 1
    torch.cuda.synchronize()
    assert fd.fdqp_last_status(fresh) == 0


@pytest.mark.parametrize("M", [1, 4])
def test_chain_through_two_layers_and_the_full_size_lm_head(M):
    """Nine steps in one launch at BASELINE sizes: the four calls of a Gemma3-4B layer twice (seeded weights of two
    different layers) and the tied LM head (K = 2560, N = 262144, seed 17).  Every output of the layer calls and a
    sample of strips spread over the LM head's outputs are checked against the oracle."""
    _, hk, hn, hseed = synthgen.GEMMA3_4B_LM_HEAD
    ctx = fd.fdqp_create(0, 8, 10240, hn)
    try:
        shapes = [(2560, 4096), (2048, 2560), (2560, 20480), (10240, 2560)]
        cases = [Case(K, N, M, seed=7700 + 10 * layer + j) for layer in range(2) for j, (K, N) in enumerate(shapes)]
        head = Case(hk, hn, M, hseed)
        outs = [torch.full((M, c.N), float("nan"), dtype=torch.float32, device="cuda") for c in cases + [head]]
        steps = [fd.chain_step(c.x_dev, c.W_dev, o, c.K, c.N) for c, o in zip(cases + [head], outs)]
        before = fd.fdqp_launch_count(ctx)
        fd.fdqp_run_chain(ctx, steps, M)
        torch.cuda.synchronize()
        assert fd.fdqp_last_status(ctx) == 0
        assert fd.fdqp_launch_count(ctx) - before == 1
        for c, o in zip(cases, outs):
            y_ref, a_ref = c.reference()
            assert_close(o.cpu().numpy(), y_ref, a_ref, f"layer call K={c.K} N={c.N} M={M}")
        y = outs[-1].cpu().numpy()
        assert np.all(np.isfinite(y))
        for n0 in (0, 4096, 99968, 131072 - 64, 200000 - 200000 % 32, hn - 128):
            y_ref, a_ref = head.reference(n0=n0, n1=n0 + 128)
            assert_close(y[:, n0:n0 + 128], y_ref, a_ref, f"LM head columns {n0}.. M={M}")
    finally:
        torch.cuda.synchronize()
        fd.fdqp_destroy(ctx)


def test_a_whole_token_of_projections_is_one_launch_and_large_chains_are_cut(fresh):
    """137 steps (34 layers of four projections and a head, here with small shapes) run as one launch; a chain whose
    steps together have more strips than the context has arrival counters is cut into shorter launches by the library."""
    M = 1
    shapes = [(256, 416), (416, 256), (256, 2048), (1024, 256)]
    cases = [Case(K, N, M, seed=4100 + i) for i, (K, N) in enumerate(shapes)]
    head = Case(256, 8192, M, seed=4105)
    steps, outs, refs = [], [], []
    for l in range(34):
        for c in cases:
            y = torch.empty((M, c.N), dtype=torch.float32, device="cuda")
            steps.append(fd.chain_step(c.x_dev, c.W_dev, y, c.K, c.N))
            outs.append(y)
            refs.append(c)
    y = torch.empty((M, head.N), dtype=torch.float32, device="cuda")
    steps.append(fd.chain_step(head.x_dev, head.W_dev, y, head.K, head.N))
    outs.append(y)
    refs.append(head)
    before = fd.fdqp_launch_count(fresh)
    fd.fdqp_run_chain(fresh, fd.make_chain(steps), M)
    torch.cuda.synchronize()
    assert fd.fdqp_last_status(fresh) == 0
    assert fd.fdqp_launch_count(fresh) - before == 1
    for y, c in zip(outs, refs):
        y_ref, a_ref = c.reference()
        assert_close(y.cpu().numpy(), y_ref, a_ref, f"K={c.K} N={c.N}")
    # 80 steps of 1024 strips each: more strips than arrival counters (65536) -> two launches, same results
    big = Case(64, 32768, M, seed=4110)
    ys = [torch.empty((M, big.N), dtype=torch.float32, device="cuda") for _ in range(80)]
    before = fd.fdqp_launch_count(fresh)
    fd.fdqp_run_chain(fresh, fd.make_chain([fd.chain_step(big.x_dev, big.W_dev, y, big.K, big.N) for y in ys]), M)
    torch.cuda.synchronize()
    assert fd.fdqp_last_status(fresh) == 0
    assert fd.fdqp_launch_count(fresh) - before == 2
    y_ref, a_ref = big.reference()
    for y in (ys[0], ys[39], ys[40], ys[79]):
        assert_close(y.cpu().numpy(), y_ref, a_ref, "cut chain")


def test_dependent_steps_begin_new_launches_by_default(fresh):
    """q, k, v (independent) -> o (depends) -> gate|up (depends, normalised, gated GELU) -> down (depends): by default the
    three independent steps are one launch and every dependent step a launch (or a single call) of its own."""
    M, D = 2, 512
    shapes = [(D, 512), (D, 256), (D, 256), (512, D), (D, 2048), (1024, D)]
    ws = [synthgen.weights(7700 + i, K, N, sigma_d=0.002, sigma_m=0.001) for i, (K, N) in enumerate(shapes)]
    ws[4] = interleave_gate_up(synthgen.weights(7710, D, 1024), synthgen.weights(7711, D, 1024))
    Ws = [dev_bytes(fd.q4nx_pack(w.codes, w.scales, w.offsets)) for w in ws]
    x0 = synthgen.activations(7720, M, D)
    gamma = synthgen.bf16_bits((0.25 * synthgen.bf16_to_f32(synthgen.activations(7721, 1, D))[0]).astype(np.float32))
    q = torch.full((M, 512), 0x7FC0, dtype=torch.int16, device="cuda")
    k = torch.full((M, 256), float("nan"), dtype=torch.float32, device="cuda")
    v = torch.full((M, 256), float("nan"), dtype=torch.float32, device="cuda")
    o = torch.full((M, D), 0x7FC0, dtype=torch.int16, device="cuda")
    act = torch.full((M, 1024), 0x7FC0, dtype=torch.int16, device="cuda")
    y = torch.full((M, D), float("nan"), dtype=torch.float32, device="cuda")
    x_dev, gamma_dev = dev_bytes(x0), dev_bytes(gamma)
    steps = [fd.chain_step(x_dev, Ws[0], q, D, 512, fd.EPI_BF16),
             fd.chain_step(x_dev, Ws[1], k, D, 256),
             fd.chain_step(x_dev, Ws[2], v, D, 256),
             fd.chain_step(q, Ws[3], o, 512, D, fd.EPI_BF16, True),
             fd.chain_step(o, Ws[4], act, D, 2048, fd.EPI_GEGLU_BF16, True, gamma_dev, 1e-6),
             fd.chain_step(act, Ws[5], y, 1024, D, fd.EPI_NONE, True)]
    outs = {}
    for in_kernel in (0, 1):
        fd.fdqp_set_param(fresh, "chain_dependent", in_kernel)
        before = fd.fdqp_launch_count(fresh)
        run_chain(fresh, steps, M)
        launches = fd.fdqp_launch_count(fresh) - before
        assert launches == 1 if in_kernel else launches >= 4
        outs[in_kernel] = (q.cpu().numpy().copy(), k.cpu().numpy().copy(), o.cpu().numpy().copy(), act.cpu().numpy().copy(), y.cpu().numpy().copy())
        # every step against the oracle's projection of the input the GPU handed on
        def check(prev_bits, w, got, bf16, label):
            y_ref, a_ref = oracle.project(prev_bits, w.codes, w.scales, w.offsets)
            g = synthgen.bf16_to_f32(got.view(np.uint16)).astype(np.float64) if bf16 else got.astype(np.float64)
            assert np.all(np.abs(g - y_ref) <= REL_TOL * a_ref + ABS_TOL + (2.0 ** -8 * np.abs(y_ref) if bf16 else 0)), label
        check(x0, ws[0], outs[in_kernel][0], True, "q")
        check(x0, ws[1], outs[in_kernel][1], False, "k")
        check(outs[in_kernel][0].view(np.uint16), ws[3], outs[in_kernel][2], True, "o")
        check(outs[in_kernel][3].view(np.uint16), ws[5], outs[in_kernel][4], False, "down")
