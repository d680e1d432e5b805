"""GPU parity of the decode attention over a KV cache (the paper's FlowKV / FlowKV-SWA) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2602_06063_b200 as fd
import synthgen

pytestmark = pytest.mark.gpu

REL, ABS = 6e-3, 1e-5   # |out - ref| <= REL * sum_j p_j |v_j| + ABS (probabilities pass through bf16: 2^-9 each)


@pytest.fixture(scope="module")
def ctx():
    h = fd.fdqp_create(0, 8, 256, 256)
    yield h
    torch.cuda.synchronize()
    fd.fdqp_destroy(h)


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda()


def make(seed, H, G, d, pitch, amp_q=1.0):
    q = synthgen.activations(seed, H, d, amp_q)
    K = synthgen.activations(seed + 1, G * pitch, d).reshape(G, pitch, d)
    V = synthgen.activations(seed + 2, G * pitch, d).reshape(G, pitch, d)
    return q, K, V


def run(ctx, q, K, V, L, window, scale):
    H, d = q.shape
    G, pitch, _ = K.shape
    out = torch.full((H, d), float("nan"), dtype=torch.float32, device="cuda")
    fd.fdqp_flowkv_decode(ctx, dev(q), dev(K), dev(V), out, H, G, d, L, pitch, window, scale)
    torch.cuda.synchronize()
    assert fd.fdqp_last_status(ctx) == 0
    return out.cpu().numpy()


# (H, G, d, L, window, pitch): Gemma3-4B heads (8 query, 4 KV, d = 256) at ragged lengths, sliding window, other groupings
CASES = [
    (8, 4, 256, 1, 0, 8), (8, 4, 256, 5, 0, 64), (8, 4, 256, 16, 0, 16), (8, 4, 256, 63, 0, 100), (8, 4, 256, 64, 0, 64),
    (8, 4, 256, 65, 0, 70), (8, 4, 256, 1000, 0, 1024), (8, 4, 256, 4113, 0, 4200), (8, 4, 256, 5000, 1024, 5000),
    (8, 4, 256, 700, 1024, 800), (8, 4, 256, 2049, 1, 2100),
    (32, 16, 128, 777, 0, 800), (16, 2, 128, 3001, 512, 3001), (4, 4, 256, 300, 0, 300), (8, 1, 128, 129, 0, 129),
    (12, 4, 256, 2500, 0, 2500), (6, 1, 128, 9000, 0, 9000), (20, 4, 128, 1500, 700, 1600), (7, 1, 256, 333, 0, 400),
]


@pytest.mark.parametrize("H,G,d,L,window,pitch", CASES)
def test_decode_attention_matches_oracle(ctx, H, G, d, L, window, pitch):
    q, K, V = make(7000 + H + G + d + L + window, H, G, d, pitch)
    scale = d ** -0.5
    out = run(ctx, q, K, V, L, window, scale)
    ref, absw = oracle.decode_attention(q, K, V, L, window, scale)
    assert np.all(np.isfinite(out))
    err = np.abs(out.astype(np.float64) - ref)
    bad = err > REL * absw + ABS
    assert not bad.any(), f"{bad.sum()} of {bad.size} outside the bound; worst {(err / (absw + 1e-30)).max():.2e}"


# Full-size caches in the launch configurations the benchmark times (one CTA per SM, every split several hundred tiles
# long): the oracle still evaluates every output (a few GFLOP in fp64).  Inputs from a seeded numpy generator, which is
# fast enough for 10^8 values; keys get a slowly varying component so that the softmax is not flat over the cache.
FULL = [(8, 4, 256, 131072, 0), (8, 4, 256, 131072, 1024), (16, 8, 256, 32768 + 17, 0), (32, 16, 128, 65536, 0),
        (4, 1, 256, 32768, 0)]


@pytest.mark.parametrize("H,G,d,L,window", FULL)
def test_full_size_caches(ctx, H, G, d, L, window):
    rng = np.random.default_rng(900 + H + L + window)
    q = synthgen.bf16_bits(rng.standard_normal((H, d), dtype=np.float32))
    Kf = rng.standard_normal((G, L, d), dtype=np.float32)
    Kf[:, :, 0] += 6.0 * np.sin(np.arange(L, dtype=np.float32) * 1e-3)[None, :]
    K = synthgen.bf16_bits(Kf)
    del Kf
    V = synthgen.bf16_bits(rng.standard_normal((G, L, d), dtype=np.float32))
    scale = d ** -0.5
    out = run(ctx, q, K, V, L, window, scale)
    ref, absw = oracle.decode_attention(q, K, V, L, window, scale)
    assert np.all(np.isfinite(out))
    err = np.abs(out.astype(np.float64) - ref)
    bad = err > REL * absw + ABS
    assert not bad.any(), f"{bad.sum()} of {bad.size} outside the bound; worst {(err / (absw + 1e-30)).max():.2e}"


@pytest.mark.parametrize("H,G,d,L,window", [(8, 4, 256, 5000, 1024), (8, 4, 256, 1024, 0), (8, 4, 256, 2048, 0), (8, 4, 256, 65, 0),
                                            (32, 16, 128, 777, 0), (16, 2, 128, 3001, 512), (7, 1, 256, 1500, 0), (8, 1, 128, 1, 0)])
def test_one_launch_and_two_launch_routes(ctx, H, G, d, L, window):
    """Short ranges run as one launch (a cluster per KV head merges its splits through distributed shared memory), or,
    with the "flowkv_cluster" parameter at 0, as the split kernel and the merge kernel; both within the bound."""
    q, K, V = make(7600 + L + H, H, G, d, L)
    scale = d ** -0.5
    ref, absw = oracle.decode_attention(q, K, V, L, window, scale)
    outs = []
    try:
        for limit in (-1, 0, 1 << 20):
            fd.fdqp_set_param(ctx, "flowkv_cluster", limit)
            before = fd.fdqp_launch_count(ctx)
            out = run(ctx, q, K, V, L, window, scale)
            n = fd.fdqp_launch_count(ctx) - before
            assert n == (2 if limit == 0 else 1)
            assert np.all(np.abs(out.astype(np.float64) - ref) <= REL * absw + ABS), f"limit {limit}"
            assert np.array_equal(out, run(ctx, q, K, V, L, window, scale))      # fixed merge order on either route
            outs.append(out)
    finally:
        fd.fdqp_set_param(ctx, "flowkv_cluster", -1)


def test_peaked_scores_and_large_magnitudes(ctx):
    # a large scale makes the distribution collapse onto few positions (running-maximum updates matter)
    H, G, d, L = 8, 4, 256, 1500
    q, K, V = make(71, H, G, d, L, amp_q=4.0)
    out = run(ctx, q, K, V, L, 0, 1.0)
    ref, absw = oracle.decode_attention(q, K, V, L, 0, 1.0)
    assert np.all(np.abs(out - ref) <= REL * absw + ABS)


def test_uniform_weights_are_exact_and_the_cache_tail_is_never_read(ctx):
    # equal keys give weights 1/64 (a power of two) and small-integer values make the mean exact in fp32; everything
    # beyond position L is poisoned with infinities
    H, G, d, L, pitch = 8, 4, 256, 64, 96
    q, K, V = make(72, H, G, d, pitch)
    K[:, :L] = K[:, :1]
    r = synthgen.u64(72, 5, G * pitch * d).reshape(G, pitch, d)
    V = synthgen.bf16_bits(((r >> np.uint64(60)).astype(np.int64) - 8).astype(np.float32))
    K[:, L:] = 0x7F80
    V[:, L:] = 0xFF80
    out = run(ctx, q, K, V, L, 0, 0.0625)
    ref, _ = oracle.decode_attention(q, K, V, L, 0, 0.0625)
    assert np.array_equal(out.astype(np.float64), ref)


def test_reruns_are_bit_identical_and_window_equals_a_shorter_cache(ctx):
    H, G, d, L, W = 8, 4, 256, 3000, 1024
    q, K, V = make(73, H, G, d, L)
    a = run(ctx, q, K, V, L, W, 0.0625)
    assert np.array_equal(a, run(ctx, q, K, V, L, W, 0.0625))
    b = run(ctx, q, np.ascontiguousarray(K[:, L - W:]), np.ascontiguousarray(V[:, L - W:]), W, 0, 0.0625)
    ref, absw = oracle.decode_attention(q, K, V, L, W, 0.0625)
    assert np.all(np.abs(a - ref) <= REL * absw + ABS) and np.all(np.abs(b - ref) <= REL * absw + ABS)


def test_argument_errors(ctx):
    lib = fd.load_library()
    q, K, V = make(74, 8, 4, 256, 32)
    o = torch.empty((8, 256), dtype=torch.float32, device="cuda")
    qd, Kd, Vd = dev(q), dev(K), dev(V)
    s = torch.cuda.current_stream().cuda_stream
    ok = (ctx, qd.data_ptr(), Kd.data_ptr(), Vd.data_ptr(), o.data_ptr())
    assert lib.fdqp_flowkv_decode(*ok, 8, 4, 256, 32, 32, 0, 0.0625, s) == 0
    assert lib.fdqp_flowkv_decode(*ok, 8, 3, 256, 32, 32, 0, 0.0625, s) == 2      # H % G
    assert lib.fdqp_flowkv_decode(*ok, 8, 4, 64, 32, 32, 0, 0.0625, s) == 2       # head dimension
    assert lib.fdqp_flowkv_decode(*ok, 8, 4, 256, 33, 32, 0, 0.0625, s) == 2      # L beyond the cache
    assert lib.fdqp_flowkv_decode(*ok, 18, 2, 256, 32, 32, 0, 0.0625, s) == 2     # more than 8 query heads per KV head
    assert lib.fdqp_flowkv_decode(ctx, qd.data_ptr() + 2, Kd.data_ptr(), Vd.data_ptr(), o.data_ptr(), 8, 4, 256, 32, 32, 0,
                                  0.0625, s) == 3
    assert lib.fdqp_flowkv_decode(ctx, None, Kd.data_ptr(), Vd.data_ptr(), o.data_ptr(), 8, 4, 256, 32, 32, 0, 0.0625, s) == 1
    torch.cuda.synchronize()
