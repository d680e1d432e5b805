"""CPU oracle for FusedDQP -- test infrastructure, not the product.

Only tests, the smoke check and the benchmark's CPU-baseline / reference arm
may import this package.  It never imports the CUDA package.

The arithmetic lives in ``oracle_q4nx.c`` (plain C, fp64); this module builds
it with gcc on first use and exposes thin numpy wrappers.  Each wrapper names
the passage of the paper its C routine follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle_q4nx.c")
_LIB = os.path.join(_HERE, "liboracle_q4nx.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction)."""
    with _lock:
        if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
            tmp = _LIB + f".tmp{os.getpid()}"
            subprocess.check_call(
                ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared",
                 "-fPIC", "-o", tmp, _SRC, "-lm"])
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, p, ci = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int
        lib.oracle_packed_bytes.restype = ctypes.c_size_t
        lib.oracle_packed_bytes.argtypes = [i64, i64]
        lib.oracle_unpack.restype = ci
        lib.oracle_unpack.argtypes = [p, i64, i64, p, p, p]
        lib.oracle_dequant.restype = ci
        lib.oracle_dequant.argtypes = [p, p, p, i64, i64, i64, i64, p, p]
        lib.oracle_project.restype = ci
        lib.oracle_project.argtypes = [p, p, p, p, i64, i64, i64, i64, i64, ci, ci, p, p]
        lib.oracle_project_packed.restype = ci
        lib.oracle_project_packed.argtypes = [p, p, i64, i64, i64, i64, i64, ci, ci, p, p]
        lib.oracle_gelu_tanh.restype = ctypes.c_double
        lib.oracle_gelu_tanh.argtypes = [ctypes.c_double]
        lib.oracle_geglu.restype = ci
        lib.oracle_geglu.argtypes = [p, i64, i64, p, p]
        lib.oracle_rmsnorm.restype = ci
        lib.oracle_rmsnorm.argtypes = [p, p, ctypes.c_double, i64, i64, p]
        lib.oracle_add_residual.restype = ci
        lib.oracle_add_residual.argtypes = [p, p, i64, i64, p]
        lib.oracle_decode_attention.restype = ci
        lib.oracle_decode_attention.argtypes = [p, p, p, i64, i64, i64, i64, i64, i64, ctypes.c_double, p, p]
        lib.oracle_fmt_packed_bytes.restype = ctypes.c_size_t
        lib.oracle_fmt_packed_bytes.argtypes = [ci, i64, i64]
        lib.oracle_fmt_unpack.restype = ci
        lib.oracle_fmt_unpack.argtypes = [ci, p, i64, i64, p, p, p]
        lib.oracle_fmt_dequant.restype = ci
        lib.oracle_fmt_dequant.argtypes = [ci, p, p, p, i64, i64, i64, i64, p, p]
        lib.oracle_fmt_project.restype = ci
        lib.oracle_fmt_project.argtypes = [ci, p, p, p, p, i64, i64, i64, i64, i64, ci, p, p]
        lib.oracle_max_threads.restype = ci
        _lib = lib
    return _lib


def _ptr(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def packed_bytes(K: int, N: int) -> int:
    """Size of a packed K x N matrix: 5 bits per weight (a 32 x 256 block is 5120 bytes)."""
    return int(_load().oracle_packed_bytes(K, N))


def max_threads() -> int:
    return int(_load().oracle_max_threads())


def unpack(packed, K: int, N: int):
    """Packed Q4NX bytes -> (codes[N,K] u8, scales[N,K/32] u16, offsets[N,K/32] u16)."""
    packed = _c(packed, np.uint8)
    if packed.size != packed_bytes(K, N) or packed.size == 0:
        raise ValueError("packed size does not match K, N")
    codes = np.empty((N, K), np.uint8)
    scales = np.empty((N, K // 32), np.uint16)
    offsets = np.empty((N, K // 32), np.uint16)
    rc = _load().oracle_unpack(_ptr(packed), K, N, _ptr(codes), _ptr(scales), _ptr(offsets))
    if rc != 0:
        raise ValueError(f"oracle_unpack failed ({rc})")
    return codes, scales, offsets


def dequant(codes, scales, offsets, n0: int = 0, n1: int | None = None):
    """Eq. 3: (w32[K, n1-n0] float32, w16[K, n1-n0] bf16 bits) for columns n0..n1."""
    codes = _c(codes, np.uint8)
    scales = _c(scales, np.uint16)
    offsets = _c(offsets, np.uint16)
    N, K = codes.shape
    n1 = N if n1 is None else n1
    w32 = np.empty((K, n1 - n0), np.float32)
    w16 = np.empty((K, n1 - n0), np.uint16)
    rc = _load().oracle_dequant(_ptr(codes), _ptr(scales), _ptr(offsets), K, N, n0, n1, _ptr(w32), _ptr(w16))
    if rc != 0:
        raise ValueError(f"oracle_dequant failed ({rc})")
    return w32, w16


def project(x_bf16, codes, scales, offsets, n0: int = 0, n1: int | None = None, use_w16: bool = False,
            nthreads: int = 1):
    """Eq. 14/15: (y[M, n1-n0] fp64, abs_sum[M, n1-n0] fp64) from unpacked weights."""
    x_bf16 = _c(x_bf16, np.uint16)
    codes = _c(codes, np.uint8)
    scales = _c(scales, np.uint16)
    offsets = _c(offsets, np.uint16)
    N, K = codes.shape
    M = x_bf16.shape[0]
    if x_bf16.shape != (M, K):
        raise ValueError("x must be [M, K]")
    n1 = N if n1 is None else n1
    y = np.empty((M, n1 - n0), np.float64)
    a = np.empty((M, n1 - n0), np.float64)
    rc = _load().oracle_project(_ptr(x_bf16), _ptr(codes), _ptr(scales), _ptr(offsets), M, K, N, n0, n1,
                                int(use_w16), nthreads, _ptr(y), _ptr(a))
    if rc != 0:
        raise ValueError(f"oracle_project failed ({rc})")
    return y, a


def project_packed(x_bf16, packed, K: int, N: int, n0: int = 0, n1: int | None = None, use_w16: bool = False,
                   nthreads: int = 1):
    """Eq. 14/15 straight from packed bytes (column range n0..n1)."""
    x_bf16 = _c(x_bf16, np.uint16)
    packed = _c(packed, np.uint8)
    M = x_bf16.shape[0]
    if x_bf16.shape != (M, K):
        raise ValueError("x must be [M, K]")
    if packed.size != packed_bytes(K, N) or packed.size == 0:
        raise ValueError("packed size does not match K, N")
    n1 = N if n1 is None else n1
    y = np.empty((M, n1 - n0), np.float64)
    a = np.empty((M, n1 - n0), np.float64)
    rc = _load().oracle_project_packed(_ptr(x_bf16), _ptr(packed), M, K, N, n0, n1, int(use_w16), nthreads,
                                       _ptr(y), _ptr(a))
    if rc != 0:
        raise ValueError(f"oracle_project_packed failed ({rc})")
    return y, a


def gelu_tanh(g: float) -> float:
    """GELU, tanh form (the reading taken for the GELU-and-multiply step the paper places after the gate and up projections)."""
    return float(_load().oracle_gelu_tanh(float(g)))


def geglu(y):
    """Gated GELU of a fused gate|up projection y [M, N] (per 32-row strip: rows 0..15 gate, 16..31 up):
    (out [M, N/2] fp64, out_bf16 [M, N/2] uint16 = RNE bf16 of the fp32 rounding)."""
    y = _c(y, np.float64)
    M, N = y.shape
    out = np.empty((M, N // 2), np.float64)
    out16 = np.empty((M, N // 2), np.uint16)
    rc = _load().oracle_geglu(_ptr(y), M, N, _ptr(out), _ptr(out16))
    if rc != 0:
        raise ValueError(f"oracle_geglu failed ({rc})")
    return out, out16


def rmsnorm(x_bf16, gamma_bf16, eps: float):
    """RMS normalisation with scale (1 + gamma): bf16 bits [M, K] in, bf16 bits [M, K] out."""
    x_bf16 = _c(x_bf16, np.uint16)
    gamma_bf16 = _c(gamma_bf16, np.uint16)
    M, K = x_bf16.shape
    if gamma_bf16.shape != (K,):
        raise ValueError("gamma must be [K]")
    out = np.empty((M, K), np.uint16)
    rc = _load().oracle_rmsnorm(_ptr(x_bf16), _ptr(gamma_bf16), float(eps), M, K, _ptr(out))
    if rc != 0:
        raise ValueError(f"oracle_rmsnorm failed ({rc})")
    return out


def add_residual(x_bf16, r_bf16):
    """The residual stream ahead of a normalisation: bf16(x + r), one rounding (bf16 bits in, bf16 bits out)."""
    x_bf16 = _c(x_bf16, np.uint16)
    r_bf16 = _c(r_bf16, np.uint16)
    if x_bf16.shape != r_bf16.shape or x_bf16.ndim != 2:
        raise ValueError("x and r must be [M, K]")
    h = np.empty_like(x_bf16)
    rc = _load().oracle_add_residual(_ptr(x_bf16), _ptr(r_bf16), x_bf16.shape[0], x_bf16.shape[1], _ptr(h))
    if rc != 0:
        raise ValueError(f"oracle_add_residual failed ({rc})")
    return h


def decode_attention(q, K, V, L: int, window: int = 0, scale: float = 1.0):
    """Attention of one new token over a KV cache (the paper's decoding-step attention; grouped queries, optional
    sliding window): q [H, d], K and V [G, pitch, d] bf16 bits -> (out [H, d] fp64, sum_j p_j |v_j| [H, d] fp64)."""
    q = _c(q, np.uint16)
    K = _c(K, np.uint16)
    V = _c(V, np.uint16)
    H, d = q.shape
    G, pitch, d2 = K.shape
    if d2 != d or V.shape != K.shape:
        raise ValueError("K and V must be [G, pitch, d] with q's d")
    out = np.empty((H, d), np.float64)
    absw = np.empty((H, d), np.float64)
    rc = _load().oracle_decode_attention(_ptr(q), _ptr(K), _ptr(V), H, G, d, L, pitch, window, float(scale), _ptr(out),
                                         _ptr(absw))
    if rc != 0:
        raise ValueError(f"oracle_decode_attention failed ({rc})")
    return out, absw


# ---- format variants of the block container (group sizes 64 / 128, MXFP4) ----------------------------------------

FMT_G64, FMT_G128, FMT_MXFP4 = 1, 2, 3
FMT_GROUP = {FMT_G64: 64, FMT_G128: 128, FMT_MXFP4: 32}


def fmt_packed_bytes(fmt: int, K: int, N: int) -> int:
    """Size of a packed K x N matrix in a variant format: 4608 (group 64) or 4352 (group 128, MXFP4) bytes per block."""
    return int(_load().oracle_fmt_packed_bytes(fmt, K, N))


def fmt_unpack(fmt: int, packed, K: int, N: int):
    """Packed bytes -> (codes[N,K] u8, scales[N,K/g] u16, offsets[N,K/g] u16 or None).  MXFP4 scales are the E8M0
    bytes widened to u16."""
    packed = _c(packed, np.uint8)
    if packed.size != fmt_packed_bytes(fmt, K, N) or packed.size == 0:
        raise ValueError("packed size does not match fmt, K, N")
    g = FMT_GROUP[fmt]
    codes = np.empty((N, K), np.uint8)
    scales = np.empty((N, K // g), np.uint16)
    offsets = None if fmt == FMT_MXFP4 else np.empty((N, K // g), np.uint16)
    rc = _load().oracle_fmt_unpack(fmt, _ptr(packed), K, N, _ptr(codes), _ptr(scales),
                                   None if offsets is None else _ptr(offsets))
    if rc != 0:
        raise ValueError(f"oracle_fmt_unpack failed ({rc})")
    return codes, scales, offsets


def fmt_dequant(fmt: int, codes, scales, offsets=None, n0: int = 0, n1: int | None = None):
    """Eq. 3 with the format's group size, or the MXFP4 element times its power-of-two scale: (w32, w16 bits)."""
    codes = _c(codes, np.uint8)
    scales = _c(scales, np.uint16)
    offsets = None if offsets is None else _c(offsets, np.uint16)
    N, K = codes.shape
    n1 = N if n1 is None else n1
    w32 = np.empty((K, n1 - n0), np.float32)
    w16 = np.empty((K, n1 - n0), np.uint16)
    rc = _load().oracle_fmt_dequant(fmt, _ptr(codes), _ptr(scales), None if offsets is None else _ptr(offsets), K, N,
                                    n0, n1, _ptr(w32), _ptr(w16))
    if rc != 0:
        raise ValueError(f"oracle_fmt_dequant failed ({rc})")
    return w32, w16


def fmt_project(fmt: int, x_bf16, codes, scales, offsets=None, n0: int = 0, n1: int | None = None, nthreads: int = 1):
    """y = x . w32 of the variant format in fp64, k ascending: (y[M, n1-n0], abs_sum[M, n1-n0])."""
    x_bf16 = _c(x_bf16, np.uint16)
    codes = _c(codes, np.uint8)
    scales = _c(scales, np.uint16)
    offsets = None if offsets is None else _c(offsets, np.uint16)
    N, K = codes.shape
    M = x_bf16.shape[0]
    if x_bf16.shape != (M, K):
        raise ValueError("x must be [M, K]")
    n1 = N if n1 is None else n1
    y = np.empty((M, n1 - n0), np.float64)
    a = np.empty((M, n1 - n0), np.float64)
    rc = _load().oracle_fmt_project(fmt, _ptr(x_bf16), _ptr(codes), _ptr(scales),
                                    None if offsets is None else _ptr(offsets), M, K, N, n0, n1, nthreads, _ptr(y),
                                    _ptr(a))
    if rc != 0:
        raise ValueError(f"oracle_fmt_project failed ({rc})")
    return y, a
