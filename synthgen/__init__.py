"""Seeded synthetic inputs for Q4NX projections (shared by all tests and the bench).

Holds only the input recipes -- none of the projection's arithmetic.  Codes are
uniform 0..15, scales are bf16(|N(0, 0.02)|), offsets bf16(N(0, 0.01)) and
activations bf16(N(0, 1)) (optionally scaled), all drawn from a counter-based
generator so that every element is a pure function of (seed, stream, index).
The shapes mirror Gemma3 projections; they stand in for trained checkpoints.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "synthgen.c")
_LIB = os.path.join(_HERE, "libsynthgen.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    with _lock:
        if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
            tmp = _LIB + f".tmp{os.getpid()}"
            subprocess.check_call(["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
                                   "-o", tmp, _SRC, "-lm"])
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u64, i64, p, dbl = ctypes.c_uint64, ctypes.c_int64, ctypes.c_void_p, ctypes.c_double
        lib.synth_u64.argtypes = [u64, u64, i64, p]
        lib.synth_codes.argtypes = [u64, i64, p]
        lib.synth_scales.argtypes = [u64, i64, dbl, p]
        lib.synth_offsets.argtypes = [u64, i64, dbl, p]
        lib.synth_x.argtypes = [u64, i64, dbl, p]
        for f in (lib.synth_u64, lib.synth_codes, lib.synth_scales, lib.synth_offsets, lib.synth_x):
            f.restype = None
        _lib = lib
    return _lib


def u64(seed: int, stream: int, count: int) -> np.ndarray:
    out = np.empty(count, np.uint64)
    _load().synth_u64(seed, stream, count, ctypes.c_void_p(out.ctypes.data))
    return out


@dataclass
class Q4NXWeights:
    """Unpacked Q4NX content: one code per byte plus raw bf16 scale/offset bits."""
    codes: np.ndarray    # [N, K] uint8, 0..15
    scales: np.ndarray   # [N, K/32] uint16 (bf16 bits)
    offsets: np.ndarray  # [N, K/32] uint16 (bf16 bits)

    @property
    def K(self) -> int:
        return self.codes.shape[1]

    @property
    def N(self) -> int:
        return self.codes.shape[0]


def weights(seed: int, K: int, N: int, sigma_d: float = 0.02, sigma_m: float = 0.01) -> Q4NXWeights:
    """Codes uniform 0..15, scale bf16(|N(0, sigma_d)|), offset bf16(N(0, sigma_m))."""
    assert K % 32 == 0 and N % 32 == 0
    lib = _load()
    codes = np.empty((N, K), np.uint8)
    scales = np.empty((N, K // 32), np.uint16)
    offsets = np.empty((N, K // 32), np.uint16)
    lib.synth_codes(seed, codes.size, ctypes.c_void_p(codes.ctypes.data))
    lib.synth_scales(seed, scales.size, sigma_d, ctypes.c_void_p(scales.ctypes.data))
    lib.synth_offsets(seed, offsets.size, sigma_m, ctypes.c_void_p(offsets.ctypes.data))
    return Q4NXWeights(codes, scales, offsets)


FMT_Q4NX, FMT_G64, FMT_G128, FMT_MXFP4 = 0, 1, 2, 3
FMT_GROUP = {FMT_Q4NX: 32, FMT_G64: 64, FMT_G128: 128, FMT_MXFP4: 32}


def weights_fmt(seed: int, K: int, N: int, fmt: int) -> Q4NXWeights:
    """Content for a format variant of the container.  Group sizes 64 / 128: the Q4NX recipe with one scale and one
    offset per larger group.  MXFP4: codes uniform 0..15 (E2M1 elements), `scales` holds the E8M0 exponent bytes
    (uniform 118..122, i.e. scales 2^-9 .. 2^-5: weights of a few hundredths like the Q4NX recipe's) widened to uint16;
    `offsets` is None."""
    assert K % 256 == 0 and N % 32 == 0
    g = FMT_GROUP[fmt]
    lib = _load()
    codes = np.empty((N, K), np.uint8)
    lib.synth_codes(seed, codes.size, ctypes.c_void_p(codes.ctypes.data))
    if fmt == FMT_MXFP4:
        e = (118 + u64(seed, 7, N * (K // g)) % np.uint64(5)).astype(np.uint16).reshape(N, K // g)
        return Q4NXWeights(codes, e, None)
    scales = np.empty((N, K // g), np.uint16)
    offsets = np.empty((N, K // g), np.uint16)
    lib.synth_scales(seed, scales.size, 0.02, ctypes.c_void_p(scales.ctypes.data))
    lib.synth_offsets(seed, offsets.size, 0.01, ctypes.c_void_p(offsets.ctypes.data))
    return Q4NXWeights(codes, scales, offsets)


def activations(seed: int, M: int, K: int, amp: float = 1.0) -> np.ndarray:
    """x[M, K] as bf16 bits, bf16(amp * N(0, 1))."""
    x = np.empty((M, K), np.uint16)
    _load().synth_x(seed, x.size, amp, ctypes.c_void_p(x.ctypes.data))
    return x


def bf16_bits(a) -> np.ndarray:
    """float array -> bf16 bit patterns (round to nearest even), for hand-built test inputs."""
    u = np.ascontiguousarray(a, np.float32).view(np.uint32).astype(np.uint64)
    return (((u + 0x7FFF + ((u >> 16) & 1)) >> 16) & 0xFFFF).astype(np.uint16)


def bf16_to_f32(bits) -> np.ndarray:
    """bf16 bit patterns -> float32 (exact)."""
    return (np.ascontiguousarray(bits, np.uint16).astype(np.uint32) << 16).view(np.float32)


# ---- the workload shapes (Gemma3 projections) ---------------------------------

GEMMA3_4B_LAYER = [  # (name, K, N, seed): one decoder layer, seeds 1..7
    ("q", 2560, 2048, 1), ("k", 2560, 1024, 2), ("v", 2560, 1024, 3), ("o", 2048, 2560, 4),
    ("gate", 2560, 10240, 5), ("up", 2560, 10240, 6), ("down", 10240, 2560, 7),
]
GEMMA3_1B_GATE = ("gate_1b", 1152, 6912, 0)
GEMMA3_12B_GATE_UP = ("gate_up_12b", 3840, 30720, 11)
GEMMA3_27B_DOWN = ("down_27b", 21504, 5376, 13)      # x scaled by 1/sqrt(K)
GEMMA3_4B_LM_HEAD = ("lm_head_4b", 2560, 262144, 17)
GEMMA3_4B_LAYERS = 34
