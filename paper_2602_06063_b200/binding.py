"""ctypes binding of the FusedDQP C ABI (see include/fdqp.h for the contract of each call).

Only marshals arguments: numpy arrays for host buffers, torch tensors (or raw integer
addresses) for device buffers, ``torch.cuda.current_stream()`` when no stream is given.
The library is built in-tree by ``build.py``; if it is missing or cannot be loaded the
import of a symbol fails loudly -- there is no Python or CPU fallback for any operation.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libfdqp.so")
_lib = None

STATUS = {
    0: "FDQP_OK", 1: "FDQP_ERR_ARG", 2: "FDQP_ERR_SHAPE", 3: "FDQP_ERR_ALIGN", 4: "FDQP_ERR_SIZE",
    5: "FDQP_ERR_ARCH", 6: "FDQP_ERR_CUDA", 7: "FDQP_ERR_NOMEM", 8: "FDQP_ERR_TIMEOUT",
}

EXPORTS = [
    "q4nx_packed_bytes", "q4nx_pack", "q4nx_unpack", "fdqp_create", "fdqp_destroy", "fdqp_run", "fdqp_run_host",
    "fdqp_run_host_async", "fdqp_run_epilogue", "fdqp_run_rmsnorm_epilogue", "fdqp_flowkv_decode", "fdqp_stream_read",
    "fdqp_dequant", "fdqp_last_status", "fdqp_last_cuda_error", "fdqp_status_string", "fdqp_set_param",
    "fdqp_launch_count", "fdqp_describe", "fdqp_run_noalloc", "q4nx_packed_bytes_fmt", "q4nx_pack_fmt",
    "q4nx_unpack_fmt", "fdqp_run_fmt", "fdqp_dequant_fmt", "fdqp_run_add_rmsnorm_epilogue",
    "fdqp_selftest_bounded_wait", "fdqp_noalloc_last_status", "fdqp_run_chain",
]


class FdqpError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        self.name = STATUS.get(code, f"status {code}")
        super().__init__(f"{where}: {self.name}" + (f" ({detail})" if detail else ""))


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Load libfdqp.so (building it first if the sources are newer)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        from . import build as _build
        _build.build()
    lib = ctypes.CDLL(_LIB_PATH)
    i64, vp, ci, sz = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    lib.q4nx_packed_bytes.restype = sz
    lib.q4nx_packed_bytes.argtypes = [i64, i64]
    lib.q4nx_pack.restype = ci
    lib.q4nx_pack.argtypes = [vp, vp, vp, i64, i64, vp, sz]
    lib.q4nx_unpack.restype = ci
    lib.q4nx_unpack.argtypes = [vp, i64, i64, vp, vp, vp]
    lib.q4nx_packed_bytes_fmt.restype = sz
    lib.q4nx_packed_bytes_fmt.argtypes = [ci, i64, i64]
    lib.q4nx_pack_fmt.restype = ci
    lib.q4nx_pack_fmt.argtypes = [ci, vp, vp, vp, i64, i64, vp, sz]
    lib.q4nx_unpack_fmt.restype = ci
    lib.q4nx_unpack_fmt.argtypes = [ci, vp, i64, i64, vp, vp, vp]
    lib.fdqp_run_fmt.restype = ci
    lib.fdqp_run_fmt.argtypes = [vp, ci, vp, vp, vp, i64, i64, i64, vp]
    lib.fdqp_dequant_fmt.restype = ci
    lib.fdqp_dequant_fmt.argtypes = [vp, ci, vp, vp, ci, i64, i64, vp]
    lib.fdqp_create.restype = ci
    lib.fdqp_create.argtypes = [ctypes.POINTER(vp), ci, i64, i64, i64]
    lib.fdqp_destroy.restype = ci
    lib.fdqp_destroy.argtypes = [vp]
    lib.fdqp_run.restype = ci
    lib.fdqp_run.argtypes = [vp, vp, vp, vp, i64, i64, i64, vp]
    lib.fdqp_run_host.restype = ci
    lib.fdqp_run_host.argtypes = [vp, vp, vp, vp, i64, i64, i64, vp]
    lib.fdqp_run_epilogue.restype = ci
    lib.fdqp_run_epilogue.argtypes = [vp, vp, vp, vp, ci, i64, i64, i64, vp]
    lib.fdqp_run_rmsnorm_epilogue.restype = ci
    lib.fdqp_run_rmsnorm_epilogue.argtypes = [vp, vp, vp, ctypes.c_float, vp, vp, ci, i64, i64, i64, vp]
    lib.fdqp_run_add_rmsnorm_epilogue.restype = ci
    lib.fdqp_run_add_rmsnorm_epilogue.argtypes = [vp, vp, vp, vp, vp, ctypes.c_float, vp, vp, ci, i64, i64, i64, vp]
    lib.fdqp_flowkv_decode.restype = ci
    lib.fdqp_flowkv_decode.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, i64, i64, i64, ctypes.c_float, vp]
    lib.fdqp_stream_read.restype = ci
    lib.fdqp_stream_read.argtypes = [vp, vp, i64, vp]
    lib.fdqp_run_host_async.restype = ci
    lib.fdqp_run_host_async.argtypes = [vp, vp, vp, vp, i64, i64, i64, vp]
    lib.fdqp_run_noalloc.restype = ci
    lib.fdqp_run_noalloc.argtypes = [vp, vp, vp, i64, i64, i64, vp]
    lib.fdqp_run_chain.restype = ci
    lib.fdqp_run_chain.argtypes = [vp, vp, i64, i64, vp]
    lib.fdqp_noalloc_last_status.restype = ci
    lib.fdqp_noalloc_last_status.argtypes = []
    lib.fdqp_dequant.restype = ci
    lib.fdqp_dequant.argtypes = [vp, vp, vp, ci, i64, i64, vp]
    lib.fdqp_last_status.restype = ci
    lib.fdqp_last_status.argtypes = [vp]
    lib.fdqp_selftest_bounded_wait.restype = ci
    lib.fdqp_selftest_bounded_wait.argtypes = [vp, ctypes.c_int64, vp]
    lib.fdqp_last_cuda_error.restype = ctypes.c_char_p
    lib.fdqp_last_cuda_error.argtypes = [vp]
    lib.fdqp_status_string.restype = ctypes.c_char_p
    lib.fdqp_status_string.argtypes = [ci]
    lib.fdqp_set_param.restype = ci
    lib.fdqp_set_param.argtypes = [vp, ctypes.c_char_p, i64]
    lib.fdqp_launch_count.restype = i64
    lib.fdqp_launch_count.argtypes = [vp]
    lib.fdqp_describe.restype = ci
    lib.fdqp_describe.argtypes = [vp, i64, i64, i64, ctypes.c_char_p, sz]
    _lib = lib
    return lib


# ---- marshalling helpers ------------------------------------------------------------------------

def _addr(buf) -> int:
    """Address of a torch tensor, a numpy array, or an integer that already is one."""
    if buf is None:
        return 0
    if isinstance(buf, int):
        return buf
    if isinstance(buf, np.ndarray):
        return buf.ctypes.data
    return int(buf.data_ptr())  # torch tensor


def _stream(stream) -> int:
    if stream is None:
        import torch
        return int(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, int):
        return stream
    return int(stream.cuda_stream)


def _check(code: int, where: str, ctx=None):
    if code != 0:
        detail = ""
        if ctx is not None and code == 6:
            detail = load_library().fdqp_last_cuda_error(ctx).decode()
        raise FdqpError(code, where, detail)


# ---- container ------------------------------------------------------------------------------------

def q4nx_packed_bytes(K: int, N: int) -> int:
    return int(load_library().q4nx_packed_bytes(K, N))


def q4nx_pack(codes: np.ndarray, scales_bf16: np.ndarray, offsets_bf16: np.ndarray) -> np.ndarray:
    """codes[N,K] u8, scales/offsets[N,K/32] u16 (bf16 bits) -> packed bytes (host numpy)."""
    codes = np.ascontiguousarray(codes, np.uint8)
    scales_bf16 = np.ascontiguousarray(scales_bf16, np.uint16)
    offsets_bf16 = np.ascontiguousarray(offsets_bf16, np.uint16)
    N, K = codes.shape
    size = q4nx_packed_bytes(K, N)
    if size == 0:
        raise FdqpError(2, "q4nx_pack")
    if scales_bf16.shape != (N, K // 32) or offsets_bf16.shape != (N, K // 32):
        raise FdqpError(2, "q4nx_pack", "scales/offsets must be [N, K/32]")
    out = np.empty(size, np.uint8)
    _check(load_library().q4nx_pack(codes.ctypes.data, scales_bf16.ctypes.data, offsets_bf16.ctypes.data, K, N,
                                    out.ctypes.data, out.size), "q4nx_pack")
    return out


def q4nx_unpack(packed: np.ndarray, K: int, N: int):
    packed = np.ascontiguousarray(packed, np.uint8)
    if q4nx_packed_bytes(K, N) == 0 or packed.size != q4nx_packed_bytes(K, N):
        raise FdqpError(2, "q4nx_unpack")
    codes = np.empty((N, K), np.uint8)
    scales = np.empty((N, K // 32), np.uint16)
    offsets = np.empty((N, K // 32), np.uint16)
    _check(load_library().q4nx_unpack(packed.ctypes.data, K, N, codes.ctypes.data, scales.ctypes.data,
                                      offsets.ctypes.data), "q4nx_unpack")
    return codes, scales, offsets


# ---- context and projection -------------------------------------------------------------------------

def fdqp_create(device: int, max_M: int, max_K: int, max_N: int) -> int:
    """Returns the context handle (an integer address); release it with fdqp_destroy."""
    h = ctypes.c_void_p()
    _check(load_library().fdqp_create(ctypes.byref(h), device, max_M, max_K, max_N), "fdqp_create")
    return h.value


def fdqp_destroy(ctx: int) -> None:
    _check(load_library().fdqp_destroy(ctx), "fdqp_destroy")


def fdqp_run(ctx: int, x_bf16, W_q4nx, y, M: int, K: int, N: int, stream=None) -> None:
    """x, W, y: device tensors (or addresses).  Asynchronous on `stream`."""
    _check(load_library().fdqp_run(ctx, _addr(x_bf16), _addr(W_q4nx), _addr(y), M, K, N, _stream(stream)),
           "fdqp_run", ctx)


EPI_NONE, EPI_BF16, EPI_GEGLU_BF16 = 0, 1, 2


def fdqp_run_epilogue(ctx: int, x_bf16, W_q4nx, out, epilogue: int, M: int, K: int, N: int, stream=None) -> None:
    """fdqp_run with the store-side epilogue fused in: EPI_NONE (fp32 [M, N]), EPI_BF16 (bf16 [M, N]) or
    EPI_GEGLU_BF16 (bf16 [M, N/2]; gate and up rows interleaved sixteen by sixteen in W, see fdqp.h)."""
    _check(load_library().fdqp_run_epilogue(ctx, _addr(x_bf16), _addr(W_q4nx), _addr(out), int(epilogue), M, K, N,
                                            _stream(stream)), "fdqp_run_epilogue", ctx)


def fdqp_run_rmsnorm_epilogue(ctx: int, x_bf16, gamma_bf16, eps: float, W_q4nx, out, epilogue: int, M: int, K: int,
                              N: int, stream=None) -> None:
    """fdqp_run_epilogue on x RMS-normalised with scale (1 + gamma) (fused into the launch where possible, see fdqp.h)."""
    _check(load_library().fdqp_run_rmsnorm_epilogue(ctx, _addr(x_bf16), _addr(gamma_bf16), float(eps), _addr(W_q4nx),
                                                    _addr(out), int(epilogue), M, K, N, _stream(stream)),
           "fdqp_run_rmsnorm_epilogue", ctx)


def fdqp_run_add_rmsnorm_epilogue(ctx: int, x_bf16, residual_bf16, h_out_bf16, gamma_bf16, eps: float, W_q4nx, out,
                                  epilogue: int, M: int, K: int, N: int, stream=None) -> None:
    """fdqp_run_rmsnorm_epilogue on h = bf16(x + residual); h is also written to h_out_bf16 unless that is None."""
    _check(load_library().fdqp_run_add_rmsnorm_epilogue(ctx, _addr(x_bf16), _addr(residual_bf16),
                                                        None if h_out_bf16 is None else _addr(h_out_bf16),
                                                        _addr(gamma_bf16), float(eps), _addr(W_q4nx), _addr(out),
                                                        int(epilogue), M, K, N, _stream(stream)),
           "fdqp_run_add_rmsnorm_epilogue", ctx)


class ChainStepC(ctypes.Structure):
    """fdqp_chain_step of include/fdqp.h."""
    _fields_ = [("x_bf16", ctypes.c_void_p), ("W_q4nx", ctypes.c_void_p), ("out", ctypes.c_void_p),
                ("K", ctypes.c_int64), ("N", ctypes.c_int64), ("epilogue", ctypes.c_int),
                ("depends_on_previous", ctypes.c_int), ("gamma_bf16", ctypes.c_void_p), ("eps", ctypes.c_float),
                ("residual_bf16", ctypes.c_void_p), ("h_out_bf16", ctypes.c_void_p)]


def chain_step(x_bf16, W_q4nx, out, K: int, N: int, epilogue: int = 0, depends_on_previous: bool = False,
               gamma_bf16=None, eps: float = 0.0, residual_bf16=None, h_out_bf16=None) -> ChainStepC:
    """One step of fdqp_run_chain (device tensors or addresses; see fdqp_chain_step in fdqp.h)."""
    return ChainStepC(_addr(x_bf16) or None, _addr(W_q4nx) or None, _addr(out) or None, K, N, int(epilogue),
                      int(bool(depends_on_previous)), _addr(gamma_bf16) or None, float(eps),
                      _addr(residual_bf16) or None, _addr(h_out_bf16) or None)


def make_chain(steps):
    """A C array of fdqp_chain_step from a list of chain_step(...) values (keep it alive for the call)."""
    return (ChainStepC * len(steps))(*steps)


def fdqp_run_chain(ctx: int, steps, M: int, stream=None) -> None:
    """Run a chain of projections (a list of chain_step(...) or an array from make_chain) at M token rows in as few
    persistent launches as possible.  Asynchronous on `stream`."""
    arr = steps if isinstance(steps, ctypes.Array) else make_chain(steps)
    _check(load_library().fdqp_run_chain(ctx, ctypes.cast(arr, ctypes.c_void_p), len(arr), M, _stream(stream)),
           "fdqp_run_chain", ctx)


def fdqp_flowkv_decode(ctx: int, q_bf16, K_bf16, V_bf16, out, H: int, G: int, d: int, L: int, pitch: int, window: int,
                       scale: float, stream=None) -> None:
    """Attention of one new token over a KV cache (q [H, d], K and V [G, pitch, d] bf16 on the device -> out [H, d]
    fp32); window > 0 restricts it to the last `window` positions."""
    _check(load_library().fdqp_flowkv_decode(ctx, _addr(q_bf16), _addr(K_bf16), _addr(V_bf16), _addr(out), H, G, d, L,
                                             pitch, window, float(scale), _stream(stream)), "fdqp_flowkv_decode", ctx)


def fdqp_stream_read(ctx: int, buf, nbytes: int, stream=None) -> None:
    """Measurement aid: reads `nbytes` of a device buffer once through the projection kernels' bulk-copy ring."""
    _check(load_library().fdqp_stream_read(ctx, _addr(buf), nbytes, _stream(stream)), "fdqp_stream_read", ctx)


def fdqp_run_host(ctx: int, x_host_bf16, W_q4nx, y_host, M: int, K: int, N: int, stream=None) -> None:
    """x, y: HOST buffers (numpy or pinned torch); W: device.  Returns after y_host is filled."""
    _check(load_library().fdqp_run_host(ctx, _addr(x_host_bf16), _addr(W_q4nx), _addr(y_host), M, K, N,
                                        _stream(stream)), "fdqp_run_host", ctx)


def fdqp_run_host_async(ctx: int, x_host_bf16, W_q4nx, y_host, M: int, K: int, N: int, stream=None) -> None:
    """fdqp_run_host without the final synchronisation: y_host is valid once the caller has synchronised the stream."""
    _check(load_library().fdqp_run_host_async(ctx, _addr(x_host_bf16), _addr(W_q4nx), _addr(y_host), M, K, N,
                                              _stream(stream)), "fdqp_run_host_async", ctx)


def fdqp_run_noalloc(x_bf16, W_q4nx, y, M: int, K: int, N: int, stream=None) -> None:
    """fdqp_run for callers that cannot allocate: no context, scratch lives in the library image (see fdqp.h).
    Runs on the current device; all calls share one scratch array, so keep them ordered on a stream."""
    _check(load_library().fdqp_run_noalloc(_addr(x_bf16), _addr(W_q4nx), _addr(y), M, K, N, _stream(stream)),
           "fdqp_run_noalloc")


def fdqp_noalloc_last_status() -> int:
    """Status word of fdqp_run_noalloc on the current device (0, or 8 once a kernel gave up on a bounded wait).
    One blocking 4-byte copy: call it after synchronising the stream."""
    return int(load_library().fdqp_noalloc_last_status())


def fdqp_dequant(ctx: int, W_q4nx, out, out_is_bf16: bool, K: int, N: int, stream=None) -> None:
    _check(load_library().fdqp_dequant(ctx, _addr(W_q4nx), _addr(out), int(out_is_bf16), K, N, _stream(stream)),
           "fdqp_dequant", ctx)


FMT_Q4NX, FMT_G64, FMT_G128, FMT_MXFP4 = 0, 1, 2, 3
_FMT_GROUP = {FMT_Q4NX: 32, FMT_G64: 64, FMT_G128: 128, FMT_MXFP4: 32}


def q4nx_packed_bytes_fmt(fmt: int, K: int, N: int) -> int:
    return int(load_library().q4nx_packed_bytes_fmt(int(fmt), K, N))


def q4nx_pack_fmt(fmt: int, codes: np.ndarray, scales: np.ndarray, offsets_bf16=None) -> np.ndarray:
    """codes[N,K] u8; scales[N,K/g]: bf16 bits (u16), or for FMT_MXFP4 the E8M0 bytes (any integer dtype, 0..254);
    offsets[N,K/g] bf16 bits (None for FMT_MXFP4) -> packed bytes (host numpy)."""
    if fmt not in _FMT_GROUP:
        raise FdqpError(1, "q4nx_pack_fmt")
    g = _FMT_GROUP[fmt]
    codes = np.ascontiguousarray(codes, np.uint8)
    N, K = codes.shape
    mx = fmt == FMT_MXFP4
    if mx and (np.asarray(scales).max(initial=0) > 255 or np.asarray(scales).min(initial=0) < 0):
        raise FdqpError(1, "q4nx_pack_fmt", "E8M0 scales are bytes")
    scales = np.ascontiguousarray(scales, np.uint8 if mx else np.uint16)
    offs = None if mx else np.ascontiguousarray(offsets_bf16, np.uint16)
    size = q4nx_packed_bytes_fmt(fmt, K, N)
    if size == 0:
        raise FdqpError(2, "q4nx_pack_fmt")
    if scales.shape != (N, K // g) or (offs is not None and offs.shape != (N, K // g)):
        raise FdqpError(2, "q4nx_pack_fmt", "scales/offsets must be [N, K/g]")
    out = np.empty(size, np.uint8)
    _check(load_library().q4nx_pack_fmt(int(fmt), codes.ctypes.data, scales.ctypes.data,
                                        None if offs is None else offs.ctypes.data, K, N, out.ctypes.data, out.size),
           "q4nx_pack_fmt")
    return out


def q4nx_unpack_fmt(fmt: int, packed: np.ndarray, K: int, N: int):
    """-> (codes[N,K] u8, scales[N,K/g] (u16 bf16 bits, or u8 E8M0 bytes for FMT_MXFP4), offsets or None)."""
    packed = np.ascontiguousarray(packed, np.uint8)
    if fmt not in _FMT_GROUP or q4nx_packed_bytes_fmt(fmt, K, N) == 0 or packed.size != q4nx_packed_bytes_fmt(fmt, K, N):
        raise FdqpError(2, "q4nx_unpack_fmt")
    g = _FMT_GROUP[fmt]
    mx = fmt == FMT_MXFP4
    codes = np.empty((N, K), np.uint8)
    scales = np.empty((N, K // g), np.uint8 if mx else np.uint16)
    offs = None if mx else np.empty((N, K // g), np.uint16)
    _check(load_library().q4nx_unpack_fmt(int(fmt), packed.ctypes.data, K, N, codes.ctypes.data, scales.ctypes.data,
                                          None if offs is None else offs.ctypes.data), "q4nx_unpack_fmt")
    return codes, scales, offs


def fdqp_run_fmt(ctx: int, fmt: int, x_bf16, W_packed, y, M: int, K: int, N: int, stream=None) -> None:
    """fdqp_run for a matrix packed in a format variant (FMT_G64, FMT_G128, FMT_MXFP4; FMT_Q4NX = fdqp_run)."""
    _check(load_library().fdqp_run_fmt(ctx, int(fmt), _addr(x_bf16), _addr(W_packed), _addr(y), M, K, N, _stream(stream)),
           "fdqp_run_fmt", ctx)


def fdqp_dequant_fmt(ctx: int, fmt: int, W_packed, out, out_is_bf16: bool, K: int, N: int, stream=None) -> None:
    _check(load_library().fdqp_dequant_fmt(ctx, int(fmt), _addr(W_packed), _addr(out), int(out_is_bf16), K, N,
                                           _stream(stream)), "fdqp_dequant_fmt", ctx)


def fdqp_last_status(ctx: int) -> int:
    return int(load_library().fdqp_last_status(ctx))


def fdqp_selftest_bounded_wait(ctx: int, limit_us: int, stream=None) -> None:
    _check(load_library().fdqp_selftest_bounded_wait(ctx, int(limit_us), _stream(stream)), "fdqp_selftest_bounded_wait", ctx)


def fdqp_last_cuda_error(ctx: int) -> str:
    return load_library().fdqp_last_cuda_error(ctx).decode()


def fdqp_status_string(code: int) -> str:
    return load_library().fdqp_status_string(code).decode()


def fdqp_set_param(ctx: int, key: str, value: int) -> None:
    _check(load_library().fdqp_set_param(ctx, key.encode(), value), f"fdqp_set_param({key})")


def fdqp_launch_count(ctx: int) -> int:
    return int(load_library().fdqp_launch_count(ctx))


def fdqp_describe(ctx: int, M: int, K: int, N: int) -> str:
    buf = ctypes.create_string_buffer(512)
    _check(load_library().fdqp_describe(ctx, M, K, N, buf, len(buf)), "fdqp_describe")
    return buf.value.decode()
