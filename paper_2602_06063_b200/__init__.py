"""FusedDQP for B200: fused Q4NX 4-bit dequantisation + projection (y = x . dequant(W)).

Thin ctypes binding over ``libfdqp.so`` -- argument marshalling only; every step of the
projection runs in the CUDA kernels of the library.  Function names match ``include/fdqp.h``.
"""
from .binding import (  # noqa: F401
    FdqpError,
    fdqp_create,
    fdqp_dequant,
    fdqp_describe,
    fdqp_destroy,
    fdqp_flowkv_decode,
    fdqp_last_cuda_error,
    fdqp_last_status,
    fdqp_launch_count,
    EPI_BF16,
    EPI_GEGLU_BF16,
    EPI_NONE,
    fdqp_run,
    fdqp_run_epilogue,
    fdqp_run_rmsnorm_epilogue,
    fdqp_run_host,
    fdqp_run_host_async,
    fdqp_run_noalloc,
    fdqp_set_param,
    fdqp_status_string,
    library_path,
    load_library,
    q4nx_pack,
    q4nx_packed_bytes,
    q4nx_unpack,
    STATUS,
)
