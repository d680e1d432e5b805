"""CPU-side checks of the library: it loads, exports what the header declares, the host packer
agrees with the oracle's reader and with the sequential writer, and argument errors are reported
without a GPU.  No kernel runs here."""
import os
import re

import numpy as np
import pytest

import oracle
import paper_2602_06063_b200 as fd
import synthgen
from paper_2602_06063_b200 import binding
from q4nx_seq import write_sequential

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    lib = fd.load_library()
    header = open(os.path.join(ROOT, "include", "fdqp.h")).read()
    declared = re.findall(r"FDQP_API\s+[\w\s\*]+?\b(\w+)\s*\(", header)
    assert sorted(declared) == sorted(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings():
    for code in range(9):
        assert fd.fdqp_status_string(code) not in ("", "unknown status")
    assert fd.fdqp_status_string(99) == "unknown status"


def test_packed_bytes():
    assert fd.q4nx_packed_bytes(256, 32) == 5120          # the paper's block
    assert fd.q4nx_packed_bytes(1152, 6912) == 4976640
    assert fd.q4nx_packed_bytes(2560, 262144) == 419430400
    for K, N in [(0, 32), (32, 0), (48, 32), (32, 48), (-32, 32)]:
        assert fd.q4nx_packed_bytes(K, N) == 0
        assert fd.q4nx_packed_bytes(K, N) == oracle.packed_bytes(K, N)


@pytest.mark.parametrize("K,N", [(32, 32), (64, 64), (256, 32), (288, 32), (544, 96), (1152, 128), (2560, 64)])
def test_pack_roundtrip_through_oracle_reader(K, N):
    w = synthgen.weights(400 + K + N, K, N)
    packed = fd.q4nx_pack(w.codes, w.scales, w.offsets)
    assert packed.size == oracle.packed_bytes(K, N)
    c, s, o = oracle.unpack(packed, K, N)                 # independent reader
    assert np.array_equal(c, w.codes) and np.array_equal(s, w.scales) and np.array_equal(o, w.offsets)
    c, s, o = fd.q4nx_unpack(packed, K, N)                # the library's own inverse
    assert np.array_equal(c, w.codes) and np.array_equal(s, w.scales) and np.array_equal(o, w.offsets)
    if K * N <= 200000:
        assert np.array_equal(packed, write_sequential(w.codes, w.scales, w.offsets))


def test_pack_golden_bytes():
    with open(os.path.join(ROOT, "tests", "golden", "q4nx_k32_n32.hex")) as f:
        want = np.frombuffer(bytes.fromhex("".join(line.split("#")[0] for line in f)), np.uint8)
    n, k = np.arange(32)[:, None], np.arange(32)[None, :]
    codes = ((k + 3 * n) % 16).astype(np.uint8)
    packed = fd.q4nx_pack(codes, np.full((32, 1), 0x3F00, np.uint16), np.full((32, 1), 0xBF80, np.uint16))
    assert np.array_equal(packed, want)


def test_pack_rejects_bad_input():
    lib = fd.load_library()
    codes = np.zeros((32, 32), np.uint8)
    sc = np.zeros((32, 1), np.uint16)
    out = np.zeros(640, np.uint8)
    args = (codes.ctypes.data, sc.ctypes.data, sc.ctypes.data)
    assert lib.q4nx_pack(*args, 32, 32, out.ctypes.data, 640) == 0
    assert lib.q4nx_pack(*args, 32, 32, out.ctypes.data, 639) == 4      # FDQP_ERR_SIZE
    assert lib.q4nx_pack(*args, 48, 32, out.ctypes.data, 640) == 2      # FDQP_ERR_SHAPE
    assert lib.q4nx_pack(None, sc.ctypes.data, sc.ctypes.data, 32, 32, out.ctypes.data, 640) == 1
    codes[3, 7] = 16
    assert lib.q4nx_pack(*args, 32, 32, out.ctypes.data, 640) == 1      # code out of range
    assert lib.q4nx_unpack(None, 32, 32, codes.ctypes.data, sc.ctypes.data, sc.ctypes.data) == 1


def test_null_and_shape_errors_without_device():
    lib = fd.load_library()
    assert lib.fdqp_create(None, 0, 1, 32, 32) == 1
    import ctypes
    h = ctypes.c_void_p()
    assert lib.fdqp_create(ctypes.byref(h), 0, 0, 32, 32) == 2
    assert lib.fdqp_create(ctypes.byref(h), 0, 1, 48, 32) == 2
    assert h.value is None
    assert lib.fdqp_run(None, None, None, None, 1, 32, 32, None) == 1
    assert lib.fdqp_destroy(None) == 0
    assert lib.fdqp_launch_count(None) == 0


def test_no_device_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    with pytest.raises(fd.FdqpError) as err:
        fd.fdqp_create(0, 1, 32, 32)
    assert err.value.code in (5, 6)   # never a silent CPU path
