"""Host code under AddressSanitizer and UndefinedBehaviorSanitizer: the library's packer / unpacker (q4nx_host.cpp) and
the oracle (oracle_q4nx.c) are compiled together with -fsanitize=address,undefined and driven through pack -> unpack
round trips, the oracle's dequantisation and projection, exact-fit output buffers and the refusal paths.  Any
out-of-bounds access or undefined behaviour in either aborts the driver, which fails this test."""
import os
import shutil
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.skipif(shutil.which("gcc") is None or shutil.which("g++") is None, reason="needs gcc and g++")
def test_packer_and_oracle_round_trips_under_asan_ubsan(tmp_path):
    san = ["-fsanitize=address,undefined", "-fno-sanitize-recover=all", "-fno-omit-frame-pointer", "-g", "-O1"]
    inc = ["-I", os.path.join(ROOT, "include")]
    objs = []
    for cc, std, src in (
        ("gcc", "-std=c11", os.path.join(ROOT, "oracle", "oracle_q4nx.c")),
        ("g++", "-std=c++17", os.path.join(ROOT, "paper_2602_06063_b200", "csrc", "q4nx_host.cpp")),
        ("gcc", "-std=c11", os.path.join(ROOT, "tests", "sanitize", "roundtrip_main.c")),
    ):
        obj = str(tmp_path / (os.path.basename(src) + ".o"))
        subprocess.check_call([cc, std] + san + inc + ["-ffp-contract=off", "-c", "-o", obj, src])
        objs.append(obj)
    exe = str(tmp_path / "roundtrip")
    subprocess.check_call(["g++"] + san + ["-o", exe] + objs + ["-lm"])
    env = dict(os.environ, ASAN_OPTIONS="detect_leaks=1:abort_on_error=0", UBSAN_OPTIONS="print_stacktrace=1")
    env.pop("LD_PRELOAD", None)
    out = subprocess.run([exe], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stdout + out.stderr
    assert "sanitized round trips ok" in out.stdout
