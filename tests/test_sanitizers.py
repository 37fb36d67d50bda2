"""The oracle and the host side of the C ABI under AddressSanitizer and UBSan.

Both are compiled from their committed sources together with a small driver program
(tests/sanitize_*_driver.*) and run as child processes: a bad access, a leak or an undefined
operation ends the child with a report and a non-zero status. No GPU is needed: without a
device the library's argument checks still run and ga_create fails with a message.
"""
import os
import shutil
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SAN = ["-fsanitize=address", "-fsanitize=undefined", "-fno-sanitize-recover=all", "-fno-omit-frame-pointer"]


def _run(exe):
    env = dict(os.environ, ASAN_OPTIONS="detect_leaks=1:abort_on_error=0", UBSAN_OPTIONS="print_stacktrace=1")
    return subprocess.run([exe], capture_output=True, text=True, env=env, timeout=300)


def test_oracle_under_sanitizers(tmp_path):
    exe = str(tmp_path / "san_oracle")
    subprocess.check_call(["g++", "-std=c++17", "-O1", "-g", "-ffp-contract=off", *SAN, "-o", exe,
                           os.path.join(ROOT, "oracle", "ga_oracle.cpp"),
                           os.path.join(ROOT, "tests", "sanitize_oracle_driver.cpp")])
    r = _run(exe)
    assert r.returncode == 0 and "sanitize driver ok" in r.stdout, r.stdout + r.stderr
    assert "runtime error" not in r.stderr and "AddressSanitizer" not in r.stderr


@pytest.mark.skipif(shutil.which("nvcc") is None, reason="needs nvcc to compile the library's source")
def test_api_host_side_under_sanitizers(tmp_path):
    exe = str(tmp_path / "san_api")
    drv = str(tmp_path / "driver.cpp")          # the driver is plain C; compiled here as C++ next to the .cu
    shutil.copy(os.path.join(ROOT, "tests", "sanitize_api_driver.c"), drv)
    cmd = ["nvcc", "-std=c++17", "-O1", "-g", "-gencode", "arch=compute_100a,code=sm_100a"]
    for f in SAN:
        cmd += ["-Xcompiler", f]
    cmd += ["-I", os.path.join(ROOT, "include"), os.path.join(ROOT, "paper_1909_10802_b200", "csrc", "ga_api.cu"),
            drv, "-o", exe]
    subprocess.check_call(cmd)
    r = _run(exe)
    assert r.returncode == 0 and "sanitize api driver ok" in r.stdout, r.stdout + r.stderr
    assert "runtime error" not in r.stderr and "AddressSanitizer" not in r.stderr
