"""The library is usable from plain C: the example links against libga.so and the CUDA runtime
only. Expected numbers: gamma = 0, constant gradient 0.5, eta 0.1 -- worker 1 makes three
unpenalised steps of 0.05 (delays 1, 1, 1); worker 0 then arrives with delay 4 and a Gap of
3*0.05 / (0.1*(0.5 + 1e-8)) + 1 = 4, so its step is 0.05 / 4: theta = 1 - 0.15 - 0.0125."""
import os
import shutil
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.gpu
def test_plain_c_program(tmp_path):
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    if not shutil.which("gcc") or not os.path.exists(os.path.join(cuda, "include", "cuda_runtime_api.h")):
        pytest.skip("no C toolchain with the CUDA runtime headers")
    exe = str(tmp_path / "ga_example")
    lib_dir = os.path.join(ROOT, "paper_1909_10802_b200")
    subprocess.check_call(["gcc", "-I", os.path.join(ROOT, "include"), "-I", os.path.join(cuda, "include"),
                           os.path.join(ROOT, "examples", "ga_example.c"), "-o", exe, "-L", lib_dir, "-lga",
                           "-L", os.path.join(cuda, "lib64"), "-lcudart", f"-Wl,-rpath,{lib_dir}",
                           f"-Wl,-rpath,{os.path.join(cuda, 'lib64')}"])
    out = subprocess.run([exe], capture_output=True, text=True, timeout=120)
    assert out.returncode == 0, out.stderr
    words = out.stdout.split()
    assert words[:5] == ["delays", "1", "1", "1", "4"]
    assert abs(float(words[6]) - (1 - 0.15 - 0.0125)) < 2e-6


@pytest.mark.gpu
def test_call_timing_program(tmp_path):
    """The small-vector timing example builds, runs and reports a plausible per-call time."""
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    if not shutil.which("gcc") or not os.path.exists(os.path.join(cuda, "include", "cuda_runtime_api.h")):
        pytest.skip("no C toolchain with the CUDA runtime headers")
    exe = str(tmp_path / "ga_call_timing")
    lib_dir = os.path.join(ROOT, "paper_1909_10802_b200")
    subprocess.check_call(["gcc", "-O2", "-I", os.path.join(ROOT, "include"), "-I", os.path.join(cuda, "include"),
                           os.path.join(ROOT, "examples", "ga_call_timing.c"), "-o", exe, "-L", lib_dir, "-lga",
                           "-L", os.path.join(cuda, "lib64"), "-lcudart", f"-Wl,-rpath,{lib_dir}",
                           f"-Wl,-rpath,{os.path.join(cuda, 'lib64')}"])
    out = subprocess.run([exe, "272474", "8", "2000"], capture_output=True, text=True, timeout=120)
    assert out.returncode == 0, out.stderr
    words = out.stdout.split()
    total = float(words[words.index("total_us_per_call") + 1])
    assert 0.5 < total < 200.0, out.stdout
