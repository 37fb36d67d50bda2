"""bench.py prints one JSON line with the agreed keys (reference arm on CPU, GPU arm on a small case)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
BASE_KEYS = {"metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
             "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e", "gpu_launches"}


def _run(*args):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True,
                         cwd=ROOT, timeout=900)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out.stdout
    return json.loads(lines[0])


def test_reference_arm_times_the_oracle():
    j = _run("--impl", "reference", "--params", "200000", "--workers", "8", "--steps", "2", "--warmup", "1")
    assert BASE_KEYS <= set(j) and j["impl"] == "reference" and j["value"] > 0
    assert j["cpu_baseline"]["kind"] == "oracle" and j["cpu_baseline"]["cores"] == 1
    assert j["cpu_baseline"]["host_cores"] >= 1 and j["cpu_baseline"]["cpu_model"]
    assert j["e2e"] == {"value": j["value"], "unit": j["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert j["metric"] == "ga_master_param_updates_per_sec" and j["higher_is_better"] is True


def test_reference_arm_other_ranks_stay_silent():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--params", "1000"],
                         capture_output=True, text=True, cwd=ROOT, env=env, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""


@pytest.mark.gpu
def test_gpu_arm_small_case():
    j = _run("--params", "300000", "--workers", "12", "--steps", "4", "--warmup", "3", "--cpu-sample-params", "100000",
             "--e2e-steps", "1", "--e2e-window", "4")
    assert BASE_KEYS | {"roofline", "clocks"} <= set(j)
    assert j["n_gpus"] == 1 and j["steps"] == 4 and j["gpu_launches"] == 4 and j["dtype"] == "f32"
    r = j["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert j["e2e"]["h2d_bytes_per_step"] > 0 and j["e2e"]["d2h_bytes_per_step"] > 0 and j["e2e"]["value"] > 0
    assert j["cpu_baseline"]["value"] > 0 and "workload" in j["config"]
    cb = j["cpu_baseline"]
    assert cb["cores"] == 1 and cb["host_cores"] >= 1 and isinstance(cb["cpu_model"], str)
    assert "all_cores" in cb and (cb["all_cores"].get("value", 0) > 0 or "unavailable" in cb["all_cores"])
    assert 0 < j["e2e"]["pcie_frac"] < 1.5 and j["e2e"]["pcie_h2d_gbs"] > 0 and j["e2e"]["pcie_d2h_gbs"] > 0
    assert "traffic" in r and "traffic_source" in r     # a capture exists for GA / 16 / exact only while the kernel is unchanged


def test_traffic_file_matches_the_kernel_source():
    """roofline.traffic comes from profiles/ga_window_kernel_dram_traffic.json; the figure is only
    reported while the kernel source has the digest recorded at capture time."""
    sys.path.insert(0, ROOT)
    import bench
    value, source = bench.measured_traffic("GA", 16, "exact")
    table = json.load(open(bench.TRAFFIC_FILE))
    entry = table["captures"]["GA/16/exact"]
    import hashlib
    digest = hashlib.sha256(open(bench.KERNEL_SOURCE, "rb").read()).hexdigest()
    if digest == entry["kernel_source_sha256"]:
        assert value == entry["dram_bytes_per_param"] and 0.9 < value / entry["algorithmic_bytes_per_param"] < 1.1
    else:
        assert value is None and "changed" in source
    assert bench.measured_traffic("SA", 16, "exact")[0] is None


@pytest.mark.gpu
def test_multi_rank_arm_runs_with_two_ranks_on_one_gpu():
    """The N > 1 arm of bench.py (replicated schedule check, barrier, max over ranks, smaller
    end-to-end leg) launched the way the contract says, with the gloo process group so that two ranks
    can share the one GPU of a test box; their kernels never wait on one another."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                          "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py"),
                          "--gpus", "2", "--backend", "gloo", "--params", "300000", "--workers", "12", "--steps", "4",
                          "--warmup", "3", "--e2e-steps", "1"],
                         capture_output=True, text=True, cwd=ROOT, timeout=900)
    assert out.returncode == 0, out.stderr[-3000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out.stdout                      # rank 0 alone prints
    j = json.loads(lines[0])
    assert BASE_KEYS | {"roofline", "clocks"} <= set(j)
    assert j["n_gpus"] == 2 and j["scaling"] == "weak" and j["value"] > 0 and j["gpu_launches"] == 4
    assert j["cpu_baseline"] is None                         # the oracle is timed at N = 1 only
    assert j["e2e"]["window"] == 2 and j["e2e"]["value"] > 0
    assert "x2" in j["config"]["parallelism"] and "NOT larger than L2" in j["config"]["l2"]
