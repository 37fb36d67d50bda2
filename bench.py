#!/usr/bin/env python
"""Benchmark of the Gap-Aware master update.

One step = one fused window of the hot path on the Transformer-LM-shaped workload (C5: 150M
fp32 parameters, 32 workers / saved copies): up to 16 consecutive arrivals applied by one
ga_push_batch call -- delay, C, Gap, penalised gradient, momentum, step, refresh of m and the
save-and-send copy for each arrival. The metric is parameter-updates per second (parameters x
arrivals applied / time). Gradients are generated on the device between steps, outside the
timed region (they are the simulated workers' job); each step is timed with CUDA events on the
launching stream around the ga_push_batch call.

    python bench.py [--gpus N --steps K --warmup W] [--impl reference]

With N > 1 (under torchrun) every rank owns one C5-sized range of an N-times larger parameter
vector; the update needs no exchange between ranges, so there is no data-path collective.
--impl reference times the CPU oracle (a deliberately plain program) on a bounded sample.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "ga_master_param_updates_per_sec"
UNIT = "param-updates/s"
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes per parameter per full window of the dominant kernel, from an ncu capture
# (dram__bytes_read.sum + dram__bytes_write.sum); the file also records a digest of the kernel
# source at capture time, and the figure is dropped once the source has changed since.
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ga_window_kernel_dram_traffic.json")
KERNEL_SOURCE = os.path.join(ROOT, "paper_1909_10802_b200", "csrc", "ga_kernels.cuh")


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=60)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="C5")
    ap.add_argument("--params", type=int, default=0, help="profiling aid: a one-segment vector of this size")
    ap.add_argument("--workers", type=int, default=32)
    ap.add_argument("--variant", default="GA", choices=["GA", "SA", "ASGD", "SA_GRAD", "DANA", "DANA_SA", "DANA_GA", "ADAM", "ADAM_SA", "ADAM_GA", "GA_LAYER"])
    ap.add_argument("--window", type=int, default=16)
    ap.add_argument("--math", default="exact", choices=["exact", "fast"])
    ap.add_argument("--e2e-steps", type=int, default=4, help="timed ga_push_batch_host calls")
    ap.add_argument("--e2e-window", type=int, default=8, help="arrivals per fused window of the e2e leg")
    ap.add_argument("--e2e-windows-per-step", type=int, default=2, help="windows handed over per call")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-sample-params", type=int, default=4_000_000)
    ap.add_argument("--backend", default="nccl", choices=["nccl", "gloo"],
                    help="process group of the multi-rank arm (barrier and max over ranks only); gloo also lets "
                         "more ranks than GPUs run, for checking that arm on a machine with one GPU")
    return ap.parse_args()


def bytes_per_param_window(variant, k):
    """Algorithmic bytes one parameter moves in a k-arrival window (fp32): theta, v (and m) in
    and out once; per arrival the gradient (and, for GA, the saved copy) in and the saved copy out."""
    if variant == "GA_LAYER":                  # one distance pass per call (8 B), then 28 B per arrival: theta, v, g and
        return 8 + 28 * k                      # the next worker's copy in; theta, v and the sent copy out
    gap = variant in ("GA", "DANA_GA", "ADAM_GA")
    state = 24 if gap else 16                  # theta, v or sum_j v^j or Adam's m (, m behind C) in and out
    if variant.startswith("ADAM"):
        state += 8                             # Adam's second moment in and out
    per_arrival = 8 + (4 if gap else 0)        # gradient in, sent copy out (, saved copy in)
    if variant.startswith("DANA"):
        per_arrival += 8                                           # the worker's v^i in and out
    return state + per_arrival * k


def measured_traffic(variant, window, math):
    """(DRAM bytes per parameter of a full window from the last ncu capture, where it came from),
    or (None, why not)."""
    import hashlib
    try:
        with open(TRAFFIC_FILE) as f:
            table = json.load(f)
        entry = table["captures"][f"{variant}/{window}/{math}"]
    except Exception:
        return None, "no ncu capture on record for this variant, window and math mode"
    with open(KERNEL_SOURCE, "rb") as f:
        digest = hashlib.sha256(f.read()).hexdigest()
    if digest != entry.get("kernel_source_sha256"):
        return None, "kernel source changed since the ncu capture"
    return float(entry["dram_bytes_per_param"]), entry.get("source", os.path.relpath(TRAFFIC_FILE, ROOT))


def host_cpu():
    """(usable cores, CPU model string) of this machine."""
    try:
        cores = len(os.sched_getaffinity(0))
    except AttributeError:
        cores = os.cpu_count() or 1
    model = "unknown"
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    model = line.split(":", 1)[1].strip()
                    break
    except OSError:
        pass
    return cores, model


def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (no MEASURED_PEAKS.json)"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                mx.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def pick_workload(args):
    import workloads as W
    if args.params:
        return W.Workload(name=f"custom{args.params}", segments=[args.params], n_workers=args.workers,
                          arrivals=500, schedule_kind="ticks", seed=W.BASE_SEED + 99)
    return W.config(args.config)


def bench_windows(wl, window, count):
    """`count` windows of the workload's schedule (the simulation is run as long as needed)."""
    import workloads as W
    need = count * window + 64
    while True:
        wins = W.windows(wl.schedule(arrivals=need), window)
        if len(wins) > count:
            return wins[:count]
        need *= 2


# ------------------------------------------------------------------------------ CPU oracle legs
def time_oracle(wl, variant, n_params, windows_list, all_cores=False):
    """The oracle, as it stands, on a contiguous slice of the workload's parameter vector.
    Only push+pull are timed (gradients are generated beforehand), like the GPU's timed region.
    all_cores: the same source built with OpenMP (loops over parameters split across threads).
    Returns (param_updates, seconds, description)."""
    import numpy as np
    import oracle
    lib = oracle.lib_openmp() if all_cores else None
    threads = host_cpu()[0] if all_cores else 1
    n_params = min(n_params, wl.d)
    j0 = max(0, wl.spec.emb_elems - n_params // 2) if wl.spec.emb_elems else 0   # straddle embedding/dense
    j0 = min(j0, wl.d - n_params)
    idx = np.arange(j0, j0 + n_params, dtype=np.int64)
    o = oracle.Oracle(n_params, wl.n_workers, wl.lr, wl.momentum, wl.c_beta,
                      oracle.VARIANTS[variant], precision=32, _lib=lib)
    o.set_params(wl.theta0(idx))
    k, updates, seconds = 0, 0, 0.0
    for win in windows_list:
        grads = [wl.grad(k + 1 + j, o.sent_f32(i), idx) for j, i in enumerate(win)]
        t0 = time.perf_counter()
        o.push_batch(win, grads)
        seconds += time.perf_counter() - t0
        k += len(win)
        updates += len(win) * n_params
    return updates, seconds, f"oracle (fp32, {threads} thread{'s' if threads > 1 else ''}) on parameters " \
                             f"[{j0}, {j0 + n_params}) of {wl.name}, {k} arrivals push+pull"


def cpu_baseline_legs(wl, variant, window, sample_params):
    """The cpu_baseline object: the oracle on one thread and, from the same source built with
    OpenMP, on all host cores, each on a bounded slice of the workload."""
    cores, model = host_cpu()
    cw = bench_windows(wl, window, 3)
    time_oracle(wl, variant, min(sample_params, wl.d) // 8, cw[:1])
    updates, seconds, sample = time_oracle(wl, variant, sample_params, cw)
    out = {"value": updates / seconds, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample,
           "host_cores": cores, "cpu_model": model}
    try:
        os.environ.setdefault("OMP_NUM_THREADS", str(cores))
        time_oracle(wl, variant, min(sample_params, wl.d), cw[:1], all_cores=True)
        u2, s2, sample2 = time_oracle(wl, variant, min(4 * sample_params, wl.d), cw, all_cores=True)
        out["all_cores"] = {"value": u2 / s2, "unit": UNIT, "cores": cores, "kind": "oracle built with OpenMP",
                            "sample": sample2}
    except Exception as exc:                      # no OpenMP runtime on this machine
        out["all_cores"] = {"unavailable": str(exc)[:200]}
    return out


def run_reference(args):
    """--impl reference: the CPU oracle on the host cores, bounded sample per step."""
    import workloads as W
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = pick_workload(args)
    n_params = min(args.cpu_sample_params // 4, wl.d)
    wins = bench_windows(wl, args.window, args.steps + args.warmup)
    time_oracle(wl, args.variant, n_params, wins[:args.warmup])
    updates, seconds, sample = time_oracle(wl, args.variant, n_params, wins[args.warmup:])
    value = updates / seconds
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * seconds / max(1, args.steps),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{wl.name}: {wl.d} fp32 params, {wl.n_workers} workers, {args.variant}, "
                               f"window {args.window}", "note": "each step = one window on a bounded slice"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample,
                         "host_cores": host_cpu()[0], "cpu_model": host_cpu()[1]},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------ GPU arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    import workloads as W
    import paper_1909_10802_b200 as P
    from paper_1909_10802_b200.runner import Run

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path); use --impl reference for the oracle")
    n_dev = torch.cuda.device_count()
    if world > 1 and args.backend == "nccl" and local_rank >= n_dev:
        raise SystemExit(f"rank {rank}: no GPU {local_rank} (NCCL wants one GPU per rank)")
    device_index = local_rank % n_dev          # gloo: ranks may share a GPU (their kernels never wait on one another)
    torch.cuda.set_device(device_index)
    if world > 1 and args.backend == "nccl":
        dist.init_process_group("nccl", device_id=torch.device("cuda", device_index))
    elif world > 1:
        dist.init_process_group("gloo")
    P.lib()

    base = pick_workload(args)
    # weak scaling: rank r owns the r-th C5-sized range of a world-times larger vector
    wl = base if world == 1 else W.Workload(
        **{**{f: getattr(base, f) for f in ("name", "segments", "n_workers", "arrivals", "schedule_kind", "lr",
                                            "momentum", "c_beta", "sigma", "quad", "emb_rows", "emb_row",
                                            "row_active_frac")}, "seed": base.seed + 1000 * rank})
    wins = bench_windows(base, args.window, args.steps + args.warmup)
    if world > 1:
        from paper_1909_10802_b200.shard import assert_same_schedule
        assert_same_schedule([i for w in wins for i in w], dist)

    opts = {P.GA_OPT_MATH: 1 if args.math == "fast" else 0}
    run = Run(wl, args.variant, args.window, options=opts)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for win in wins[:args.warmup]:
        run.step(win)
    barrier()
    sampler = ClockSampler(device_index)
    if rank == 0:
        sampler.start()
    events, launches0 = [], run.launches
    wall0 = time.perf_counter()
    for win in wins[args.warmup:]:
        run.generate(win)                               # the workers' side: outside the timed events
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        run.apply(win)                                  # ga_push_batch: the hot path
        e1.record(stream)
        events.append((e0, e1, len(win)))
    barrier()
    wall = time.perf_counter() - wall0
    clocks = sampler.stop() if rank == 0 else None
    ms = [e0.elapsed_time(e1) for e0, e1, _ in events]
    total_ms = sum(ms)
    if world > 1:
        t = torch.tensor([total_ms], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    arrivals = sum(n for _, _, n in events)
    launches = run.launches - launches0
    updates_all = arrivals * wl.d * world
    value = updates_all / (total_ms * 1e-3)

    # roofline of the dominant kernel (the fused window kernel): algorithmic bytes / device time
    alg_bytes = sum(bytes_per_param_window(args.variant, n) * wl.d for _, _, n in events)
    achieved = alg_bytes / (sum(ms) * 1e-3) / 1e9
    peak, peak_src = hbm_peak()
    full = [(m, n) for m, (_, _, n) in zip(ms, events) if n == args.window]
    traffic_pp, traffic_src = measured_traffic(args.variant, args.window, args.math)
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                # measured DRAM bytes of a full window, scaled to the average launch of this run
                # (windows cut short by a repeated worker move proportionally fewer bytes)
                "traffic": (traffic_pp * wl.d * (alg_bytes / max(1, launches)) /
                            (bytes_per_param_window(args.variant, args.window) * wl.d)) if traffic_pp else None,
                "traffic_source": traffic_src, "peak_source": peak_src,
                "kernel": "ga_window_kernel", "algorithmic_bytes_per_launch": alg_bytes / max(1, launches),
                "avg_launch_ms": sum(ms) / max(1, launches),
                "frac_of_nominal_8TBs": achieved / 8000.0,
                "full_window_ms": statistics.median(m for m, _ in full) if full else None}

    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(args, run, wl, base, world, dist if world > 1 else None, barrier)
    run.close()
    torch.cuda.empty_cache()

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = cpu_baseline_legs(base, args.variant, args.window, args.cpu_sample_params)

    per_step_gb = alg_bytes / max(1, len(events)) / 1e9
    state_mb = wl.d * 4 * (3 + wl.n_workers) / 1e6           # theta, v, m and the saved copies
    if per_step_gb * 1e3 > 2 * 126 and state_mb > 2 * 126:
        l2_note = f"inputs larger than L2 (each step streams {per_step_gb:.2f} GB; state {state_mb / 1e3:.1f} GB)"
    else:
        l2_note = (f"NOT larger than L2: each step streams {per_step_gb * 1e3:.0f} MB over a state of {state_mb:.0f} MB "
                   "and L2 is not flushed between steps, so GB/s here is not a DRAM figure")
    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": total_ms / max(1, args.steps), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"{wl.name}: {wl.d} fp32 params per GPU, {wl.n_workers} workers "
                                   f"({wl.n_workers} saved copies), {args.variant}, window {args.window}, "
                                   f"{args.math} math",
                       "arrivals_timed": arrivals, "parallelism": f"range-sharded x{world}, no collective",
                       "l2": l2_note,
                       "timed": "CUDA events around each ga_push_batch call; gradient generation between "
                                "steps is outside the events", "wall_s_incl_generation": wall},
            "roofline": roofline, "cpu_baseline": cpu_baseline, "e2e": e2e, "gpu_launches": launches,
            "clocks": clocks,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def pcie_rates(host_in, dev_in, dev_out, host_out, repeats=3):
    """What plain copies reach on this machine: one pinned host->device copy and one device->pinned
    host copy of whole vectors running at the same time on two streams (the traffic pattern of the
    end-to-end path). Returns (host->device GB/s, device->host GB/s), best of `repeats`."""
    import torch
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    best = [0.0, 0.0]
    nbytes = host_in.numel() * 4
    for _ in range(repeats + 1):
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        with torch.cuda.stream(s_in):
            ev[0].record(s_in)
            dev_in.copy_(host_in, non_blocking=True)
            ev[1].record(s_in)
        with torch.cuda.stream(s_out):
            ev[2].record(s_out)
            host_out.copy_(dev_out, non_blocking=True)
            ev[3].record(s_out)
        torch.cuda.synchronize()
        best[0] = max(best[0], nbytes / (ev[0].elapsed_time(ev[1]) * 1e-3) / 1e9)
        best[1] = max(best[1], nbytes / (ev[2].elapsed_time(ev[3]) * 1e-3) / 1e9)
    return best[0], best[1]


def run_e2e(args, run, wl, base, world, dist, barrier):
    """Same metric through ga_push_batch_host: gradients start in pinned host memory and the
    parameters sent back to each worker end in pinned host memory, copies inside the timed region.
    One step = one call that hands over several fused windows."""
    import torch
    k = min(args.e2e_window, args.window)
    wps = args.e2e_windows_per_step
    if world > 1:            # every rank pins its own buffers: keep the node's pinned memory small
        k, wps = min(k, 2), 2
    wins = bench_windows(base, k, (args.e2e_steps + 1) * wps)      # the replicated schedule
    steps = [[i for w in wins[q * wps:(q + 1) * wps] for i in w] for q in range(args.e2e_steps + 1)]
    grads = [torch.empty(wl.d, dtype=torch.float32).pin_memory() for _ in range(k)]
    outs = [torch.empty(wl.d, dtype=torch.float32).pin_memory() for _ in range(k)]
    for j, g in enumerate(grads):                     # synthetic gradients, generated on the device
        run.dev.grad_ptr(run.k + 1 + j, run.engine.saved_ptr(wins[0][j % len(wins[0])]), run.grads[0].data_ptr())
        g.copy_(run.grads[0])
    torch.cuda.synchronize()

    def call(sched):
        n = len(sched)
        run.engine.push_batch_host(sched, [grads[q % k] for q in range(n)], [outs[q % k] for q in range(n)])
        return n

    call(steps[0])                                    # warm-up (allocates the staging buffers)
    barrier()
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    arrivals = 0
    t0 = time.perf_counter()
    e0.record(stream)
    for sched in steps[1:]:
        arrivals += call(sched)
    e1.record(stream)
    barrier()
    seconds = max(e0.elapsed_time(e1) * 1e-3, time.perf_counter() - t0 if world == 1 else 0.0)
    if dist is not None:
        t = torch.tensor([seconds], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        seconds = float(t.item())
    per_step = arrivals / max(1, args.e2e_steps)
    bytes_each_way = arrivals * wl.d * 4
    h2d, d2h = pcie_rates(grads[0], run.grads[0], run.grads[-1], outs[0])   # outside the timed region
    bound = max(bytes_each_way / (h2d * 1e9), bytes_each_way / (d2h * 1e9))
    return {"value": arrivals * wl.d * world / seconds, "unit": UNIT,
            "h2d_bytes_per_step": int(per_step * wl.d * 4), "d2h_bytes_per_step": int(per_step * wl.d * 4),
            "steps": args.e2e_steps, "window": k, "windows_per_step": wps,
            "pcie_h2d_gbs": h2d, "pcie_d2h_gbs": d2h, "pcie_frac": bound / seconds,
            "pcie_note": "plain pinned copies of one vector each way, concurrently on two streams, best of 3; "
                         "pcie_frac = time those rates need for this leg's bytes / measured time",
            "note": "ga_push_batch_host: pinned host gradients in, sent parameters out, chunked overlap"}


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
