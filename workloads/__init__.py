"""Seeded synthetic workloads for the parameter-server update.

Input generation only: parameter-vector shapes (layer segments), arrival schedules of N
simulated asynchronous workers, initial parameters and the stand-in worker gradient. None of
the master's update arithmetic lives here. Both the CPU oracle's tests and the CUDA library's
callers draw their inputs from this module. The per-element generators exist twice, written
separately from one definition: wl_cpu.c (plain C, feeds the oracle) and wl_gen.h + wl_cuda.cu
(device); this module's own mix64/key/word in Python is a third statement used by the tests.

The five workloads take the SHAPES of the models the paper trains (CIFAR ResNet-20, ImageNet
ResNet-50, WRN-16-4, a Transformer language model); no dataset, model or weight is involved.
"""
import ctypes
import heapq
import math
import os
import subprocess
from dataclasses import dataclass, field

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_CPU_LIB = os.path.join(_HERE, "libwl_cpu.so")
_CUDA_LIB = os.path.join(_HERE, "libwl_cuda.so")

NOISE, CURV, TARGET, INIT, ROW, SIGMA, TIME, SPEED = range(8)
_M64 = (1 << 64) - 1
_GOLD = 0x9E3779B97F4A7C15
BASE_SEED = 190910802


# ----------------------------------------------------------------------------- hash (host)
def mix64(z):
    z &= _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def key(seed, tag, a):
    return mix64(mix64(seed + _GOLD * (tag + 1)) + a)


def word(k, b):
    return mix64(k + _GOLD * (b + 1))


def hash4(seed, tag, a, b):
    return word(key(seed, tag, a), b)


def unit_double(w):
    """53-bit uniform in (0, 1) for host-side schedule draws."""
    return ((w >> 11) + 0.5) * 2.0 ** -53


# ----------------------------------------------------------------------------- shapes
def resnet20_segments():
    """CIFAR ResNet-20 with 1x1 projection shortcuts: 65 tensors, 272,474 parameters."""
    seg = [3 * 3 * 3 * 16, 16, 16]
    c_in = 16
    for w in (16, 32, 64):
        for b in range(3):
            seg += [3 * 3 * c_in * w, w, w, 3 * 3 * w * w, w, w]
            if b == 0 and c_in != w:
                seg += [c_in * w, w, w]
            c_in = w
    seg += [64 * 10, 10]
    return seg


def resnet50_segments():
    """ImageNet ResNet-50: 161 tensors, 25,557,032 parameters."""
    seg = [7 * 7 * 3 * 64, 64, 64]
    c_in = 64
    for w, blocks in ((64, 3), (128, 4), (256, 6), (512, 3)):
        for b in range(blocks):
            seg += [c_in * w, w, w, 9 * w * w, w, w, w * 4 * w, 4 * w, 4 * w]
            if b == 0:
                seg += [c_in * 4 * w, 4 * w, 4 * w]
            c_in = 4 * w
    seg += [2048 * 1000, 1000]
    return seg


def wrn16_4_segments():
    """WideResNet-16-4, 10 classes, pre-activation blocks: 2,748,890 parameters."""
    seg = [3 * 3 * 3 * 16]
    c_in = 16
    for w in (64, 128, 256):
        for b in range(2):
            seg += [c_in, c_in, 9 * c_in * w, w, w, 9 * w * w]
            if b == 0:
                seg += [c_in * w]
            c_in = w
    seg += [256, 256, 256 * 10, 10]
    return seg


def transformer_lm_segments():
    """Embedding 267,735 x 512, then 16 equal blocks filling up to 150,000,000 parameters."""
    emb = 267735 * 512
    rest = 150_000_000 - emb
    assert rest % 16 == 0
    return [emb] + [rest // 16] * 16


# ----------------------------------------------------------------------------- schedules
def _simulate(n_workers, arrivals, draw):
    """All workers pull at time 0 in id order; a worker that finishes pushes, pulls at once
    and starts its next task. Next arrival = smallest finish time, ties to the lower id.
    draw(worker, nth_task) -> compute time. Returns the list of arriving workers."""
    heap = [(draw(i, 0), i) for i in range(n_workers)]
    heapq.heapify(heap)
    count = [1] * n_workers
    out = []
    for _ in range(arrivals):
        t, i = heapq.heappop(heap)
        out.append(i)
        nxt = draw(i, count[i])
        if nxt is None:          # the caller's table of task times ran out
            return None
        heapq.heappush(heap, (t + nxt, i))
        count[i] += 1
    return out


def schedule_uniform_ticks(seed, n_workers, arrivals):
    """Equal-speed workers; each compute time is an integer uniform in {1, 2, 3} ticks."""
    keys = [key(seed, TIME, i) for i in range(n_workers)]
    return _simulate(n_workers, arrivals, lambda i, n: 1 + ((word(keys[i], n) >> 32) * 3 >> 32))


def schedule_lognormal(seed, n_workers, arrivals, s=0.5):
    """Worker i always takes exp(s * z_i) per task, z_i standard normal (Box-Muller)."""
    k = key(seed, SPEED, 0)
    f = []
    for i in range(n_workers):
        u1, u2 = unit_double(word(k, 2 * i)), unit_double(word(k, 2 * i + 1))
        z = math.sqrt(-2.0 * math.log(u1)) * math.cos(2.0 * math.pi * u2)
        f.append(math.exp(s * z))
    return _simulate(n_workers, arrivals, lambda i, n: f[i])


def schedule_exponential_stragglers(seed, n_workers, arrivals, frac=0.1, slow=5.0):
    """Exponential task times; the ceil(frac*N) workers of smallest hash rank are `slow` x slower."""
    k = key(seed, SPEED, 0)
    rank = sorted(range(n_workers), key=lambda i: (word(k, i), i))
    n_slow = math.ceil(frac * n_workers)
    scale = [1.0] * n_workers
    for i in rank[:n_slow]:
        scale[i] = slow
    keys = [key(seed, TIME, i) for i in range(n_workers)]
    return _simulate(n_workers, arrivals,
                     lambda i, n: -scale[i] * math.log(1.0 - unit_double(word(keys[i], n))))


def gamma_task_times(seed, n_workers, tasks_per_worker, batch=128, heterogeneous=False, v_task=0.1,
                     v_mach=None):
    """Execution times of the paper's gamma-distributed cluster model (Appendix "Gamma
    Distribution", Algorithms "Task execution time - homogeneous / heterogeneous machines").
    Returns an (n_workers, tasks_per_worker) array. Mean time = `batch` simulated units (the
    figure's 128 for B = 128; the text's mu = B*V_mach^2 contradicts its own figure).
    V_mach = 0.1 (homogeneous) or 0.6 (heterogeneous), V_task = 0.1; alpha = 1/V^2."""
    rng = np.random.Generator(np.random.PCG64(seed))
    v_mach = (0.6 if heterogeneous else 0.1) if v_mach is None else v_mach
    a_task, a_mach, mu = 1.0 / v_task ** 2, 1.0 / v_mach ** 2, float(batch)
    if heterogeneous:
        p = rng.gamma(a_mach, mu / a_mach, size=n_workers)             # mean time of each machine
        return rng.gamma(a_task, p[:, None] / a_task, size=(n_workers, tasks_per_worker))
    q = rng.gamma(a_task, mu / a_task)                                  # drawn once
    return rng.gamma(a_mach, q / a_mach, size=(n_workers, tasks_per_worker))


def schedule_gamma(seed, n_workers, arrivals, heterogeneous=False, batch=128):
    """Arrival order under the gamma execution-time model."""
    per = arrivals // n_workers + 8
    while True:
        t = gamma_task_times(seed, n_workers, per, batch, heterogeneous)
        sched = _simulate(n_workers, arrivals, lambda i, n: float(t[i, n]) if n < per else None)
        if sched is not None:
            return sched
        per *= 2


def schedule_round_robin(n_workers, arrivals):
    return [k % n_workers for k in range(arrivals)]


def windows(schedule, k_max):
    """Cut a schedule into consecutive windows of at most k_max arrivals in which no worker
    appears twice (a worker's second gradient needs the parameters sent after its first)."""
    out, cur, seen = [], [], set()
    for i in schedule:
        if len(cur) == k_max or i in seen:
            out.append(cur)
            cur, seen = [], set()
        cur.append(i)
        seen.add(i)
    if cur:
        out.append(cur)
    return out


# ----------------------------------------------------------------------------- bindings
class _Spec(ctypes.Structure):
    _fields_ = [("seed", ctypes.c_uint64), ("d", ctypes.c_int64), ("quad", ctypes.c_int32),
                ("n_seg", ctypes.c_int32), ("emb_elems", ctypes.c_int64),
                ("emb_row", ctypes.c_int64), ("row_thresh", ctypes.c_uint64)]


def build_cpu(force=False):
    srcs = [os.path.join(_HERE, "wl_cpu.c")]
    if not force and os.path.exists(_CPU_LIB) and all(
            os.path.getmtime(_CPU_LIB) >= os.path.getmtime(s) for s in srcs):
        return _CPU_LIB
    tmp = f"{_CPU_LIB}.{os.getpid()}.tmp"
    try:
        subprocess.check_call(["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fPIC", "-shared", "-Wall",
                               "-o", tmp, srcs[0], "-lm"])
    except OSError:   # the compiler itself is missing
        if os.path.exists(_CPU_LIB) and not force:
            return _CPU_LIB
        raise
    os.replace(tmp, _CPU_LIB)
    return _CPU_LIB


def build_cuda(force=False):
    srcs = [os.path.join(_HERE, "wl_cuda.cu"), os.path.join(_HERE, "wl_gen.h")]
    if not force and os.path.exists(_CUDA_LIB) and all(
            os.path.getmtime(_CUDA_LIB) >= os.path.getmtime(s) for s in srcs):
        return _CUDA_LIB
    tmp = f"{_CUDA_LIB}.{os.getpid()}.tmp"
    try:
        subprocess.check_call(["nvcc", "-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a",
                               "-lineinfo", "-fmad=false", "-Xcompiler", "-fPIC", "-shared",
                               "-o", tmp, srcs[0]])
    except OSError:   # the compiler itself is missing
        if os.path.exists(_CUDA_LIB) and not force:
            return _CUDA_LIB
        raise
    os.replace(tmp, _CUDA_LIB)
    return _CUDA_LIB


_cpu = None
_cuda = None


def cpu_lib():
    global _cpu
    if _cpu is None:
        l = ctypes.CDLL(build_cpu())
        c = ctypes
        l.wl_cpu_mix64.restype = c.c_uint64
        l.wl_cpu_mix64.argtypes = [c.c_uint64]
        l.wl_cpu_hash.restype = c.c_uint64
        l.wl_cpu_hash.argtypes = [c.c_uint64] * 4
        l.wl_cpu_uniform.restype = c.c_float
        l.wl_cpu_uniform.argtypes = [c.c_uint64]
        l.wl_cpu_xi.restype = c.c_float
        l.wl_cpu_xi.argtypes = [c.c_uint64]
        for f in (l.wl_cpu_init, l.wl_cpu_target, l.wl_cpu_curv):
            f.argtypes = [c.c_uint64, c.c_void_p, c.c_int64, c.c_void_p]
        l.wl_cpu_grad.argtypes = [c.POINTER(_Spec), c.c_void_p, c.c_void_p, c.c_int64, c.c_void_p,
                                  c.c_int64, c.c_void_p, c.c_void_p]
        _cpu = l
    return _cpu


def cuda_lib():
    """The device generator. Fails loudly when the library was not built."""
    global _cuda
    if _cuda is None:
        if not os.path.exists(_CUDA_LIB):
            raise RuntimeError(f"{_CUDA_LIB} is missing: run __graft_entry__.build() first")
        l = ctypes.CDLL(_CUDA_LIB)
        c = ctypes
        l.wl_cuda_init.restype = c.c_int
        l.wl_cuda_init.argtypes = [c.c_uint64, c.c_int64, c.c_int64, c.c_void_p, c.c_void_p]
        l.wl_cuda_grad.restype = c.c_int
        l.wl_cuda_grad.argtypes = [c.POINTER(_Spec), c.c_void_p, c.c_void_p, c.c_int64, c.c_int64,
                                   c.c_int64, c.c_void_p, c.c_void_p, c.c_void_p]
        _cuda = l
    return _cuda


# ----------------------------------------------------------------------------- workloads
@dataclass
class Workload:
    name: str
    segments: list
    n_workers: int
    arrivals: int
    schedule_kind: str            # "ticks" | "lognormal" | "exp_stragglers" | "round_robin" | "gamma" | "gamma_hetero"
    seed: int
    lr: float = 0.1
    momentum: float = 0.9
    c_beta: float = 0.999
    sigma: object = 0.01          # float, or "loguniform" for 10^(-3+2u) per segment
    quad: bool = True             # g has the a*(s - theta*) term
    emb_rows: int = 0             # leading rows of emb_row elements with sparse activity
    emb_row: int = 0
    row_active_frac: float = 1.0
    variants: tuple = ("GA",)
    _sched: list = field(default=None, repr=False)

    def __post_init__(self):
        self.d = int(sum(self.segments))
        self.seg_off = np.zeros(len(self.segments) + 1, dtype=np.int64)
        self.seg_off[1:] = np.cumsum(self.segments)
        if self.sigma == "loguniform":
            k = key(self.seed, SIGMA, 0)
            sig = [10.0 ** (-3.0 + 2.0 * unit_double(word(k, l))) for l in range(len(self.segments))]
        else:
            sig = [float(self.sigma)] * len(self.segments)
        self.seg_sigma = np.asarray(sig, dtype=np.float32)
        thresh = _M64 if self.row_active_frac >= 1.0 else (1 << 64) * int(self.row_active_frac * 1000) // 1000
        self.spec = _Spec(self.seed, self.d, int(self.quad), len(self.segments),
                          self.emb_rows * self.emb_row, max(self.emb_row, 1), thresh)

    # -- host-side inputs
    def schedule(self, arrivals=None):
        """The workload's arrival schedule; `arrivals` asks for a longer (or shorter) run of
        the same simulation (the first self.arrivals entries are the workload's own)."""
        if arrivals is not None:
            return self._simulate(arrivals)
        if self._sched is None:
            self._sched = self._simulate(self.arrivals)
        return self._sched

    def _simulate(self, a):
        kind, n = self.schedule_kind, self.n_workers
        if kind == "ticks":
            return schedule_uniform_ticks(self.seed, n, a)
        if kind == "lognormal":
            return schedule_lognormal(self.seed, n, a)
        if kind == "exp_stragglers":
            return schedule_exponential_stragglers(self.seed, n, a)
        if kind == "round_robin":
            return schedule_round_robin(n, a)
        if kind in ("gamma", "gamma_hetero"):
            return schedule_gamma(self.seed, n, a, heterogeneous=(kind == "gamma_hetero"))
        raise ValueError(kind)

    def sample_indices(self, n, extra_seed=0):
        """Global element indices for a sampled parity check: both ends of every segment,
        the vector's last elements, and hashed picks; sorted and unique."""
        picks = set()
        for l in range(len(self.segments)):
            picks.update((int(self.seg_off[l]), int(self.seg_off[l + 1]) - 1))
        picks.update(range(max(0, self.d - 9), self.d))
        picks.update(range(0, min(self.d, 9)))
        k = key(self.seed ^ 0x5A17, 99, extra_seed)
        t = 0
        while len(picks) < min(n, self.d):
            picks.add(word(k, t) % self.d)
            t += 1
        return np.asarray(sorted(picks), dtype=np.int64)

    # -- CPU generators (global indices; idx=None is the dense vector)
    def _vec(self, fn, idx):
        n = self.d if idx is None else len(idx)
        out = np.empty(n, dtype=np.float32)
        p = None if idx is None else np.ascontiguousarray(idx, dtype=np.int64).ctypes.data
        fn(self.seed, p, n, out.ctypes.data)
        return out

    def theta0(self, idx=None):
        return self._vec(cpu_lib().wl_cpu_init, idx)

    def theta_star(self, idx=None):
        return self._vec(cpu_lib().wl_cpu_target, idx)

    def curvature(self, idx=None):
        return self._vec(cpu_lib().wl_cpu_curv, idx)

    def grad(self, k, sent, idx=None):
        """Gradient of arrival k (1-based) from the fp32 parameters the worker was sent."""
        sent = np.ascontiguousarray(sent, dtype=np.float32)
        n = self.d if idx is None else len(idx)
        assert sent.shape == (n,)
        out = np.empty(n, dtype=np.float32)
        idx_c = None if idx is None else np.ascontiguousarray(idx, dtype=np.int64)
        cpu_lib().wl_cpu_grad(ctypes.byref(self.spec), self.seg_off.ctypes.data,
                              self.seg_sigma.ctypes.data, k,
                              None if idx_c is None else idx_c.ctypes.data, n,
                              sent.ctypes.data, out.ctypes.data)
        return out

    # -- device generators
    def device(self, torch_device="cuda", j0=0, n=None):
        return DeviceWorkload(self, torch_device, j0, n)


class DeviceWorkload:
    """Device-side twin of Workload's generators (torch only holds the memory)."""

    def __init__(self, wl, torch_device, j0=0, n=None):
        import torch
        self.wl = wl
        self.j0 = int(j0)                                  # this holder covers [j0, j0 + n)
        self.n = int(wl.d - j0 if n is None else n)
        assert 0 <= self.j0 and self.j0 + self.n <= wl.d
        self._torch = torch
        self.seg_off = torch.from_numpy(wl.seg_off).to(torch_device)
        self.seg_sigma = torch.from_numpy(wl.seg_sigma).to(torch_device)
        self.lib = cuda_lib()
        self._spec_ref = ctypes.byref(wl.spec)
        self._seg_off_p = ctypes.c_void_p(self.seg_off.data_ptr())
        self._seg_sigma_p = ctypes.c_void_p(self.seg_sigma.data_ptr())

    def _stream(self):
        return ctypes.c_void_p(self._torch.cuda.current_stream().cuda_stream)

    def theta0(self, out):
        assert out.dtype == self._torch.float32 and out.numel() >= self.n and out.is_contiguous()
        rc = self.lib.wl_cuda_init(self.wl.seed, self.j0, self.n, ctypes.c_void_p(out.data_ptr()), self._stream())
        if rc:
            raise RuntimeError(f"wl_cuda_init: CUDA error {rc}")
        return out

    def grad_ptr(self, k, sent_ptr, out_ptr):
        rc = self.lib.wl_cuda_grad(self._spec_ref, self._seg_off_p, self._seg_sigma_p, k, self.j0, self.n,
                                   sent_ptr, out_ptr, self._stream())
        if rc:
            raise RuntimeError(f"wl_cuda_grad: CUDA error {rc}")


def _cfg(idx, **kw):
    return Workload(seed=BASE_SEED + idx, **kw)


def config(name):
    """The five workloads, by name C1..C5, plus 'mini' (a seconds-scale case for smoke checks)."""
    if name == "C1":
        return _cfg(1, name="C1", segments=resnet20_segments(), n_workers=8, arrivals=1000,
                    schedule_kind="ticks")
    if name == "C2":
        return _cfg(2, name="C2", segments=resnet20_segments(), n_workers=32, arrivals=20000,
                    schedule_kind="lognormal", variants=("GA", "SA", "ASGD"))
    if name == "C3":
        return _cfg(3, name="C3", segments=resnet50_segments(), n_workers=64, arrivals=2000,
                    schedule_kind="ticks", sigma="loguniform")
    if name == "C4":
        return _cfg(4, name="C4", segments=wrn16_4_segments(), n_workers=128, arrivals=50000,
                    schedule_kind="exp_stragglers")
    if name == "C5":
        return _cfg(5, name="C5", segments=transformer_lm_segments(), n_workers=32, arrivals=500,
                    schedule_kind="ticks", quad=False, emb_rows=267735, emb_row=512,
                    row_active_frac=0.1)
    if name == "mini":
        return _cfg(0, name="mini", segments=[1000, 37, 4099, 2, 515], n_workers=5, arrivals=60,
                    schedule_kind="ticks", sigma="loguniform")
    raise KeyError(name)
