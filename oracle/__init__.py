"""ctypes binding of the CPU oracle (oracle/ga_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the CPU-baseline leg
of the benchmark. The CUDA library never imports or links this package.
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ga_oracle.cpp")
_LIB = os.path.join(_HERE, "libga_oracle.so")

ASGD, SA, GA, SA_GRAD, DANA, DANA_SA, DANA_GA, ADAM, ADAM_SA, ADAM_GA, GA_LAYER = range(11)
VARIANTS = {"ASGD": ASGD, "SA": SA, "GA": GA, "SA_GRAD": SA_GRAD, "DANA": DANA, "DANA_SA": DANA_SA,
            "DANA_GA": DANA_GA, "ADAM": ADAM, "ADAM_SA": ADAM_SA, "ADAM_GA": ADAM_GA, "GA_LAYER": GA_LAYER}
CXXFLAGS = ["-std=c++17", "-O2", "-ffp-contract=off", "-fPIC", "-shared", "-Wall", "-Wextra"]


def build(force=False, src=_SRC, out=_LIB):
    """Compile the oracle with g++ (no fast-math, no FMA contraction)."""
    if not force and os.path.exists(out) and os.path.getmtime(out) >= os.path.getmtime(src):
        return out
    tmp = f"{out}.{os.getpid()}.tmp"          # several test workers may build at once
    try:
        subprocess.check_call(["g++", *CXXFLAGS, "-o", tmp, src])
    except OSError:   # the compiler itself is missing
        if os.path.exists(out) and not force:  # no compiler here: the library that travelled with the tree
            return out
        raise
    os.replace(tmp, out)
    return out


def _bind(path):
    lib = ctypes.CDLL(path)
    c = ctypes
    lib.gao_create.restype = c.c_void_p
    lib.gao_create.argtypes = [c.c_int64, c.c_int, c.c_double, c.c_double, c.c_double, c.c_int, c.c_int]
    lib.gao_destroy.argtypes = [c.c_void_p]
    lib.gao_set_c_order.argtypes = [c.c_void_p, c.c_int]
    lib.gao_set_eps.argtypes = [c.c_void_p, c.c_double]
    lib.gao_set_lr.argtypes = [c.c_void_p, c.c_double]
    lib.gao_set_weight_decay.argtypes = [c.c_void_p, c.c_double]
    lib.gao_set_nesterov.argtypes = [c.c_void_p, c.c_int]
    lib.gao_set_params.argtypes = [c.c_void_p, c.c_void_p]
    lib.gao_pull.argtypes = [c.c_void_p, c.c_int]
    lib.gao_push.restype = c.c_int64
    lib.gao_push.argtypes = [c.c_void_p, c.c_int, c.c_void_p]
    lib.gao_gap.argtypes = [c.c_void_p, c.c_int, c.c_void_p]
    lib.gao_k_done.restype = c.c_int64
    lib.gao_k_done.argtypes = [c.c_void_p]
    lib.gao_iter.restype = c.c_int64
    lib.gao_iter.argtypes = [c.c_void_p, c.c_int]
    lib.gao_set_state.argtypes = [c.c_void_p] * 6 + [c.c_int64, c.c_int64, c.c_void_p]
    lib.gao_set_dana_sum.argtypes = [c.c_void_p, c.c_int]
    lib.gao_set_layers.restype = c.c_int
    lib.gao_set_layers.argtypes = [c.c_void_p, c.c_void_p, c.c_int]
    lib.gao_layer_state.argtypes = [c.c_void_p, c.c_void_p, c.c_void_p]
    lib.gao_set_adam.argtypes = [c.c_void_p, c.c_double, c.c_double]
    lib.gao_k_c.restype = c.c_int64
    lib.gao_k_c.argtypes = [c.c_void_p]
    lib.gao_stats.argtypes = [c.c_void_p, c.c_void_p, c.c_void_p]
    lib.gao_get.restype = c.c_int
    lib.gao_get.argtypes = [c.c_void_p, c.c_int, c.c_void_p]
    lib.gao_sent_f32.argtypes = [c.c_void_p, c.c_int, c.c_void_p]
    return lib


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = _bind(build())
    return _lib


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


class Oracle:
    """One simulated master. precision=32 computes in fp32 (the parity reference for the
    fp32 CUDA path); precision=64 runs the same steps in fp64."""

    THETA, V, M, C = 0, 1, 2, 3

    def __init__(self, n_params, n_workers, lr, momentum, c_beta, variant, precision=32,
                 c_order=0, eps=None, dana_sum=1, beta2=0.999, adam_eps=1e-8, _lib=None):
        """For the Adam variants `momentum` is beta_1."""
        self._l = _lib if _lib is not None else lib()
        self.d, self.n = int(n_params), int(n_workers)
        self._h = self._l.gao_create(self.d, self.n, lr, momentum, c_beta, variant, precision)
        if not self._h:
            raise ValueError("gao_create failed")
        self.variant = variant
        self._l.gao_set_c_order(self._h, c_order)
        self._l.gao_set_dana_sum(self._h, dana_sum)
        self._l.gao_set_adam(self._h, beta2, adam_eps)
        if eps is not None:
            self._l.gao_set_eps(self._h, eps)

    def __del__(self):
        if getattr(self, "_h", None):
            self._l.gao_destroy(self._h)
            self._h = None

    def set_params(self, theta0):
        a = _f32(theta0)
        assert a.shape == (self.d,)
        self._l.gao_set_params(self._h, a.ctypes.data)

    def set_layers(self, offsets):
        """GA_LAYER: layer p = elements [offsets[p], offsets[p+1]); default is one layer (global Gap)."""
        off = np.ascontiguousarray(offsets, dtype=np.int64)
        assert self._l.gao_set_layers(self._h, off.ctypes.data, len(off) - 1) == 0, "bad layer offsets"
        self.n_layers = len(off) - 1

    def layer_state(self):
        """(Gap of every layer at the last arrival, m_p of every layer)."""
        n = getattr(self, "n_layers", 1)
        g, m = np.empty(n), np.empty(n)
        self._l.gao_layer_state(self._h, g.ctypes.data, m.ctypes.data)
        return g, m

    def set_nesterov(self, on=True):
        self._l.gao_set_nesterov(self._h, int(on))

    def set_weight_decay(self, wd):
        self._l.gao_set_weight_decay(self._h, wd)

    def set_lr(self, lr):
        self._l.gao_set_lr(self._h, lr)

    def pull(self, worker):
        assert 0 <= worker < self.n
        self._l.gao_pull(self._h, worker)

    def push(self, worker, grad):
        assert 0 <= worker < self.n
        g = _f32(grad)
        assert g.shape == (self.d,)
        return int(self._l.gao_push(self._h, worker, g.ctypes.data))

    def push_batch(self, schedule, grads):
        """push(i, g) then pull(i) for each arrival, in order. Returns the delays."""
        delays = []
        for i, g in zip(schedule, grads):
            delays.append(self.push(i, g))
            self.pull(i)
        return delays

    def get(self, which):
        out = np.empty(self.d, dtype=np.float64)
        rc = self._l.gao_get(self._h, which, out.ctypes.data)
        assert rc == 0
        return out

    def saved(self, worker):
        return self.get(4 + worker)

    def worker_momentum(self, worker):
        """DANA: v^worker."""
        return self.get(100000 + worker)

    def second_moment(self):
        """Adam: v (the first moment is get(V))."""
        return self.get(200000)

    @property
    def is_adam(self):
        return self.variant in (ADAM, ADAM_SA, ADAM_GA)

    @property
    def is_dana(self):
        return self.variant in (DANA, DANA_SA, DANA_GA)

    def sent_f32(self, worker):
        out = np.empty(self.d, dtype=np.float32)
        self._l.gao_sent_f32(self._h, worker, out.ctypes.data)
        return out

    def gap(self, worker):
        out = np.empty(self.d, dtype=np.float64)
        self._l.gao_gap(self._h, worker, out.ctypes.data)
        return out

    def stats(self):
        s, m = ctypes.c_double(), ctypes.c_double()
        self._l.gao_stats(self._h, ctypes.byref(s), ctypes.byref(m))
        return s.value, m.value

    def state(self):
        """(theta, v, m, saved[N][d], iter[N], k_done, k_c); vectors as float64."""
        saved = np.stack([self.saved(i) for i in range(self.n)])
        iters = np.asarray([self.iter(i) for i in range(self.n)], dtype=np.int64)
        out = (self.get(self.THETA), self.get(self.V), self.get(self.M), saved, iters,
               self.k_done, int(self._l.gao_k_c(self._h)))
        if self.is_dana:
            out += (np.stack([self.worker_momentum(i) for i in range(self.n)]),)
        if self.is_adam:
            out += (self.second_moment(),)
        return out

    def set_state(self, theta, v, m, saved, iters, k_done, k_c, v_workers=None):
        a = [np.ascontiguousarray(x, dtype=np.float64) for x in (theta, v, m, saved)]
        assert a[0].shape == (self.d,) and a[3].shape == (self.n, self.d)
        it = np.ascontiguousarray(iters, dtype=np.int64)
        vw = None
        if self.is_dana:
            vw = np.ascontiguousarray(v_workers, dtype=np.float64)
            assert vw.shape == (self.n, self.d)
        if self.is_adam:      # the extra array is Adam's second moment
            vw = np.ascontiguousarray(v_workers, dtype=np.float64)
            assert vw.shape == (self.d,)
        self._l.gao_set_state(self._h, *(x.ctypes.data for x in a), it.ctypes.data, k_done, k_c,
                              None if vw is None else vw.ctypes.data)

    @property
    def k_done(self):
        return int(self._l.gao_k_done(self._h))

    def iter(self, worker):
        return int(self._l.gao_iter(self._h, worker))


_LIB_OMP = os.path.join(_HERE, "libga_oracle_omp.so")


def build_openmp(force=False):
    """The same source split across threads (-fopenmp -DGAO_OPENMP): only for timing the oracle
    on all host cores; parity always uses the single-threaded build."""
    if not force and os.path.exists(_LIB_OMP) and os.path.getmtime(_LIB_OMP) >= os.path.getmtime(_SRC):
        return _LIB_OMP
    tmp = f"{_LIB_OMP}.{os.getpid()}.tmp"
    try:
        subprocess.check_call(["g++", *CXXFLAGS, "-fopenmp", "-DGAO_OPENMP", "-o", tmp, _SRC])
    except OSError:
        if os.path.exists(_LIB_OMP) and not force:
            return _LIB_OMP
        raise
    os.replace(tmp, _LIB_OMP)
    return _LIB_OMP


def lib_openmp():
    return _bind(build_openmp())
