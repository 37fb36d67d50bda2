"""Python binding of the Gap-Aware master library (include/ga.h).

Argument marshalling only: every step of the update runs in the CUDA kernels of libga.so.
There is no CPU fallback -- importing works anywhere (so the exported symbols can be checked),
but creating an engine without the library or without a CUDA device raises.

    eng = Engine(n_params, n_workers, lr=0.1, momentum=0.9, c_beta=0.999, variant=GA_GA)
    eng.set_params(theta0)                      # torch.float32 CUDA tensor
    delays = eng.push_batch(workers, grads)     # grads: list of CUDA tensors
    theta = eng.get(GA_THETA)
"""
import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("GA_LIBRARY") or os.path.join(_HERE, "libga.so")   # GA_LIBRARY: another build

(GA_ASGD, GA_SA, GA_GA, GA_SA_GRAD, GA_DANA, GA_DANA_SA, GA_DANA_GA, GA_ADAM, GA_ADAM_SA,
 GA_ADAM_GA, GA_GA_LAYER) = range(11)
GA_OK, GA_ERR_ARG, GA_ERR_STATE, GA_ERR_OOM, GA_ERR_CUDA = 0, -1, -2, -3, -4
GA_THETA, GA_V, GA_M, GA_C, GA_V2 = 0, 1, 2, 3, 4
(GA_OPT_C_ORDER, GA_OPT_MATH, GA_OPT_STATS, GA_OPT_WINDOW, GA_OPT_ADAM_BETA2, GA_OPT_ADAM_EPS,
 GA_OPT_WEIGHT_DECAY, GA_OPT_NESTEROV) = range(8)
GA_MAX_WINDOW = 16
GA_NOALLOC_MAX_PARAMS = 1 << 28
GA_STATS_LOG = 4096
VARIANTS = {"ASGD": GA_ASGD, "SA": GA_SA, "GA": GA_GA, "SA_GRAD": GA_SA_GRAD, "DANA": GA_DANA,
            "DANA_SA": GA_DANA_SA, "DANA_GA": GA_DANA_GA, "ADAM": GA_ADAM, "ADAM_SA": GA_ADAM_SA,
            "ADAM_GA": GA_ADAM_GA, "GA_LAYER": GA_GA_LAYER}

# every symbol include/ga.h declares: name -> (restype, argtypes)
_c = ctypes
_SIGNATURES = {
    "ga_create": (_c.c_void_p, [_c.c_size_t, _c.c_int, _c.c_float, _c.c_float, _c.c_float, _c.c_int]),
    "ga_workspace_bytes": (_c.c_size_t, [_c.c_size_t, _c.c_int, _c.c_int]),
    "ga_create_in": (_c.c_void_p, [_c.c_size_t, _c.c_int, _c.c_float, _c.c_float, _c.c_float, _c.c_int, _c.c_void_p,
                                   _c.c_size_t]),
    "ga_destroy": (None, [_c.c_void_p]),
    "ga_set_stream": (_c.c_int, [_c.c_void_p, _c.c_void_p]),
    "ga_set_lr": (_c.c_int, [_c.c_void_p, _c.c_float]),
    "ga_set_layers": (_c.c_int, [_c.c_void_p, _c.c_void_p, _c.c_int]),
    "ga_num_layers": (_c.c_int, [_c.c_void_p]),
    "ga_get_layer_state": (_c.c_int, [_c.c_void_p, _c.c_void_p, _c.c_void_p]),
    "ga_set_params": (_c.c_int, [_c.c_void_p, _c.c_void_p]),
    "ga_pull": (_c.c_void_p, [_c.c_void_p, _c.c_int]),
    "ga_saved": (_c.c_void_p, [_c.c_void_p, _c.c_int]),
    "ga_push": (_c.c_int64, [_c.c_void_p, _c.c_int, _c.c_void_p]),
    "ga_push_batch": (_c.c_int, [_c.c_void_p, _c.c_void_p, _c.c_void_p, _c.c_int, _c.c_void_p]),
    "ga_push_batch_host": (_c.c_int, [_c.c_void_p, _c.c_void_p, _c.c_void_p, _c.c_int, _c.c_void_p, _c.c_void_p]),
    "ga_get": (_c.c_int, [_c.c_void_p, _c.c_int, _c.c_void_p]),
    "ga_get_worker_momentum": (_c.c_int, [_c.c_void_p, _c.c_int, _c.c_void_p]),
    "ga_gap": (_c.c_int, [_c.c_void_p, _c.c_int, _c.c_void_p]),
    "ga_set_option": (_c.c_int, [_c.c_void_p, _c.c_int, _c.c_double]),
    "ga_get_stats": (_c.c_int, [_c.c_void_p, _c.c_void_p, _c.c_void_p]),
    "ga_get_stats_window": (_c.c_int, [_c.c_void_p, _c.c_void_p, _c.c_void_p, _c.c_int]),
    "ga_num_arrivals": (_c.c_int64, [_c.c_void_p]),
    "ga_worker_iter": (_c.c_int64, [_c.c_void_p, _c.c_int]),
    "ga_export_state": (_c.c_size_t, [_c.c_void_p, _c.c_void_p, _c.c_size_t]),
    "ga_import_state": (_c.c_int, [_c.c_void_p, _c.c_void_p, _c.c_size_t]),
    "ga_gap_stats_noalloc": (_c.c_int, [_c.c_void_p, _c.c_void_p, _c.c_void_p, _c.c_size_t, _c.c_float, _c.c_float,
                                        _c.c_int64, _c.c_void_p, _c.c_void_p]),
    "ga_selftest_exact_forms": (_c.c_int64, [_c.c_int, _c.c_void_p]),
    "ga_selftest_bounded_wait": (_c.c_int, [_c.c_void_p, _c.c_void_p]),
    "ga_last_error": (_c.c_char_p, []),
}

_lib = None


class GaError(RuntimeError):
    def __init__(self, code, message):
        super().__init__(f"[{code}] {message}")
        self.code = code


def lib():
    """The loaded C library. Raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_1909_10802_b200.build`")
        l = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(l, name)
            fn.restype = res
            fn.argtypes = args
        _lib = l
    return _lib


def last_error():
    return lib().ga_last_error().decode()


def _check(rc):
    if rc < 0:
        raise GaError(rc, last_error())
    return rc


def _ptr(t):
    """Device (or host) address of a tensor, an int address, or None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def gap_stats_noalloc(theta, saved, m, lr_max, c_beta, n_refreshes, out, stream=None):
    """ga_gap_stats_noalloc: sum and max of the parameter-wise Gap from three CUDA float32
    tensors into `out` (two float64 on the device). Allocates nothing, needs no Engine; meant for
    callers that must not touch the device allocator (see include/ga.h)."""
    import torch
    n = theta.numel()
    assert saved.numel() >= n and m.numel() >= n
    assert out.is_cuda and out.dtype == torch.float64 and out.numel() >= 2
    raw = (stream if stream is not None else torch.cuda.current_stream()).cuda_stream
    _check(lib().ga_gap_stats_noalloc(theta.data_ptr(), saved.data_ptr(), m.data_ptr(), n, lr_max, c_beta,
                                      n_refreshes, out.data_ptr(), raw))
    return out


def workspace_bytes(n_params, n_workers, variant=GA_GA):
    """ga_workspace_bytes: device bytes an Engine(..., workspace=...) of this shape needs."""
    if isinstance(variant, str):
        variant = VARIANTS[variant]
    n = lib().ga_workspace_bytes(int(n_params), int(n_workers), variant)
    if n == 0:
        raise GaError(GA_ERR_ARG, last_error())
    return n


def selftest_exact_forms(level=0, stream=None):
    """ga_selftest_exact_forms: operands on which the kernels' short exact forms differ from the
    IEEE routines on the current device (0 = they agree everywhere they are used)."""
    import torch
    raw = (stream if stream is not None else torch.cuda.current_stream()).cuda_stream
    return _check(lib().ga_selftest_exact_forms(level, raw))


class Engine:
    """One master. Thin wrapper: methods carry the names of the C calls without the prefix."""

    def __init__(self, n_params, n_workers, lr=0.1, momentum=0.9, c_beta=0.999, variant=GA_GA,
                 stream=None, workspace=None):
        """workspace: a CUDA tensor (any dtype) of at least workspace_bytes(...) bytes in which the
        engine keeps its state (ga_create_in); the engine holds a reference to it."""
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("the Gap-Aware master needs a CUDA device; there is no CPU path")
        self._torch = torch
        self._l = lib()
        if isinstance(variant, str):
            variant = VARIANTS[variant]
        self.n_params, self.n_workers, self.variant = int(n_params), int(n_workers), variant
        torch.cuda.init()
        torch.zeros(1, device="cuda")      # make sure a context exists on the current device
        self._workspace = workspace
        if workspace is None:
            self._h = self._l.ga_create(self.n_params, self.n_workers, lr, momentum, c_beta, variant)
        else:
            assert workspace.is_cuda and workspace.is_contiguous()
            self._h = self._l.ga_create_in(self.n_params, self.n_workers, lr, momentum, c_beta, variant,
                                           workspace.data_ptr(), workspace.numel() * workspace.element_size())
        if not self._h:
            raise GaError(GA_ERR_ARG, last_error())
        self.set_stream(stream if stream is not None else torch.cuda.current_stream())

    def close(self):
        if getattr(self, "_h", None):
            self._l.ga_destroy(self._h)
            self._h = None

    __del__ = close

    # -- plumbing
    def set_stream(self, stream):
        raw = stream if isinstance(stream, int) else stream.cuda_stream
        _check(self._l.ga_set_stream(self._h, raw))

    def set_layers(self, offsets):
        import numpy as np
        off = np.ascontiguousarray(offsets, dtype=np.int64)
        _check(self._l.ga_set_layers(self._h, off.ctypes.data, len(off) - 1))

    @property
    def n_layers(self):
        return _check(self._l.ga_num_layers(self._h))

    def get_layer_state(self):
        """(Gap of every layer at the last arrival, m_p of every layer) as numpy arrays."""
        import numpy as np
        n = self.n_layers
        g, m = np.empty(n, np.float32), np.empty(n, np.float32)
        _check(self._l.ga_get_layer_state(self._h, g.ctypes.data, m.ctypes.data))
        return g, m

    def set_lr(self, lr):
        _check(self._l.ga_set_lr(self._h, lr))

    def set_option(self, key, value):
        _check(self._l.ga_set_option(self._h, key, float(value)))

    def _grad_ok(self, g):
        if not isinstance(g, int):
            assert g.is_cuda and g.dtype == self._torch.float32 and g.is_contiguous()
            assert g.numel() >= self.n_params

    # -- the master's calls
    def set_params(self, theta0):
        self._grad_ok(theta0)
        _check(self._l.ga_set_params(self._h, _ptr(theta0)))

    def pull(self, worker):
        """Returns a torch view (n_params floats) of the worker's saved copy."""
        p = self._l.ga_pull(self._h, worker)
        if not p:
            raise GaError(GA_ERR_ARG, last_error())
        return self.saved_view(p)

    def saved_ptr(self, worker):
        p = self._l.ga_saved(self._h, worker)
        if not p:
            raise GaError(GA_ERR_ARG, last_error())
        return p

    def saved(self, worker):
        return self.saved_view(self.saved_ptr(worker))

    def saved_view(self, address):
        torch = self._torch
        iface = {"shape": (self.n_params,), "typestr": "<f4", "data": (address, False), "version": 2}

        class _Holder:
            __cuda_array_interface__ = iface

        return torch.as_tensor(_Holder(), device="cuda")

    def push(self, worker, grad):
        self._grad_ok(grad)
        return _check(self._l.ga_push(self._h, worker, _ptr(grad)))

    def push_batch(self, schedule, grads, return_launches=False):
        k = len(schedule)
        assert len(grads) == k
        for g in grads:
            self._grad_ok(g)
        sched = (ctypes.c_int * k)(*schedule)
        ptrs = (ctypes.c_void_p * k)(*[_ptr(g) for g in grads])
        delays = (ctypes.c_int64 * k)()
        launches = _check(self._l.ga_push_batch(self._h, sched, ptrs, k, delays))
        return (list(delays), launches) if return_launches else list(delays)

    def push_batch_raw(self, sched_array, ptr_array, k, delays_array):
        """ga_push_batch on caller-kept ctypes arrays (c_int[k], c_void_p[k], c_int64[k]): the
        lean path for loops over small vectors, where building arrays per call would dominate.
        Returns the number of launches."""
        rc = self._l.ga_push_batch(self._h, sched_array, ptr_array, k, delays_array)
        if rc < 0:
            raise GaError(rc, last_error())
        return rc

    def push_batch_host(self, schedule, grads_host, sent_out_host=None):
        """grads_host / sent_out_host: CPU tensors (pinned for speed) of n_params floats."""
        k = len(schedule)
        torch = self._torch
        for t in list(grads_host) + list(sent_out_host or []):
            assert not t.is_cuda and t.dtype == torch.float32 and t.is_contiguous() and t.numel() >= self.n_params
        sched = (ctypes.c_int * k)(*schedule)
        ptrs = (ctypes.c_void_p * k)(*[t.data_ptr() for t in grads_host])
        outs = (ctypes.c_void_p * k)(*[t.data_ptr() for t in sent_out_host]) if sent_out_host else None
        delays = (ctypes.c_int64 * k)()
        launches = _check(self._l.ga_push_batch_host(self._h, sched, ptrs, k, delays, outs))
        return list(delays), launches

    def get(self, which, out=None):
        torch = self._torch
        if out is None:
            out = torch.empty(self.n_params, dtype=torch.float32, device="cuda")
        _check(self._l.ga_get(self._h, which, _ptr(out)))
        return out

    def get_worker_momentum(self, worker, out=None):
        torch = self._torch
        if out is None:
            out = torch.empty(self.n_params, dtype=torch.float32, device="cuda")
        _check(self._l.ga_get_worker_momentum(self._h, worker, _ptr(out)))
        return out

    def gap(self, worker, out=None):
        torch = self._torch
        if out is None:
            out = torch.empty(self.n_params, dtype=torch.float32, device="cuda")
        _check(self._l.ga_gap(self._h, worker, _ptr(out)))
        return out

    def get_stats(self):
        s, m = ctypes.c_double(), ctypes.c_double()
        _check(self._l.ga_get_stats(self._h, ctypes.byref(s), ctypes.byref(m)))
        return s.value, m.value

    def get_stats_window(self, cap=GA_STATS_LOG):
        """[(sum of the Gap, max of the Gap)] for every arrival of the most recent push call, oldest first."""
        s, m = (ctypes.c_double * cap)(), (ctypes.c_double * cap)()
        n = _check(self._l.ga_get_stats_window(self._h, s, m, cap))
        return list(zip(s[:n], m[:n]))

    @property
    def num_arrivals(self):
        return _check(self._l.ga_num_arrivals(self._h))

    def worker_iter(self, worker):
        return _check(self._l.ga_worker_iter(self._h, worker))

    def export_state(self):
        need = self._l.ga_export_state(self._h, None, 0)
        if need == 0:
            raise GaError(GA_ERR_CUDA, last_error())
        buf = ctypes.create_string_buffer(need)
        if self._l.ga_export_state(self._h, buf, need) != need:
            raise GaError(GA_ERR_CUDA, last_error())
        return buf.raw

    def import_state(self, blob):
        _check(self._l.ga_import_state(self._h, blob, len(blob)))


# ---- checkpoint blobs (layout of ga_export_state): header, iter[N], theta, v, m, saved[N][d]
_HEADER = "<IIqqqqffffiiiiiiffff"
_MAGIC = 0x47415331


def unpack_state(blob):
    """Checkpoint blob -> dict of header fields and numpy arrays (copies)."""
    import struct

    import numpy as np
    hs = struct.calcsize(_HEADER)
    (magic, version, d, n, k_done, k_c, lr, gamma, beta, eps, variant, c_order, fast_math, stats,
     window, nesterov, beta2, adam_eps, lr_max, weight_decay) = struct.unpack_from(_HEADER, blob, 0)
    if magic != _MAGIC or version != 2:
        raise ValueError("not a Gap-Aware master checkpoint")
    off = hs
    iters = np.frombuffer(blob, dtype=np.int64, count=n, offset=off).copy()
    off += 8 * n
    dana = variant in (GA_DANA, GA_DANA_SA, GA_DANA_GA)
    adam = variant in (GA_ADAM, GA_ADAM_SA, GA_ADAM_GA)
    rows = 3 + n * (2 if dana else 1) + (1 if adam else 0)
    vecs = np.frombuffer(blob, dtype=np.float32, count=rows * d, offset=off).reshape(rows, d).copy()
    extra = {"v_workers": vecs[3 + n:]} if dana else {"v2": vecs[3 + n]} if adam else {}
    extra.update(beta2=beta2, adam_eps=adam_eps, lr_max=lr_max, weight_decay=weight_decay, nesterov=nesterov)
    if variant == GA_GA_LAYER:
        at = off + 4 * rows * d
        nl = int(np.frombuffer(blob, dtype=np.int64, count=1, offset=at)[0])
        extra["layer_offsets"] = np.frombuffer(blob, dtype=np.int64, count=nl + 1, offset=at + 8).copy()
        extra["m_layer"] = np.frombuffer(blob, dtype=np.float32, count=nl, offset=at + 8 * (nl + 2)).copy()
    return dict(**extra, d=d, n_workers=n, k_done=k_done, k_c=k_c, lr=lr, momentum=gamma, c_beta=beta, eps=eps,
                variant=variant, c_order=c_order, fast_math=fast_math, stats=stats, window=window,
                iter=iters, theta=vecs[0], v=vecs[1], m=vecs[2], saved=vecs[3:3 + n])


def pack_state(st):
    """Inverse of unpack_state."""
    import struct

    import numpy as np
    head = struct.pack(_HEADER, _MAGIC, 2, st["d"], st["n_workers"], st["k_done"], st["k_c"], st["lr"],
                       st["momentum"], st["c_beta"], st["eps"], st["variant"], st["c_order"],
                       st["fast_math"], st["stats"], st["window"], st.get("nesterov", 0), st.get("beta2", 0.999),
                       st.get("adam_eps", 1e-8), st.get("lr_max", st["lr"]), st.get("weight_decay", 0.0))
    parts = [head, np.ascontiguousarray(st["iter"], dtype=np.int64).tobytes()]
    for name in ("theta", "v", "m", "saved") + tuple(x for x in ("v_workers", "v2") if x in st):
        a = np.ascontiguousarray(st[name], dtype=np.float32)
        parts.append(a.tobytes())
    if "layer_offsets" in st:
        lo = np.ascontiguousarray(st["layer_offsets"], dtype=np.int64)
        parts += [np.int64(len(lo) - 1).tobytes(), lo.tobytes(),
                  np.ascontiguousarray(st["m_layer"], dtype=np.float32).tobytes()]
    return b"".join(parts)
