"""Drives an Engine through a synthetic workload: the simulated workers' side of the loop.

For every window of the arrival schedule the stand-in gradients are generated on the device
from the parameters each worker was last sent, then the window goes to ga_push_batch. The
generators come from the `workloads` module; no update arithmetic happens here.
"""
import ctypes

import workloads as W

from . import Engine, GA_MAX_WINDOW, GA_OPT_WINDOW, VARIANTS


class Run:
    def __init__(self, wl, variant="GA", window=GA_MAX_WINDOW, options=None, torch_device="cuda",
                 shard=None, workspace=None):
        """shard = (j0, n): this engine holds parameters [j0, j0+n) of the workload's vector
        (every step is independent per parameter, so ranks need no exchange)."""
        import torch
        self.torch = torch
        self.wl = wl
        self.j0, self.n = shard if shard is not None else (0, wl.d)
        self.dev = wl.device(torch_device, self.j0, self.n)
        self.window = window
        self.engine = Engine(self.n, wl.n_workers, wl.lr, wl.momentum, wl.c_beta, VARIANTS[variant],
                             workspace=workspace)    # workspace: a CUDA tensor that holds the engine's state
        self.engine.set_option(GA_OPT_WINDOW, window)
        if variant == "GA_LAYER":          # the workload's tensors are the layers
            # a layer's norm needs the whole layer on one rank: a shard must begin and end on layer
            # boundaries (shard.layer_shard_range), and holds the layers in between
            off = [int(x) for x in wl.seg_off]
            if self.j0 not in off or self.j0 + self.n not in off:
                raise ValueError("a shard of the layer-wise Gap must consist of whole layers")
            l0, l1 = off.index(self.j0), off.index(self.j0 + self.n)
            self.engine.set_layers([x - self.j0 for x in off[l0:l1 + 1]])
        for key, value in (options or {}).items():
            self.engine.set_option(key, value)
        theta0 = torch.empty(self.n, dtype=torch.float32, device=torch_device)
        self.dev.theta0(theta0)
        self.engine.set_params(theta0)
        del theta0
        self.grads = [torch.empty(self.n, dtype=torch.float32, device=torch_device) for _ in range(window)]
        self._rows = [self.engine.saved_ptr(i) for i in range(wl.n_workers)]   # stable for the engine's life
        self._grad_ptrs = [g.data_ptr() for g in self.grads]
        # arrays handed to ga_push_batch, kept across calls (the gradient buffers never move)
        self._sched = (ctypes.c_int * window)()
        self._ptrs = (ctypes.c_void_p * window)(*self._grad_ptrs)
        self._delays = (ctypes.c_int64 * window)()
        self.k = 0            # arrivals applied
        self.delays = []
        self.launches = 0

    def generate(self, workers):
        """Gradients of the next len(workers) arrivals into the gradient buffers."""
        for j, i in enumerate(workers):
            self.dev.grad_ptr(self.k + 1 + j, self._rows[i], self._grad_ptrs[j])

    def apply(self, workers):
        n = len(workers)
        self._sched[:n] = workers
        self.launches += self.engine.push_batch_raw(self._sched, self._ptrs, n, self._delays)
        delays = self._delays[:n]
        self.k += n
        self.delays += delays
        return delays

    def step(self, workers):
        self.generate(workers)
        return self.apply(workers)

    def run(self, n_arrivals=None):
        sched = self.wl.schedule()[self.k:n_arrivals if n_arrivals is not None else self.wl.arrivals]
        for win in W.windows(sched, self.window):
            self.step(win)
        return self.delays

    def close(self):
        self.engine.close()
        self.grads = []
