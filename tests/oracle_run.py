"""Runs the CPU oracle through a synthetic workload (test infrastructure)."""
import numpy as np

import oracle


def run_oracle(wl, variant, n_arrivals=None, idx=None, precision=32, c_order=0, checkpoints=(),
               schedule=None):
    """Push+pull every arrival of the workload's schedule through the oracle, restricted to the
    global element indices `idx` (None = all). Returns (oracle, delays, {arrival: snapshot of
    (theta, v, m)} for the requested checkpoints)."""
    d = wl.d if idx is None else len(idx)
    o = oracle.Oracle(d, wl.n_workers, wl.lr, wl.momentum, wl.c_beta,
                      oracle.VARIANTS[variant],
                      precision=precision, c_order=c_order)
    if variant == "GA_LAYER":
        if idx is None:
            o.set_layers(wl.seg_off)
        else:                        # a contiguous range made of whole layers: those layers alone
            off = [int(x) for x in wl.seg_off]
            j0, j1 = int(idx[0]), int(idx[-1]) + 1
            assert len(idx) == j1 - j0 and j0 in off and j1 in off, "layer norms need whole layers"
            o.set_layers([x - j0 for x in off[off.index(j0):off.index(j1) + 1]])
    o.set_params(wl.theta0(idx))
    sched = (schedule if schedule is not None else wl.schedule())
    sched = sched[:n_arrivals if n_arrivals is not None else len(sched)]
    delays, snaps = [], {}
    for k, i in enumerate(sched, start=1):
        g = wl.grad(k, o.sent_f32(i), idx)
        delays.append(o.push(i, g))
        o.pull(i)
        if k in checkpoints:
            snaps[k] = (o.get(o.THETA), o.get(o.V), o.get(o.M))
    return o, delays, snaps


def within(got, ref, tol=1e-5):
    """max |got - ref| <= tol * (1 + |ref|), elementwise."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    return bool(np.all(np.abs(got - ref) <= tol * (1.0 + np.abs(ref))))


def worst(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    return float(np.max(np.abs(got - ref) / (1.0 + np.abs(ref))))
