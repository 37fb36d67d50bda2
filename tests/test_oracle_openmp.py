"""The all-cores build of the oracle (-fopenmp -DGAO_OPENMP, timed by the benchmark's CPU leg)
against the single-threaded parity build: same source, loops over parameters split across
threads, so every vector must come out bit for bit the same."""
import numpy as np
import pytest

import oracle
import workloads as W


@pytest.mark.parametrize("variant", ["GA", "SA", "ASGD", "SA_GRAD", "DANA_GA", "DANA_SA", "ADAM_GA", "ADAM"])
def test_openmp_build_equals_single_thread(variant):
    wl = W.config("mini")
    omp = oracle.lib_openmp()
    res = []
    for lib in (None, omp):
        for c_order in ((0, 1) if variant in ("GA", "DANA_GA", "ADAM_GA") else (0,)):
            o = oracle.Oracle(wl.d, wl.n_workers, wl.lr, wl.momentum, wl.c_beta, oracle.VARIANTS[variant],
                              c_order=c_order, _lib=lib)
            o.set_params(wl.theta0())
            delays, stats = [], []
            for k, i in enumerate(wl.schedule(), start=1):
                delays.append(o.push(i, wl.grad(k, o.sent_f32(i))))
                stats.append(o.stats())
                o.pull(i)
            vecs = [o.get(o.THETA), o.get(o.V), o.get(o.M)] + [o.saved(i) for i in range(wl.n_workers)]
            res.append((delays, stats, vecs))
    half = len(res) // 2
    for (d1, s1, v1), (d2, s2, v2) in zip(res[:half], res[half:]):
        assert d1 == d2
        for a, b in zip(v1, v2):
            assert np.array_equal(a, b, equal_nan=True)
        for (sa, ma), (sb, mb) in zip(s1, s2):        # the fp64 sum is taken in another order
            assert ma == mb and abs(sa - sb) <= 1e-12 * max(1.0, abs(sa))
