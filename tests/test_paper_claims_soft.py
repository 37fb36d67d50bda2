"""Qualitative statements of the paper checked on the synthetic workloads (CPU oracle only).

These are sanity checks of behaviour, not parity pins: Section 5.1 says E[G] = tau only if all
updates point the same way and that empirically E[G] < tau; Section 6 says GA penalises less
than SA, which divides by tau itself.
"""
import numpy as np
import pytest

import oracle
import workloads as W


@pytest.mark.parametrize("name,arrivals", [("C3", 500), ("C4", 2500), ("C5", 400)])
def test_mean_gap_is_below_the_delay(name, arrivals):
    wl = W.config(name)
    idx = wl.sample_indices(1024)
    o = oracle.Oracle(len(idx), wl.n_workers, wl.lr, wl.momentum, wl.c_beta, oracle.GA)
    o.set_params(wl.theta0(idx))
    gaps, taus = [], []
    for k, i in enumerate(wl.schedule()[:arrivals], start=1):
        taus.append(o.push(i, wl.grad(k, o.sent_f32(i), idx)))
        o.pull(i)
        gaps.append(o.stats()[0] / len(idx))
    half = arrivals // 2                      # after every worker has reported at least once
    assert 1.0 < np.mean(gaps[half:]) < np.mean(taus[half:])
    assert min(gaps) >= 1.0
