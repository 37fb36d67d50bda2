"""Parity of the CUDA library (through its C ABI) against the CPU oracle.

The fp32 oracle rounds exactly as the kernels' exact mode does, so whole trajectories are
compared element by element and must agree within 1e-5*(1+|ref|) -- and, as measured, bit for
bit. (The synthetic quadratic is unstable under the simulated delays for several of the
configurations, so a trajectory-level tolerance would be meaningless for anything but an
implementation that rounds identically; single arrivals from identical states are also
compared with the fp64 oracle, and fast-math mode is held to the tolerance the same way.)
"""
import numpy as np
import pytest

import oracle
import workloads as W
from tests.oracle_run import run_oracle, within, worst

pytestmark = pytest.mark.gpu

TOL = 1e-5     # max |gpu - ref| <= TOL * (1 + |ref|)


@pytest.fixture(scope="module")
def P():
    import torch
    assert torch.cuda.is_available()
    import paper_1909_10802_b200 as pkg
    pkg.lib()
    W.cuda_lib()
    return pkg


def _np(t):
    return t.detach().cpu().numpy()


def _same(a, b):
    """Equal element by element; NaN equals NaN (payload bits differ between CPU and GPU)."""
    return np.array_equal(np.asarray(a, dtype=np.float32), np.asarray(b, dtype=np.float32), equal_nan=True)


def _close(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    fin = np.isfinite(ref)
    if not np.array_equal(np.isnan(got), np.isnan(ref)):
        return False
    if not np.array_equal(got[~fin & ~np.isnan(ref)], ref[~fin & ~np.isnan(ref)]):
        return False
    return within(got[fin], ref[fin], TOL)


def _compare_engine(P, run, o, idx=None, label=""):
    """theta, v, m and derived C of the engine against the oracle (at idx if given)."""
    import torch
    sel = None if idx is None else torch.as_tensor(idx, device="cuda")
    names = (("theta", P.GA_THETA, o.THETA), ("v", P.GA_V, o.V))
    if run.engine.variant in (P.GA_GA, P.GA_DANA_GA, P.GA_ADAM_GA):
        names += (("m", P.GA_M, o.M), ("C", P.GA_C, o.C))
    if run.engine.variant in (P.GA_ADAM, P.GA_ADAM_SA, P.GA_ADAM_GA):
        names += (("v2", ("v2", 0), None),)
    if run.engine.variant in (P.GA_DANA, P.GA_DANA_SA, P.GA_DANA_GA):
        names += tuple((f"v^{i}", ("vw", i), None) for i in range(run.engine.n_workers))
    names += tuple((f"sent^{i}", ("sent", i), None) for i in range(min(run.engine.n_workers, 8)))
    if run.engine.variant == P.GA_GA_LAYER:
        gaps, m_layer = run.engine.get_layer_state()
        ogaps, om = o.layer_state()
        assert np.array_equal(gaps, ogaps.astype(np.float32)), f"{label}layer Gaps differ"
        assert np.array_equal(m_layer, om.astype(np.float32)), f"{label}layer m differ"
    for name, which, owhich in names:
        if isinstance(which, tuple):
            kind, i = which
            got = (run.engine.get_worker_momentum(i) if kind == "vw" else
                   run.engine.get(P.GA_V2) if kind == "v2" else run.engine.saved(i))
            ref = o.worker_momentum(i) if kind == "vw" else o.second_moment() if kind == "v2" else o.saved(i)
        else:
            got = run.engine.get(which)
            ref = o.get(owhich)
        got = _np(got if sel is None else got[sel])
        assert _close(got, ref), f"{label}{name}: outside {TOL}*(1+|ref|)"
        nbad = int(np.sum(~((got == ref.astype(np.float32)) | (np.isnan(got) & np.isnan(ref)))))
        assert nbad == 0, f"{label}{name}: {nbad} elements differ from the fp32 oracle in some bit"


# ----------------------------------------------------------------------------- generators
@pytest.mark.parametrize("name", ["mini", "C1"])
def test_device_generator_matches_cpu(P, name):
    import torch
    wl = W.config(name)
    dev = wl.device()
    t0 = torch.empty(wl.d, dtype=torch.float32, device="cuda")
    dev.theta0(t0)
    assert np.array_equal(_np(t0), wl.theta0())
    g = torch.empty_like(t0)
    for k in (1, 7):
        dev.grad_ptr(k, t0.data_ptr(), g.data_ptr())
        assert np.array_equal(_np(g), wl.grad(k, wl.theta0()))


def test_device_generator_sparse_rows_and_subrange(P):
    import torch
    wl = W.Workload(name="emb", segments=[64 * 300, 5000], n_workers=2, arrivals=4, schedule_kind="ticks",
                    seed=11, quad=False, emb_rows=300, emb_row=64, row_active_frac=0.1)
    dev = wl.device()
    z = torch.zeros(wl.d, dtype=torch.float32, device="cuda")
    g = torch.empty_like(z)
    dev.grad_ptr(3, z.data_ptr(), g.data_ptr())
    ref = wl.grad(3, np.zeros(wl.d, np.float32))
    assert np.array_equal(_np(g), ref) and 0.02 < (ref[:64 * 300] != 0).mean() < 0.25
    sub = wl.device(j0=1000, n=7777)
    gs = torch.empty(7777, dtype=torch.float32, device="cuda")
    sub.grad_ptr(3, z.data_ptr(), gs.data_ptr())
    assert np.array_equal(_np(gs), ref[1000:8777])


# ----------------------------------------------------------------------------- small, exhaustive
ALL_VARIANTS = ["GA", "SA", "ASGD", "SA_GRAD", "DANA", "DANA_SA", "DANA_GA", "ADAM", "ADAM_SA", "ADAM_GA",
                "GA_LAYER"]


@pytest.mark.parametrize("variant", ALL_VARIANTS)
@pytest.mark.parametrize("window", [1, 4, 16])
def test_mini_trajectory(P, variant, window):
    from paper_1909_10802_b200.runner import Run
    wl = W.config("mini")
    for c_order in ((0, 1) if variant in ("GA", "DANA_GA", "ADAM_GA") else (0,)):
        run = Run(wl, variant, window, options={P.GA_OPT_C_ORDER: c_order})
        delays = run.run()
        o, odelays, _ = run_oracle(wl, variant, c_order=c_order)
        assert delays == odelays
        _compare_engine(P, run, o, label=f"{variant}/c_order={c_order}/K={window}: ")
        for i in range(wl.n_workers):
            assert _same(_np(run.engine.saved(i)), o.saved(i))
            assert run.engine.worker_iter(i) == o.iter(i)
        run.close()


@pytest.mark.parametrize("d", [1, 3, 4, 5, 31, 33, 255, 1025])
def test_ragged_sizes(P, d):
    from paper_1909_10802_b200.runner import Run
    wl = W.Workload(name=f"d{d}", segments=[d], n_workers=3, arrivals=20, schedule_kind="ticks", seed=100 + d)
    run = Run(wl, "GA", 16)
    delays = run.run()
    o, odelays, _ = run_oracle(wl, "GA")
    assert delays == odelays
    _compare_engine(P, run, o)
    run.close()


# ----------------------------------------------------------------------------- the five workloads
def test_c1_full_with_checkpoints(P):
    """C1 (ResNet-20 shape, 8 workers, 1000 arrivals), every element, 3 checkpoints + the end."""
    from paper_1909_10802_b200.runner import Run
    wl = W.config("C1")
    cps = (250, 500, 750)
    o, odelays, snaps = run_oracle(wl, "GA", checkpoints=cps)
    run = Run(wl, "GA", 16)
    for cp in cps:
        run.run(cp)
        for which, ref in zip((P.GA_THETA, P.GA_V, P.GA_M), snaps[cp]):
            got = _np(run.engine.get(which))
            assert _close(got, ref) and _same(got, ref), f"checkpoint {cp}, vector {which}"
    run.run()
    assert run.delays == odelays
    _compare_engine(P, run, o)
    run.close()


def _sampled(P, name, variant, window, n_sample=4096, n_arrivals=None, options=None):
    from paper_1909_10802_b200.runner import Run
    wl = W.config(name)
    idx = wl.sample_indices(n_sample)
    run = Run(wl, variant, window, options=options)
    run.run(n_arrivals)
    o, odelays, _ = run_oracle(wl, variant, n_arrivals=n_arrivals, idx=idx)
    assert run.delays == odelays, "delays must be identical integers"
    _compare_engine(P, run, o, idx=idx, label=f"{name}/{variant}/K={window}: ")
    return run


@pytest.mark.parametrize("variant", ["GA", "SA", "ASGD"])
def test_c2_heterogeneous_workers(P, variant):
    _sampled(P, "C2", variant, 16).close()


@pytest.mark.parametrize("variant", ["DANA_GA", "ADAM_GA", "ADAM_SA", "SA_GRAD", "DANA_SA"])
def test_c2_heterogeneous_workers_other_masters(P, variant):
    """6,000 arrivals with widely spread delays (32 workers of log-normal speed) on the ResNet-20
    shape -- short enough for the two-parameters-per-thread layout -- for the appendix's masters."""
    _sampled(P, "C2", variant, 16, n_arrivals=6000).close()


def test_c3_window_invariance(P):
    """ResNet-50 shape: K = 1, 4, 16 all match the oracle and each other, bit for bit."""
    import torch
    ref = None
    for window in (16, 4, 1):
        run = _sampled(P, "C3", "GA", window, n_arrivals=2000 if window == 16 else 300)
        if window != 16:
            full = [run.engine.get(w).clone() for w in (P.GA_THETA, P.GA_V, P.GA_M)]
            if ref is None:
                ref = full
            else:
                assert all(torch.equal(a, b) for a, b in zip(ref, full)), "K=1 and K=4 disagree"
        run.close()
        torch.cuda.empty_cache()


@pytest.mark.parametrize("variant", ["DANA_GA", "DANA", "DANA_SA", "SA_GRAD", "ADAM", "ADAM_SA", "ADAM_GA"])
def test_c3_appendix_masters(P, variant):
    """The appendix's masters on the ResNet-50 shape (64 workers), fused windows of 16."""
    import torch
    _sampled(P, "C3", variant, 16, n_arrivals=400).close()
    torch.cuda.empty_cache()


def test_dana_push_then_pull_and_checkpoint(P):
    """DANA-GA through the stand-alone calls (the pull computes the look-ahead estimate) and
    through export/import (the workers' momentum vectors travel with the state)."""
    import torch
    eng, o, rng = _small_engine(P, n=3, variant=P.GA_DANA_GA)
    for step, i in enumerate([0, 1, 1, 2, 0]):
        g = rng.normal(size=eng.n_params).astype(np.float32)
        assert eng.push(i, torch.from_numpy(g).cuda()) == o.push(i, g)
        if step != 1:
            sent = eng.pull(i)
            o.pull(i)
            assert _same(_np(sent), o.saved(i))
    blob = eng.export_state()
    other = P.Engine(eng.n_params, 3, 0.1, 0.9, 0.999, P.GA_DANA_GA)
    other.import_state(blob)
    wrong = P.Engine(eng.n_params, 3, 0.1, 0.9, 0.999, P.GA_GA)
    with pytest.raises(P.GaError):
        wrong.import_state(blob)
    wrong.close()
    g = rng.normal(size=eng.n_params).astype(np.float32)
    for e_ in (eng, other):
        assert e_.push_batch([2], [torch.from_numpy(g).cuda()]) == [2]
    o.push_batch([2], [g])
    for e_ in (eng, other):
        for which, ow in ((P.GA_THETA, o.THETA), (P.GA_V, o.V), (P.GA_M, o.M)):
            assert _same(_np(e_.get(which)), o.get(ow))
        for i in range(3):
            assert _same(_np(e_.get_worker_momentum(i)), o.worker_momentum(i))
            assert _same(_np(e_.saved(i)), o.saved(i))
        e_.close()
    with pytest.raises(P.GaError):
        plain = P.Engine(100, 2)
        try:
            plain.get_worker_momentum(0)
        finally:
            plain.close()


def test_adam_options_and_checkpoint(P):
    """Adam-GA with non-default beta_2 / epsilon, stand-alone push + pull, export/import."""
    import torch
    d, n = 4099, 3
    rng = np.random.default_rng(9)
    th0 = rng.normal(size=d).astype(np.float32)
    eng = P.Engine(d, n, 0.01, 0.8, 0.99, P.GA_ADAM_GA)
    eng.set_option(P.GA_OPT_ADAM_BETA2, 0.95)
    eng.set_option(P.GA_OPT_ADAM_EPS, 1e-6)
    eng.set_params(torch.from_numpy(th0).cuda())
    o = oracle.Oracle(d, n, 0.01, 0.8, 0.99, oracle.ADAM_GA, beta2=0.95, adam_eps=1e-6)
    o.set_params(th0)
    for i in [0, 1, 2, 1, 0, 0]:
        g = rng.normal(size=d).astype(np.float32)
        assert eng.push(i, torch.from_numpy(g).cuda()) == o.push(i, g)
        assert _same(_np(eng.pull(i)), (o.pull(i), o.saved(i))[1])
    with pytest.raises(P.GaError):
        eng.set_option(P.GA_OPT_ADAM_BETA2, 0.9)          # not after the first arrival
    other = P.Engine(d, n, 0.5, 0.1, 0.5, P.GA_ADAM_GA)   # hyper-parameters come with the state
    other.import_state(eng.export_state())
    g = rng.normal(size=d).astype(np.float32)
    o.push_batch([2], [g])
    for e_ in (eng, other):
        e_.push_batch([2], [torch.from_numpy(g).cuda()])
        for which, ref in ((P.GA_THETA, o.get(o.THETA)), (P.GA_V, o.get(o.V)), (P.GA_V2, o.second_moment()),
                           (P.GA_M, o.get(o.M)), (P.GA_C, o.get(o.C))):
            assert _same(_np(e_.get(which)), ref), which
        e_.close()
    plain = P.Engine(64, 2)
    with pytest.raises(P.GaError):
        plain.get(P.GA_V2)
    plain.close()


@pytest.mark.parametrize("variant", ["GA", "SA", "DANA_GA", "ADAM_GA"])
def test_learning_rate_schedule(P, variant):
    """ga_set_lr between windows (a warm-up then a decay): eta_k changes, eta_max does not."""
    import torch
    wl = W.config("mini")
    from paper_1909_10802_b200.runner import Run
    run = Run(wl, variant, 4)
    o = oracle.Oracle(wl.d, wl.n_workers, wl.lr, wl.momentum, wl.c_beta, oracle.VARIANTS[variant])
    o.set_params(wl.theta0())
    sched = wl.schedule()
    k = 0
    for lr, upto in ((wl.lr / wl.n_workers, 12), (wl.lr, 36), (wl.lr * 0.1, 60)):
        run.engine.set_lr(lr)
        o.set_lr(lr)
        run.run(upto)
        while k < upto:
            i = sched[k]
            o.push(i, wl.grad(k + 1, o.sent_f32(i)))
            o.pull(i)
            k += 1
    _compare_engine(P, run, o, label=f"{variant} with schedule: ")
    blob = run.engine.export_state()
    assert abs(P.unpack_state(blob)["lr_max"] - np.float32(wl.lr)) < 1e-9
    assert abs(P.unpack_state(blob)["lr"] - np.float32(wl.lr * 0.1)) < 1e-9
    assert run.engine._l.ga_set_lr(run.engine._h, -1.0) == P.GA_ERR_ARG
    run.close()


def test_layer_gap_shapes(P):
    """Layer-wise Gap on real layer tables: ResNet-20 (65 tensors, some of 10 or 16 elements,
    odd offsets at the end) for 300 arrivals and ResNet-50 (161 tensors, 25.5M parameters, tiles
    of 4096) for 40 arrivals; the oracle runs on whole vectors."""
    import torch
    from paper_1909_10802_b200.runner import Run
    c1 = W.config("C1")
    r50 = W.Workload(name="r50x8", segments=W.resnet50_segments(), n_workers=8, arrivals=40,
                     schedule_kind="ticks", seed=77, sigma="loguniform")
    for wl, n in ((c1, 300), (r50, 40)):
        run = Run(wl, "GA_LAYER", 16)
        run.run(n)
        o, odelays, _ = run_oracle(wl, "GA_LAYER", n_arrivals=n)
        assert run.delays == odelays
        _compare_engine(P, run, o, label=f"{wl.name}/layer-wise: ")
        gaps = run.engine.get_layer_state()[0]
        assert gaps.min() >= 1.0 and gaps.max() > 1.5
        run.close()
        torch.cuda.empty_cache()


def test_layer_gap_special_cases_and_checkpoint(P):
    """One parameter per layer equals the parameter-wise kernel bit for bit; no layer table
    means the global Gap; the state (layer table and m_p included) survives export/import."""
    import torch
    d, n = 1537, 3
    rng = np.random.default_rng(12)
    th0 = torch.from_numpy(rng.normal(size=d).astype(np.float32)).cuda()
    sched = [0, 1, 2, 1, 0, 2, 2]
    grads = [torch.from_numpy(rng.normal(size=d).astype(np.float32)).cuda() for _ in sched]
    a = P.Engine(d, n, 0.1, 0.9, 0.999, P.GA_GA_LAYER)
    a.set_layers(np.arange(d + 1))
    b = P.Engine(d, n, 0.1, 0.9, 0.999, P.GA_GA)
    for e_ in (a, b):
        e_.set_params(th0)
    assert a.push_batch(sched, grads) == b.push_batch(sched, grads)
    assert torch.equal(a.get(P.GA_THETA), b.get(P.GA_THETA)) and torch.equal(a.get(P.GA_V), b.get(P.GA_V))
    assert np.array_equal(a.get_layer_state()[1], _np(b.get(P.GA_M)))
    a.close()
    b.close()
    # global Gap + checkpoint
    g = P.Engine(d, n, 0.1, 0.9, 0.999, P.GA_GA_LAYER)
    o = oracle.Oracle(d, n, 0.1, 0.9, 0.999, oracle.GA_LAYER)
    g.set_params(th0)
    o.set_params(_np(th0))
    g.push_batch(sched[:4], grads[:4])
    o.push_batch(sched[:4], [_np(x) for x in grads[:4]])
    h = P.Engine(d, n, 0.1, 0.9, 0.999, P.GA_GA_LAYER)
    h.set_layers([0, 100, d])                # replaced by the table in the state
    blob = g.export_state()
    h.import_state(blob)
    st = P.unpack_state(blob)
    assert list(st["layer_offsets"]) == [0, d] and P.pack_state(st) == blob
    o.push_batch(sched[4:], [_np(x) for x in grads[4:]])
    for e_ in (g, h):
        e_.push_batch(sched[4:], grads[4:])
        assert _same(_np(e_.get(P.GA_THETA)), o.get(o.THETA))
        assert np.array_equal(e_.get_layer_state()[0], o.layer_state()[0].astype(np.float32))
    # what this variant does not offer comes back as an error, not a fault
    l = P.lib()
    assert l.ga_set_layers(g._h, None, 1) == P.GA_ERR_STATE            # after the first arrival
    assert l.ga_gap(g._h, 0, th0.data_ptr()) == P.GA_ERR_STATE
    assert l.ga_set_option(h._h, P.GA_OPT_C_ORDER, 1.0) == P.GA_ERR_STATE
    plain = P.Engine(64, 2)
    assert l.ga_set_layers(plain._h, None, 1) == P.GA_ERR_STATE
    fresh = P.Engine(d, n, 0.1, 0.9, 0.999, P.GA_GA_LAYER)
    import ctypes
    bad = (ctypes.c_int64 * 3)(0, 50, d - 1)
    assert l.ga_set_layers(fresh._h, bad, 2) == P.GA_ERR_ARG
    for e_ in (g, h, plain, fresh):
        e_.close()


def test_sharded_runs_equal_the_whole(P):
    """The N > 1 layout on one GPU, one shard after the other: each rank owns a 128-byte aligned
    range of the vector; put together the shards are the single-engine result bit for bit."""
    import torch
    from paper_1909_10802_b200.runner import Run
    from paper_1909_10802_b200.shard import shard_range
    wl = W.config("mini")
    whole = Run(wl, "DANA_GA", 16)
    whole.run()
    parts = []
    for rank in range(3):
        j0, n = shard_range(wl.d, rank, 3)
        part = Run(wl, "DANA_GA", 16, shard=(j0, n))
        assert part.run() == whole.delays
        parts.append((part.engine.get(P.GA_THETA), part.engine.get(P.GA_M), part.engine.saved(1).clone()))
        part.close()
    for q, ref in enumerate((whole.engine.get(P.GA_THETA), whole.engine.get(P.GA_M), whole.engine.saved(1))):
        assert torch.equal(torch.cat([p[q] for p in parts]), ref)
    whole.close()


@pytest.mark.parametrize("variant", ["GA", "SA", "DANA_GA", "ADAM_GA", "GA_LAYER"])
def test_weight_decay(P, variant):
    """GA_OPT_WEIGHT_DECAY: lambda * theta_k joins the gradient before the penalty."""
    from paper_1909_10802_b200.runner import Run
    wl = W.config("mini")
    run = Run(wl, variant, 16, options={P.GA_OPT_WEIGHT_DECAY: 5e-4})
    run.run()
    o = oracle.Oracle(wl.d, wl.n_workers, wl.lr, wl.momentum, wl.c_beta, oracle.VARIANTS[variant])
    if variant == "GA_LAYER":
        o.set_layers(wl.seg_off)
    o.set_weight_decay(5e-4)
    o.set_params(wl.theta0())
    for k, i in enumerate(wl.schedule(), start=1):
        o.push(i, wl.grad(k, o.sent_f32(i)))
        o.pull(i)
    _compare_engine(P, run, o, label=f"{variant} with weight decay: ")
    assert abs(P.unpack_state(run.engine.export_state())["weight_decay"] - np.float32(5e-4)) < 1e-10
    assert run.engine._l.ga_set_option(run.engine._h, P.GA_OPT_WEIGHT_DECAY, -1.0) == P.GA_ERR_ARG
    run.close()


@pytest.mark.parametrize("variant", ["GA", "SA", "ASGD", "SA_GRAD", "GA_LAYER"])
def test_nesterov_step(P, variant):
    """GA_OPT_NESTEROV (with weight decay on top, the usual recipe of the paper's CIFAR runs)."""
    from paper_1909_10802_b200.runner import Run
    wl = W.config("mini")
    run = Run(wl, variant, 16, options={P.GA_OPT_NESTEROV: 1, P.GA_OPT_WEIGHT_DECAY: 1e-4})
    run.run()
    o = oracle.Oracle(wl.d, wl.n_workers, wl.lr, wl.momentum, wl.c_beta, oracle.VARIANTS[variant])
    if variant == "GA_LAYER":
        o.set_layers(wl.seg_off)
    o.set_nesterov()
    o.set_weight_decay(1e-4)
    o.set_params(wl.theta0())
    for k, i in enumerate(wl.schedule(), start=1):
        o.push(i, wl.grad(k, o.sent_f32(i)))
        o.pull(i)
    _compare_engine(P, run, o, label=f"{variant}, Nesterov: ")
    assert P.unpack_state(run.engine.export_state())["nesterov"] == 1
    run.close()
    dana = P.Engine(64, 2, 0.1, 0.9, 0.999, P.GA_DANA)
    assert dana._l.ga_set_option(dana._h, P.GA_OPT_NESTEROV, 1.0) == P.GA_ERR_STATE
    dana.close()


def test_c4_stragglers(P):
    import torch
    _sampled(P, "C4", "GA", 16).close()
    torch.cuda.empty_cache()


def test_c5_transformer_lm_full_size(P):
    """The benchmark configuration itself: 150M parameters, 32 saved copies, K = 16."""
    import torch
    _sampled(P, "C5", "GA", 16).close()
    torch.cuda.empty_cache()


@pytest.mark.parametrize("variant", ["DANA_GA", "ADAM_GA", "SA_GRAD"])
def test_c5_full_size_other_masters(P, variant):
    """150M parameters, 32 workers, K = 16 for the appendix's masters (DANA-GA adds 19 GB of
    per-worker momentum); 96 arrivals, sampled parameters against the oracle."""
    import torch
    _sampled(P, "C5", variant, 16, n_arrivals=96).close()
    torch.cuda.empty_cache()


# ----------------------------------------------------------------------------- single calls
def _small_engine(P, d=5003, n=4, variant=None, seed=5):
    import torch
    rng = np.random.default_rng(seed)
    th0 = rng.normal(size=d).astype(np.float32)
    eng = P.Engine(d, n, 0.1, 0.9, 0.999, P.GA_GA if variant is None else variant)
    eng.set_params(torch.from_numpy(th0).cuda())
    o = oracle.Oracle(d, n, 0.1, 0.9, 0.999, variant if variant is not None else oracle.GA)
    o.set_params(th0)
    return eng, o, rng


def test_push_then_pull_equals_batch_of_one(P):
    """ga_push + ga_pull (TMA bulk copy) as separate calls, including a second push without
    a pull in between."""
    import torch
    eng, o, rng = _small_engine(P)
    for step, i in enumerate([0, 1, 1, 2, 0, 3, 3]):
        g = rng.normal(size=eng.n_params).astype(np.float32)
        assert eng.push(i, torch.from_numpy(g).cuda()) == o.push(i, g)
        if step != 1:
            sent = eng.pull(i)
            o.pull(i)
            assert _same(_np(sent), o.saved(i))
    for which, ow in ((P.GA_THETA, o.THETA), (P.GA_V, o.V), (P.GA_M, o.M), (P.GA_C, o.C)):
        assert _same(_np(eng.get(which)), o.get(ow))
    for i in range(4):
        assert _same(_np(eng.saved(i)), o.saved(i)) and eng.worker_iter(i) == o.iter(i)
        assert _same(_np(eng.gap(i)), o.gap(i))
    eng.close()


def test_pull_bulk_copy_large(P):
    """A pull of a vector spanning many 16 KB bulk copies and a ragged last one."""
    import torch
    d = 3_000_017
    eng = P.Engine(d, 2, 0.1, 0.9, 0.999, P.GA_ASGD)
    th0 = torch.randn(d, device="cuda")
    eng.set_params(th0)
    g = torch.randn(d, device="cuda")
    eng.push(0, g)
    sent = eng.pull(1)
    assert torch.equal(sent, eng.get(P.GA_THETA)) and torch.equal(eng.saved(0), th0)
    eng.close()


def test_batch_with_repeated_workers_and_empty_batch(P):
    import torch
    eng, o, rng = _small_engine(P, n=3)
    sched = [0, 1, 0, 0, 2, 1, 2, 2]
    grads = [rng.normal(size=eng.n_params).astype(np.float32) for _ in sched]
    delays, launches = eng.push_batch(sched, [torch.from_numpy(g).cuda() for g in grads], return_launches=True)
    assert delays == o.push_batch(sched, grads)
    assert launches == len(W.windows(sched, 16)) == 5
    assert eng.push_batch([], []) == []
    for which, ow in ((P.GA_THETA, o.THETA), (P.GA_V, o.V), (P.GA_M, o.M)):
        assert _same(_np(eng.get(which)), o.get(ow))
    eng.close()


def test_gap_statistics(P):
    import torch
    eng, o, rng = _small_engine(P, d=70001, n=3)
    eng.set_option(P.GA_OPT_STATS, 1)
    with pytest.raises(P.GaError):
        eng.get_stats()
    sched = [0, 1, 2, 1, 0]
    grads = [rng.normal(size=eng.n_params).astype(np.float32) for _ in sched]
    dev = [torch.from_numpy(g).cuda() for g in grads]
    for j, (i, g) in enumerate(zip(sched, grads)):          # one arrival at a time
        eng.push_batch([i], [dev[j]])
        o.push(i, g)
        o.pull(i)
        s, m = eng.get_stats()
        os_, om = o.stats()
        assert abs(s - os_) <= 1e-9 * os_ and m == om
    # a fused window reports the statistics of its last arrival
    eng.push_batch([0, 1, 2], dev[:3])
    o.push_batch([0, 1, 2], grads[:3])
    s, m = eng.get_stats()
    assert abs(s - o.stats()[0]) <= 1e-9 * o.stats()[0] and m == o.stats()[1]
    assert _same(_np(eng.get(P.GA_THETA)), o.get(o.THETA))
    eng.close()


def test_checkpoint_resume_is_bit_identical(P):
    from paper_1909_10802_b200.runner import Run
    import torch
    wl = W.config("mini")
    a = Run(wl, "GA", 4)
    a.run(30)
    blob = a.engine.export_state()
    b = Run(wl, "GA", 4)
    b.engine.import_state(blob)
    b.k = 30
    a.run()
    b.run()
    for which in (P.GA_THETA, P.GA_V, P.GA_M, P.GA_C):
        assert torch.equal(a.engine.get(which), b.engine.get(which))
    assert a.delays[30:] == b.delays
    st = P.unpack_state(blob)
    assert st["k_done"] == 30 and P.pack_state(st) == blob
    with pytest.raises(P.GaError):
        b.engine.import_state(blob[:100])
    a.close()
    b.close()


def test_host_buffer_path_equals_device_path(P):
    import torch
    d, n = 9_000_011, 3      # three chunks of the host path, ragged end
    rng = np.random.default_rng(3)
    th0 = torch.from_numpy(rng.normal(size=d).astype(np.float32)).cuda()
    sched = [2, 0, 1, 0]
    grads = [torch.from_numpy(rng.normal(size=d).astype(np.float32)).pin_memory() for _ in sched]
    outs = [torch.empty(d, dtype=torch.float32).pin_memory() for _ in sched]
    a = P.Engine(d, n, 0.1, 0.9, 0.999, P.GA_GA)
    b = P.Engine(d, n, 0.1, 0.9, 0.999, P.GA_GA)
    a.set_params(th0)
    b.set_params(th0)
    da, _ = a.push_batch_host(sched, grads, outs)
    sent_dev = []
    db = []
    for i, g in zip(sched, grads):
        db += b.push_batch([i], [g.cuda()])
        sent_dev.append(b.saved(i).clone())
    assert da == db
    for which in (P.GA_THETA, P.GA_V, P.GA_M):
        assert torch.equal(a.get(which), b.get(which))
    for o_host, s_dev in zip(outs, sent_dev):
        assert torch.equal(o_host.cuda(), s_dev)
    a.close()
    b.close()


# ----------------------------------------------------------------------------- fp64 and fast mode
def test_adam_ga_fast_math_single_arrival(P):
    """Adam-GA's fast form against the fp64 oracle, one arrival from an identical fp32 state."""
    import torch
    wl = W.Workload(name="adamfast", segments=[30_000], n_workers=4, arrivals=40, schedule_kind="ticks",
                    seed=321, lr=0.01)
    sched = wl.schedule()
    for start in (0, 25):
        o32, _, _ = run_oracle(wl, "ADAM_GA", n_arrivals=start)
        state = o32.state()
        o64 = oracle.Oracle(wl.d, wl.n_workers, wl.lr, wl.momentum, wl.c_beta, oracle.ADAM_GA, precision=64)
        o64.set_state(*state[:7], v_workers=state[7])
        eng = P.Engine(wl.d, wl.n_workers, wl.lr, wl.momentum, wl.c_beta, P.GA_ADAM_GA)
        eng.set_option(P.GA_OPT_MATH, 1)
        st = P.unpack_state(eng.export_state())
        st.update(theta=state[0], v=state[1], m=state[2], saved=state[3], iter=state[4], k_done=state[5],
                  k_c=state[6], v2=state[7])
        eng.import_state(P.pack_state(st))
        i = sched[start]
        g = wl.grad(start + 1, o32.sent_f32(i))
        assert eng.push_batch([i], [torch.from_numpy(g).cuda()]) == [o64.push(i, g)]
        for which, ref in ((P.GA_THETA, o64.get(o64.THETA)), (P.GA_V, o64.get(o64.V)), (P.GA_V2, o64.second_moment()),
                           (P.GA_M, o64.get(o64.M))):
            got = _np(eng.get(which))
            assert within(got, ref, TOL), (start, which, worst(got, ref))
        eng.close()


@pytest.mark.parametrize("math_mode", [0, 1])
def test_single_arrival_against_fp64(P, math_mode):
    """From one fp32 state, one arrival on the GPU (exact or fast math) and in the fp64 oracle."""
    import torch
    wl = W.config("C1")
    idx = wl.sample_indices(20000)
    d = len(idx)
    sched = wl.schedule()
    for start in (0, 40, 300):
        o32, _, _ = run_oracle(wl, "GA", n_arrivals=start, idx=idx)
        th, v, m, saved, iters, k_done, k_c = o32.state()
        o64 = oracle.Oracle(d, wl.n_workers, wl.lr, wl.momentum, wl.c_beta, oracle.GA, precision=64)
        o64.set_state(th, v, m, saved, iters, k_done, k_c)
        eng = P.Engine(d, wl.n_workers, wl.lr, wl.momentum, wl.c_beta, P.GA_GA)
        eng.set_option(P.GA_OPT_MATH, math_mode)
        st = P.unpack_state(eng.export_state())
        st.update(theta=th, v=v, m=m, saved=saved, iter=iters, k_done=k_done, k_c=k_c)
        eng.import_state(P.pack_state(st))
        i = sched[start]
        g = wl.grad(start + 1, o32.sent_f32(i), idx)
        assert eng.push_batch([i], [torch.from_numpy(g).cuda()]) == [o64.push(i, g)]
        o64.pull(i)
        for which, ow in ((P.GA_THETA, o64.THETA), (P.GA_V, o64.V), (P.GA_M, o64.M)):
            got, ref = _np(eng.get(which)), o64.get(ow)
            assert within(got, ref, TOL), (start, which, worst(got, ref))
        eng.close()


@pytest.mark.parametrize("variant", ["GA", "DANA_GA", "ADAM_GA", "ADAM_SA", "SA_GRAD", "GA_LAYER"])
def test_extreme_values_round_like_the_oracle(P, variant):
    """States and gradients spanning the whole fp32 range -- subnormals, zeros of both signs,
    1e-42 .. 1e38, infinities, NaNs -- imported into both sides; a window of three arrivals must
    still agree element for element (the IEEE division / square-root / reciprocal paths and
    their zero shortcuts are all exercised)."""
    import torch
    d, n = 60_000, 3
    rng = np.random.default_rng(99)

    def wild(nonneg=False):
        x = (10.0 ** rng.uniform(-44, 38, size=d)) * (1 if nonneg else rng.choice([-1.0, 1.0], size=d))
        x = x.astype(np.float32)
        kind = rng.integers(0, 40, size=d)
        x[kind == 0] = 0.0
        x[kind == 1] = 0.0 if nonneg else -0.0
        x[kind == 2] = np.inf
        x[kind == 3] = np.inf if nonneg else -np.inf
        x[kind == 4] = np.nan
        x[kind == 5] = np.float32(1e-45)          # smallest subnormal
        return x

    var = oracle.VARIANTS[variant]
    o = oracle.Oracle(d, n, 0.1, 0.9, 0.999, var)
    eng = P.Engine(d, n, 0.1, 0.9, 0.999, var)
    theta, v, m = wild(), wild(), wild(nonneg=True)
    saved = np.stack([wild() for _ in range(n)])
    saved[0, ::3] = theta[::3]                     # plenty of exact "copy equals master"
    iters = np.array([2, 0, 4], dtype=np.int64)
    extra = {}
    if variant == "DANA_GA":
        extra = dict(v_workers=np.stack([wild() for _ in range(n)]))
    if variant.startswith("ADAM"):
        extra = dict(v_workers=wild(nonneg=True))
    o.set_state(theta, v, m, saved, iters, 5, 5, **extra)
    if variant == "GA_LAYER":                      # three layers; their m_p start at 0 on both sides
        o.set_layers([0, 7, 30_001, d])
        eng.set_layers([0, 7, 30_001, d])
    st = P.unpack_state(eng.export_state())
    st.update(theta=theta, v=v, m=m, saved=saved, iter=iters, k_done=5, k_c=5)
    if variant == "DANA_GA":
        st["v_workers"] = extra["v_workers"]
    if variant.startswith("ADAM"):
        st["v2"] = extra["v_workers"]
    eng.import_state(P.pack_state(st))
    grads = [wild() for _ in range(3)]
    sched = [1, 0, 2]
    assert eng.push_batch(sched, [torch.from_numpy(g).cuda() for g in grads]) == o.push_batch(sched, grads)
    pairs = [(P.GA_THETA, o.get(o.THETA)), (P.GA_V, o.get(o.V))]
    if variant in ("GA", "DANA_GA", "ADAM_GA"):
        pairs.append((P.GA_M, o.get(o.M)))
    if variant.startswith("ADAM"):
        pairs.append((P.GA_V2, o.second_moment()))
    for which, ref in pairs:
        got = _np(eng.get(which))
        bad = ~((got == ref.astype(np.float32)) | (np.isnan(got) & np.isnan(ref)))
        assert not bad.any(), (variant, which, int(bad.sum()), got[bad][:4], ref[bad][:4])
    for i in range(n):
        assert _same(_np(eng.saved(i)), o.saved(i))
    eng.close()


# ----------------------------------------------------------------------------- errors
def test_bad_arguments_return_errors(P):
    import ctypes
    import torch
    l = P.lib()
    assert not l.ga_create(0, 4, 0.1, 0.9, 0.999, P.GA_GA) and "n_params" in P.last_error()
    assert not l.ga_create(10, 0, 0.1, 0.9, 0.999, P.GA_GA)
    assert not l.ga_create(10, 4, -1.0, 0.9, 0.999, P.GA_GA)
    assert not l.ga_create(10, 4, 0.1, 1.0, 0.999, P.GA_GA)
    assert not l.ga_create(10, 4, 0.1, 0.9, 1.0, P.GA_GA)
    assert not l.ga_create(10, 4, 0.1, 0.9, 0.999, 11) and "variant" in P.last_error()
    assert l.ga_push(None, 0, None) == P.GA_ERR_ARG
    l.ga_destroy(None)
    eng = P.Engine(1000, 4, 0.1, -0.5, 0.999, P.GA_GA)     # negative momentum is legal
    g = torch.zeros(1004, device="cuda")
    h = eng._h
    assert l.ga_push(h, 4, g.data_ptr()) == P.GA_ERR_ARG and "worker" in P.last_error()
    assert l.ga_push(h, -1, g.data_ptr()) == P.GA_ERR_ARG
    assert l.ga_push(h, 0, None) == P.GA_ERR_ARG
    assert l.ga_push(h, 0, g.data_ptr() + 4) == P.GA_ERR_ARG and "aligned" in P.last_error()
    assert not l.ga_pull(h, 99)
    assert l.ga_set_option(h, 99, 1.0) == P.GA_ERR_ARG
    assert l.ga_set_option(h, P.GA_OPT_WINDOW, 17.0) == P.GA_ERR_ARG
    sched = (ctypes.c_int * 2)(0, 9)
    ptrs = (ctypes.c_void_p * 2)(g.data_ptr(), g.data_ptr())
    assert l.ga_push_batch(h, sched, ptrs, 2, None) == P.GA_ERR_ARG
    assert eng.num_arrivals == 0, "a rejected batch applies nothing"
    assert l.ga_push_batch(h, sched, ptrs, -1, None) == P.GA_ERR_ARG
    assert eng.push(0, g) == 1 and eng.num_arrivals == 1     # still usable
    assert l.ga_set_option(h, P.GA_OPT_C_ORDER, 1.0) == P.GA_ERR_STATE
    # ordinary host memory handed over as device memory is refused before any kernel could touch it
    import numpy as np
    host = np.zeros(1024 + 8, dtype=np.float32)
    addr = (host.ctypes.data + 15) // 16 * 16
    assert l.ga_push(h, 0, addr) == P.GA_ERR_ARG and "host memory" in P.last_error()
    ptrs = (ctypes.c_void_p * 2)(g.data_ptr(), addr)
    sched = (ctypes.c_int * 2)(0, 1)
    assert l.ga_push_batch(h, sched, ptrs, 2, None) == P.GA_ERR_ARG and "gradient 1" in P.last_error()
    assert l.ga_get(h, P.GA_THETA, addr) == P.GA_ERR_ARG
    assert l.ga_set_params(h, addr) == P.GA_ERR_ARG
    assert eng.num_arrivals == 1
    pinned = torch.zeros(1000).pin_memory()                 # pinned host memory is reachable from the device
    assert l.ga_push(h, 1, pinned.data_ptr()) == 2
    # and device memory where the host-buffer call expects host memory
    hp = (ctypes.c_void_p * 1)(g.data_ptr())
    one = (ctypes.c_int * 1)(2)
    assert l.ga_push_batch_host(h, one, hp, 1, None, None) == P.GA_ERR_ARG and "device memory" in P.last_error()
    assert eng.num_arrivals == 2
    pageable = (ctypes.c_void_p * 1)(addr)                   # ordinary host memory is fine there
    assert l.ga_push_batch_host(h, one, pageable, 1, None, None) >= 1 and eng.num_arrivals == 3
    assert torch.isfinite(eng.get(P.GA_THETA)).all()
    eng.close()


def test_no_write_outside_the_callers_buffers(P):
    """Canary words around every caller-owned buffer (ragged d, so the last vector is partial):
    outputs are written for exactly n_params floats, gradients are never written at all."""
    import torch
    d, pad = 10_007, 64
    canary = 12345.0

    def guarded():
        t = torch.full((d + 2 * pad,), canary, device="cuda")
        return t, t[pad:pad + d]

    def intact(t):
        return bool((t[:pad] == canary).all() and (t[pad + d:] == canary).all())

    for variant in (P.GA_GA, P.GA_DANA_GA, P.GA_ADAM_GA, P.GA_GA_LAYER):
        eng = P.Engine(d, 3, 0.1, 0.9, 0.999, variant)
        full0, th0 = guarded()
        th0.normal_()
        eng.set_params(th0)
        grads = [guarded() for _ in range(3)]
        for _, g in grads:
            g.normal_()
        before = [full.clone() for full, _ in grads]
        eng.push_batch([0, 1, 2], [g for _, g in grads])
        eng.push(1, grads[0][1])
        eng.pull(1)
        assert all(torch.equal(full, b) for (full, _), b in zip(grads, before)) and intact(full0)
        outs = []
        for which in (P.GA_THETA, P.GA_V, P.GA_M) + ((P.GA_C,) if variant != P.GA_GA_LAYER else ()):
            full, view = guarded()
            eng.get(which, view)
            outs.append(full)
        if variant != P.GA_GA_LAYER:
            full, view = guarded()
            eng.gap(2, view)
            outs.append(full)
        if variant == P.GA_DANA_GA:
            full, view = guarded()
            eng.get_worker_momentum(0, view)
            outs.append(full)
        assert all(intact(o) for o in outs)
        eng.close()


def test_non_finite_gradient_propagates(P):
    import torch
    eng, o, rng = _small_engine(P, d=257, n=2)
    g = rng.normal(size=257).astype(np.float32)
    g[3], g[100], g[200] = np.nan, np.inf, -np.inf
    assert eng.push_batch([0], [torch.from_numpy(g).cuda()]) == o.push_batch([0], [g])
    g2 = rng.normal(size=257).astype(np.float32)
    assert eng.push_batch([1], [torch.from_numpy(g2).cuda()]) == o.push_batch([1], [g2])
    for which, ow in ((P.GA_THETA, o.THETA), (P.GA_V, o.V), (P.GA_M, o.M)):
        assert _same(_np(eng.get(which)), o.get(ow))
    eng.close()
