"""More parity cases through the C ABI: Gap statistics of every arrival of a call (all three
parameter-wise Gap-Aware masters, fused windows, the host-buffer path, range shards), the
host-buffer path for the DANA and Adam masters, DANA-GA's fast-math form, the shared-memory ring
against the register path over a whole ResNet-50-sized vector, and what ga_import_state and
ga_create must refuse.
"""
import ctypes
import struct

import numpy as np
import pytest

import oracle
import workloads as W
from tests.oracle_run import run_oracle, within, worst

pytestmark = pytest.mark.gpu

TOL = 1e-5     # max |gpu - ref| <= TOL * (1 + |ref|)
GAP_VARIANTS = ["GA", "DANA_GA", "ADAM_GA"]


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


def _oracle_stats(wl, variant, c_order=0, n_arrivals=None):
    """(sum of the Gap, max of the Gap) of every arrival, from the oracle, and the oracle itself."""
    o = oracle.Oracle(wl.d, wl.n_workers, wl.lr, wl.momentum, wl.c_beta, oracle.VARIANTS[variant], c_order=c_order)
    o.set_params(wl.theta0())
    pairs, delays = [], []
    sched = wl.schedule()[:n_arrivals]
    for k, i in enumerate(sched, start=1):
        delays.append(o.push(i, wl.grad(k, o.sent_f32(i))))
        pairs.append(o.stats())
        o.pull(i)
    return pairs, delays, o


# ----------------------------------------------------------------------------- Gap statistics
@pytest.mark.parametrize("variant", GAP_VARIANTS)
@pytest.mark.parametrize("c_order", [0, 1])
def test_stats_of_every_arrival_of_a_call(P, variant, c_order):
    """Appendix "Gap and Delay" logs the average Gap over all updates: through the whole mini
    schedule (60 arrivals, a dozen fused windows) every arrival's sum and max of the Gap must come
    back, not only those of a window's last arrival."""
    from paper_1909_10802_b200.runner import Run
    wl = W.config("mini")
    want, odelays, o = _oracle_stats(wl, variant, c_order)
    run = Run(wl, variant, 16, options={P.GA_OPT_C_ORDER: c_order, P.GA_OPT_STATS: 1})
    assert run.engine.get_stats_window() == []                      # nothing applied yet
    wins = W.windows(wl.schedule(), 16)
    got = []
    for win in wins:                          # gradients need the copies sent so far: one window per call
        run.step(win)
        got += run.engine.get_stats_window()
    assert run.delays == odelays and len(got) == len(want) == wl.arrivals
    for k, ((s, m), (os_, om)) in enumerate(zip(got, want)):
        assert abs(s - os_) <= 1e-9 * os_ and m == om, (variant, k, s, os_, m, om)
    assert run.engine.get_stats() == got[-1]
    assert len(run.engine.get_stats_window(cap=2)) == min(2, len(wins[-1]))
    run.close()


@pytest.mark.parametrize("variant", GAP_VARIANTS)
def test_stats_of_a_multi_window_call(P, variant):
    """One call whose schedule splits into three launches (a worker repeats twice): the log must
    hold all eight arrivals in order. Gradients are fixed vectors here, so the whole schedule can
    go into one ga_push_batch."""
    import torch
    d, n = 70_001, 3
    rng = np.random.default_rng(17)
    th0 = rng.normal(size=d).astype(np.float32)
    sched = [0, 1, 2, 1, 0, 2, 2, 1]
    grads = [rng.normal(size=d).astype(np.float32) for _ in sched]
    var = oracle.VARIANTS[variant]
    lr = 0.01 if variant == "ADAM_GA" else 0.1
    o = oracle.Oracle(d, n, lr, 0.9, 0.999, var)
    o.set_params(th0)
    eng = P.Engine(d, n, lr, 0.9, 0.999, var)
    eng.set_option(P.GA_OPT_STATS, 1)
    eng.set_params(torch.from_numpy(th0).cuda())
    want = []
    for i, g in zip(sched, grads):
        o.push(i, g)
        want.append(o.stats())
        o.pull(i)
    delays, launches = eng.push_batch(sched, [torch.from_numpy(g).cuda() for g in grads], return_launches=True)
    assert launches == len(W.windows(sched, 16)) == 3
    got = eng.get_stats_window()
    assert len(got) == len(sched)
    for (s, m), (os_, om) in zip(got, want):
        assert abs(s - os_) <= 1e-9 * os_ and m == om
    # a single push is a call of one arrival
    g = rng.normal(size=d).astype(np.float32)
    eng.push(1, torch.from_numpy(g).cuda())
    o.push(1, g)
    (s, m), = eng.get_stats_window()
    assert abs(s - o.stats()[0]) <= 1e-9 * o.stats()[0] and m == o.stats()[1]
    # switched off: nothing to read
    eng.set_option(P.GA_OPT_STATS, 0)
    with pytest.raises(P.GaError):
        eng.get_stats_window()
    eng.close()
    plain = P.Engine(64, 2, 0.1, 0.9, 0.999, P.GA_SA)
    plain.set_option(P.GA_OPT_STATS, 1)
    with pytest.raises(P.GaError):
        plain.get_stats_window()
    plain.close()


def test_stats_log_keeps_the_most_recent_arrivals(P):
    """A call longer than the log (GA_STATS_LOG arrivals): the newest entries survive, in order."""
    import torch
    d, n = 257, 2
    rng = np.random.default_rng(2)
    eng = P.Engine(d, n, 0.1, 0.9, 0.999, P.GA_GA)
    eng.set_option(P.GA_OPT_STATS, 1)
    th0 = rng.normal(size=d).astype(np.float32)
    eng.set_params(torch.from_numpy(th0).cuda())
    o = oracle.Oracle(d, n, 0.1, 0.9, 0.999, oracle.GA)
    o.set_params(th0)
    g = (0.01 * rng.normal(size=d)).astype(np.float32)
    gd = torch.from_numpy(g).cuda()
    K = P.GA_STATS_LOG + 37
    sched = [k % n for k in range(K)]
    want = []
    for i in sched:
        o.push(i, g)
        want.append(o.stats())
        o.pull(i)
    eng.push_batch(sched, [gd] * K)
    got = eng.get_stats_window()
    assert len(got) == P.GA_STATS_LOG
    for (s, m), (os_, om) in zip(got, want[-P.GA_STATS_LOG:]):
        assert abs(s - os_) <= 1e-9 * os_ and m == om
    eng.close()


def test_stats_of_range_shards_combine_to_the_whole(P):
    """Three engines that each own a 128-byte aligned range of the vector: the sum of their sums
    and the maximum of their maxima are the whole engine's statistics (what
    shard.combine_gap_stats computes with two all-reduces)."""
    from paper_1909_10802_b200.runner import Run
    from paper_1909_10802_b200.shard import shard_range
    wl = W.config("mini")
    opts = {P.GA_OPT_STATS: 1}
    whole = Run(wl, "GA", 16, options=opts)
    wins = W.windows(wl.schedule(), 16)
    parts = [Run(wl, "GA", 16, options=opts, shard=shard_range(wl.d, r, 3)) for r in range(3)]
    for win in wins:
        whole.step(win)
        ref = whole.engine.get_stats_window()
        shards = []
        for part in parts:
            part.step(win)
            shards.append(part.engine.get_stats_window())
        for k, (s, m) in enumerate(ref):
            assert abs(sum(sh[k][0] for sh in shards) - s) <= 1e-12 * s
            assert max(sh[k][1] for sh in shards) == m
    for r in parts + [whole]:
        r.close()


def test_mean_gap_below_mean_delay_on_resnet50_shape(P):
    """Section 5.1 (soft check, on the GPU and over ALL 25.5M parameters): the average Gap stays
    above 1 and below the average delay."""
    import torch
    from paper_1909_10802_b200.runner import Run
    wl = W.config("C3")
    run = Run(wl, "GA", 16, options={P.GA_OPT_STATS: 1})
    gaps = []
    for win in W.windows(wl.schedule()[:320], 16):
        run.step(win)
        gaps += [s / wl.d for s, _ in run.engine.get_stats_window()]
    taus = run.delays
    assert len(gaps) == len(taus) == 320 and min(gaps) >= 1.0
    assert 1.0 < np.mean(gaps[160:]) < np.mean(taus[160:])
    run.close()
    torch.cuda.empty_cache()


# ----------------------------------------------------------------------------- host-buffer path
@pytest.mark.parametrize("variant", ["GA", "DANA_GA", "ADAM_GA", "DANA", "SA"])
def test_host_buffer_path_all_families(P, variant):
    """ga_push_batch_host on three chunks with a ragged end, two windows in one call (worker 0
    repeats), against the device path arrival by arrival: state, sent parameters, delays and the
    Gap statistics (merged chunk by chunk) must agree."""
    import torch
    d, n = 9_000_011, 3
    rng = np.random.default_rng(3)
    th0 = torch.from_numpy(rng.normal(size=d).astype(np.float32)).cuda()
    sched = [2, 0, 1, 0, 2]
    grads = [torch.from_numpy((0.1 * rng.normal(size=d)).astype(np.float32)).pin_memory() for _ in sched]
    outs = [torch.empty(d, dtype=torch.float32).pin_memory() for _ in sched]
    var = P.VARIANTS[variant]
    lr = 0.01 if variant == "ADAM_GA" else 0.1
    a = P.Engine(d, n, lr, 0.9, 0.999, var)
    b = P.Engine(d, n, lr, 0.9, 0.999, var)
    gap = variant in GAP_VARIANTS
    for e_ in (a, b):
        e_.set_params(th0)
        if gap:
            e_.set_option(P.GA_OPT_STATS, 1)
    da, launches = a.push_batch_host(sched, grads, outs)
    assert launches == 2 * 3
    sent_dev, db, stats_b = [], [], []
    for i, g in zip(sched, grads):
        db += b.push_batch([i], [g.cuda()])
        sent_dev.append(b.saved(i).clone())
        if gap:
            stats_b += b.get_stats_window()
    assert da == db
    vectors = [P.GA_THETA, P.GA_V] + ([P.GA_M] if gap else []) + ([P.GA_V2] if variant.startswith("ADAM") else [])
    for which in vectors:
        assert torch.equal(a.get(which), b.get(which)), which
    if variant.startswith("DANA"):
        for i in range(n):
            assert torch.equal(a.get_worker_momentum(i), b.get_worker_momentum(i))
    for o_host, s_dev in zip(outs, sent_dev):
        assert torch.equal(o_host.cuda(), s_dev)
    if gap:
        stats_a = a.get_stats_window()
        assert len(stats_a) == len(stats_b) == len(sched)
        for (s, m), (sb, mb) in zip(stats_a, stats_b):
            assert abs(s - sb) <= 1e-12 * sb and m == mb
    # without result buffers (nothing is copied back) the state still advances identically
    a.push_batch_host([1, 2], grads[:2], None)
    b.push_batch([1, 2], [g.cuda() for g in grads[:2]])
    assert torch.equal(a.get(P.GA_THETA), b.get(P.GA_THETA))
    a.close()
    b.close()


# ----------------------------------------------------------------------------- ring path vs register path
def test_c3_ring_path_equals_register_path_everywhere(P):
    """ResNet-50 shape, 64 workers: after the same 208 arrivals the K = 16 launches (shared-memory
    ring) and the K = 1 launches (register loads) must leave every element of theta, v, m and of
    two saved copies identical -- all 200k blocks, not a sample."""
    import torch
    from paper_1909_10802_b200.runner import Run
    wl = W.config("C3")
    keep = None
    for window in (16, 1):
        run = Run(wl, "GA", window)
        run.run(208)
        last = run.wl.schedule()[207]
        vecs = [run.engine.get(w) for w in (P.GA_THETA, P.GA_V, P.GA_M)]
        vecs += [run.engine.saved(last).clone(), run.engine.saved(wl.schedule()[100]).clone()]
        delays = list(run.delays)
        run.close()
        torch.cuda.empty_cache()
        if keep is None:
            keep = (vecs, delays)
        else:
            assert delays == keep[1]
            for q, (x, y) in enumerate(zip(keep[0], vecs)):
                assert torch.equal(x, y), f"vector {q} differs between K = 16 and K = 1"


# ----------------------------------------------------------------------------- fast math, DANA-GA
def test_dana_ga_fast_math_single_arrival(P):
    """DANA-GA's fast form (GA_OPT_MATH = 1) against the fp64 oracle, one arrival from an
    identical fp32 state, at the start and deep into a run."""
    import torch
    wl = W.Workload(name="danafast", segments=[30_000], n_workers=4, arrivals=40, schedule_kind="ticks", seed=123)
    sched = wl.schedule()
    for start in (0, 25):
        o32, _, _ = run_oracle(wl, "DANA_GA", n_arrivals=start)
        state = o32.state()
        o64 = oracle.Oracle(wl.d, wl.n_workers, wl.lr, wl.momentum, wl.c_beta, oracle.DANA_GA, precision=64)
        o64.set_state(*state[:7], v_workers=state[7])
        eng = P.Engine(wl.d, wl.n_workers, wl.lr, wl.momentum, wl.c_beta, P.GA_DANA_GA)
        eng.set_option(P.GA_OPT_MATH, 1)
        st = P.unpack_state(eng.export_state())
        st.update(theta=state[0], v=state[1], m=state[2], saved=state[3], iter=state[4], k_done=state[5],
                  k_c=state[6], v_workers=state[7])
        eng.import_state(P.pack_state(st))
        i = sched[start]
        g = wl.grad(start + 1, o32.sent_f32(i))
        assert eng.push_batch([i], [torch.from_numpy(g).cuda()]) == [o64.push(i, g)]
        o64.pull(i)
        pairs = [(eng.get(P.GA_THETA), o64.get(o64.THETA)), (eng.get(P.GA_V), o64.get(o64.V)),
                 (eng.get(P.GA_M), o64.get(o64.M)), (eng.get_worker_momentum(i), o64.worker_momentum(i)),
                 (eng.saved(i), o64.saved(i))]
        for q, (got, ref) in enumerate(pairs):
            assert within(_np(got), ref, TOL), (start, q, worst(_np(got), ref))
        eng.close()


# ----------------------------------------------------------------------------- what must be refused
def test_lr_too_small_for_c_is_refused(P):
    """C = eta_max (sqrt(m_hat) + 1e-8) must stay positive: a rate for which eta_max * 1e-8 rounds
    to zero would make the Gap 0/0, so ga_create refuses it; the smallest accepted rates work."""
    import torch
    l = P.lib()
    assert not l.ga_create(16, 2, 1e-38, 0.9, 0.999, P.GA_GA) and "rounds to zero" in P.last_error()
    eng = P.Engine(1000, 2, 2e-37, 0.9, 0.999, P.GA_GA)        # eta_max * 1e-8 is a subnormal, still > 0
    o = oracle.Oracle(1000, 2, 2e-37, 0.9, 0.999, oracle.GA)
    rng = np.random.default_rng(4)
    th0 = rng.normal(size=1000).astype(np.float32)
    eng.set_params(torch.from_numpy(th0).cuda())
    o.set_params(th0)
    for i in (0, 1, 0):
        g = rng.normal(size=1000).astype(np.float32)
        assert eng.push_batch([i], [torch.from_numpy(g).cuda()]) == o.push_batch([i], [g])
    for which, ow in ((P.GA_THETA, o.THETA), (P.GA_V, o.V), (P.GA_M, o.M), (P.GA_C, o.C)):
        got, ref = _np(eng.get(which)), o.get(ow).astype(np.float32)
        assert np.array_equal(got, ref, equal_nan=True), which
    assert l.ga_set_option(eng._h, P.GA_OPT_ADAM_EPS, 1e-60) == P.GA_ERR_ARG    # zero as a float
    eng.close()


def test_import_state_refuses_inconsistent_headers(P):
    """Every header field and iter[] entry that a later push relies on is checked before device
    state is touched: a doctored checkpoint comes back as GA_ERR_ARG and the engine continues
    exactly as if the call had not been made."""
    import torch
    from paper_1909_10802_b200.runner import Run
    wl = W.config("mini")
    a = Run(wl, "GA", 4)
    b = Run(wl, "GA", 4)
    a.run(30)
    b.run(30)
    blob = a.engine.export_state()
    fmt = "<IIqqqqffffiiiiiiffff"
    names = ("magic version d n_workers k_done k_c lr gamma beta eps variant c_order fast_math stats window nesterov "
             "beta2 adam_eps lr_max weight_decay").split()
    head = list(struct.unpack_from(fmt, blob, 0))
    hs = struct.calcsize(fmt)
    bad_values = {"k_done": -1, "k_c": 31, "lr": 0.0, "gamma": 1.5, "beta": 1.0, "eps": 0.0, "c_order": 2,
                  "fast_math": -1, "stats": 7, "window": 0, "nesterov": 3, "beta2": -0.1, "adam_eps": 0.0,
                  "lr_max": float("inf"), "weight_decay": -1.0, "variant": P.GA_SA, "d": wl.d + 1, "magic": 1}
    for name, value in bad_values.items():
        h = list(head)
        h[names.index(name)] = value
        doctored = struct.pack(fmt, *h) + blob[hs:]
        assert a.engine._l.ga_import_state(a.engine._h, doctored, len(doctored)) == P.GA_ERR_ARG, name
    for worker, value in ((0, 31), (2, -1)):      # a pull in the future would give a delay <= 0
        iters = np.frombuffer(blob, dtype=np.int64, count=wl.n_workers, offset=hs).copy()
        iters[worker] = value
        doctored = blob[:hs] + iters.tobytes() + blob[hs + 8 * wl.n_workers:]
        assert a.engine._l.ga_import_state(a.engine._h, doctored, len(doctored)) == P.GA_ERR_ARG
        assert "iter" in P.last_error()
    # a second moment is a running average of squares: a negative entry is refused
    st = P.unpack_state(blob)
    st["m"] = st["m"].copy()
    st["m"][17] = -1e-6
    doctored = P.pack_state(st)
    assert a.engine._l.ga_import_state(a.engine._h, doctored, len(doctored)) == P.GA_ERR_ARG
    assert "second moment" in P.last_error()
    a.run()
    b.run()
    for which in (P.GA_THETA, P.GA_V, P.GA_M):
        assert torch.equal(a.engine.get(which), b.engine.get(which))
    assert a.delays == b.delays
    a.close()
    b.close()


# ----------------------------------------------------------------------------- exact arithmetic
def test_short_exact_forms_agree_with_ieee_on_this_device(P):
    """Exact mode evaluates roots, divisions and reciprocals by short sequences wherever their
    operands lie in proven ranges. The library's self-test compares them with the IEEE routines on
    this GPU: every reciprocal operand in [2^-100, 2^100], every radicand in [2^-100, FLT_MAX],
    2 x 10^9 random divisions over all exponent pairs of the windows in use, constant numerators over
    every divisor in [1, 2^100]. Not one operand may differ."""
    assert P.selftest_exact_forms(0) == 0
    assert P.lib().ga_selftest_exact_forms(7, None) == P.GA_ERR_ARG


@pytest.mark.parametrize("variant", ["GA", "DANA_GA", "ADAM_GA", "ADAM", "ADAM_SA"])
def test_short_forms_and_ieee_fallback_give_the_same_bits(P, variant):
    """The same three arrivals with hyper-parameters inside the proven ranges (short forms on) and
    from a checkpoint whose eta_max lies outside them (every element takes the IEEE routines): both
    must equal the oracle bit for bit, on values spanning tiny, ordinary and huge magnitudes."""
    import torch
    d, n = 40_000, 3
    rng = np.random.default_rng(5)
    var = oracle.VARIANTS[variant]

    def spread(nonneg=False):
        x = (10.0 ** rng.uniform(-30, 20, size=d)) * (1 if nonneg else rng.choice([-1.0, 1.0], size=d))
        x = x.astype(np.float32)
        x[rng.integers(0, 10, size=d) == 0] = 0.0
        return x

    for lr_max in (0.1, 1e-20):                    # 1e-20 < 2^-49: outside the short forms' range
        o = oracle.Oracle(d, n, lr_max, 0.9, 0.999, var)
        eng = P.Engine(d, n, lr_max, 0.9, 0.999, var)
        theta, v, m = spread(), spread(), spread(nonneg=True)
        saved = np.stack([spread() for _ in range(n)])
        saved[1, ::2] = theta[::2]
        iters = np.array([1, 0, 3], dtype=np.int64)
        extra = {}
        if variant == "DANA_GA":
            extra = dict(v_workers=np.stack([spread() for _ in range(n)]))
        if variant.startswith("ADAM"):
            extra = dict(v_workers=spread(nonneg=True))
        o.set_state(theta, v, m, saved, iters, 4, 4, **extra)
        st = P.unpack_state(eng.export_state())
        st.update(theta=theta, v=v, m=m, saved=saved, iter=iters, k_done=4, k_c=4)
        if variant == "DANA_GA":
            st["v_workers"] = extra["v_workers"]
        if variant.startswith("ADAM"):
            st["v2"] = extra["v_workers"]
        eng.import_state(P.pack_state(st))
        grads = [spread() for _ in range(3)]
        sched = [1, 0, 2]
        assert eng.push_batch(sched, [torch.from_numpy(g).cuda() for g in grads]) == o.push_batch(sched, grads)
        pairs = [(P.GA_THETA, o.get(o.THETA)), (P.GA_V, o.get(o.V))]
        if variant not in ("ADAM", "ADAM_SA"):
            pairs.append((P.GA_M, o.get(o.M)))
        if variant.startswith("ADAM"):
            pairs.append((P.GA_V2, o.second_moment()))
        for which, ref in pairs:
            got = _np(eng.get(which))
            bad = ~((got == ref.astype(np.float32)) | (np.isnan(got) & np.isnan(ref)))
            assert not bad.any(), (variant, lr_max, which, int(bad.sum()), got[bad][:4], ref[bad][:4])
        eng.close()


# ----------------------------------------------------------------------------- bounded waits
def test_a_wait_that_nothing_satisfies_gives_up_and_reports(P):
    """The layer-wise kernels wait for per-layer counters; such a wait must end by itself. One block
    waits for a counter nothing advances: the wait runs out, the error flag is raised, the kernel
    returns and the context stays usable (a second engine runs right after)."""
    import time
    import torch
    t0 = time.time()
    assert P.lib().ga_selftest_bounded_wait(None, None) == P.GA_OK, P.last_error()
    assert time.time() - t0 < 30.0
    eng = P.Engine(1000, 2, 0.1, 0.9, 0.999, P.GA_GA_LAYER)
    eng.set_params(torch.zeros(1000, device="cuda"))
    assert eng.push_batch([0, 1], [torch.ones(1000, device="cuda")] * 2) == [1, 2]
    assert torch.isfinite(eng.get(P.GA_THETA)).all()
    # the same through an engine's own flag: the host learns of the lost wait at the next
    # synchronising call, and the engine stays failed (every later call says so) while others work on
    assert P.lib().ga_selftest_bounded_wait(eng._h, None) == P.GA_OK, P.last_error()
    out = torch.empty(1000, device="cuda")
    assert P.lib().ga_get(eng._h, P.GA_THETA, out.data_ptr()) == P.GA_ERR_CUDA and "waiting" in P.last_error()
    assert P.lib().ga_push(eng._h, 0, out.data_ptr()) == P.GA_ERR_CUDA
    eng.close()
    other = P.Engine(1000, 2, 0.1, 0.9, 0.999, P.GA_GA)
    other.set_params(torch.zeros(1000, device="cuda"))
    assert other.push_batch([0], [torch.ones(1000, device="cuda")]) == [1]
    assert torch.isfinite(other.get(P.GA_THETA)).all()
    other.close()


# ----------------------------------------------------------------------------- caller-owned memory
@pytest.mark.parametrize("variant", ["GA", "DANA_GA", "ADAM_GA", "GA_LAYER"])
def test_engine_inside_a_callers_workspace(P, variant):
    """ga_create_in: the engine's state laid out in a torch tensor must behave exactly like an
    engine that allocated for itself (oracle parity, statistics), must not write outside the bytes
    ga_workspace_bytes asked for, and must leave the tensor alone after ga_destroy."""
    import torch
    from paper_1909_10802_b200.runner import Run
    wl = W.config("mini")
    need = P.workspace_bytes(wl.d, wl.n_workers, variant)
    state_floats = wl.d * (3 + wl.n_workers * (2 if variant == "DANA_GA" else 1) + (1 if variant == "ADAM_GA" else 0))
    assert 4 * state_floats < need < 4 * state_floats + (2 << 20)
    pad = 4096
    ws = torch.full((need + 2 * pad,), 0x5A, dtype=torch.uint8, device="cuda")
    inner = ws[pad:pad + need]
    assert inner.data_ptr() % 256 == 0

    run = Run(wl, variant, 16, options={P.GA_OPT_STATS: 1} if variant != "GA_LAYER" else None, workspace=inner)
    delays = run.run()
    o, odelays, _ = run_oracle(wl, variant)
    assert delays == odelays
    for which, ow in ((P.GA_THETA, o.THETA), (P.GA_V, o.V)):
        assert np.array_equal(_np(run.engine.get(which)), o.get(ow).astype(np.float32), equal_nan=True)
    for i in range(wl.n_workers):
        assert np.array_equal(_np(run.engine.saved(i)), o.saved(i).astype(np.float32), equal_nan=True)
    if variant != "GA_LAYER":
        s, m = run.engine.get_stats()
        assert abs(s - o.stats()[0]) <= 1e-9 * o.stats()[0] and m == o.stats()[1]
    theta_addr = run.engine.saved_ptr(0)
    assert inner.data_ptr() <= theta_addr < inner.data_ptr() + need          # the copies live in the tensor
    assert bool((ws[:pad] == 0x5A).all()) and bool((ws[pad + need:] == 0x5A).all())
    run.close()
    snapshot = ws.clone()
    torch.cuda.synchronize()
    assert torch.equal(ws, snapshot)
    # too small, misaligned or missing workspaces are refused
    l = P.lib()
    assert not l.ga_create_in(wl.d, wl.n_workers, 0.1, 0.9, 0.999, P.VARIANTS[variant], inner.data_ptr(), need - 1)
    assert "ga_workspace_bytes" in P.last_error()
    assert not l.ga_create_in(wl.d, wl.n_workers, 0.1, 0.9, 0.999, P.VARIANTS[variant], inner.data_ptr() + 16, need)
    assert not l.ga_create_in(wl.d, wl.n_workers, 0.1, 0.9, 0.999, P.VARIANTS[variant], None, need)
    assert l.ga_workspace_bytes(0, 4, P.GA_GA) == 0


def test_statistics_notice_non_finite_values(P):
    """Nothing traps on a diverged run; with GA_OPT_STATS the sum of the Gap turns non-finite as soon
    as one parameter's Gap does (here: a NaN gradient poisons theta, so the next Gap taken against
    that theta is NaN)."""
    import math
    import torch
    d = 3000
    eng = P.Engine(d, 2, 0.1, 0.9, 0.999, P.GA_GA)
    eng.set_option(P.GA_OPT_STATS, 1)
    eng.set_params(torch.zeros(d, device="cuda"))
    g = torch.full((d,), 0.01, device="cuda")
    eng.push_batch([0, 1], [g, g])
    assert all(math.isfinite(s) for s, _ in eng.get_stats_window())
    bad = g.clone()
    bad[1234] = float("nan")
    eng.push_batch([0], [bad])                 # theta[1234] becomes NaN
    eng.push_batch([1], [g])                   # worker 1's Gap at 1234 is |NaN - s| / C + 1
    (s, _), = eng.get_stats_window()
    assert math.isnan(s)
    assert int(torch.isnan(eng.get(P.GA_THETA)).sum()) == 1
    eng.close()


def test_layer_gap_one_long_call(P):
    """One ga_push_batch call of 45 arrivals with the layer-wise Gap: the call spans three arrival
    tables of 16, so the second and third run 'primed' (their first Gap was prepared by the launch
    before), workers repeat back to back (distance exactly 0) and at random. Every launch is
    chained to the one before; the result must still equal the oracle's bit for bit."""
    import torch
    d, n = 50_003, 4
    offsets = [0, 7, 4_100, 4_101, 30_000, d]
    rng = np.random.default_rng(21)
    th0 = rng.normal(size=d).astype(np.float32)
    pool = [(0.1 * rng.normal(size=d)).astype(np.float32) for _ in range(5)]
    sched = [int(x) for x in rng.integers(0, n, size=45)]
    sched[10] = sched[11] = sched[12] = 2          # the same worker three times in a row
    sched[15] = sched[16] = 1                      # ... and across the boundary of two tables
    grads = [pool[k % 5] for k in range(len(sched))]
    o = oracle.Oracle(d, n, 0.05, 0.9, 0.999, oracle.GA_LAYER)
    o.set_layers(offsets)
    o.set_params(th0)
    eng = P.Engine(d, n, 0.05, 0.9, 0.999, P.GA_GA_LAYER)
    eng.set_layers(offsets)
    eng.set_params(torch.from_numpy(th0).cuda())
    dev = [torch.from_numpy(g).cuda() for g in pool]
    delays, launches = eng.push_batch(sched, [dev[k % 5] for k in range(len(sched))], return_launches=True)
    assert delays == o.push_batch(sched, grads) and launches == len(sched) + 1
    assert np.array_equal(_np(eng.get(P.GA_THETA)), o.get(o.THETA).astype(np.float32))
    assert np.array_equal(_np(eng.get(P.GA_V)), o.get(o.V).astype(np.float32))
    gaps, m_layer = eng.get_layer_state()
    ogaps, om = o.layer_state()
    assert np.array_equal(gaps, ogaps.astype(np.float32)) and np.array_equal(m_layer, om.astype(np.float32))
    for i in range(n):
        assert np.array_equal(_np(eng.saved(i)), o.saved(i).astype(np.float32))
    # a second call continues from there (its distance pass runs after the chain has drained)
    more = [3, 3, 0]
    assert eng.push_batch(more, dev[:3]) == o.push_batch(more, pool[:3])
    assert np.array_equal(_np(eng.get(P.GA_THETA)), o.get(o.THETA).astype(np.float32))
    eng.close()


@pytest.mark.parametrize("variant", ["GA", "ADAM_GA"])
def test_host_buffer_path_on_a_short_vector(P, variant):
    """The host-buffer path on a vector short enough for the two-parameters-per-thread layout (one
    chunk, ragged end), statistics on: equal to the device path and to the oracle."""
    import torch
    d, n = 10_007, 3
    rng = np.random.default_rng(8)
    th0 = rng.normal(size=d).astype(np.float32)
    sched = [1, 0, 2, 0]
    grads = [(0.1 * rng.normal(size=d)).astype(np.float32) for _ in sched]
    var = P.VARIANTS[variant]
    lr = 0.01 if variant == "ADAM_GA" else 0.1
    o = oracle.Oracle(d, n, lr, 0.9, 0.999, oracle.VARIANTS[variant])
    o.set_params(th0)
    want = []
    for i, g in zip(sched, grads):
        o.push(i, g)
        want.append(o.stats())
        o.pull(i)
    eng = P.Engine(d, n, lr, 0.9, 0.999, var)
    eng.set_option(P.GA_OPT_STATS, 1)
    eng.set_params(torch.from_numpy(th0).cuda())
    outs = [torch.empty(d, dtype=torch.float32).pin_memory() for _ in sched]
    eng.push_batch_host(sched, [torch.from_numpy(g).pin_memory() for g in grads], outs)
    assert np.array_equal(_np(eng.get(P.GA_THETA)), o.get(o.THETA).astype(np.float32))
    assert np.array_equal(_np(eng.get(P.GA_M)), o.get(o.M).astype(np.float32))
    assert np.array_equal(outs[-1].numpy(), o.saved(0).astype(np.float32))
    for (s, m), (os_, om) in zip(eng.get_stats_window(), want):
        assert abs(s - os_) <= 1e-9 * os_ and m == om
    eng.close()


@pytest.mark.parametrize("variant,d", [("GA", 272_474), ("GA", 3_000_001), ("DANA_GA", 272_474), ("ADAM_GA", 50_003),
                                       ("SA", 272_474)])
def test_calls_back_to_back_without_a_host_wait(P, variant, d):
    """Window launches are made so that the next one may be scheduled under the tail of the one before
    it (the kernel then waits for that launch to complete before it reads anything). Sixty calls of
    one to eight arrivals on fixed gradients, nothing between them on the stream and no host wait:
    the state and every saved copy equal the oracle's bit for bit."""
    import torch
    n = 8
    rng = np.random.default_rng(d % 1000 + len(variant))
    th0 = rng.normal(size=d).astype(np.float32)
    pool = [(0.1 * rng.normal(size=d)).astype(np.float32) for _ in range(n)]
    dev = [torch.from_numpy(g).cuda() for g in pool]
    lr = 0.01 if variant.startswith("ADAM") else 0.1
    o = oracle.Oracle(d, n, lr, 0.9, 0.999, oracle.VARIANTS[variant])
    o.set_params(th0)
    eng = P.Engine(d, n, lr, 0.9, 0.999, P.VARIANTS[variant])
    eng.set_params(torch.from_numpy(th0).cuda())
    calls = [[int(w) for w in rng.permutation(n)[: 1 + c % 8]] for c in range(60)]
    got = [eng.push_batch(c, [dev[w] for w in c]) for c in calls]           # enqueued in one go
    want = [o.push_batch(c, [pool[w] for w in c]) for c in calls]
    assert got == want
    for which, ow in ((P.GA_THETA, o.THETA), (P.GA_V, o.V), (P.GA_M, o.M)):
        if which == P.GA_M and variant == "SA":
            continue
        assert np.array_equal(_np(eng.get(which)), o.get(ow).astype(np.float32)), (variant, which)
    for w in range(n):
        assert np.array_equal(_np(eng.saved(w)), o.saved(w).astype(np.float32)), w
    eng.close()


@pytest.mark.parametrize("config,world,n_arrivals", [("mini", 2, None), ("C1", 3, 120)])
def test_layer_wise_gap_on_shards_of_whole_layers(P, config, world, n_arrivals):
    """The layer-wise Gap (Section 5.3) with the vector split over ranks at layer boundaries: each
    engine holds whole layers and needs nothing from the others. One shard after the other on one
    GPU; parameters, momentum, a saved copy, the per-layer Gaps and second moments, put together,
    equal the oracle's run over the whole vector bit for bit."""
    from paper_1909_10802_b200.runner import Run
    from paper_1909_10802_b200.shard import layer_shard_range
    wl = W.config(config)
    o, odelays, _ = run_oracle(wl, "GA_LAYER", n_arrivals=n_arrivals)
    ogap, om = o.layer_state()
    theta, vel, saved, gaps, ms = [], [], [], [], []
    for rank in range(world):
        l0, l1, j0, n = layer_shard_range(wl.seg_off, rank, world)
        part = Run(wl, "GA_LAYER", 16, shard=(j0, n))
        assert part.engine.n_layers == l1 - l0
        assert part.run(n_arrivals) == odelays
        theta.append(_np(part.engine.get(P.GA_THETA)))
        vel.append(_np(part.engine.get(P.GA_V)))
        saved.append(_np(part.engine.saved(1)))
        g, m = part.engine.get_layer_state()
        gaps.append(g)
        ms.append(m)
        part.close()
    assert np.array_equal(np.concatenate(theta), o.get(o.THETA).astype(np.float32))
    assert np.array_equal(np.concatenate(vel), o.get(o.V).astype(np.float32))
    assert np.array_equal(np.concatenate(saved), o.saved(1).astype(np.float32))
    assert np.array_equal(np.concatenate(gaps), ogap.astype(np.float32))
    assert np.array_equal(np.concatenate(ms), om.astype(np.float32))
    with pytest.raises(ValueError):           # a range that cuts a layer is refused
        Run(wl, "GA_LAYER", 16, shard=(0, int(wl.seg_off[1]) + 1))


def test_host_buffer_path_with_the_layer_wise_gap(P):
    """ga_push_batch_host for the layer-wise Gap (Section 5.3): whole gradients are staged a few
    arrivals at a time. Eleven arrivals with workers that repeat (next to one another and further
    apart), a ragged vector in five layers: the parameters sent after every arrival, the state and
    the per-layer Gaps and second moments equal the oracle's, and so does a second call."""
    import torch
    d, n = 20_011, 4
    layers = [0, 4096, 4100, 12_000, 12_001, d]
    rng = np.random.default_rng(21)
    th0 = rng.normal(size=d).astype(np.float32)
    sched = [1, 0, 2, 3, 3, 0, 1, 2, 0, 0, 3]
    grads = [(0.1 * rng.normal(size=d)).astype(np.float32) for _ in sched]
    o = oracle.Oracle(d, n, 0.1, 0.9, 0.999, oracle.GA_LAYER)
    o.set_layers(layers)
    o.set_params(th0)
    eng = P.Engine(d, n, 0.1, 0.9, 0.999, P.GA_GA_LAYER)
    eng.set_layers(layers)
    eng.set_params(torch.from_numpy(th0).cuda())
    for call in range(2):
        want_sent, want_delays = [], []
        for i, g in zip(sched, grads):
            want_delays.append(o.push(i, g))
            o.pull(i)
            want_sent.append(o.saved(i).astype(np.float32))
        outs = [torch.empty(d, dtype=torch.float32).pin_memory() for _ in sched]
        got_delays, launches = eng.push_batch_host(sched, [torch.from_numpy(g).pin_memory() for g in grads], outs)
        assert got_delays == want_delays and launches > len(sched)      # one launch per arrival + distance passes
        for j, (got, want) in enumerate(zip(outs, want_sent)):
            assert np.array_equal(got.numpy(), want), (call, j)
        assert np.array_equal(_np(eng.get(P.GA_THETA)), o.get(o.THETA).astype(np.float32))
        assert np.array_equal(_np(eng.get(P.GA_V)), o.get(o.V).astype(np.float32))
        ogap, om = o.layer_state()
        gap, m = eng.get_layer_state()
        assert np.array_equal(gap, ogap.astype(np.float32)) and np.array_equal(m, om.astype(np.float32))
    # without copies back to the host, and then the device path carries on from there
    got_delays, _ = eng.push_batch_host([0, 0, 2], [torch.from_numpy(g).pin_memory() for g in grads[3:6]])
    assert got_delays == o.push_batch([0, 0, 2], grads[3:6])
    dev = [torch.from_numpy(g).cuda() for g in grads[:3]]
    assert eng.push_batch([2, 2, 1], dev) == o.push_batch([2, 2, 1], grads[:3])
    assert np.array_equal(_np(eng.get(P.GA_THETA)), o.get(o.THETA).astype(np.float32))
    assert np.array_equal(_np(eng.saved(0)), o.saved(0).astype(np.float32))
    eng.close()


def test_engines_give_their_memory_back(P):
    """Create, use (device path, host-buffer path with its staging buffers and streams, layer tables,
    statistics) and destroy engines of every kind many times: the device's free memory afterwards is
    what it was before."""
    import torch
    d, n = 300_001, 3
    g = torch.ones(d, device="cuda")
    gh = torch.ones(d).pin_memory()
    out = torch.empty(d).pin_memory()

    def cycle(variant):
        eng = P.Engine(d, n, 0.01, 0.9, 0.999, P.VARIANTS[variant])
        if variant == "GA_LAYER":
            eng.set_layers([0, 1000, 200_000, d])
        elif variant in GAP_VARIANTS:
            eng.set_option(P.GA_OPT_STATS, 1)
        eng.set_params(g)
        eng.push_batch([0, 1], [g, g])
        eng.push_batch_host([2, 0], [gh, gh], [out, out])
        eng.pull(1)
        eng.close()

    kinds = ["GA", "SA", "DANA_GA", "ADAM_GA", "GA_LAYER"]
    for v in kinds:
        cycle(v)                              # first use: lazily created contexts, module loading
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(40):
        for v in kinds:
            cycle(v)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 >= free0 - (8 << 20), (free0, free1)      # nothing of the 200 engines (tens of MB each) is left


@pytest.mark.parametrize("variant", ["GA", "GA_LAYER"])
def test_a_change_of_stream_keeps_the_engines_launches_in_order(P, variant):
    """ga_set_stream while work is still queued on the old stream: the new stream waits for it, so
    windows enqueued on alternating streams, with no host wait in between, give the oracle's result."""
    import torch
    d, n = 6_000_011, 4
    rng = np.random.default_rng(33)
    th0 = rng.normal(size=d).astype(np.float32)
    pool = [(0.1 * rng.normal(size=d)).astype(np.float32) for _ in range(n)]
    dev = [torch.from_numpy(g).cuda() for g in pool]
    o = oracle.Oracle(d, n, 0.1, 0.9, 0.999, oracle.VARIANTS[variant])
    o.set_params(th0)
    eng = P.Engine(d, n, 0.1, 0.9, 0.999, P.VARIANTS[variant])
    eng.set_params(torch.from_numpy(th0).cuda())
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    calls = [[0, 1, 2, 3], [2, 0], [3, 1, 0], [1], [0, 2, 3, 1], [3, 0]]
    for c, call in enumerate(calls):
        eng.set_stream(streams[c % 2])
        assert eng.push_batch(call, [dev[w] for w in call]) == o.push_batch(call, [pool[w] for w in call])
    assert np.array_equal(_np(eng.get(P.GA_THETA)), o.get(o.THETA).astype(np.float32))
    assert np.array_equal(_np(eng.get(P.GA_V)), o.get(o.V).astype(np.float32))
    for w in range(n):
        assert np.array_equal(_np(eng.saved(w)), o.saved(w).astype(np.float32))
    eng.close()
