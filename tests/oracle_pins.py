"""Pins that tie the CPU oracle to what the paper and the mathematics fix.

Each pin takes `make`, a factory with the signature of oracle.Oracle, so the same checks can
be run against a deliberately broken build of the oracle (tests/test_oracle_mutants.py).
Nothing here restates the oracle's loop: a pin is a closed form, an invariant, a special case
that collapses to a textbook routine, a hand-worked value, or an exact-arithmetic brute force.
"""
import os
from decimal import Decimal, getcontext
from fractions import Fraction

import numpy as np

ASGD, SA, GA, SA_GRAD, DANA, DANA_SA, DANA_GA, ADAM, ADAM_SA, ADAM_GA, GA_LAYER = range(11)
THETA, V, M, C = 0, 1, 2, 3
GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _rng(seed):
    return np.random.default_rng(seed)


def _f32(x):
    return np.asarray(x, dtype=np.float32)


# --------------------------------------------------------------------------------------
def pin_gap_is_one_where_copy_equals_master(make):
    """Definition 1 / Section 4.1 'Over-Penalizing': where theta_k equals the saved copy the
    Gap is exactly 1 and the gradient goes through unpenalised, while SA still divides by tau."""
    d, eta = 64, 0.1
    r = _rng(1)
    th0 = _f32(r.normal(size=d))
    g1 = _f32(r.normal(size=d))
    g1[1::2] = 0.0                      # worker 1 moves only the even elements
    g0 = _f32(r.normal(size=d))
    res = {}
    for variant in (GA, ASGD, SA):
        o = make(d, 2, eta, 0.9, 0.999, variant, precision=32)
        o.set_params(th0)
        assert o.push(1, g1) == 1
        o.pull(1)
        if variant == GA:
            G = o.gap(0)
            assert np.all(G >= 1.0)
            assert np.all(G[1::2] == 1.0), "Gap must be exactly 1 where the copy equals the master"
            assert np.all(G[0::2][g1[0::2] != 0] > 1.0)
        assert o.push(0, g0) == 2       # delay 2 although the odd elements never moved
        res[variant] = (o.get(THETA), o.get(V))
    odd = slice(1, None, 2)
    # GA == unpenalised momentum step, bit for bit, on the untouched elements ...
    assert np.array_equal(res[GA][0][odd], res[ASGD][0][odd])
    assert np.array_equal(res[GA][1][odd], res[ASGD][1][odd])
    # ... and that step is theta0 - eta*g0 (v was 0 there)
    want = th0.astype(np.float64)[odd] - np.float64(np.float32(eta)) * g0.astype(np.float64)[odd]
    assert np.allclose(res[GA][0][odd], want, rtol=0, atol=2e-7)
    # SA halves the step there (tau = 2): over-penalised
    want_sa = th0.astype(np.float64)[odd] - np.float64(np.float32(eta)) / 2 * g0.astype(np.float64)[odd]
    assert np.allclose(res[SA][0][odd], want_sa, rtol=0, atol=2e-7)
    # on the moved elements GA penalises: |step| strictly smaller than the unpenalised one
    ev = slice(0, None, 2)
    moved = g1[ev] != 0
    v_prev = g1.astype(np.float64)[ev]
    pen = np.abs(res[GA][1][ev] - 0.9 * v_prev)[moved]      # |g_hat|
    raw = np.abs(res[ASGD][1][ev] - 0.9 * v_prev)[moved]    # |g|
    assert np.all(pen < raw + 1e-12) and np.any(pen < 0.9 * raw)


def pin_one_worker_is_heavy_ball(make):
    """Section 3: with one worker (push, pull, push, ...) every delay is 1 and the saved copy is
    always current, so GA, SA and ASGD are the momentum method without dampening -- checked
    against torch.optim.SGD(momentum) and against the closed form for a constant gradient."""
    import torch
    d, eta, gam, steps = 33, 0.05, 0.9, 25
    r = _rng(2)
    th0 = _f32(r.normal(size=d))
    grads = [_f32(r.normal(size=d)) for _ in range(steps)]
    out = {}
    for variant in (GA, SA, ASGD):
        for prec in (32, 64):
            o = make(d, 1, eta, gam, 0.999, variant, precision=prec)
            o.set_params(th0)
            for g in grads:
                assert o.push(0, g) == 1
                o.pull(0)
            out[(variant, prec)] = (o.get(THETA), o.get(V))
    for prec in (32, 64):
        for variant in (GA, SA):
            assert np.array_equal(out[(variant, prec)][0], out[(ASGD, prec)][0])
            assert np.array_equal(out[(variant, prec)][1], out[(ASGD, prec)][1])
    p = torch.tensor(th0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.SGD([p], lr=float(np.float32(eta)), momentum=float(np.float32(gam)), dampening=0.0)
    for g in grads:
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
    assert np.allclose(out[(ASGD, 64)][0], p.detach().numpy(), rtol=1e-12, atol=1e-13)
    assert np.allclose(out[(ASGD, 32)][0], p.detach().numpy(), rtol=1e-5, atol=1e-5)
    # constant gradient c: v_k = c (1-gam^k)/(1-gam); theta_k = theta_0 - eta * sum_t v_t
    c = _f32(r.normal(size=d))
    o = make(d, 1, eta, gam, 0.999, ASGD, precision=64)
    o.set_params(th0)
    e, g_ = float(np.float32(eta)), float(np.float32(gam))
    for k in range(1, 12):
        o.push(0, c)
        o.pull(0)
        vk = c.astype(np.float64) * (1 - g_ ** k) / (1 - g_)
        sk = c.astype(np.float64) * (k - g_ * (1 - g_ ** k) / (1 - g_)) / (1 - g_)
        assert np.allclose(o.get(V), vk, rtol=1e-12, atol=1e-14)
        assert np.allclose(o.get(THETA), th0.astype(np.float64) - e * sk, rtol=1e-12, atol=1e-13)


def pin_sa_two_step_expansion(make):
    """Section 4.1 'Under-Penalizing': theta_{k+2} = theta_{k+1} - (eta/tau_{k+1})
    (gam^2 v_k + gam g_k + g_{k+1}), and theta_{k+1} = theta_k - (eta/tau_k)(gam v_k + g_k);
    delays for the schedule 0,1,2,0,2 worked by hand: 1,2,3,3,2."""
    d, eta, gam = 17, 0.1, 0.9
    r = _rng(3)
    th0 = _f32(r.normal(size=d))
    sched, want_tau = [0, 1, 2, 0, 2], [1, 2, 3, 3, 2]
    grads = [_f32(r.normal(size=d)) for _ in sched]
    o = make(d, 3, eta, gam, 0.999, SA, precision=64)
    o.set_params(th0)
    th, v = [o.get(THETA)], [o.get(V)]
    taus = []
    for i, g in zip(sched, grads):
        taus.append(o.push(i, g))
        o.pull(i)
        th.append(o.get(THETA))
        v.append(o.get(V))
    assert taus == want_tau
    e, g_ = float(np.float32(eta)), float(np.float32(gam))
    G = [g.astype(np.float64) for g in grads]
    for k in range(len(sched)):
        one = th[k] - e / want_tau[k] * (g_ * v[k] + G[k])
        assert np.allclose(th[k + 1], one, rtol=1e-13, atol=1e-14)
    for k in range(len(sched) - 1):
        two = th[k + 1] - e / want_tau[k + 1] * (g_ * g_ * v[k] + g_ * G[k] + G[k + 1])
        assert np.allclose(th[k + 2], two, rtol=1e-13, atol=1e-14)
    # and the fp32 build agrees to rounding
    o32 = make(d, 3, eta, gam, 0.999, SA, precision=32)
    o32.set_params(th0)
    assert o32.push_batch(sched, grads) == want_tau
    assert np.allclose(o32.get(THETA), th[-1], rtol=1e-5, atol=1e-6)


def pin_zero_momentum(make):
    """Section 6 'ASGD': gamma = 0 leaves theta <- theta - eta * g_hat and v = g_hat."""
    d, eta = 21, 0.2
    r = _rng(4)
    th0 = _f32(r.normal(size=d))
    o = make(d, 2, eta, 0.0, 0.999, ASGD, precision=64)
    o.set_params(th0)
    acc = th0.astype(np.float64)
    for k in range(6):
        g = _f32(r.normal(size=d))
        o.push(k % 2, g)
        o.pull(k % 2)
        acc = acc - float(np.float32(eta)) * g.astype(np.float64)
        assert np.array_equal(o.get(V), g.astype(np.float64))
        assert np.allclose(o.get(THETA), acc, rtol=1e-14, atol=1e-15)
    # SA with gamma = 0: plain SGD with the step divided by the delay
    o = make(d, 3, eta, 0.0, 0.999, SA, precision=64)
    o.set_params(th0)
    acc = th0.astype(np.float64)
    for k, (i, tau) in enumerate(zip([0, 1, 2, 1], [1, 2, 3, 2])):
        g = _f32(r.normal(size=d))
        assert o.push(i, g) == tau
        o.pull(i)
        acc = acc - float(np.float32(eta)) / tau * g.astype(np.float64)
        assert np.allclose(o.get(THETA), acc, rtol=1e-14, atol=1e-15)


def pin_constant_magnitude_gives_constant_C(make):
    """C Coefficient algorithm: if |v| = c at every step, the bias-corrected second moment is
    c^2 at every k, so C = eta_max (c + eps) from the first refresh on (the Adam-style
    correction with exponent k = number of refreshes)."""
    d, eta, beta, eps = 16, 0.1, 0.999, 1e-8
    c = _f32(np.linspace(0.01, 3.0, d))
    sign = np.ones(d, dtype=np.float32)
    for c_order in (0, 1):
        o = make(d, 1, eta, 0.0, beta, GA, precision=64, c_order=c_order)
        o.set_params(np.zeros(d, np.float32))
        want = float(np.float32(eta)) * (c.astype(np.float64) + eps)
        for k in range(1, 40):
            sign = -sign if k % 3 == 0 else sign
            o.push(0, c * sign)
            o.pull(0)
            assert np.allclose(o.get(C), want, rtol=1e-11, atol=0), f"C drifted at k={k}"
    # fp32 build: same to fp32 rounding
    o = make(d, 1, eta, 0.0, beta, GA, precision=32)
    o.set_params(np.zeros(d, np.float32))
    for k in range(1, 40):
        o.push(0, c)
        o.pull(0)
        assert np.allclose(o.get(C), want, rtol=3e-5, atol=0)


def pin_first_refresh(make):
    """C Coefficient algorithm at k = 1: m_hat = v^2, so C = eta_max (|v| + eps); before any
    refresh C = eta_max * eps (the reading of 'Initialize C <- 0')."""
    d, eta = 12, 0.25
    r = _rng(6)
    th0 = _f32(r.normal(size=d))
    g = _f32(r.normal(size=d))
    o = make(d, 2, eta, 0.9, 0.75, GA, precision=64)
    o.set_params(th0)
    assert np.allclose(o.get(C), 0.25 * 1e-8, rtol=1e-12)
    assert np.array_equal(o.gap(0), np.ones(d))
    o.push(0, g)
    assert np.allclose(o.get(V), g.astype(np.float64), rtol=0, atol=0)
    assert np.allclose(o.get(M), 0.25 * g.astype(np.float64) ** 2, rtol=1e-14)
    assert np.allclose(o.get(C), 0.25 * (np.abs(g.astype(np.float64)) + 1e-8), rtol=1e-12)


def pin_same_direction_steps_give_gap_tau(make):
    """Section 5.1: E[G] = tau exactly when all tau updates went the same way. Worker B makes t
    unpenalised steps of eta*c each (gamma = 0, its own copy always current) while worker A
    holds theta_0: A's Gap is t + 1 = A's delay, and A's gradient is divided by it."""
    d, eta, t = 8, 0.1, 6
    c = _f32(np.linspace(0.5, 4.0, d))
    o = make(d, 2, eta, 0.0, 0.999, GA, precision=64)
    o.set_params(np.zeros(d, np.float32))
    for k in range(t):
        assert o.push(1, c) == (1 if k else 1)
        o.pull(1)
        assert np.array_equal(o.gap(1), np.ones(d))
    e = float(np.float32(eta))
    assert np.allclose(o.get(THETA), -t * e * c.astype(np.float64), rtol=1e-13)
    G = o.gap(0)
    assert np.allclose(G, t + 1, rtol=1e-6), G       # eps makes it a hair below t+1
    assert np.all(G < t + 1) and np.all(G > t + 1 - 1e-5)
    before = o.get(THETA)
    assert o.push(0, c) == t + 1
    assert np.allclose(o.get(V), c.astype(np.float64) / G, rtol=1e-13)
    assert np.allclose(before - o.get(THETA), e * c.astype(np.float64) / G, rtol=1e-11)


def pin_round_robin_delays(make):
    """Staleness-Aware master: tau_k = k - iter[i]. N equal workers in round robin give
    tau = k for the first N arrivals and N from then on ('tau scales linearly with N')."""
    d, n = 4, 7
    g = np.ones(d, np.float32)
    for variant in (ASGD, SA, GA):
        o = make(d, n, 0.01, 0.5, 0.999, variant, precision=32)
        o.set_params(np.zeros(d, np.float32))
        taus = o.push_batch([k % n for k in range(3 * n)], [g] * (3 * n))
        assert taus == [k + 1 for k in range(n)] + [n] * (2 * n)
        assert o.k_done == 3 * n
    # a second push with no pull in between keeps measuring against the old copy
    o = make(d, 2, 0.01, 0.5, 0.999, SA, precision=32)
    o.set_params(np.zeros(d, np.float32))
    assert [o.push(0, g), o.push(0, g), o.push(1, g), o.push(0, g)] == [1, 2, 3, 4]
    o.pull(0)
    assert o.iter(0) == 4 and o.push(0, g) == 1


def pin_pull_saves_master(make):
    """'Save and send current parameters': after pull(i) the saved copy of worker i is the
    master's theta; other workers' copies are untouched; set_params seeds every copy."""
    d = 9
    r = _rng(8)
    th0 = _f32(r.normal(size=d))
    o = make(d, 3, 0.1, 0.9, 0.999, GA, precision=32)
    o.set_params(th0)
    for i in range(3):
        assert np.array_equal(o.saved(i), th0.astype(np.float64))
    o.push(0, _f32(r.normal(size=d)))
    th1 = o.get(THETA)
    assert not np.array_equal(th1, th0.astype(np.float64))
    o.pull(2)
    assert np.array_equal(o.saved(2), th1)
    assert np.array_equal(o.saved(0), th0.astype(np.float64))
    assert np.array_equal(o.saved(1), th0.astype(np.float64))
    assert np.array_equal(o.sent_f32(2).astype(np.float64), th1)
    # set_params starts a new run: v = m = 0, no arrivals counted, every copy = theta_0
    o.set_params(th0)
    assert not o.get(V).any() and not o.get(M).any() and o.k_done == 0 and o.iter(2) == 0
    assert np.array_equal(o.saved(2), th0.astype(np.float64))


def pin_hand_worked_example(make):
    """Two arrivals worked by hand in exact fractions (tests/golden/ga_two_arrivals.txt)."""
    vals = {}
    with open(os.path.join(GOLDEN, "ga_two_arrivals.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split("=")
                vals[k.strip()] = Fraction(v.strip())
    o = make(1, 2, float(vals["eta"]), float(vals["gamma"]), float(vals["beta"]), GA,
             precision=64, eps=float(vals["eps"]))
    o.set_params(_f32([float(vals["theta0"])]))
    assert o.push(0, _f32([float(vals["g1"])])) == 1
    o.pull(0)
    for name, which in (("theta1", THETA), ("v1", V), ("m1", M), ("C1", C)):
        assert abs(o.get(which)[0] - float(vals[name])) <= 1e-15 * max(1, abs(float(vals[name]))), name
    assert abs(o.gap(1)[0] - float(vals["G2"])) < 1e-15 * 4
    assert o.push(1, _f32([float(vals["g2"])])) == 2
    for name, which in (("theta2", THETA), ("v2", V), ("m2", M)):
        assert abs(o.get(which)[0] - float(vals[name])) <= 4e-16 * max(1, abs(float(vals[name]))), name
    assert o.stats()[1] == o.stats()[0] and abs(o.stats()[0] - float(vals["G2"])) < 1e-15


# ------------------------------------------------------------------ exact brute force
def _sqrt_fraction(x):
    getcontext().prec = 90
    if x == 0:
        return Fraction(0)
    s = (Decimal(x.numerator) / Decimal(x.denominator)).sqrt()
    return Fraction(s)


def brute_force(th0, sched, grads, n, eta, gam, beta, eps, variant, c_order):
    """The master algorithms of the paper in exact rational arithmetic (square roots to 90
    digits), scalar by scalar. push followed by pull for each arrival."""
    d = len(th0)
    th = [Fraction(float(x)) for x in th0]
    v = [Fraction(0)] * d
    m = [Fraction(0)] * d
    saved = [list(th) for _ in range(n)]
    it = [0] * n
    refreshes = 0
    taus, gaps = [], []
    for k, (i, g) in enumerate(zip(sched, grads), start=1):
        g = [Fraction(float(x)) for x in g]
        tau = k - it[i]
        taus.append(tau)
        for j in range(d):
            if variant == ASGD:
                v[j] = gam * v[j] + g[j]
                th[j] = th[j] - eta * v[j]
            elif variant == SA:
                v[j] = gam * v[j] + g[j]
                th[j] = th[j] - eta / tau * v[j]
            else:
                r = refreshes
                mj = m[j]
                if c_order == 1:
                    u = gam * v[j] + g[j]
                    mj = beta * mj + (1 - beta) * u * u
                    r += 1
                    m[j] = mj
                Cj = eta * eps if r == 0 else eta * (_sqrt_fraction(mj / (1 - beta ** r)) + eps)
                Gj = abs(th[j] - saved[i][j]) / Cj + 1
                v[j] = gam * v[j] + g[j] / Gj
                th[j] = th[j] - eta * v[j]
                if c_order == 0:
                    m[j] = beta * m[j] + (1 - beta) * v[j] * v[j]
                if j == d - 1:
                    gaps.append(Gj)
        if variant == GA:
            refreshes += 1
        saved[i] = list(th)
        it[i] = k
    return th, v, m, taus


def pin_exact_brute_force(make):
    """Algorithms 'Momentum-ASGD', 'Staleness-Aware', 'Gap-Aware: master' and 'C Coefficient
    Calculation' evaluated in exact arithmetic on d = 3, N = 3, 6 arrivals."""
    r = _rng(10)
    d, n = 3, 3
    th0 = _f32(r.normal(size=d))
    sched = [0, 1, 0, 2, 1, 0]
    grads = [_f32(r.normal(size=d)) for _ in sched]
    eta, gam, beta, eps = 0.125, 0.75, 0.875, 1e-8      # dyadic: exact as fp32 and as fractions
    F = Fraction
    for variant in (ASGD, SA, GA):
        for c_order in ((0, 1) if variant == GA else (0,)):
            th, v, m, taus = brute_force(th0, sched, grads, n, F(eta), F(gam), F(beta), F(eps),
                                         variant, c_order)
            for prec, tol in ((64, 2e-13), (32, 2e-5)):
                o = make(d, n, eta, gam, beta, variant, precision=prec, c_order=c_order, eps=eps)
                o.set_params(th0)
                assert o.push_batch(sched, grads) == taus
                for which, ref in ((THETA, th), (V, v), (M, m)):
                    got = o.get(which)
                    want = np.array([float(x) for x in ref])
                    assert np.all(np.abs(got - want) <= tol * (1 + np.abs(want))), \
                        (variant, c_order, prec, which, got, want)


# ------------------------------------------------------------------ SA-Gradient and DANA
def pin_sa_gradient_two_step(make):
    """Algorithm 'Staleness-Aware-Gradient: master': v <- gamma v + g/tau, theta <- theta - eta v.
    Unrolled twice: theta_{k+2} = theta_{k+1} - eta (gamma^2 v_k + gamma g_k/tau_k + g_{k+1}/tau_{k+1}),
    which differs from the Section 4.1 form where the whole step is divided by tau_{k+1}."""
    d, eta, gam = 13, 0.1, 0.9
    r = _rng(21)
    th0 = _f32(r.normal(size=d))
    sched, want_tau = [0, 1, 2, 0, 2], [1, 2, 3, 3, 2]
    grads = [_f32(r.normal(size=d)) for _ in sched]
    o = make(d, 3, eta, gam, 0.999, SA_GRAD, precision=64)
    o.set_params(th0)
    th, v, taus = [o.get(THETA)], [o.get(V)], []
    for i, g in zip(sched, grads):
        taus.append(o.push(i, g))
        o.pull(i)
        th.append(o.get(THETA))
        v.append(o.get(V))
    assert taus == want_tau
    e, g_ = float(np.float32(eta)), float(np.float32(gam))
    G = [g.astype(np.float64) for g in grads]
    for k in range(len(sched) - 1):
        two = th[k + 1] - e * (g_ * g_ * v[k] + g_ * G[k] / want_tau[k] + G[k + 1] / want_tau[k + 1])
        assert np.allclose(th[k + 2], two, rtol=1e-13, atol=1e-14)
    # all delays 1 (one worker): the same as plain momentum, bit for bit
    a = make(d, 1, eta, gam, 0.999, SA_GRAD, precision=32)
    b = make(d, 1, eta, gam, 0.999, ASGD, precision=32)
    for o_ in (a, b):
        o_.set_params(th0)
        for g in grads:
            assert o_.push(0, g) == 1
            o_.pull(0)
    assert np.array_equal(a.get(THETA), b.get(THETA))


def pin_dana_one_worker_is_nesterov(make):
    """Algorithm 'DANA: master' with one worker: the worker is always sent theta - eta gamma v,
    the look-ahead point of Nesterov's accelerated gradient. On a quadratic the points sent are
    exactly the iterates of torch.optim.SGD(nesterov=True), which stores that look-ahead point."""
    import torch
    d, eta, gam, steps = 19, 0.05, 0.9, 30
    r = _rng(22)
    th0 = _f32(r.normal(size=d))
    a = r.uniform(0.5, 2.0, size=d)
    target = r.normal(size=d)
    p = torch.tensor(th0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.SGD([p], lr=float(np.float32(eta)), momentum=float(np.float32(gam)), nesterov=True)
    o = make(d, 1, eta, gam, 0.999, DANA, precision=64)
    o.set_params(th0)
    for _ in range(steps):
        sent = o.saved(0)
        assert np.allclose(sent, p.detach().numpy(), rtol=1e-11, atol=1e-12)
        g = _f32(a * (sent - target))            # gradient at the point the worker was sent
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        assert o.push(0, g) == 1
        o.pull(0)
    assert np.allclose(o.saved(0), p.detach().numpy(), rtol=1e-10, atol=1e-11)
    assert not np.allclose(o.saved(0), o.get(THETA), rtol=1e-3, atol=1e-6), "the estimate is not theta itself"


def pin_dana_zero_momentum_reduces(make):
    """gamma = 0: the estimate is theta itself and every DANA master is its plain counterpart
    (DANA = ASGD, DANA-SA = SA-Gradient, DANA-GA = GA), bit for bit."""
    d, n, eta = 23, 3, 0.1
    r = _rng(23)
    th0 = _f32(r.normal(size=d))
    sched = [0, 1, 2, 1, 0, 2, 2, 0]
    grads = [_f32(r.normal(size=d)) for _ in sched]
    for dana, plain in ((DANA, ASGD), (DANA_SA, SA_GRAD), (DANA_GA, GA)):
        a = make(d, n, eta, 0.0, 0.999, dana, precision=32)
        b = make(d, n, eta, 0.0, 0.999, plain, precision=32)
        a.set_params(th0)
        b.set_params(th0)
        assert a.push_batch(sched, grads) == b.push_batch(sched, grads)
        assert np.array_equal(a.get(THETA), b.get(THETA)), (dana, plain)
        for i in range(n):
            assert np.array_equal(a.saved(i), b.saved(i))
        if dana == DANA_GA:
            assert np.array_equal(a.get(M), b.get(M)) and a.stats() == b.stats()


def pin_dana_structure(make):
    """DANA masters, step by step: only the arriving worker's momentum changes, v^i <- gamma v^i
    + g (DANA) or g/tau (DANA-SA); the master moves by -eta v^i; the running sum equals the sum
    of the N momentum vectors; the worker is sent theta - eta gamma sum_j v^j; summing the v^j
    afresh at every send (the printed form) gives the same trajectory."""
    d, n, eta, gam = 11, 4, 0.1, 0.9
    r = _rng(24)
    th0 = _f32(r.normal(size=d))
    sched = [0, 1, 2, 3, 1, 0, 3, 3, 2, 1]
    want_tau = [1, 2, 3, 4, 3, 5, 3, 1, 6, 5]
    grads = [_f32(r.normal(size=d)) for _ in sched]
    e, g_ = float(np.float32(eta)), float(np.float32(gam))
    for variant in (DANA, DANA_SA):
        o = make(d, n, eta, gam, 0.999, variant, precision=64)
        o.set_params(th0)
        vw = [np.zeros(d) for _ in range(n)]
        th = th0.astype(np.float64)
        for i, g, tau in zip(sched, grads, want_tau):
            assert o.push(i, g) == tau
            gg = g.astype(np.float64) / (tau if variant == DANA_SA else 1)
            vw[i] = g_ * vw[i] + gg
            th = th - e * vw[i]
            for w in range(n):
                assert np.allclose(o.worker_momentum(w), vw[w], rtol=1e-13, atol=1e-15)
            assert np.allclose(o.get(THETA), th, rtol=1e-13, atol=1e-14)
            assert np.allclose(o.get(V), sum(vw), rtol=1e-12, atol=1e-14)
            o.pull(i)
            assert np.allclose(o.saved(i), th - e * g_ * sum(vw), rtol=1e-12, atol=1e-14)
    # constant gradient, round robin: worker's momentum after t pushes is c (1-gam^t)/(1-gam)
    c = _f32(r.normal(size=d))
    o = make(d, 3, eta, gam, 0.999, DANA, precision=64)
    o.set_params(th0)
    o.push_batch([k % 3 for k in range(9)], [c] * 9)
    geo = [(1 - g_ ** t) / (1 - g_) for t in (1, 2, 3)]
    assert np.allclose(o.worker_momentum(1), c.astype(np.float64) * geo[2], rtol=1e-13)
    assert np.allclose(o.get(THETA), th0.astype(np.float64) - e * 3 * sum(geo) * c.astype(np.float64), rtol=1e-12, atol=1e-13)
    # running sum versus the printed sum over j
    for variant in (DANA, DANA_SA, DANA_GA):
        a = make(d, n, eta, gam, 0.999, variant, precision=64, dana_sum=1)
        b = make(d, n, eta, gam, 0.999, variant, precision=64, dana_sum=0)
        a.set_params(th0)
        b.set_params(th0)
        assert a.push_batch(sched, grads) == b.push_batch(sched, grads) == want_tau
        assert np.allclose(a.get(THETA), b.get(THETA), rtol=1e-12, atol=1e-13)
        for i in range(n):
            assert np.allclose(a.saved(i), b.saved(i), rtol=1e-12, atol=1e-13)


def pin_dana_gap(make):
    """Algorithm 'DANA-Gap-Aware: master': the Gap is measured against the ESTIMATE that was
    saved when sent; where the master happens to sit on that estimate the gradient passes
    unpenalised; elsewhere it is divided by |theta - theta^i|/C + 1 with the same C as GA."""
    d, eta, gam = 10, 0.1, 0.5
    r = _rng(25)
    th0 = _f32(r.normal(size=d))
    g0 = _f32(r.normal(size=d))
    o = make(d, 2, eta, gam, 0.75, DANA_GA, precision=64)
    o.set_params(th0)
    assert o.push(0, g0) == 1            # G = 1 (copy = theta_0 = master); v^0 = g0
    assert np.array_equal(o.worker_momentum(0), g0.astype(np.float64))
    o.pull(0)
    e, g_ = float(np.float32(eta)), float(np.float32(gam))
    th1 = th0.astype(np.float64) - e * g0.astype(np.float64)
    est = th1 - e * g_ * g0.astype(np.float64)
    assert np.allclose(o.saved(0), est, rtol=1e-14)
    # Gap of worker 0 now: |theta_1 - estimate| / C + 1 with C = eta (|v| + eps) after one refresh
    Cw = e * (np.abs(g0.astype(np.float64)) + 1e-8)
    assert np.allclose(o.get(C), Cw, rtol=1e-12)
    assert np.allclose(o.gap(0), np.abs(th1 - est) / Cw + 1, rtol=1e-12)
    assert np.allclose(o.gap(0), g_ + 1, rtol=1e-6)       # eta gamma |v| / (eta |v|) + 1
    # worker 1 still holds theta_0: its Gap is |theta_1 - theta_0| / C + 1 = 2
    assert np.allclose(o.gap(1), 2.0, rtol=1e-6)
    g1 = _f32(r.normal(size=d))
    G1 = o.gap(1)
    assert o.push(1, g1) == 2
    assert np.allclose(o.worker_momentum(1), g1.astype(np.float64) / G1, rtol=1e-13)
    assert np.allclose(o.get(THETA), th1 - e * g1.astype(np.float64) / G1, rtol=1e-13)


def brute_force_dana(th0, sched, grads, n, eta, gam, beta, eps, variant, c_order):
    """The three DANA masters in exact rational arithmetic; the sum over workers is the printed one."""
    d = len(th0)
    th = [Fraction(float(x)) for x in th0]
    vw = [[Fraction(0)] * d for _ in range(n)]
    m = [Fraction(0)] * d
    saved = [list(th) for _ in range(n)]
    it = [0] * n
    refreshes = 0
    taus = []
    for k, (i, g) in enumerate(zip(sched, grads), start=1):
        g = [Fraction(float(x)) for x in g]
        tau = k - it[i]
        taus.append(tau)
        for j in range(d):
            gp = g[j]
            if variant == DANA_SA:
                gp = g[j] / tau
            elif variant == DANA_GA:
                r, mj = refreshes, m[j]
                if c_order == 1:
                    u = gam * vw[i][j] + g[j]
                    mj = beta * mj + (1 - beta) * u * u
                    r += 1
                    m[j] = mj
                Cj = eta * eps if r == 0 else eta * (_sqrt_fraction(mj / (1 - beta ** r)) + eps)
                gp = g[j] / (abs(th[j] - saved[i][j]) / Cj + 1)
            vw[i][j] = gam * vw[i][j] + gp
            th[j] = th[j] - eta * vw[i][j]
            if variant == DANA_GA and c_order == 0:
                m[j] = beta * m[j] + (1 - beta) * vw[i][j] * vw[i][j]
        if variant == DANA_GA:
            refreshes += 1
        saved[i] = [th[j] - eta * gam * sum(vw[w][j] for w in range(n)) for j in range(d)]
        it[i] = k
    return th, vw, m, saved, taus


def pin_dana_exact_brute_force(make):
    """Algorithms 'DANA', 'DANA-Staleness-Aware', 'DANA-Gap-Aware: master' in exact arithmetic."""
    r = _rng(26)
    d, n = 3, 3
    th0 = _f32(r.normal(size=d))
    sched = [0, 1, 0, 2, 1, 0, 2]
    grads = [_f32(r.normal(size=d)) for _ in sched]
    eta, gam, beta, eps = 0.125, 0.75, 0.875, 1e-8
    F = Fraction
    for variant in (DANA, DANA_SA, DANA_GA):
        for c_order in ((0, 1) if variant == DANA_GA else (0,)):
            th, vw, m, saved, taus = brute_force_dana(th0, sched, grads, n, F(eta), F(gam), F(beta), F(eps),
                                                      variant, c_order)
            for prec, tol in ((64, 2e-13), (32, 2e-5)):
                for dana_sum in (0, 1):
                    o = make(d, n, eta, gam, beta, variant, precision=prec, c_order=c_order, eps=eps,
                             dana_sum=dana_sum)
                    o.set_params(th0)
                    assert o.push_batch(sched, grads) == taus
                    pairs = [(o.get(THETA), th), (o.get(M), m)]
                    pairs += [(o.worker_momentum(w), vw[w]) for w in range(n)]
                    pairs += [(o.saved(w), saved[w]) for w in range(n)]
                    for got, ref in pairs:
                        want = np.array([float(x) for x in ref])
                        assert np.all(np.abs(got - want) <= tol * (1 + np.abs(want))), (variant, c_order, prec)


# ------------------------------------------------------------------ Adam masters
def pin_adam_is_torch_adam(make):
    """Algorithm 'Adam: master' ignores staleness altogether: whatever the schedule it is the
    textbook Adam, checked against torch.optim.Adam; its first step moves every parameter by
    eta * g / (|g| + eps)."""
    import torch
    d, eta, b1, b2, eps = 29, 0.01, 0.9, 0.999, 1e-8
    r = _rng(31)
    th0 = _f32(r.normal(size=d))
    sched = [0, 1, 2, 0, 2, 1, 1, 0, 2, 2, 0, 1]
    grads = [_f32(r.normal(size=d)) for _ in sched]
    o = make(d, 3, eta, b1, 0.999, ADAM, precision=64, beta2=b2, adam_eps=eps)
    o.set_params(th0)
    p = torch.tensor(th0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([p], lr=float(np.float32(eta)), betas=(float(np.float32(b1)), float(np.float32(b2))),
                           eps=float(np.float32(eps)))
    for k, (i, g) in enumerate(zip(sched, grads)):
        o.push(i, g)
        o.pull(i)
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        if k == 0:
            g64 = g.astype(np.float64)
            step1 = float(np.float32(eta)) * g64 / (np.abs(g64) + float(np.float32(eps)))
            assert np.allclose(o.get(THETA), th0.astype(np.float64) - step1, rtol=1e-12, atol=1e-14)
        assert np.allclose(o.get(THETA), p.detach().numpy(), rtol=1e-10, atol=1e-12), k
    st = opt.state[p]
    assert np.allclose(o.get(V), st["exp_avg"].numpy(), rtol=1e-12, atol=1e-15)
    assert np.allclose(o.second_moment(), st["exp_avg_sq"].numpy(), rtol=1e-12, atol=1e-18)
    o32 = make(d, 3, eta, b1, 0.999, ADAM, precision=32, beta2=b2, adam_eps=eps)
    o32.set_params(th0)
    o32.push_batch(sched, grads)
    assert np.allclose(o32.get(THETA), p.detach().numpy(), rtol=1e-4, atol=1e-5)


def pin_adam_penalty_on_first_moment_only(make):
    """Algorithms 'Adam-Staleness-Aware' and 'Adam-Gap-Aware': the second moment is that of
    plain Adam, bit for bit; the first moment accumulates (1-beta1) g / tau (SA), resp.
    ((1-beta1)/G) g (GA). One worker (tau = 1) makes Adam-SA plain Adam; where the master still
    equals the saved copy Adam-GA adds exactly (1-beta1) g."""
    d, n, eta, b1 = 16, 3, 0.01, 0.9
    r = _rng(32)
    th0 = _f32(r.normal(size=d))
    sched, want_tau = [0, 1, 2, 0, 2], [1, 2, 3, 3, 2]
    grads = [_f32(r.normal(size=d)) for _ in sched]
    runs = {}
    for variant in (ADAM, ADAM_SA, ADAM_GA):
        o = make(d, n, eta, b1, 0.999, variant, precision=64)
        o.set_params(th0)
        assert o.push_batch(sched, grads) == want_tau
        runs[variant] = o
    for variant in (ADAM_SA, ADAM_GA):
        assert np.array_equal(runs[variant].second_moment(), runs[ADAM].second_moment())
    B1 = float(np.float32(b1))
    m_sa = np.zeros(d)
    for g, tau in zip(grads, want_tau):
        m_sa = B1 * m_sa + (1 - B1) * g.astype(np.float64) / tau
    assert np.allclose(runs[ADAM_SA].get(V), m_sa, rtol=1e-12, atol=1e-16)
    assert not np.allclose(runs[ADAM_SA].get(V), runs[ADAM].get(V), rtol=1e-3)
    # one worker: every delay is 1
    a = make(d, 1, eta, b1, 0.999, ADAM_SA, precision=32)
    b = make(d, 1, eta, b1, 0.999, ADAM, precision=32)
    for o in (a, b):
        o.set_params(th0)
        o.push_batch([0] * 5, grads)
    assert np.array_equal(a.get(THETA), b.get(THETA))
    # Adam-GA, first arrival of each worker's untouched elements: G = 1 there
    g1 = grads[0].copy()
    g1[1::2] = 0.0
    ga = make(d, 2, eta, b1, 0.999, ADAM_GA, precision=32)
    ad = make(d, 2, eta, b1, 0.999, ADAM, precision=32)
    for o in (ga, ad):
        o.set_params(th0)
        o.push(1, g1)
        o.pull(1)
    G = ga.gap(0)
    assert np.all(G[1::2] == 1.0) and np.all(G[0::2] > 1.0)
    for o in (ga, ad):
        o.push(0, grads[1])
    assert np.array_equal(ga.get(V)[1::2], ad.get(V)[1::2])
    assert np.array_equal(ga.get(THETA)[1::2], ad.get(THETA)[1::2])
    # penalised elements: first moment is beta1 m + ((1-beta1)/G) g with the G read before the push
    m_prev = (1 - B1) * g1.astype(np.float64)
    want = B1 * m_prev + (1 - B1) / G * grads[1].astype(np.float64)
    assert np.allclose(ga.get(V), want, rtol=1e-5, atol=1e-9)


def pin_adam_ga_coefficient(make):
    """Adam-GA's C: the C algorithm with gamma = 0. A gradient of constant magnitude c gives
    C = eta_max (c + eps) from the first refresh on, whatever Adam's own moments do."""
    d, eta = 12, 0.01
    c = _f32(np.linspace(0.02, 2.0, d))
    for c_order in (0, 1):
        o = make(d, 1, eta, 0.9, 0.999, ADAM_GA, precision=64, c_order=c_order)
        o.set_params(np.zeros(d, np.float32))
        sign = 1.0
        for k in range(1, 25):
            sign = -sign if k % 4 == 0 else sign
            o.push(0, _f32(c * sign))
            o.pull(0)
            assert np.allclose(o.get(C), float(np.float32(eta)) * (c.astype(np.float64) + 1e-8), rtol=1e-11)


def brute_force_adam(th0, sched, grads, n, eta, b1, b2, eps_adam, beta, eps, variant, c_order):
    d = len(th0)
    th = [Fraction(float(x)) for x in th0]
    m1 = [Fraction(0)] * d
    v2 = [Fraction(0)] * d
    mc = [Fraction(0)] * d
    saved = [list(th) for _ in range(n)]
    it = [0] * n
    refreshes = 0
    taus = []
    for k, (i, g) in enumerate(zip(sched, grads), start=1):
        g = [Fraction(float(x)) for x in g]
        tau = k - it[i]
        taus.append(tau)
        for j in range(d):
            if variant == ADAM:
                first = (1 - b1) * g[j]
            elif variant == ADAM_SA:
                first = (1 - b1) * g[j] / tau
            else:
                r, mj = refreshes, mc[j]
                if c_order == 1:
                    mj = beta * mj + (1 - beta) * g[j] * g[j]
                    r += 1
                    mc[j] = mj
                Cj = eta * eps if r == 0 else eta * (_sqrt_fraction(mj / (1 - beta ** r)) + eps)
                Gj = abs(th[j] - saved[i][j]) / Cj + 1
                first = (1 - b1) / Gj * g[j]
                if c_order == 0:
                    mc[j] = beta * mc[j] + (1 - beta) * g[j] * g[j]
            m1[j] = b1 * m1[j] + first
            v2[j] = b2 * v2[j] + (1 - b2) * g[j] * g[j]
            m_hat = m1[j] / (1 - b1 ** k)
            v_hat = v2[j] / (1 - b2 ** k)
            th[j] = th[j] - eta * m_hat / (_sqrt_fraction(v_hat) + eps_adam)
        if variant == ADAM_GA:
            refreshes += 1
        saved[i] = list(th)
        it[i] = k
    return th, m1, v2, mc, taus


def pin_adam_exact_brute_force(make):
    """Algorithms 'Adam', 'Adam-Staleness-Aware', 'Adam-Gap-Aware: master' in exact arithmetic."""
    r = _rng(33)
    d, n = 3, 3
    th0 = _f32(r.normal(size=d))
    sched = [0, 1, 0, 2, 1, 0]
    grads = [_f32(r.normal(size=d)) for _ in sched]
    eta, b1, b2, beta, eps = 0.0625, 0.75, 0.875, 0.9375, 2.0 ** -20
    F = Fraction
    for variant in (ADAM, ADAM_SA, ADAM_GA):
        for c_order in ((0, 1) if variant == ADAM_GA else (0,)):
            th, m1, v2, mc, taus = brute_force_adam(th0, sched, grads, n, F(eta), F(b1), F(b2), F(eps), F(beta),
                                                    F(eps), variant, c_order)
            for prec, tol in ((64, 5e-13), (32, 5e-5)):
                o = make(d, n, eta, b1, beta, variant, precision=prec, c_order=c_order, eps=eps, beta2=b2,
                         adam_eps=eps)
                o.set_params(th0)
                assert o.push_batch(sched, grads) == taus
                for got, ref in ((o.get(THETA), th), (o.get(V), m1), (o.second_moment(), v2), (o.get(M), mc)):
                    want = np.array([float(x) for x in ref])
                    assert np.all(np.abs(got - want) <= tol * (1 + np.abs(want))), (variant, c_order, prec)


# ------------------------------------------------------------------ layer-wise and global Gap
def pin_layer_gap_with_one_parameter_per_layer_is_parameter_wise(make):
    """Section 5.3: with every parameter a layer of its own the layer-wise Gap IS the
    parameter-wise Gap (the norm of one number is its absolute value), bit for bit."""
    d, n = 9, 3
    r = _rng(51)
    th0 = _f32(r.normal(size=d))
    sched = [0, 1, 2, 0, 0, 2, 1]
    grads = [_f32(r.normal(size=d)) for _ in sched]
    for prec in (32, 64):
        a = make(d, n, 0.1, 0.9, 0.999, GA_LAYER, precision=prec)
        a.set_layers(np.arange(d + 1))
        b = make(d, n, 0.1, 0.9, 0.999, GA, precision=prec)
        for o in (a, b):
            o.set_params(th0)
        assert a.push_batch(sched, grads) == b.push_batch(sched, grads)
        assert np.array_equal(a.get(THETA), b.get(THETA)) and np.array_equal(a.get(V), b.get(V))
        assert np.array_equal(a.layer_state()[1], b.get(M))


def pin_global_gap_definition(make):
    """Definition 1: G = ||theta_k - theta_{k-tau}|| / C + 1 with C = eta_max E||grad||: one number
    for the whole vector. After t same-direction unpenalised steps G = t + 1 = the delay
    (Section 5.1); the whole gradient is divided by that one number; the value follows from
    the norms directly."""
    d, eta, t = 6, 0.1, 5
    c = _f32(np.linspace(0.5, 3.0, d))
    o = make(d, 2, eta, 0.0, 0.999, GA_LAYER, precision=64)        # default: one layer = global
    o.set_params(np.zeros(d, np.float32))
    for _ in range(t):
        o.push(1, c)
        o.pull(1)
        assert o.layer_state()[0][0] == 1.0
    e = float(np.float32(eta))
    c64 = c.astype(np.float64)
    want_G = np.linalg.norm(t * e * c64) / (e * (np.linalg.norm(c64) + 1e-8)) + 1
    assert abs(want_G - (t + 1)) < 1e-6
    before = o.get(THETA)
    g = _f32(np.linspace(-1, 1, d))
    assert o.push(0, g) == t + 1
    assert abs(o.layer_state()[0][0] - want_G) < 1e-12
    assert np.allclose(before - o.get(THETA), e * g.astype(np.float64) / want_G, rtol=1e-12)
    # m is the running average of the squared NORM of the update vector
    m1 = o.layer_state()[1][0]
    b = float(np.float32(0.999))
    m_t = (1 - b ** t) * np.dot(c64, c64)                      # t refreshes with ||c||^2
    want_m = b * m_t + (1 - b) * np.dot(g.astype(np.float64) / want_G, g.astype(np.float64) / want_G)
    assert abs(m1 - want_m) <= 1e-12 * want_m


def pin_layers_are_penalised_independently(make):
    """Layer-wise Gap: 'every layer is penalized differently and independently'. A layer the
    master has not moved since the worker pulled passes its gradient unpenalised (bitwise the
    plain momentum step); a moved layer is scaled by one common factor 1/G_p."""
    off = [0, 5, 12, 20]
    d, eta = 20, 0.1
    r = _rng(53)
    th0 = _f32(r.normal(size=d))
    g1 = _f32(r.normal(size=d))
    g1[5:12] = 0.0                        # worker 1 leaves layer 1 alone
    g0 = _f32(r.normal(size=d))
    res = {}
    for variant in (GA_LAYER, ASGD):
        o = make(d, 2, eta, 0.9, 0.999, variant, precision=32)
        if variant == GA_LAYER:
            o.set_layers(off)
        o.set_params(th0)
        o.push(1, g1)
        o.pull(1)
        o.push(0, g0)
        res[variant] = o
    G = res[GA_LAYER].layer_state()[0]
    assert G[1] == 1.0 and G[0] > 1.0 and G[2] > 1.0
    assert np.array_equal(res[GA_LAYER].get(THETA)[5:12], res[ASGD].get(THETA)[5:12])
    v_prev = g1.astype(np.float64)
    for p, (lo, hi) in enumerate(zip(off[:-1], off[1:])):
        ratio = (res[GA_LAYER].get(V)[lo:hi] - 0.9 * v_prev[lo:hi]) / g0.astype(np.float64)[lo:hi]
        assert np.allclose(ratio, 1.0 / G[p], rtol=2e-5), p    # one factor per layer
    # duplicating a layer's content leaves its Gap unchanged (both norms grow by sqrt 2)
    a = make(10, 2, eta, 0.9, 0.999, GA_LAYER, precision=64)
    b = make(20, 2, eta, 0.9, 0.999, GA_LAYER, precision=64)
    h0, h1, h2 = th0[:10], g1[:10] + 1, g0[:10]
    a.set_params(h0)
    b.set_params(np.concatenate([h0, h0]))
    for o, k in ((a, 1), (b, 2)):
        o.push(1, np.concatenate([h1] * k)); o.pull(1); o.push(0, np.concatenate([h2] * k))
    assert abs(a.layer_state()[0][0] - b.layer_state()[0][0]) < 1e-9
    assert np.allclose(b.get(THETA)[:10], a.get(THETA), rtol=1e-9) and np.array_equal(b.get(THETA)[:10], b.get(THETA)[10:])


def pin_layer_gap_exact_brute_force(make):
    """Layer-wise Gap-Aware master in exact rational arithmetic (norms via exact sums)."""
    r = _rng(54)
    d, n, off = 5, 3, [0, 2, 5]
    th0 = _f32(r.normal(size=d))
    sched = [0, 1, 0, 2, 1, 0]
    grads = [_f32(r.normal(size=d)) for _ in sched]
    eta, gam, beta, eps = 0.125, 0.75, 0.875, 1e-8
    F = Fraction
    th = [F(float(x)) for x in th0]
    v = [F(0)] * d
    mp = [F(0)] * (len(off) - 1)
    saved = [list(th) for _ in range(n)]
    refreshes = 0
    for i, g in zip(sched, grads):
        g = [F(float(x)) for x in g]
        for p in range(len(off) - 1):
            js = range(off[p], off[p + 1])
            dist = _sqrt_fraction(sum((th[j] - saved[i][j]) ** 2 for j in js))
            Cp = F(eta) * F(eps) if refreshes == 0 else F(eta) * (_sqrt_fraction(mp[p] / (1 - F(beta) ** refreshes)) + F(eps))
            Gp = dist / Cp + 1
            for j in js:
                v[j] = F(gam) * v[j] + g[j] / Gp
                th[j] = th[j] - F(eta) * v[j]
            mp[p] = F(beta) * mp[p] + (1 - F(beta)) * sum(v[j] ** 2 for j in js)
        refreshes += 1
        saved[i] = list(th)
    for prec, tol in ((64, 2e-13), (32, 2e-5)):
        o = make(d, n, eta, gam, beta, GA_LAYER, precision=prec, eps=eps)
        o.set_layers(off)
        o.set_params(th0)
        o.push_batch(sched, grads)
        for got, ref in ((o.get(THETA), th), (o.get(V), v), (o.layer_state()[1], mp)):
            want = np.array([float(x) for x in ref])
            assert np.all(np.abs(got - want) <= tol * (1 + np.abs(want))), prec


def pin_learning_rate_schedule(make):
    """Section 5.1: the staleness penalty should shrink as eta decays, so C keeps the MAXIMAL
    rate (C = eta_max E|grad|) while the step uses eta_k. After the rate is cut by 10 the
    coefficient is unchanged, the same displacement counts as the same Gap, and steps are 10x
    shorter; for Adam and DANA the new rate enters the step / the estimate the same way."""
    d, eta = 14, 0.1
    r = _rng(41)
    th0 = _f32(r.normal(size=d))
    g = [_f32(r.normal(size=d)) for _ in range(4)]
    o = make(d, 2, eta, 0.0, 0.999, GA, precision=64)
    o.set_params(th0)
    o.push(0, g[0]); o.pull(0)
    C_before = o.get(C)
    o.set_lr(eta / 10)
    assert np.array_equal(o.get(C), C_before)
    th_before, G = o.get(THETA), o.gap(1)
    o.push(1, g[1])
    e10 = float(np.float32(eta / 10))
    assert np.allclose(th_before - o.get(THETA), e10 * g[1].astype(np.float64) / G, rtol=1e-12)
    # SA: eta_k / tau
    o = make(d, 2, eta, 0.0, 0.999, SA, precision=64)
    o.set_params(th0)
    o.push(0, g[0]); o.pull(0)
    o.set_lr(eta / 10)
    th_before = o.get(THETA)
    assert o.push(1, g[1]) == 2
    assert np.allclose(th_before - o.get(THETA), e10 / 2 * g[1].astype(np.float64), rtol=1e-12)
    # DANA: the estimate uses the current rate
    o = make(d, 1, eta, 0.5, 0.999, DANA, precision=64)
    o.set_params(th0)
    o.push(0, g[0])
    o.set_lr(eta / 10)
    o.pull(0)
    assert np.allclose(o.saved(0), o.get(THETA) - e10 * 0.5 * g[0].astype(np.float64), rtol=1e-13)
    # Adam: first step at the new rate
    o = make(d, 1, eta, 0.9, 0.999, ADAM, precision=64)
    o.set_params(th0)
    o.set_lr(eta / 10)
    o.push(0, g[0])
    g64 = g[0].astype(np.float64)
    assert np.allclose(th0.astype(np.float64) - o.get(THETA), e10 * g64 / (np.abs(g64) + 1e-8), rtol=1e-6)


def pin_weight_decay_is_part_of_the_gradient(make):
    """Appendix "Weight Decay": the decay element belongs to the gradient and is divided by the
    Gap with it. A master with decay lambda fed g equals a master without decay fed
    g + lambda * theta_k (theta_k = its parameters at that arrival), for every family; and the
    textbook case: one worker, momentum SGD with weight_decay in torch."""
    import torch
    d, n, lam = 12, 3, 0.05
    r = _rng(61)
    th0 = _f32(r.normal(size=d))
    sched = [0, 1, 2, 1, 0, 2, 0]
    grads = [_f32(r.normal(size=d)) for _ in sched]
    for variant in (ASGD, SA, GA, SA_GRAD, DANA_GA, ADAM_GA, GA_LAYER):
        a = make(d, n, 0.1, 0.9, 0.999, variant, precision=64)
        b = make(d, n, 0.1, 0.9, 0.999, variant, precision=64)
        a.set_weight_decay(lam)
        for o in (a, b):
            o.set_params(th0)
        for i, g in zip(sched, grads):
            folded = g.astype(np.float64) + float(np.float32(lam)) * b.get(THETA)
            # b is fed fp32 inputs: compare at fp32 resolution of the folded gradient
            ta, tb = a.push(i, g), b.push(i, _f32(folded))
            assert ta == tb
            a.pull(i); b.pull(i)
        assert np.allclose(a.get(THETA), b.get(THETA), rtol=2e-5, atol=2e-6), variant
    p = torch.tensor(th0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.SGD([p], lr=float(np.float32(0.1)), momentum=float(np.float32(0.9)),
                          weight_decay=float(np.float32(lam)))
    o = make(d, 1, 0.1, 0.9, 0.999, GA, precision=64)
    o.set_weight_decay(lam)
    o.set_params(th0)
    for g in grads:
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        o.push(0, g); o.pull(0)
    assert np.allclose(o.get(THETA), p.detach().numpy(), rtol=1e-12, atol=1e-13)


def pin_nesterov_step(make):
    """The Nesterov form of the momentum step, theta - eta (g_hat + gamma v_{k+1}): one worker
    is torch.optim.SGD(nesterov=True); under GA the look-ahead uses the PENALISED gradient; the
    momentum vector itself (and hence C) is that of the plain form."""
    import torch
    d, eta, gam = 15, 0.05, 0.9
    r = _rng(71)
    th0 = _f32(r.normal(size=d))
    grads = [_f32(r.normal(size=d)) for _ in range(12)]
    for variant in (ASGD, SA, GA, SA_GRAD, GA_LAYER):
        p = torch.tensor(th0, dtype=torch.float64, requires_grad=True)
        opt = torch.optim.SGD([p], lr=float(np.float32(eta)), momentum=float(np.float32(gam)), nesterov=True)
        o = make(d, 1, eta, gam, 0.999, variant, precision=64)
        o.set_nesterov()
        o.set_params(th0)
        for g in grads:
            p.grad = torch.tensor(g, dtype=torch.float64)
            opt.step()
            o.push(0, g); o.pull(0)
        assert np.allclose(o.get(THETA), p.detach().numpy(), rtol=1e-12, atol=1e-13), variant
        assert np.allclose(o.get(V), opt.state[p]["momentum_buffer"].numpy(), rtol=1e-12, atol=1e-14)
    # two workers under GA: theta moves by eta (g/G + gamma v_new), v_new = gamma v + g/G
    a = make(d, 2, eta, gam, 0.999, GA, precision=64)
    a.set_nesterov()
    a.set_params(th0)
    a.push(1, grads[0]); a.pull(1)
    G, v_old, th_old = a.gap(0), a.get(V), a.get(THETA)
    a.push(0, grads[1])
    g_hat = grads[1].astype(np.float64) / G
    v_new = float(np.float32(gam)) * v_old + g_hat
    assert np.allclose(a.get(V), v_new, rtol=1e-13)
    assert np.allclose(th_old - a.get(THETA), float(np.float32(eta)) * (g_hat + float(np.float32(gam)) * v_new), rtol=1e-11)
    assert np.any(G > 1.5)


ALL_PINS = [
    pin_gap_is_one_where_copy_equals_master,
    pin_one_worker_is_heavy_ball,
    pin_sa_two_step_expansion,
    pin_zero_momentum,
    pin_constant_magnitude_gives_constant_C,
    pin_first_refresh,
    pin_same_direction_steps_give_gap_tau,
    pin_round_robin_delays,
    pin_pull_saves_master,
    pin_hand_worked_example,
    pin_exact_brute_force,
    pin_sa_gradient_two_step,
    pin_dana_one_worker_is_nesterov,
    pin_dana_zero_momentum_reduces,
    pin_dana_structure,
    pin_dana_gap,
    pin_dana_exact_brute_force,
    pin_adam_is_torch_adam,
    pin_adam_penalty_on_first_moment_only,
    pin_adam_ga_coefficient,
    pin_adam_exact_brute_force,
    pin_learning_rate_schedule,
    pin_layer_gap_with_one_parameter_per_layer_is_parameter_wise,
    pin_global_gap_definition,
    pin_layers_are_penalised_independently,
    pin_layer_gap_exact_brute_force,
    pin_weight_decay_is_part_of_the_gradient,
    pin_nesterov_step,
]
