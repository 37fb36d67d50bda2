"""Synthetic-input generators: hash, shapes, schedules, gradients (CPU side)."""
import numpy as np

import workloads as W


def test_splitmix64_published_outputs():
    # word(key, b) is output b of SplitMix64 seeded with `key`; these are the generator's
    # widely published first outputs for seed 1234567.
    assert [W.word(1234567, b) for b in range(5)] == [
        6457827717110365317, 3203168211198807973, 9817491932198370423,
        4593380528125082431, 16408922859458223821]


def test_c_and_python_hash_agree():
    lib = W.cpu_lib()
    rng = np.random.default_rng(0)
    for _ in range(200):
        seed, tag, a, b = (int(x) for x in rng.integers(0, 2**63, size=4))
        assert lib.wl_cpu_hash(seed, tag % 8, a, b) == W.hash4(seed, tag % 8, a, b)
        assert lib.wl_cpu_mix64(seed) == W.mix64(seed)


def test_uniform_and_noise_fields():
    lib = W.cpu_lib()
    assert lib.wl_cpu_uniform(0) == np.float32(2.0 ** -24)
    assert lib.wl_cpu_uniform(2**64 - 1) == np.float32(1.0 - 2.0 ** -24)
    scale = np.float32(np.sqrt(3.0) / 65536)
    assert lib.wl_cpu_xi(0) == np.float32(-131070) * scale
    assert lib.wl_cpu_xi(2**64 - 1) == np.float32(131070) * scale
    assert lib.wl_cpu_xi(0x0001_0002_0003_0004) == np.float32(10 - 131070) * scale


def test_shapes_match_the_models():
    assert (len(W.resnet20_segments()), sum(W.resnet20_segments())) == (65, 272_474)
    assert (len(W.resnet50_segments()), sum(W.resnet50_segments())) == (161, 25_557_032)
    assert sum(W.wrn16_4_segments()) == 2_748_890
    seg = W.transformer_lm_segments()
    assert seg[0] == 267_735 * 512 and sum(seg) == 150_000_000 and len(seg) == 17
    for name, n, arrivals in (("C1", 8, 1000), ("C2", 32, 20000), ("C3", 64, 2000),
                              ("C4", 128, 50000), ("C5", 32, 500)):
        w = W.config(name)
        assert (w.n_workers, w.arrivals) == (n, arrivals)


def test_static_vectors_have_the_stated_distributions():
    w = W.config("C1")
    a, ts, t0 = w.curvature(), w.theta_star(), w.theta0()
    assert 0.5 <= a.min() and a.max() <= 2.0 and abs(a.mean() - 1.25) < 0.01
    assert abs(ts.std() - 0.1) < 2e-3 and abs(ts.mean()) < 1e-3
    assert abs(t0.std() - 0.05) < 1e-3 and abs(t0.mean()) < 1e-3
    idx = w.sample_indices(500)
    assert np.array_equal(w.theta0(idx), t0[idx])
    assert np.array_equal(w.curvature(idx), a[idx])


def test_gradient_is_the_quadratic_model():
    w = W.config("C1")
    sent = w.theta0()
    g = w.grad(7, sent)
    a, ts = w.curvature().astype(np.float64), w.theta_star().astype(np.float64)
    noise = g.astype(np.float64) - a * (sent.astype(np.float64) - ts)
    assert abs(noise.std() - 0.01) < 2e-4 and abs(noise.mean()) < 1e-4
    # another arrival draws other noise; sampled indices reproduce the dense values
    assert not np.array_equal(w.grad(8, sent), g)
    idx = w.sample_indices(777)
    assert np.array_equal(w.grad(7, sent[idx], idx), g[idx])
    # gradient at the minimiser is noise only
    g_star = w.grad(7, w.theta_star())
    assert abs(g_star.std() - 0.01) < 2e-4


def test_per_segment_noise_scale():
    w = W.config("mini")
    assert w.seg_sigma.min() >= 1e-3 and w.seg_sigma.max() <= 1e-1
    g = w.grad(3, w.theta_star()).astype(np.float64)
    for l in (0, 2):
        lo, hi = w.seg_off[l], w.seg_off[l + 1]
        assert abs(g[lo:hi].std() / w.seg_sigma[l] - 1) < 0.1


def test_sparse_embedding_rows():
    w = W.config("C5")
    rows = np.arange(0, 20000, dtype=np.int64)
    idx = rows * 512 + 5
    g1 = w.grad(1, np.zeros(len(idx), np.float32), idx)
    active = g1 != 0
    assert abs(active.mean() - 0.1) < 0.01
    # a whole row shares its activity
    idx2 = rows * 512 + 300
    g2 = w.grad(1, np.zeros(len(idx), np.float32), idx2)
    assert np.array_equal(g2 != 0, active)
    # other arrival, other rows
    g3 = w.grad(2, np.zeros(len(idx), np.float32), idx)
    assert not np.array_equal(g3 != 0, active)
    # dense region: never exactly sparse, std 0.01; independent of the sent parameters
    tail = np.arange(w.d - 50000, w.d, dtype=np.int64)
    gt = w.grad(1, np.zeros(len(tail), np.float32), tail)
    assert abs(gt.std() - 0.01) < 3e-4 and (gt == 0).mean() < 1e-3
    assert np.array_equal(gt, w.grad(1, np.ones(len(tail), np.float32), tail))


def test_schedules():
    for name in ("C1", "C2", "C4"):
        w = W.config(name)
        s = w.schedule()
        assert len(s) == w.arrivals and set(s) <= set(range(w.n_workers))
        assert len(set(s)) == w.n_workers, "every worker arrives at least once"
        assert s == W.config(name).schedule(), "deterministic"
    # equal speeds with 1..3 tick jitter: nobody laps anybody by much
    s = W.config("C1").schedule()
    counts = np.bincount(s, minlength=8)
    assert counts.max() - counts.min() < 0.2 * counts.mean()
    # stragglers: the 13 slow workers of C4 arrive about 5x less often
    s = W.config("C4").schedule()
    counts = np.sort(np.bincount(s, minlength=128))
    assert 3.5 < counts[13:].mean() / counts[:13].mean() < 7
    # log-normal: constant per-worker speed => strictly periodic arrivals of each worker
    s = np.asarray(W.config("C2").schedule())
    assert np.bincount(s).max() / np.bincount(s).min() > 2
    assert W.schedule_round_robin(3, 7) == [0, 1, 2, 0, 1, 2, 0]


def test_windows_never_repeat_a_worker():
    s = W.config("C2").schedule()[:3000]
    for k_max in (1, 4, 16):
        ws = W.windows(s, k_max)
        assert [i for w in ws for i in w] == s
        assert all(len(w) <= k_max and len(set(w)) == len(w) for w in ws)
    assert W.windows([0, 1, 0, 0, 2], 16) == [[0, 1], [0], [0, 2]]


def test_gamma_execution_time_model_matches_the_papers_figures():
    """Appendix "Gamma Distribution": both settings have mean 128; an iteration takes at least
    1.25x the mean with probability 1% (homogeneous) and 27.9% (heterogeneous)."""
    homo = np.concatenate([W.gamma_task_times(s, 64, 2000).ravel() / W.gamma_task_times(s, 64, 2000).mean()
                           for s in range(20)])
    assert abs((homo >= 1.25).mean() - 0.01) < 0.003
    het = np.concatenate([W.gamma_task_times(s, 512, 200, heterogeneous=True).ravel() for s in range(20)])
    assert abs(het.mean() / 128 - 1) < 0.03
    assert abs((het >= 160).mean() - 0.279) < 0.015
    t = W.gamma_task_times(3, 16, 50000)
    assert abs(t.std() / t.mean() - 0.1) < 0.005            # V_mach = 0.1
    # heterogeneous machines keep their own mean for the whole run; homogeneous ones do not
    th = W.gamma_task_times(4, 32, 4000, heterogeneous=True)
    assert th.mean(axis=1).std() / th.mean() > 0.3 and t.mean(axis=1).std() / t.mean() < 0.01
    s1 = W.schedule_gamma(5, 8, 500)
    assert len(s1) == 500 and set(s1) == set(range(8)) and s1 == W.schedule_gamma(5, 8, 500)
    counts = np.bincount(W.schedule_gamma(5, 16, 4000, heterogeneous=True), minlength=16)
    assert counts.max() / max(1, counts.min()) > 2


# ----------------------------------------------------------------------------- exact pins of the C generator
def _round_f32(q):
    """The fp32 value nearest to the exact rational q (ties to even), via exact comparisons."""
    from fractions import Fraction
    f = np.float32(float(q))
    best = None
    for c in (np.nextafter(f, np.float32(-np.inf)), f, np.nextafter(f, np.float32(np.inf))):
        err = abs(Fraction(float(c)) - q)
        even = (int(np.float32(c).view(np.uint32)) & 1) == 0
        if best is None or err < best[0] or (err == best[0] and even):
            best = (err, np.float32(c))
    return best[1]


def _exact_uniform(w):
    from fractions import Fraction
    return Fraction(2 * (w >> 41) + 1, 1 << 24)


def _xi_f32(w):
    from fractions import Fraction
    fields = sum((w >> (16 * f)) & 0xFFFF for f in range(4)) - 131070
    scale = np.float32(np.sqrt(3.0) / 65536.0)
    return _round_f32(Fraction(fields) * Fraction(float(scale)))


def test_generator_values_against_exact_arithmetic():
    """Initial parameters, targets, curvature and gradients of the C generator at a handful of
    elements, recomputed here from the Python statement of the hash and exact rational
    arithmetic rounded once per operation: pins the C code to the written definition
    independently of the device generator."""
    from fractions import Fraction as F
    wl = W.config("mini")
    idx = np.array([0, 1, 999, 1000, 1036, 1037, 5135, 5136, 5137, 5652], dtype=np.int64)
    t0, ts, a = wl.theta0(idx), wl.theta_star(idx), wl.curvature(idx)
    sent = (t0 * np.float32(1.25)).astype(np.float32)
    for k in (1, 9):
        g = wl.grad(k, sent, idx)
        for q, j in enumerate(int(x) for x in idx):
            xi0 = _xi_f32(W.hash4(wl.seed, W.INIT, 0, j))
            assert t0[q] == _round_f32(F(float(np.float32(0.05))) * F(float(xi0)))
            xit = _xi_f32(W.hash4(wl.seed, W.TARGET, 0, j))
            target = _round_f32(F(float(np.float32(0.1))) * F(float(xit)))
            assert ts[q] == target
            u = _exact_uniform(W.hash4(wl.seed, W.CURV, 0, j))
            assert float(u) == float(np.float32(float(u)))          # the uniform is exact in fp32
            curv = _round_f32(F(3, 2) * u + F(1, 2))
            assert a[q] == curv
            seg = int(np.searchsorted(wl.seg_off, j, side="right") - 1)
            noise = _round_f32(F(float(wl.seg_sigma[seg])) * F(float(_xi_f32(W.hash4(wl.seed, W.NOISE, k, j)))))
            diff = _round_f32(F(float(sent[q])) - F(float(target)))
            want = _round_f32(F(float(curv)) * F(float(diff)) + F(float(noise)))       # one fused operation
            assert g[q] == want, (k, j)


def test_sparse_rows_follow_the_row_hash():
    wl = W.Workload(name="emb", segments=[64 * 50, 500], n_workers=2, arrivals=4, schedule_kind="ticks",
                    seed=11, quad=False, emb_rows=50, emb_row=64, row_active_frac=0.3)
    g = wl.grad(3, np.zeros(wl.d, np.float32))
    thresh = (1 << 64) * 300 // 1000
    for r in range(50):
        active = W.hash4(wl.seed, W.ROW, 3, r) < thresh
        row = g[64 * r:64 * (r + 1)]
        if active:
            for c in (0, 63):
                j = 64 * r + c
                assert row[c] == np.float32(wl.seg_sigma[0]) * _xi_f32(W.hash4(wl.seed, W.NOISE, 3, j))
        else:
            assert not row.any()
    assert (g[64 * 50:] != 0).mean() > 0.99
