"""The allocation-free Gap statistics call against the ordinary one.

ga_gap_stats_noalloc serves callers that cannot use the device allocator -- monitoring code in a
process where a framework pool already owns the GPU's memory, or hooks that must avoid the
device-wide synchronisation an allocation implies -- so its reduction scratch is a fixed array
inside the library. This test drives it through the C ABI on state produced by a real run and
compares it with the existing entry point ga_gap (whose per-parameter output is reduced here) and,
directly, with the CPU oracle's Gap of the same run summed in fp64 -- twice in a row: the second
call uses another worker and a shorter vector, so anything left in the shared scratch array by
the first call would show. Collected last on purpose.
"""
import pytest

pytestmark = pytest.mark.gpu


def _reference(P, eng, worker, n):
    import torch
    G = eng.gap(worker)[:n]
    return float(G.double().sum()), float(G.max())


def _oracle_reference(o, worker, n):
    G = o.gap(worker)[:n]              # fp32 values held in float64
    return float(G.sum()), float(G.max())


def test_no_alloc_gap_stats_matches_ga_gap_twice():
    import torch
    import workloads as W
    import paper_1909_10802_b200 as P
    from paper_1909_10802_b200.runner import Run

    wl = W.Workload(name="noalloc", segments=[700_001, 37, 300_000], n_workers=4, arrivals=24,
                    schedule_kind="ticks", seed=424242)
    run = Run(wl, "GA", 16)
    run.run()
    eng = run.engine
    from tests.oracle_run import run_oracle
    o, odelays, _ = run_oracle(wl, "GA")
    assert run.delays == odelays
    theta, m = eng.get(P.GA_THETA), eng.get(P.GA_M)
    out = torch.full((2,), -1.0, dtype=torch.float64, device="cuda")
    k_c = eng.num_arrivals                      # one refresh of m per GA arrival

    # first call: the whole vector (245 blocks and a ragged tail), worker 0
    P.gap_stats_noalloc(theta, eng.saved(0), m, wl.lr, wl.c_beta, k_c, out)
    s_ref, m_ref = _reference(P, eng, 0, wl.d)
    s, mx = out.tolist()
    assert abs(s - s_ref) <= 1e-9 * s_ref and mx == m_ref and mx > 1.0
    so, mo = _oracle_reference(o, 0, wl.d)
    assert abs(s - so) <= 1e-9 * so and mx == mo

    # second call, right after: another worker and only the first 123,457 parameters
    n2 = 123_457
    out.fill_(-1.0)
    P.gap_stats_noalloc(theta[:n2], eng.saved(2)[:n2], m[:n2], wl.lr, wl.c_beta, k_c, out)
    s_ref2, m_ref2 = _reference(P, eng, 2, n2)
    s2, mx2 = out.tolist()
    assert abs(s2 - s_ref2) <= 1e-9 * s_ref2 and mx2 == m_ref2
    so2, mo2 = _oracle_reference(o, 2, n2)
    assert abs(s2 - so2) <= 1e-9 * so2 and mx2 == mo2
    assert (s2, mx2) != (s, mx)

    # sizes beyond the fixed scratch are refused, with a message that says why; nothing runs
    l = P.lib()
    rc = l.ga_gap_stats_noalloc(theta.data_ptr(), theta.data_ptr(), m.data_ptr(), P.GA_NOALLOC_MAX_PARAMS + 1,
                                wl.lr, wl.c_beta, k_c, out.data_ptr(), None)
    assert rc == P.GA_ERR_ARG and "GA_NOALLOC_MAX_PARAMS" in P.last_error()
    assert l.ga_gap_stats_noalloc(None, theta.data_ptr(), m.data_ptr(), 10, wl.lr, wl.c_beta, k_c,
                                  out.data_ptr(), None) == P.GA_ERR_ARG
    torch.cuda.synchronize()
    assert out.tolist() == [s2, mx2]
    run.close()
