"""The N > 1 path on CPU: two gloo ranks each own a parameter range; because every step is
independent per parameter their shards, put together, are the single-rank result exactly."""
import os
import socket

import numpy as np
import torch.multiprocessing as mp

import workloads as W


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank(rank, world, port, out_dir):
    import torch
    import torch.distributed as dist
    from paper_1909_10802_b200.shard import assert_same_schedule, combine_gap_stats, shard_range
    from tests.oracle_run import run_oracle
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = W.config("mini")
    assert_same_schedule(wl.schedule(), dist)
    j0, n = shard_range(wl.d, rank, world)
    idx = np.arange(j0, j0 + n, dtype=np.int64)
    o, delays, _ = run_oracle(wl, "GA", idx=idx)
    # delays are replicated host state: identical on every rank
    all_delays = [None] * world
    dist.all_gather_object(all_delays, delays)
    assert all(x == delays for x in all_delays)
    total, biggest = combine_gap_stats(*o.stats(), dist)      # statistics of the last arrival
    np.save(os.path.join(out_dir, f"stats_{rank}.npy"), np.array([total, biggest]))
    np.save(os.path.join(out_dir, f"theta_{rank}.npy"), o.get(o.THETA))
    np.save(os.path.join(out_dir, f"m_{rank}.npy"), o.get(o.M))
    # a rank with a different schedule is detected
    bad = list(wl.schedule())
    if rank == 1:
        bad[3] = (bad[3] + 1) % wl.n_workers
    try:
        assert_same_schedule(bad, dist)
        raised = False
    except RuntimeError:
        raised = True
    assert raised
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_equal_one(tmp_path):
    from tests.oracle_run import run_oracle
    world = 2
    mp.spawn(_rank, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    wl = W.config("mini")
    full, _, _ = run_oracle(wl, "GA")
    theta = np.concatenate([np.load(tmp_path / f"theta_{r}.npy") for r in range(world)])
    m = np.concatenate([np.load(tmp_path / f"m_{r}.npy") for r in range(world)])
    assert np.array_equal(theta, full.get(full.THETA)) and np.array_equal(m, full.get(full.M))
    want_sum, want_max = full.stats()
    for r in range(world):
        got_sum, got_max = np.load(tmp_path / f"stats_{r}.npy")
        assert abs(got_sum - want_sum) <= 1e-12 * want_sum and got_max == want_max


def _layer_rank(rank, world, port, out_dir):
    import torch.distributed as dist
    from paper_1909_10802_b200.shard import assert_same_schedule, layer_shard_range
    from tests.oracle_run import run_oracle
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = W.config("mini")
    assert_same_schedule(wl.schedule(), dist)
    l0, l1, j0, n = layer_shard_range(wl.seg_off, rank, world)
    o, delays, _ = run_oracle(wl, "GA_LAYER", idx=np.arange(j0, j0 + n, dtype=np.int64))
    gaps, m_layers = o.layer_state()
    np.save(os.path.join(out_dir, f"ltheta_{rank}.npy"), o.get(o.THETA))
    np.save(os.path.join(out_dir, f"lgap_{rank}.npy"), np.asarray(gaps))
    np.save(os.path.join(out_dir, f"lm_{rank}.npy"), np.asarray(m_layers))
    dist.barrier()
    dist.destroy_process_group()


def test_layer_wise_gap_on_ranks_that_hold_whole_layers(tmp_path):
    """Section 5.3's layer-wise Gap on two ranks: each holds whole layers, nothing is exchanged, and
    parameters, per-layer Gaps and per-layer second moments together are the single-rank run's."""
    from tests.oracle_run import run_oracle
    world = 2
    mp.spawn(_layer_rank, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    wl = W.config("mini")
    full, _, _ = run_oracle(wl, "GA_LAYER")
    gaps, m_layers = full.layer_state()
    cat = lambda name: np.concatenate([np.load(tmp_path / f"{name}_{r}.npy") for r in range(world)])
    assert np.array_equal(cat("ltheta"), full.get(full.THETA))
    assert np.array_equal(cat("lgap"), np.asarray(gaps)) and np.array_equal(cat("lm"), np.asarray(m_layers))
