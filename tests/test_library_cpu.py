"""Host-side checks that need no GPU: the C ABI exports what the header declares, argument
errors come back as codes, checkpoint blobs round-trip, shards tile the vector."""
import os
import re

import numpy as np
import pytest

import paper_1909_10802_b200 as P
from paper_1909_10802_b200 import build as ga_build
from paper_1909_10802_b200.shard import shard_range

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    ga_build.build()
    return P.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "ga.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ga_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert len(names) >= 18 and "ga_push_batch" in names
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in ga.h but not exported"
    assert set(names) == set(P._SIGNATURES), "binding and header list different calls"


def test_errors_without_touching_the_gpu(lib):
    assert lib.ga_push(None, 0, None) == P.GA_ERR_ARG
    assert "NULL" in P.last_error()
    assert lib.ga_set_stream(None, None) == P.GA_ERR_ARG
    assert not lib.ga_pull(None, 0)
    assert lib.ga_export_state(None, None, 0) == 0
    lib.ga_destroy(None)
    assert not lib.ga_create(0, 1, 0.1, 0.9, 0.999, P.GA_GA)
    assert "n_params" in P.last_error()


def test_no_cpu_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(RuntimeError, match="CUDA"):
        P.Engine(10, 2)


def test_state_blob_round_trip():
    rng = np.random.default_rng(0)
    d, n = 37, 3
    st = dict(d=d, n_workers=n, k_done=12, k_c=12, lr=np.float32(0.1), momentum=np.float32(0.9),
              c_beta=np.float32(0.999), eps=np.float32(1e-8), variant=2, c_order=0, fast_math=0, stats=0,
              window=16, iter=np.array([3, 12, 7]), theta=rng.normal(size=d), v=rng.normal(size=d),
              m=rng.random(size=d), saved=rng.normal(size=(n, d)))
    blob = P.pack_state(st)
    back = P.unpack_state(blob)
    assert back["k_done"] == 12 and list(back["iter"]) == [3, 12, 7]
    assert np.array_equal(back["saved"], st["saved"].astype(np.float32))
    assert P.pack_state(back) == blob


@pytest.mark.parametrize("d,world", [(272474, 2), (150_000_000, 8), (5, 4), (33, 2), (1, 3)])
def test_shards_tile_the_vector(d, world):
    pos = 0
    for r in range(world):
        j0, n = shard_range(d, r, world)
        assert j0 == pos and n >= 0 and (j0 % 32 == 0 or n == 0)
        pos += n
    assert pos == d


@pytest.mark.parametrize("config,world", [("C1", 2), ("C1", 3), ("C3", 8), ("C3", 5), ("C4", 4), ("C5", 2), ("mini", 2)])
def test_layer_shards_hold_whole_layers_and_tile_the_vector(config, world):
    """Ranks of the layer-wise Gap own whole layers: consecutive, non-empty, covering every layer once;
    where no layer dominates (the ResNet shapes) no rank is more than one layer away from an equal share."""
    import workloads as W
    from paper_1909_10802_b200.shard import layer_shard_range
    off = [int(x) for x in W.config(config).seg_off]
    d, biggest = off[-1], max(b - a for a, b in zip(off, off[1:]))
    pos_l, pos_j = 0, 0
    for r in range(world):
        l0, l1, j0, n = layer_shard_range(off, r, world)
        assert l0 == pos_l and l1 > l0 and j0 == pos_j == off[l0] and n == off[l1] - off[l0]
        if config in ("C1", "C3", "C4"):
            assert abs(n - d / world) <= biggest
        pos_l, pos_j = l1, j0 + n
    assert pos_l == len(off) - 1 and pos_j == d


def test_layer_shards_refuse_what_cannot_be_split():
    from paper_1909_10802_b200.shard import layer_shard_range
    with pytest.raises(ValueError):
        layer_shard_range([0, 10, 20], 0, 3)          # more ranks than layers
    with pytest.raises(ValueError):
        layer_shard_range([0, 10, 10], 0, 1)          # an empty layer
    with pytest.raises(ValueError):
        layer_shard_range([0, 10, 20], 2, 2)
    assert layer_shard_range([0, 10, 20], 1, 2) == (1, 2, 10, 10)
    assert layer_shard_range([0, 1, 2, 1000], 0, 2) == (0, 2, 0, 2)      # a dominant layer stays whole
