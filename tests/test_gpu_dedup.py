"""The three ways of finding first occurrences for dedup + relabel (direct-address table, batch-sized
hash table, radix sort + unique) must give the same blocks: each alternative is compared with the CPU
oracle element by element, on the named workloads, on random configurations, with grids capped at one
and two blocks (every block then walks many tiles of the sort and of the hash insert), and on the
device-detected errors (needs a B200)."""
import numpy as np
import pytest
import torch

from workloads import batch_seeds, get_config

pytestmark = pytest.mark.gpu

METHODS = {"direct": 0, "hash": 1, "sort": 2}


def _pair(name, method):
    from parity import Pair
    pair = Pair(get_config(name))
    pair.dedup = METHODS[method]
    return pair


@pytest.mark.parametrize("method", ["hash", "sort"])
def test_tiny_every_mode(method):
    pair = _pair("tiny", method)
    pair.run("otf", 0.25, 6)
    pair.run("fcr", 0.0, 2)
    pair.run("fbl", 0.0, 2)
    pair.run("fetch", 0.5, 2)
    pair.run("otf", 0.25, 2, host_api=True)
    pair.run("otf", 0.25, 2, theta=16)


@pytest.mark.parametrize("method", ["hash", "sort"])
def test_mid_and_shared(method):
    pair = _pair("mid", method)
    pair.run("otf", 0.3, 2, rows=2000)
    pair.run("fcr", 0.0, 1, rows=2000)
    pair = _pair("shared", method)
    pair.run("otf", 0.3, 2, rows=2000)


@pytest.mark.parametrize("method", ["hash", "sort"])
@pytest.mark.parametrize("cap", [1, 2])
def test_mid_with_capped_grids(method, cap):
    import paper_2406_17918_b200 as gs
    pair = _pair("mid", method)
    gs.gs_debug_set_grid_cap(cap)
    try:
        pair.run("otf", 0.1, 1, rows=500, features=False)
    finally:
        gs.gs_debug_set_grid_cap(0)


@pytest.mark.parametrize("method", ["hash", "sort"])
@pytest.mark.parametrize("case", range(12))
def test_random_configurations(method, case):
    from parity import Pair
    from test_gpu_parity import _random_graph

    rng = np.random.default_rng(7000 + case)
    indptr, indices = _random_graph(rng)
    n = len(indptr) - 1
    L = int(rng.integers(1, 5))
    W = int(rng.choice([1, 2, 8, 20, 32]))
    fanouts = [int(rng.integers(1, W + 1)) for _ in range(L)]
    shared = bool(rng.random() < 0.3)
    theta = None if rng.random() < 0.6 else int(rng.integers(W, 129))
    pair = Pair.from_csr(indptr, indices, fanouts, W, shared=shared, seed=int(rng.integers(1, 2**63)))
    pair.dedup = METHODS[method]
    B = int(rng.integers(1, min(n, 300) + 1))
    C, ws, O = pair.samplers(B, theta=theta)
    for b in range(4):
        mode = str(rng.choice(["otf", "otf", "fcr", "fetch", "fbl"]))
        rate = float(rng.choice([0.0, 0.1, 0.25, 0.5, 1.0]))
        seeds = torch.from_numpy(rng.choice(n, size=int(rng.integers(1, B + 1)), replace=False).astype(np.int32))
        pair.check_batch(C, ws, O, seeds, mode, rate, 20 + b, features=False)
    pair.check_rows(C, O, np.arange(n))


@pytest.mark.parametrize("method", ["hash", "sort"])
def test_device_detected_errors(method):
    import paper_2406_17918_b200 as gs
    pair = _pair("tiny", method)
    B = 16
    C, ws, O = pair.samplers(B)
    good = batch_seeds(pair.perm, 0, B)
    bad = good.clone()
    bad[5] = pair.cfg["num_nodes"] + 3
    gs.gs_sample_batch(C, bad.cuda(), gs.GS_MODE_OTF, 0.25, 1, ws)
    with pytest.raises(gs.GsError) as e:
        gs.gs_batch_counts(C)
    assert e.value.status == 3
    dup = good.clone()
    dup[7] = dup[2]
    gs.gs_sample_batch(C, dup.cuda(), gs.GS_MODE_OTF, 0.25, 1, ws)
    with pytest.raises(gs.GsError) as e:
        gs.gs_batch_counts(C)
    assert e.value.status == 5
    # the rejected batches refreshed nothing (duplicates are caught at the seeds, before the first refresh)
    pair.check_batch(C, ws, O, good, "otf", 0.25, 1)


def test_switching_methods_between_batches():
    """The direct table keeps stamps of earlier batches; batches run with another method in between must not disturb it."""
    import paper_2406_17918_b200 as gs
    from parity import Pair
    pair = Pair(get_config("tiny"))
    C, ws, O = pair.samplers(pair.cfg["batch"])
    for b, method in enumerate([0, 1, 0, 2, 2, 0, 1, 3, 0]):
        gs.gs_cache_set_dedup(C, method)
        pair.check_batch(C, ws, O, batch_seeds(pair.perm, b, pair.cfg["batch"]), "otf", 0.25, b + 1)
    with pytest.raises(gs.GsError):
        gs.gs_cache_set_dedup(C, 7)
