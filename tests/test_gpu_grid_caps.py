"""Every kernel walks its work with a grid-stride or work-counter loop, so that the host can size
grids from upper bounds only.  With the designed grids most of those loops run once per block: a
block of the first-occurrence scan only takes a second tile above 9.7 M picks per hop.  Here the
grids are capped at 1, 2 and 3 blocks (the library's test knob), so every block walks many tiles
and the last-block hand-over happens after a long walk, and everything is compared with the CPU
oracle element by element (needs a B200)."""
import numpy as np
import pytest
import torch

from workloads import batch_seeds, get_config

pytestmark = pytest.mark.gpu


@pytest.fixture
def grid_cap():
    import paper_2406_17918_b200 as gs

    def set_cap(n):
        gs.gs_debug_set_grid_cap(n)

    yield set_cap
    gs.gs_debug_set_grid_cap(0)


@pytest.fixture(scope="module")
def mid():
    from parity import Pair
    return Pair(get_config("mid"))


@pytest.mark.parametrize("cap", [1, 2, 3])
def test_mid_batches_with_capped_grids(mid, grid_cap, cap):
    """Mid: up to 67 K frontier nodes (66 tiles of the row-count scan) and 1 M picks (247 tiles of the
    first-occurrence scan) per hop, walked by `cap` blocks; pre-sample included."""
    grid_cap(cap)
    C, ws, O = mid.samplers(mid.cfg["batch"])
    rng = np.random.default_rng(cap)
    mid.check_rows(C, O, rng.integers(0, mid.cfg["num_nodes"], 3000).astype(np.int32))
    for b, (mode, gamma) in enumerate([("otf", 0.3), ("fcr", 0.0), ("otf", 0.1)]):
        seeds = batch_seeds(mid.perm, b, mid.cfg["batch"])
        mid.check_batch(C, ws, O, seeds, mode, gamma, b + 1, rows=2000)


def test_capped_and_designed_grids_give_the_same_bits(mid, grid_cap):
    """The same batch with a cap of 2 blocks and with the designed grids, output arrays compared directly."""
    import paper_2406_17918_b200 as gs

    outs = []
    for cap in (2, 0):
        grid_cap(cap)
        C, ws, _ = mid.samplers(mid.cfg["batch"])
        seeds = batch_seeds(mid.perm, 0, mid.cfg["batch"]).cuda()
        blocks, input_nodes, cnt = gs.gs_sample_batch(C, seeds, gs.GS_MODE_OTF, 0.3, 1, ws)
        n, m = gs.gs_batch_counts(C)
        L = mid.L
        feats = torch.empty((n[L], mid.X.shape[1]), dtype=mid.X.dtype, device="cuda")
        gs.gs_gather_features(mid.G, input_nodes, cnt, feats)
        outs.append((n, m, input_nodes[: n[L]].clone(), [blocks[l].indptr(n[L - 1 - l]).clone() for l in range(L)],
                     [blocks[l].indices(m[l]).clone() for l in range(L)], feats))
    a, b = outs
    assert a[0] == b[0] and a[1] == b[1]
    assert torch.equal(a[2], b[2])
    for x, y in zip(a[3] + a[4], b[3] + b[4]):
        assert torch.equal(x, y)
    assert torch.equal(a[5].view(torch.int32), b[5].view(torch.int32))


@pytest.mark.parametrize("case", range(12))
def test_random_configurations_with_capped_grids(grid_cap, case):
    """Seeded random graphs, shapes, modes, rates and splits under caps of 1-3 blocks."""
    from parity import Pair
    from test_gpu_parity import _random_graph

    rng = np.random.default_rng(5000 + case)
    grid_cap(1 + case % 3)
    indptr, indices = _random_graph(rng)
    n = len(indptr) - 1
    L = int(rng.integers(1, 4))
    W = int(rng.choice([2, 8, 20, 32]))
    fanouts = [int(rng.integers(1, W + 1)) for _ in range(L)]
    shared = bool(rng.random() < 0.3)
    theta = None if rng.random() < 0.6 else int(rng.integers(W, 129))
    pair = Pair.from_csr(indptr, indices, fanouts, W, shared=shared, seed=int(rng.integers(1, 2**63)))
    B = int(rng.integers(1, min(n, 300) + 1))
    C, ws, O = pair.samplers(B, theta=theta)
    pair.check_rows(C, O, np.arange(n))
    for b in range(3):
        mode = str(rng.choice(["otf", "otf", "fcr", "fetch", "fbl"]))
        rate = float(rng.choice([0.0, 0.1, 0.25, 0.5, 1.0]))
        seeds = torch.from_numpy(rng.choice(n, size=int(rng.integers(1, B + 1)), replace=False).astype(np.int32))
        pair.check_batch(C, ws, O, seeds, mode, rate, 10 + b, features=False)
    pair.check_rows(C, O, np.arange(n))
