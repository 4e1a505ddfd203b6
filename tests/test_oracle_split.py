"""Pins of the oracle's dense/sparse split by degree threshold theta."""
import numpy as np

import oracle
from workloads import batch_seeds, build_graph, get_config, seed_permutation


def _setup():
    cfg = get_config("tiny")
    g = build_graph(cfg)
    return cfg, g.indptr.numpy(), g.indices.numpy(), seed_permutation(cfg)


def test_theta_above_every_degree_is_full_batch_load():
    cfg, indptr, indices, perm = _setup()
    W = cfg["cache_width"]
    a = oracle.Sampler(indptr, indices, cfg["fanouts"], W, seed=6)
    b = oracle.Sampler(indptr, indices, cfg["fanouts"], W, seed=6)
    a.set_theta(int((indptr[1:] - indptr[:-1]).max()))
    for t in range(3):
        seeds = batch_seeds(perm, t, cfg["batch"]).numpy()
        fa, na, ba = a.sample_batch(seeds, oracle.MODE_OTF, 0.25, t + 1)
        fb, nb, bb = b.sample_batch(seeds, oracle.MODE_FBL, 0.0, t + 1)
        assert np.array_equal(fa, fb) and na == nb
        assert all(np.array_equal(x.indices, y.indices) for x, y in zip(ba, bb))


def test_split_invariants_and_dense_rows_follow_the_unsplit_rule():
    cfg, indptr, indices, perm = _setup()
    deg = indptr[1:] - indptr[:-1]
    L, W, N = len(cfg["fanouts"]), cfg["cache_width"], cfg["num_nodes"]
    theta = 2 * W
    adj = [set(indices[indptr[v]:indptr[v + 1]].tolist()) for v in range(N)]
    s = oracle.Sampler(indptr, indices, cfg["fanouts"], W, seed=6)
    s.set_theta(theta)
    ref = oracle.Sampler(indptr, indices, cfg["fanouts"], W, seed=6)      # unsplit, driven node by node
    r = oracle.refresh_count(oracle.MODE_OTF, 0.25, W)
    frozen = [s.cache_rows(l, np.nonzero(deg <= theta)[0]) for l in range(L)]
    for t in range(3):
        seeds = batch_seeds(perm, t, cfg["batch"]).numpy()
        fr, n, blocks = s.sample_batch(seeds, oracle.MODE_OTF, 0.25, t + 1)
        for layer in range(L):
            k = L - 1 - layer
            b = blocks[layer]
            dst = fr[: n[k]]
            assert np.array_equal(np.diff(b.indptr), np.minimum(cfg["fanouts"][layer], deg[dst]))
            for p in range(n[k]):
                v = dst[p]
                row = b.picked[b.indptr[p]:b.indptr[p + 1]]
                assert len(set(row.tolist())) == len(row) and set(row.tolist()) <= adj[v]
                if deg[v] <= theta:       # sparse: the FBL rule, ascending offsets
                    assert list(row) == list(ref.fbl_node(layer, v, t + 1))
                else:                     # dense: refresh + pick exactly as without a split
                    ref.refresh_node(layer, v, t + 1, r)
                    assert list(row) == list(ref.pick_node(layer, v, t + 1))
                    assert np.array_equal(s.cache_row(layer, v), ref.cache_row(layer, v))
    # sparse rows were never refreshed
    for l in range(L):
        assert np.array_equal(s.cache_rows(l, np.nonzero(deg <= theta)[0]), frozen[l])
    refreshed, _ = s.stats()
    assert refreshed > 0
