"""Pins of the oracle's whole-cache periodic refresh (the periodic branch of Algorithms 2 and 3, taken every T-th batch)."""
import numpy as np
import pytest

import oracle
from helpers import csr_from_rows, golden_json, star_graph
from workloads import batch_seeds, build_graph, get_config, seed_permutation

PURPOSE = {oracle.FILL: "fill", oracle.EVICT: "evict", oracle.PICK: "pick"}


def test_worked_periodic_example():
    ex = golden_json("worked_periodic_example.json")
    indptr, indices = csr_from_rows(ex["rows"])
    s = oracle.Sampler(indptr, indices, ex["fanouts"], ex["cache_width"], seed=1)
    s.set_key_fn(lambda purpose, tag, v, step, i: ex["keys"]["%s/%d/%d/%d" % (PURPOSE[purpose], tag, v, step)][i])

    def check(want):
        for layer in (0, 1):
            for v in (0, 1):
                assert list(s.cache_row(layer, v)) == want[str(layer)][v], (layer, v)
            for v in (2, 3, 4, 5):
                assert list(s.cache_row(layer, v)) == ex["low_rows"]

    check(ex["presample"])
    s.refresh_all(oracle.MODE_OTF, ex["after_otf_refresh_step_2"]["gamma"], 2)
    check(ex["after_otf_refresh_step_2"])
    b = ex["batch_step_3"]
    fr, n, blocks = s.sample_batch(np.array(b["seeds"], dtype=np.int32), oracle.MODE_OTF, 0.0, 3)
    assert list(fr) == b["frontier"]
    assert list(blocks[1].picked) == b["picked_layer_1"] and list(blocks[0].picked) == b["picked_layer_0"]
    check(ex["after_otf_refresh_step_2"])          # sampling between two refreshes leaves the cache alone
    s.refresh_all(oracle.MODE_FCR, 0.0, 4)
    check(ex["after_fcr_refresh_step_4"])


def test_full_refresh_of_every_row_is_a_presample_with_that_steps_keys():
    """FCR replaces the whole row, so the result cannot depend on the row before: it is the W edge
    offsets first in FILL order at that step, recomputed here from raw Philox calls."""
    d, W, seed, step = 37, 6, 0xFEEDFACE12345678, 9
    indptr, indices = star_graph(d)
    s = oracle.Sampler(indptr, indices, [3, 2], W, seed)
    s.refresh_all(oracle.MODE_OTF, 0.5, 4)           # some other state first
    s.refresh_all(oracle.MODE_FCR, 0.0, step)
    for layer in (0, 1):
        keys = []
        for i in range(d):
            out = oracle.philox4x32_10([i >> 2, 0, step, (oracle.FILL << 8) | layer], [seed & 0xFFFFFFFF, seed >> 32])
            keys.append((out[i & 3], i))
        assert list(s.cache_row(layer, 0)) == [indices[i] for _, i in sorted(keys)[:W]]


@pytest.mark.parametrize("shared", [False, True])
def test_periodic_schedule_invariants(shared):
    cfg = get_config("tiny")
    g = build_graph(cfg)
    indptr, indices = g.indptr.numpy(), g.indices.numpy()
    deg = indptr[1:] - indptr[:-1]
    perm = seed_permutation(cfg)
    N, W, L = cfg["num_nodes"], cfg["cache_width"], len(cfg["fanouts"])
    caches = 1 if shared else L
    adj = [set(indices[indptr[v]:indptr[v + 1]].tolist()) for v in range(N)]
    s = oracle.Sampler(indptr, indices, cfg["fanouts"], W, 11, shared)
    ref = oracle.Sampler(indptr, indices, cfg["fanouts"], W, 11, shared)    # driven row by row
    T, gamma = 3, 0.3
    r = oracle.refresh_count(oracle.MODE_OTF, gamma, W)
    nodes = np.arange(N)
    before = [s.cache_rows(l, nodes) for l in range(caches)]
    for t in range(1, 8):
        if t % T == 0:
            s.refresh_all(oracle.MODE_OTF, gamma, t)
            refreshed, scanned = s.stats()
            after = [s.cache_rows(l, nodes) for l in range(caches)]
            for l in range(caches):
                changed = (after[l] != before[l]).sum(axis=1)
                assert (changed <= r).all() and changed.max() > 0
                assert (changed[deg <= W] == 0).all()
                for v in range(N):
                    row = after[l][v][after[l][v] >= 0]
                    assert len(set(row.tolist())) == len(row) == min(W, deg[v]) and set(row.tolist()) <= adj[v]
                    ref.refresh_node(l, v, t, r)
                assert np.array_equal(ref.cache_rows(l, nodes), after[l])
            before = after
        seeds = batch_seeds(perm, t, cfg["batch"]).numpy()
        s.sample_batch(seeds, oracle.MODE_OTF, 0.0, t)
        for l in range(caches):
            assert np.array_equal(s.cache_rows(l, nodes), before[l])          # frozen between refreshes


def test_refresh_all_respects_the_dense_sparse_split_and_rejects_bad_arguments():
    cfg = get_config("tiny")
    g = build_graph(cfg)
    indptr, indices = g.indptr.numpy(), g.indices.numpy()
    deg = indptr[1:] - indptr[:-1]
    W = cfg["cache_width"]
    s = oracle.Sampler(indptr, indices, cfg["fanouts"], W, 11)
    s.set_theta(2 * W)
    nodes = np.arange(cfg["num_nodes"])
    before = s.cache_rows(0, nodes)
    s.refresh_all(oracle.MODE_FCR, 0.0, 5)
    after = s.cache_rows(0, nodes)
    changed = (after != before).any(axis=1)
    assert not changed[deg <= 2 * W].any() and changed[deg > 2 * W].any()
    for bad in [(oracle.MODE_FBL, 0.0, 1), (oracle.MODE_OTF_FETCH, 0.5, 1), (oracle.MODE_OTF, 1.5, 1), (oracle.MODE_FCR, 0.0, 0)]:
        with pytest.raises(ValueError):
            s.refresh_all(*bad)
