"""Pins of the oracle's OTF Fetch mode: hand-worked example, special cases that reduce to the
other modes, exact enumeration, invariants."""
import itertools
import math
from collections import Counter

import numpy as np
import pytest

import oracle
from helpers import csr_from_rows, golden_json, star_graph
from workloads import batch_seeds, build_graph, get_config, seed_permutation


def test_worked_fetch_example():
    ex = golden_json("worked_fetch_example.json")
    rows = [[] for _ in range(ex["num_nodes"])]
    rows[ex["node"]] = ex["neighbours"]
    indptr, indices = csr_from_rows(rows)
    s = oracle.Sampler(indptr, indices, [ex["fanout"]], ex["cache_width"], seed=1)
    table = {(oracle.FILL, 0): ex["fill_keys_step0"]}
    for c in ex["cases"]:
        table[(oracle.PICK, c["step"])] = c["pick_keys"]
        table[(oracle.FETCH, c["step"])] = c["fetch_keys"]
    s.set_key_fn(lambda purpose, tag, v, step, i: table[(purpose, step)][i])
    assert list(s.cache_row(0, 0)) == ex["row"]
    for c in ex["cases"]:
        assert list(s.fetch_node(0, 0, c["step"], c["n_fetch"])) == c["picks"], c
        assert list(s.cache_row(0, 0)) == ex["row"]                 # the cache is never modified


@pytest.mark.parametrize("delta,f,n", [(0.0, 10, 0), (0.3, 10, 3), (0.25, 10, 3), (0.5, 5, 3), (1.0, 7, 7), (0.04, 10, 0)])
def test_fetch_count(delta, f, n):
    assert oracle.fetch_count(delta, f) == n


def test_fetch_enumeration_uniform_given_cache_part():
    """With the cache part fixed, every n_fetch-subset of the remaining neighbours is equally likely,
    in every order."""
    d, W, f, n_fetch = 6, 3, 3, 2
    indptr, indices = star_graph(d)
    s = oracle.Sampler(indptr, indices, [f], W, seed=0)
    keys = {oracle.FILL: list(range(d)), oracle.PICK: [2, 0, 1], oracle.FETCH: None}
    s.set_key_fn(lambda purpose, tag, v, step, i: keys[purpose][i])
    assert list(s.cache_row(0, 0)) == [1, 2, 3]
    counts = Counter()
    for perm in itertools.permutations(range(d)):
        keys[oracle.FETCH] = perm
        picks = list(s.fetch_node(0, 0, 1, n_fetch))
        assert picks[0] == 2                                        # slot 1 has the smallest PICK key
        rest = [i for i in sorted(range(d), key=lambda i: perm[i]) if i + 1 != 2][:n_fetch]
        assert picks[1:] == [i + 1 for i in rest]
        counts[tuple(picks[1:])] += 1
    assert len(counts) == math.perm(d - 1, n_fetch) and len(set(counts.values())) == 1


def test_fetch_special_cases_on_a_batch():
    cfg = get_config("tiny")
    g = build_graph(cfg)
    indptr, indices = g.indptr.numpy(), g.indices.numpy()
    deg = indptr[1:] - indptr[:-1]
    adj = [set(indices[indptr[v]:indptr[v + 1]].tolist()) for v in range(cfg["num_nodes"])]
    perm = seed_permutation(cfg)
    L, W, N = len(cfg["fanouts"]), cfg["cache_width"], cfg["num_nodes"]
    seeds = batch_seeds(perm, 0, cfg["batch"]).numpy()
    a = oracle.Sampler(indptr, indices, cfg["fanouts"], W, seed=4)
    b = oracle.Sampler(indptr, indices, cfg["fanouts"], W, seed=4)
    # delta = 0 is sampling from the untouched cache (= OTF with gamma 0)
    fa, na, ba = a.sample_batch(seeds, oracle.MODE_OTF_FETCH, 0.0, 1)
    fb, nb, bb = b.sample_batch(seeds, oracle.MODE_OTF, 0.0, 1)
    assert np.array_equal(fa, fb) and all(np.array_equal(x.indices, y.indices) for x, y in zip(ba, bb))
    # delta = 1: for rows larger than the cache the same neighbours as Full Batch Load (same FETCH keys)
    hubs = np.nonzero(deg > W)[0][:40]
    for v in hubs:
        for l in range(L):
            f = cfg["fanouts"][l]
            assert set(a.fetch_node(l, v, 3, f).tolist()) == set(a.fbl_node(l, v, 3).tolist())
    # invariants at an intermediate rate, cache frozen
    frozen = [a.cache_rows(l, range(N)) for l in range(L)]
    fr, n, blocks = a.sample_batch(seeds, oracle.MODE_OTF_FETCH, 0.4, 2)
    for layer in range(L):
        k = L - 1 - layer
        bl = blocks[layer]
        dst = fr[: n[k]]
        assert np.array_equal(np.diff(bl.indptr), np.minimum(cfg["fanouts"][layer], deg[dst]))
        for p in range(n[k]):
            row = bl.picked[bl.indptr[p]:bl.indptr[p + 1]]
            assert len(set(row.tolist())) == len(row) and set(row.tolist()) <= adj[dst[p]]
            if deg[dst[p]] > W:
                n_cache = cfg["fanouts"][layer] - oracle.fetch_count(0.4, cfg["fanouts"][layer])
                assert set(row[:n_cache].tolist()) <= set(frozen[layer][dst[p]].tolist())
    for l in range(L):
        assert np.array_equal(a.cache_rows(l, range(N)), frozen[l])


def test_fetch_of_every_sample_with_fanout_equal_to_width_leaves_the_cache_alone():
    """f = W and delta = 1: as many neighbours are fetched as a row has slots; the row is still not written."""
    cfg = get_config("tiny", fanouts=[10, 10], cache_width=10)
    g = build_graph(cfg)
    indptr, indices = g.indptr.numpy(), g.indices.numpy()
    perm = seed_permutation(cfg)
    N = cfg["num_nodes"]
    a = oracle.Sampler(indptr, indices, cfg["fanouts"], 10, seed=8)
    frozen = [a.cache_rows(l, range(N)) for l in range(2)]
    fr, n, blocks = a.sample_batch(batch_seeds(perm, 0, cfg["batch"]).numpy(), oracle.MODE_OTF_FETCH, 1.0, 1)
    b = oracle.Sampler(indptr, indices, cfg["fanouts"], 10, seed=8)
    fb, nb, bb = b.sample_batch(batch_seeds(perm, 0, cfg["batch"]).numpy(), oracle.MODE_FBL, 0.0, 1)
    for l in range(2):
        assert np.array_equal(a.cache_rows(l, range(N)), frozen[l])
        assert blocks[l].num_edges == bb[l].num_edges
    # the same neighbours as Full Batch Load (only the order inside a row, and with it the order in which new
    # nodes enter the frontier, differs: key order here, offset order there)
    assert n == nb and set(fr.tolist()) == set(fb.tolist())
