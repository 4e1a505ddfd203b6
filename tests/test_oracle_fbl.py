"""Pins of the oracle's Full Batch Load mode (no cache): hand-worked example, exact enumeration,
invariants on a whole batch, and independence from the cache."""
import itertools
import math
from collections import Counter

import numpy as np

import oracle
from helpers import csr_from_rows, golden_json, star_graph
from workloads import batch_seeds, build_graph, get_config, seed_permutation


def test_worked_fbl_example():
    ex = golden_json("worked_fbl_example.json")
    rows = [[] for _ in range(ex["num_nodes"])]
    rows[ex["node"]] = ex["neighbours"]
    rows[ex["small_node"]] = ex["small_neighbours"]
    indptr, indices = csr_from_rows(rows)
    s = oracle.Sampler(indptr, indices, [ex["fanout"]], ex["cache_width"], seed=1)
    table = {c["step"]: c["fetch_keys"] for c in ex["cases"]}
    s.set_key_fn(lambda purpose, tag, v, step, i: table[step][i] if purpose == oracle.FETCH else 0)
    for c in ex["cases"]:
        assert list(s.fbl_node(0, ex["node"], c["step"])) == c["picks"]
    assert list(s.fbl_node(0, ex["small_node"], 1)) == ex["small_picks"]


def test_fbl_enumeration_uniform_subsets():
    d, f = 6, 3
    indptr, indices = star_graph(d)
    s = oracle.Sampler(indptr, indices, [f], 4, seed=0)
    counts = Counter()
    for perm in itertools.permutations(range(d)):
        s.set_key_fn(lambda purpose, tag, v, step, i: perm[i])
        picks = list(s.fbl_node(0, 0, 1))
        assert picks == sorted(picks) and len(set(picks)) == f
        assert set(picks) == {1 + i for i in sorted(range(d), key=lambda i: perm[i])[:f]}
        counts[tuple(picks)] += 1
    assert len(counts) == math.comb(d, f) and len(set(counts.values())) == 1


def test_fbl_batch_invariants_and_cache_untouched():
    cfg = get_config("tiny")
    g = build_graph(cfg)
    indptr, indices = g.indptr.numpy(), g.indices.numpy()
    deg = indptr[1:] - indptr[:-1]
    adj = [set(indices[indptr[v]:indptr[v + 1]].tolist()) for v in range(cfg["num_nodes"])]
    perm = seed_permutation(cfg)
    L, W, N = len(cfg["fanouts"]), cfg["cache_width"], cfg["num_nodes"]
    s = oracle.Sampler(indptr, indices, cfg["fanouts"], W, seed=13)
    frozen = [s.cache_rows(l, range(N)) for l in range(L)]
    seen = []
    for t in range(3):
        seeds = batch_seeds(perm, 0, cfg["batch"]).numpy()          # same seeds every step
        frontier, n, blocks = s.sample_batch(seeds, oracle.MODE_FBL, 0.0, t + 1)
        for layer in range(L):
            k = L - 1 - layer
            b = blocks[layer]
            dst = frontier[: n[k]]
            assert np.array_equal(np.diff(b.indptr), np.minimum(cfg["fanouts"][layer], deg[dst]))
            assert np.array_equal(frontier[b.indices], b.picked)
            for p in range(n[k]):
                row = b.picked[b.indptr[p]:b.indptr[p + 1]]
                assert list(row) == sorted(row) and len(set(row.tolist())) == len(row)
                assert set(row.tolist()) <= adj[dst[p]]
                if deg[dst[p]] <= cfg["fanouts"][layer]:
                    assert list(row) == list(indices[indptr[dst[p]]:indptr[dst[p] + 1]])
        seen.append(frontier.copy())
        for l in range(L):
            assert np.array_equal(s.cache_rows(l, range(N)), frozen[l])
    assert not np.array_equal(seen[0], seen[1])                     # the step changes the sample


def test_fbl_marginals_real_philox():
    d, f, T = 9, 4, 30000
    indptr, indices = star_graph(d)
    s = oracle.Sampler(indptr, indices, [f], 4, seed=99)
    occ = np.zeros(d + 1)
    for t in range(1, T + 1):
        occ[s.fbl_node(0, 0, t)] += 1
    assert np.all(np.abs(occ[1:] / T - f / d) < 0.02)
