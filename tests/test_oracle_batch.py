"""Whole-batch pins of the CPU oracle: invariants of the method, the BFS special case, and an
independent recomposition of SampleBlocks from the per-node primitives (no GPU involved)."""
import numpy as np
import pytest
import scipy.sparse as sp

import oracle
from workloads import batch_seeds, build_graph, get_config, seed_permutation


@pytest.fixture(scope="module")
def tiny():
    cfg = get_config("tiny")
    g = build_graph(cfg)
    perm = seed_permutation(cfg)
    return cfg, g.indptr.numpy(), g.indices.numpy(), perm


def _adj_sets(indptr, indices):
    return [set(indices[indptr[v]:indptr[v + 1]].tolist()) for v in range(len(indptr) - 1)]


def _relabel_by_sorting(frontier_k, picked):
    """First-appearance relabel written differently from the oracle: numpy unique + argsort."""
    allids = np.concatenate([frontier_k, picked])
    uniq, first = np.unique(allids, return_index=True)
    order = np.argsort(first, kind="stable")
    new_frontier = uniq[order]
    rank = np.empty(len(uniq), dtype=np.int64)
    rank[order] = np.arange(len(uniq))
    local = rank[np.searchsorted(uniq, picked)]
    return new_frontier.astype(np.int32), local.astype(np.int32)


def _check_batch(cfg, indptr, indices, adj, s, seeds, frontier, n, blocks):
    L, W = len(cfg["fanouts"]), cfg["cache_width"]
    deg = indptr[1:] - indptr[:-1]
    assert n[0] == len(seeds) and list(frontier[: n[0]]) == list(seeds)
    assert len(np.unique(frontier)) == len(frontier) == n[L]
    for layer in range(L):
        k = L - 1 - layer
        b = blocks[layer]
        f = cfg["fanouts"][layer]
        assert (b.num_dst, b.num_src) == (n[k], n[k + 1])
        assert b.indptr[0] == 0 and b.indptr[-1] == b.num_edges and np.all(np.diff(b.indptr) >= 0)
        dst = frontier[: n[k]]
        assert np.array_equal(np.diff(b.indptr), np.minimum(f, deg[dst]))          # deg < f => all neighbours
        assert np.array_equal(frontier[b.indices], b.picked)
        want_frontier, want_local = _relabel_by_sorting(frontier[: n[k]], b.picked)
        assert np.array_equal(want_frontier, frontier[: n[k + 1]])
        assert np.array_equal(want_local, b.indices)
        for p in range(n[k]):
            row = b.picked[b.indptr[p]:b.indptr[p + 1]]
            assert len(set(row.tolist())) == len(row)                              # no duplicate neighbour
            assert set(row.tolist()) <= adj[dst[p]]                               # every edge exists
            if deg[dst[p]] <= f:
                assert list(row) == list(indices[indptr[dst[p]]:indptr[dst[p] + 1]])


def test_invariants_over_batches(tiny):
    cfg, indptr, indices, perm = tiny
    adj = _adj_sets(indptr, indices)
    L, W = len(cfg["fanouts"]), cfg["cache_width"]
    deg = indptr[1:] - indptr[:-1]
    s = oracle.Sampler(indptr, indices, cfg["fanouts"], W, seed=11)
    r = oracle.refresh_count(oracle.MODE_OTF, 0.25, W)
    for b in range(6):
        seeds = batch_seeds(perm, b, cfg["batch"]).numpy()
        before = {l: s.cache_rows(l, range(cfg["num_nodes"])) for l in range(L)}
        frontier, n, blocks = s.sample_batch(seeds, oracle.MODE_OTF, 0.25, b + 1)
        _check_batch(cfg, indptr, indices, adj, s, seeds, frontier, n, blocks)
        for l in range(L):
            k = L - 1 - l
            after = s.cache_rows(l, range(cfg["num_nodes"]))
            touched = set(frontier[: n[k]].tolist())
            for v in range(cfg["num_nodes"]):
                changed = int(np.sum(before[l][v] != after[v]))
                if v not in touched or deg[v] <= W:
                    assert changed == 0
                else:
                    assert changed <= r
                valid = after[v][after[v] >= 0]
                assert len(valid) == min(deg[v], W) and len(set(valid.tolist())) == len(valid)
                assert set(valid.tolist()) <= adj[v]
                if deg[v] <= W:
                    assert list(valid) == list(indices[indptr[v]:indptr[v + 1]])


def test_otf_gamma_one_equals_fcr_and_gamma_zero_freezes(tiny):
    cfg, indptr, indices, perm = tiny
    L, W, N = len(cfg["fanouts"]), cfg["cache_width"], cfg["num_nodes"]
    a = oracle.Sampler(indptr, indices, cfg["fanouts"], W, seed=5)
    b = oracle.Sampler(indptr, indices, cfg["fanouts"], W, seed=5)
    z = oracle.Sampler(indptr, indices, cfg["fanouts"], W, seed=5)
    frozen = [z.cache_rows(l, range(N)) for l in range(L)]
    for t in range(4):
        seeds = batch_seeds(perm, t, cfg["batch"]).numpy()
        fa, na, ba = a.sample_batch(seeds, oracle.MODE_FCR, 0.0, t + 1)
        fb, nb, bb = b.sample_batch(seeds, oracle.MODE_OTF, 1.0, t + 1)
        assert np.array_equal(fa, fb) and na == nb
        for x, y in zip(ba, bb):
            assert np.array_equal(x.indptr, y.indptr) and np.array_equal(x.indices, y.indices)
        for l in range(L):
            assert np.array_equal(a.cache_rows(l, range(N)), b.cache_rows(l, range(N)))
        fz, nz, bz = z.sample_batch(seeds, oracle.MODE_OTF, 0.0, t + 1)
        for l in range(L):
            assert np.array_equal(z.cache_rows(l, range(N)), frozen[l])
            # gamma = 0: picks come from the untouched pre-sampled rows
            k = L - 1 - l
            for p in range(0, nz[k], 7):
                row = bz[l].picked[bz[l].indptr[p]:bz[l].indptr[p + 1]]
                assert set(row.tolist()) <= set(frozen[l][fz[p]].tolist())
    # the two modes really do differ from the frozen cache
    assert any(not np.array_equal(a.cache_rows(l, range(N)), frozen[l]) for l in range(L))


def test_layers_have_independent_caches_and_keys(tiny):
    cfg, indptr, indices, perm = tiny
    deg = indptr[1:] - indptr[:-1]
    W = cfg["cache_width"]
    s = oracle.Sampler(indptr, indices, [5, 5], W, seed=3)
    hubs = np.nonzero(deg > 3 * W)[0]
    assert len(hubs) > 3
    assert any(not np.array_equal(s.cache_row(0, v), s.cache_row(1, v)) for v in hubs)
    sh = oracle.Sampler(indptr, indices, [5, 5], W, seed=3, shared=True)
    assert all(np.array_equal(sh.cache_row(0, v), sh.cache_row(1, v)) for v in hubs)
    t = oracle.Sampler(indptr, indices, [5, 5], W, seed=4)
    assert any(not np.array_equal(s.cache_row(0, v), t.cache_row(0, v)) for v in hubs)   # the seed matters


def test_bfs_special_case(tiny):
    """W and every fan-out >= max degree: frontier_k is the BFS ball of radius k (any mode, any gamma)."""
    cfg = get_config("tiny", num_nodes=600, undirected_edges=900)
    g = build_graph(cfg)
    indptr, indices = g.indptr.numpy(), g.indices.numpy()
    maxdeg = int((indptr[1:] - indptr[:-1]).max())
    assert 10 < maxdeg <= 64
    N = cfg["num_nodes"]
    A = sp.csr_matrix((np.ones(len(indices), dtype=np.int8), indices, indptr), shape=(N, N))
    seeds = seed_permutation(cfg)[:5].numpy()
    for mode, gamma, shared in ((oracle.MODE_FCR, 0, False), (oracle.MODE_OTF, 0.3, False), (oracle.MODE_OTF, 0.3, True)):
        s = oracle.Sampler(indptr, indices, [maxdeg] * 3, maxdeg, seed=9, shared=shared)
        frontier, n, blocks = s.sample_batch(seeds, mode, gamma, 1)
        x = np.zeros(N, dtype=np.int8)
        x[seeds] = 1
        for k in range(1, 4):
            # row v of A lists in-neighbours of v: one hop adds every u with A[v,u] != 0 for v in the ball
            x = ((A.T @ x + x) > 0).astype(np.int8)
            assert set(np.nonzero(x)[0].tolist()) == set(frontier[: n[k]].tolist())


def _recompose(s, cfg, seeds, step, r, shared):
    """SampleBlocks rebuilt in Python from the per-node primitives, in the order Algorithm 2 states
    (refresh the frontier's rows, then sample from the cache, then S <- N), with a dict relabel."""
    L = len(cfg["fanouts"])
    frontier = list(seeds)
    pos = {v: p for p, v in enumerate(frontier)}
    n = [len(frontier)]
    blocks = [None] * L
    for k in range(L):
        l = L - 1 - k
        refresh_from = n[k - 1] if (shared and k > 0) else 0
        indptr, picked = [0], []
        for p in range(n[k]):
            v = frontier[p]
            if p >= refresh_from:
                s.refresh_node(l, v, step, r)
            picked += s.pick_node(l, v, step).tolist()
            indptr.append(len(picked))
        local = []
        for u in picked:
            if u not in pos:
                pos[u] = len(frontier)
                frontier.append(u)
            local.append(pos[u])
        n.append(len(frontier))
        blocks[l] = (indptr, local)
    return frontier, n, blocks


@pytest.mark.parametrize("shared", [False, True])
def test_batch_equals_recomposition(tiny, shared):
    cfg, indptr, indices, perm = tiny
    W = cfg["cache_width"]
    a = oracle.Sampler(indptr, indices, cfg["fanouts"], W, seed=21, shared=shared)
    b = oracle.Sampler(indptr, indices, cfg["fanouts"], W, seed=21, shared=shared)
    r = oracle.refresh_count(oracle.MODE_OTF, 0.25, W)
    for t in range(3):
        seeds = batch_seeds(perm, t, cfg["batch"]).numpy()
        frontier, n, blocks = a.sample_batch(seeds, oracle.MODE_OTF, 0.25, t + 1)
        f2, n2, b2 = _recompose(b, cfg, seeds.tolist(), t + 1, r, shared)
        assert list(frontier) == f2 and n == n2
        for l in range(len(cfg["fanouts"])):
            assert list(blocks[l].indptr) == b2[l][0] and list(blocks[l].indices) == b2[l][1]
        for l in range(len(cfg["fanouts"])):
            assert np.array_equal(a.cache_rows(l, range(cfg["num_nodes"])), b.cache_rows(l, range(cfg["num_nodes"])))


def test_shared_cache_refreshes_each_node_once(tiny):
    cfg, indptr, indices, perm = tiny
    W = cfg["cache_width"]
    deg = indptr[1:] - indptr[:-1]
    s = oracle.Sampler(indptr, indices, cfg["fanouts"], W, seed=2, shared=True)
    u = oracle.Sampler(indptr, indices, cfg["fanouts"], W, seed=2, shared=False)
    seeds = batch_seeds(perm, 0, cfg["batch"]).numpy()
    frontier, n, _ = s.sample_batch(seeds, oracle.MODE_OTF, 0.25, 1)
    L = len(cfg["fanouts"])
    refreshed, scanned = s.stats()
    dst_last = frontier[: n[L - 1]]                 # every node that was ever a destination
    assert refreshed == int(np.sum(deg[dst_last] > W))
    assert scanned == int(np.sum(deg[dst_last][deg[dst_last] > W]))
    fu, nu, _ = u.sample_batch(seeds, oracle.MODE_OTF, 0.25, 1)
    ref_u, _ = u.stats()
    assert ref_u == sum(int(np.sum(deg[fu[: nu[k]]] > W)) for k in range(L))


def test_resume_from_exported_rows(tiny):
    cfg, indptr, indices, perm = tiny
    L, W, N = len(cfg["fanouts"]), cfg["cache_width"], cfg["num_nodes"]
    a = oracle.Sampler(indptr, indices, cfg["fanouts"], W, seed=8)
    outs = []
    for t in range(6):
        seeds = batch_seeds(perm, t, cfg["batch"]).numpy()
        if t == 3:
            b = oracle.Sampler(indptr, indices, cfg["fanouts"], W, seed=8)
            for l in range(L):
                rows = a.cache_rows(l, range(N))
                for v in range(N):
                    b.cache_set_row(l, v, rows[v])
        fa, na, ba = a.sample_batch(seeds, oracle.MODE_OTF, 0.25, t + 1)
        if t >= 3:
            fb, nb, bb = b.sample_batch(seeds, oracle.MODE_OTF, 0.25, t + 1)
            assert np.array_equal(fa, fb) and na == nb
            assert all(np.array_equal(x.indices, y.indices) for x, y in zip(ba, bb))
