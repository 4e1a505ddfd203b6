"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU involved)."""
import itertools
import math
import os
from collections import Counter

import numpy as np
import pytest

import oracle
from helpers import GOLDEN, csr_from_rows, golden_json, star_graph


# ------------------------------------------------------------------ Philox known answers
def test_philox_known_answer_vectors():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 3
    for w in rows:
        v = [int(x, 16) for x in w]
        assert oracle.philox4x32_10(v[0:4], v[4:6]) == v[6:10]


def test_default_keys_are_philox_words():
    """key32(i) is word (i & 3) of Philox(counter=(i>>2, v, step, purpose<<8|tag), key=seed words):
    checked through the pre-sample of a node whose order the test recomputes from raw Philox calls."""
    d, W, seed = 23, 5, 0x0123456789ABCDEF
    indptr, indices = star_graph(d)
    s = oracle.Sampler(indptr, indices, [3], W, seed)
    keys = []
    for i in range(d):
        out = oracle.philox4x32_10([i >> 2, 0, 0, (oracle.FILL << 8) | 0], [seed & 0xFFFFFFFF, seed >> 32])
        keys.append((out[i & 3], i))
    want = [indices[i] for _, i in sorted(keys)[:W]]
    assert list(s.cache_row(0, 0)) == want


# ------------------------------------------------------------------ hand-worked example
def test_worked_refresh_example():
    ex = golden_json("worked_refresh_example.json")
    rows = [[] for _ in range(ex["num_nodes"])]
    rows[ex["node"]] = ex["neighbours"]
    indptr, indices = csr_from_rows(rows)
    s = oracle.Sampler(indptr, indices, [ex["fanout"]], ex["cache_width"], seed=1)
    table = {}
    for st in ex["steps"]:
        table[(oracle.FILL, st["step"])] = st["fill_keys"]
        if "evict_keys" in st:
            table[(oracle.EVICT, st["step"])] = st["evict_keys"]
            table[(oracle.PICK, st["step"])] = st["pick_keys"]
    s.set_key_fn(lambda purpose, tag, v, step, i: table[(purpose, step)][i])
    v = ex["node"]
    for st in ex["steps"]:
        if st["what"] == "presample":
            assert list(s.cache_row(0, v)) == st["row_after"]
            continue
        s.refresh_node(0, v, st["step"], st["r"])
        assert list(s.cache_row(0, v)) == st["row_after"], st
        assert list(s.pick_node(0, v, st["step"])) == st["picks"], st


def test_worked_blocks_example():
    ex = golden_json("worked_blocks_example.json")
    indptr, indices = csr_from_rows(ex["rows"])
    for mode, gamma in ((oracle.MODE_OTF, 0.5), (oracle.MODE_FCR, 0.0), (oracle.MODE_OTF, 0.0)):
        s = oracle.Sampler(indptr, indices, ex["fanouts"], ex["cache_width"], seed=7)
        frontier, n, blocks = s.sample_batch(ex["seeds"], mode, gamma, step=1)
        assert list(frontier) == ex["frontier"] and n == ex["n"]
        for want in ex["blocks_by_layer"]:
            b = blocks[want["layer"]]
            assert list(b.indptr) == want["indptr"]
            assert list(b.picked) == want["picked"]
            assert list(b.indices) == want["indices"]


# ------------------------------------------------------------------ refresh count
@pytest.mark.parametrize("gamma,W,r", [(0.25, 10, 3), (0.1, 32, 3), (0.3, 32, 10), (0.2, 20, 4), (0.5, 20, 10),
                                       (0.1, 20, 2), (0.3, 20, 6), (0.0, 20, 0), (1.0, 20, 20)])
def test_refresh_count(gamma, W, r):
    assert oracle.refresh_count(oracle.MODE_OTF, gamma, W) == r
    assert oracle.refresh_count(oracle.MODE_FCR, gamma, W) == W


# ------------------------------------------------------------------ exact enumeration of the selection law
def _rank_keys(perm_by_purpose):
    def fn(purpose, tag, v, step, i):
        return perm_by_purpose[purpose][i]
    return fn


def test_presample_enumeration_uniform_ordered():
    """Over all d! rank assignments every ordered W-arrangement of neighbours appears equally often."""
    d, W = 5, 3
    indptr, indices = star_graph(d)
    counts = Counter()
    for perm in itertools.permutations(range(d)):
        s = oracle.Sampler(indptr, indices, [2], W, seed=0)
        s.set_key_fn(_rank_keys({oracle.FILL: perm}))
        counts[tuple(s.cache_row(0, 0))] += 1
        s.close()
    assert len(counts) == math.perm(d, W)
    assert set(counts.values()) == {math.factorial(d) // math.perm(d, W)}


def test_pick_enumeration_uniform_and_ascending():
    d, W, f = 6, 4, 2
    indptr, indices = star_graph(d)
    s = oracle.Sampler(indptr, indices, [f], W, seed=0)
    s.set_key_fn(_rank_keys({oracle.FILL: list(range(d))}))
    row = list(s.cache_row(0, 0))
    counts = Counter()
    for perm in itertools.permutations(range(W)):
        s.set_key_fn(_rank_keys({oracle.FILL: list(range(d)), oracle.PICK: perm}))
        picks = list(s.pick_node(0, 0, 1))
        slots = [row.index(u) for u in picks]
        assert slots == sorted(slots) and len(set(picks)) == f
        # the picked slots are exactly the f slots of smallest rank
        assert sorted(slots) == sorted(sorted(range(W), key=lambda j: perm[j])[:f])
        counts[tuple(picks)] += 1
    assert len(counts) == math.comb(W, f)
    assert set(counts.values()) == {math.factorial(W) // math.comb(W, f)}


@pytest.mark.parametrize("r", [1, 2, 3])
def test_refresh_enumeration_stationary(r):
    """Uniform W-subsets stay uniform under evict-r / refill-r: starting from every W-subset and
    enumerating all EVICT and FILL rank assignments, every W-subset results equally often, the
    retained slots never move, and exactly the evicted positions are rewritten."""
    d, W = 5, 3
    indptr, indices = star_graph(d)
    nb = list(range(1, d + 1))
    counts = Counter()
    s = oracle.Sampler(indptr, indices, [2], W, seed=0)
    for start in itertools.permutations(nb, W):
        for ev in itertools.permutations(range(W)):
            evicted = set(sorted(range(W), key=lambda j: ev[j])[:r])
            for fl in itertools.permutations(range(d)):
                s.cache_set_row(0, 0, np.array(start, dtype=np.int32))
                s.set_key_fn(_rank_keys({oracle.EVICT: ev, oracle.FILL: fl}))
                s.refresh_node(0, 0, 1, r)
                row = list(s.cache_row(0, 0))
                for j in range(W):
                    if j not in evicted:
                        assert row[j] == start[j]
                assert len(set(row)) == W and set(row) <= set(nb)
                # refill = the r best-ranked offsets whose neighbour is not retained, into ascending evicted slots
                retained = {start[j] for j in range(W) if j not in evicted}
                cand = [i for i in sorted(range(d), key=lambda i: fl[i]) if nb[i] not in retained][:r]
                assert [row[j] for j in sorted(evicted)] == [nb[i] for i in cand]
                counts[frozenset(row)] += 1
    assert len(counts) == math.comb(d, W)
    assert len(set(counts.values())) == 1


def test_ties_break_by_index():
    d, W = 6, 3
    indptr, indices = star_graph(d)
    s = oracle.Sampler(indptr, indices, [2], W, seed=0)
    s.set_key_fn(lambda purpose, tag, v, step, i: 5)
    assert list(s.cache_row(0, 0)) == [1, 2, 3]
    assert list(s.pick_node(0, 0, 1)) == [1, 2]
    s.refresh_node(0, 0, 1, 1)           # evicts slot 0; candidates offsets 0,3,4,5 -> offset 0 again
    assert list(s.cache_row(0, 0)) == [1, 2, 3]


# ------------------------------------------------------------------ statistics with the real keys
def _chi2(counts, total, cells):
    exp = total / cells
    return sum((c - exp) ** 2 / exp for c in counts) + (cells - len(counts)) * exp


def test_fcr_subsets_chi_square_real_philox():
    d, W, T = 8, 4, 70000
    indptr, indices = star_graph(d)
    s = oracle.Sampler(indptr, indices, [2], W, seed=0xC0FFEE)
    counts = Counter()
    for t in range(1, T + 1):
        s.refresh_node(0, 0, t, W)
        counts[frozenset(s.cache_row(0, 0))] += 1
    cells = math.comb(d, W)                       # 70 cells, 69 degrees of freedom
    assert _chi2(counts.values(), T, cells) < 69 + 5 * math.sqrt(2 * 69)


def test_otf_marginal_presence_is_W_over_d_real_philox():
    d, W, T = 9, 4, 40000
    indptr, indices = star_graph(d)
    s = oracle.Sampler(indptr, indices, [2], W, seed=42)
    occ = np.zeros(d + 1)
    pick_occ = np.zeros(d + 1)
    for t in range(1, T + 1):
        s.refresh_node(0, 0, t, 1)
        occ[s.cache_row(0, 0)] += 1
        pick_occ[s.pick_node(0, 0, t)] += 1
    p = occ[1:] / T
    assert np.all(np.abs(p - W / d) < 0.02), p
    q = pick_occ[1:] / T
    assert np.all(np.abs(q - 2 / d) < 0.02), q


# ------------------------------------------------------------------ feature gather
def test_gather_equals_indexing():
    rng = np.random.default_rng(0)
    for dtype, d in ((np.float32, 100), (np.uint16, 128), (np.float32, 1433), (np.uint8, 7)):
        X = rng.integers(0, 255, size=(50, d)).astype(dtype)
        ids = rng.integers(0, 50, size=77).astype(np.int32)
        assert np.array_equal(oracle.gather(X, ids), X[ids])
    assert oracle.gather(X, np.empty(0, np.int32)).shape == (0, 7)


# ------------------------------------------------------------------ argument checks
def test_bad_arguments():
    indptr, indices = star_graph(4)
    with pytest.raises(ValueError):
        oracle.Sampler(indptr, indices, [5], 4, 0)            # fan-out above the cache width
    s = oracle.Sampler(indptr, indices, [2], 3, 0)
    with pytest.raises(ValueError):
        s.sample_batch([0], oracle.MODE_OTF, 0.5, 0)            # step 0 is the pre-sample
    with pytest.raises(ValueError):
        s.sample_batch([9], oracle.MODE_OTF, 0.5, 1)            # seed out of range
    with pytest.raises(ValueError):
        s.sample_batch([1, 1], oracle.MODE_OTF, 0.5, 1)         # duplicate seeds
    with pytest.raises(ValueError):
        s.sample_batch([1], oracle.MODE_OTF, 1.5, 1)
    s.sample_batch([1, 0], oracle.MODE_OTF, 0.5, 1)             # still usable afterwards
