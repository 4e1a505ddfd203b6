"""The synthetic input generators: shapes, CSR contract, determinism (no GPU involved)."""
import numpy as np
import pytest
import torch

from workloads import batch_seeds, build_features, build_graph, feature_rows, get_config, seed_permutation


def _check_csr(g, symmetric):
    deg = g.degrees()
    assert g.indptr.dtype == torch.int64 and g.indices.dtype == torch.int32
    assert int(g.indptr[0]) == 0 and int(g.indptr[-1]) == g.num_edges == g.indices.numel()
    rows = torch.repeat_interleave(torch.arange(g.num_nodes), deg)
    keys = (rows << 32) | g.indices.long()
    assert bool((keys[1:] > keys[:-1]).all())                 # rows ascending, no duplicate neighbour
    assert bool((g.indices.long() != rows).all())             # no self-loops
    assert int(g.indices.min()) >= 0 and int(g.indices.max()) < g.num_nodes
    if symmetric:
        rev = torch.sort((g.indices.long() << 32) | rows).values
        assert torch.equal(rev, keys)


def test_tiny_shape():
    cfg = get_config("tiny")
    g = build_graph(cfg)
    assert (g.num_nodes, g.num_edges) == (2708, 10556)
    _check_csr(g, True)
    X = build_features(cfg)
    assert X.shape == (2708, 1433) and X.dtype == torch.float32
    assert set(torch.unique(X).tolist()) == {0.0, 1.0}
    assert 10 < float(X.sum(1).mean()) < 26


def test_mid_shape():
    cfg = get_config("mid")
    g = build_graph(cfg)
    assert (g.num_nodes, g.num_edges) == (169343, 2332486)
    _check_csr(g, True)
    assert int(g.degrees().max()) > 500                       # heavy tail


def test_rmat_small_is_deterministic_and_bucket_independent():
    from workloads import graphs
    cfg = get_config("shared", rmat_scale=14, num_nodes=12000, draws=150000)
    a = build_graph(cfg)
    b = graphs._rmat(cfg, torch.device("cpu"), chunk=1 << 12, buckets=4)
    assert torch.equal(a.indptr, b.indptr) and torch.equal(a.indices, b.indices)
    _check_csr(a, True)
    deg = a.degrees()
    assert int(deg.max()) > 40 * float(deg.float().mean())    # skewed
    assert int((deg == 0).sum()) > 0                          # isolated nodes exist
    c = build_graph(get_config("scale", rmat_scale=12, num_nodes=1 << 12, draws=1 << 16))
    _check_csr(c, False)


@pytest.mark.parametrize("name", ["large", "shared"])
def test_hash_features_row_evaluation(name):
    cfg = get_config(name, num_nodes=5000)
    X = build_features(cfg, rows_per_chunk=1024)
    ids = torch.tensor([0, 1, 1023, 1024, 4999])
    bits = torch.int32 if cfg["feat_dtype"] == "f32" else torch.int16
    assert torch.equal(feature_rows(cfg, ids).view(bits), X[ids].view(bits))
    assert bool(torch.isfinite(X.float()).all()) and float(X.float().abs().max()) < 2.0
    assert float(X.float().abs().min()) >= 2.0 ** -7


def test_seed_batches_are_distinct_and_sharded():
    cfg = get_config("tiny")
    perm = seed_permutation(cfg)
    assert sorted(perm.tolist()) == list(range(cfg["num_nodes"]))
    b0 = batch_seeds(perm, 0, 64)
    assert len(set(b0.tolist())) == 64
    wrap = batch_seeds(perm, 42, 64)                          # 42*64 = 2688: wraps past 2708
    assert len(set(wrap.tolist())) == 64
    # two ranks interleave windows of the one-rank sequence
    assert torch.equal(batch_seeds(perm, 1, 64, rank=1, world=2), batch_seeds(perm, 3, 64))
    assert torch.equal(batch_seeds(perm, 1, 64, rank=0, world=2), batch_seeds(perm, 2, 64))
