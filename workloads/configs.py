"""The five workload shapes (stand-ins for the public datasets the paper measures on).

Fan-outs are listed input-layer-first: the hop that starts from the seeds uses
the LAST entry (the paper's sampling loop runs l = L down to 1, Algorithm 2).
"""
from __future__ import annotations

import copy

GRAPH_SEED_BASE = 0x5EED0000

CONFIGS = {
    # Cora-shaped: small power-law graph, wide binary bag-of-words features.
    "tiny": dict(
        index=0, kind="chunglu", num_nodes=2708, undirected_edges=5278, symmetric=True,
        feat_dtype="f32", feat_dim=1433, feat_kind="bow",
        fanouts=[5, 5], cache_width=10, shared=False,
        runs=[("otf", 0.25)], batch=64, batches=20,
    ),
    # ogbn-arxiv-shaped citation graph, symmetrised.
    "mid": dict(
        index=1, kind="chunglu", num_nodes=169343, undirected_edges=1166243, symmetric=True,
        feat_dtype="f32", feat_dim=128, feat_kind="normal",
        fanouts=[15, 10, 5], cache_width=20, shared=False,
        runs=[("fcr", 1.0), ("otf", 0.1), ("otf", 0.3), ("otf", 0.5)], batch=1024, batches=10,
    ),
    # ogbn-products-shaped co-purchase graph: R-MAT, symmetric.
    # `draws` was tuned once: it yields exactly 123,679,916 directed edges (target 123.7M).
    "large": dict(
        index=2, kind="rmat", rmat_scale=22, num_nodes=2449029, draws=83_448_488, symmetric=True,
        feat_dtype="f32", feat_dim=100, feat_kind="hash",
        fanouts=[15, 10, 5], cache_width=20, shared=False,
        runs=[("otf", 0.2)], batch=4096, batches=3,
    ),
    # ogbn-mag-shaped, one cache shared by all hops (cache width is not given by the
    # workload statement; 32 = one 128-byte line and >= the largest fan-out).
    "shared": dict(
        index=3, kind="rmat", rmat_scale=20, num_nodes=736389, draws=6_391_012, symmetric=True,
        feat_dtype="bf16", feat_dim=128, feat_kind="hash",
        fanouts=[25, 10], cache_width=32, shared=True,
        runs=[("otf", 0.3)], batch=2048, batches=3,
    ),
    # Scale: 2^26 nodes, 2^31 directed draws (average degree 32 before de-duplication).
    "scale": dict(
        index=4, kind="rmat", rmat_scale=26, num_nodes=1 << 26, draws=1 << 31, symmetric=False,
        feat_dtype="bf16", feat_dim=128, feat_kind="hash",
        fanouts=[20, 15, 10], cache_width=32, shared=False,
        runs=[("otf", 0.1)], batch=8192, batches=3,
    ),
}


def config_names():
    return list(CONFIGS.keys())


def get_config(name: str, **overrides) -> dict:
    """A copy of a named config; `overrides` replace keys (used by reduced-size test variants)."""
    cfg = copy.deepcopy(CONFIGS[name])
    cfg["name"] = name
    cfg.update(overrides)
    cfg.setdefault("graph_seed", GRAPH_SEED_BASE + cfg["index"])
    return cfg
