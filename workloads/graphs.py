"""Seeded synthetic graphs in CSR form (rows sorted ascending, no duplicate neighbour).

Row v lists the nodes whose messages flow to v (in-neighbours).  Two recipes:

* ``chunglu``  - Chung-Lu power law (exponent 2.5), exactly `undirected_edges` distinct
  undirected edges, symmetrised.  Uses float64 for the inverse CDF, so it is generated on
  the host only and the resulting bytes are what both sides consume.
* ``rmat``     - R-MAT (a=.57, b=c=.19, d=.05), integer-only, identical on CPU and CUDA.
  Endpoints >= num_nodes and self-loops are rejected, ids are permuted, duplicates removed.
  On a CUDA device the edge keys are bucketed by source range so that no single sort
  exceeds ~2^28 keys (the 2^31-draw graph is built this way).
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

from .hashing import hash_u64, lsr, permutation

# 16-bit thresholds of the four R-MAT quadrants (a | b | c | d).
_TA = int(round(0.57 * 65536))
_TB = _TA + int(round(0.19 * 65536))
_TC = _TB + int(round(0.19 * 65536))

_STREAM_EDGE = 1
_STREAM_PERM = 2


@dataclass
class Graph:
    num_nodes: int
    num_edges: int          # directed edges stored
    indptr: torch.Tensor    # int64 [N+1]
    indices: torch.Tensor   # int32 [E]

    def to(self, device) -> "Graph":
        return Graph(self.num_nodes, self.num_edges, self.indptr.to(device), self.indices.to(device))

    def degrees(self) -> torch.Tensor:
        return self.indptr[1:] - self.indptr[:-1]


def csr_from_keys(keys_sorted_unique: torch.Tensor, num_nodes: int) -> Graph:
    """keys = (row << 32) | col, sorted ascending and distinct -> CSR."""
    rows = keys_sorted_unique >> 32
    indices = (keys_sorted_unique & 0xFFFFFFFF).to(torch.int32)
    deg = torch.bincount(rows, minlength=num_nodes)
    indptr = torch.zeros(num_nodes + 1, dtype=torch.int64, device=keys_sorted_unique.device)
    torch.cumsum(deg, 0, out=indptr[1:])
    return Graph(num_nodes, int(indices.numel()), indptr, indices)


def csr_from_edges(dst: torch.Tensor, src: torch.Tensor, num_nodes: int) -> Graph:
    """Directed edges src->dst (row = dst) -> sorted, de-duplicated CSR."""
    keys = (dst.to(torch.int64) << 32) | src.to(torch.int64)
    keys = torch.unique(keys)  # sorted ascending
    return csr_from_keys(keys, num_nodes)


# ----------------------------------------------------------------------------- Chung-Lu

def _chunglu(cfg: dict) -> Graph:
    n = cfg["num_nodes"]
    m = cfg["undirected_edges"]
    seed = cfg["graph_seed"]
    i = torch.arange(n, dtype=torch.float64)
    w = (i + 10.0) ** (-1.0 / 1.5)          # exponent beta = 2.5  ->  -1/(beta-1)
    cdf = torch.cumsum(w, 0)
    cdf = cdf / cdf[-1]
    have = torch.empty(0, dtype=torch.int64)
    drawn = 0
    while True:
        k = max(1024, int(1.5 * (m - have.numel())) + 1024)
        e = torch.arange(drawn, drawn + k, dtype=torch.int64)
        drawn += k
        ua = lsr(hash_u64(seed, _STREAM_EDGE, 2 * e), 11).to(torch.float64) * (1.0 / (1 << 53))
        ub = lsr(hash_u64(seed, _STREAM_EDGE, 2 * e + 1), 11).to(torch.float64) * (1.0 / (1 << 53))
        a = torch.searchsorted(cdf, ua, right=True).clamp_(max=n - 1)
        b = torch.searchsorted(cdf, ub, right=True).clamp_(max=n - 1)
        keep = a != b
        lo = torch.minimum(a, b)[keep]
        hi = torch.maximum(a, b)[keep]
        cand = torch.cat([have, (lo << 32) | hi])
        # distinct keys in order of first appearance
        uniq, inv = torch.unique(cand, return_inverse=True)
        first = torch.full((uniq.numel(),), cand.numel(), dtype=torch.int64)
        first.scatter_reduce_(0, inv, torch.arange(cand.numel(), dtype=torch.int64), reduce="amin")
        order = torch.argsort(first)
        have = uniq[order]
        if have.numel() >= m:
            have = have[:m]
            break
    perm = permutation(seed, _STREAM_PERM, n)
    a = perm[have >> 32]
    b = perm[have & 0xFFFFFFFF]
    return csr_from_edges(torch.cat([a, b]), torch.cat([b, a]), n)


# ----------------------------------------------------------------------------- R-MAT

def _rmat_chunk(seed: int, scale: int, e: torch.Tensor):
    """Raw R-MAT endpoints (src, dst) in [0, 2^scale) for draw indices `e` (int64)."""
    src = torch.zeros_like(e)
    dst = torch.zeros_like(e)
    words = (scale + 3) // 4
    h = None
    for level in range(scale):
        if level % 4 == 0:
            h = hash_u64(seed, _STREAM_EDGE, e * words + (level // 4))
        bits = (h >> (16 * (level % 4))) & 0xFFFF
        sbit = bits >= _TB                                   # quadrants c, d
        dbit = ((bits >= _TA) & (bits < _TB)) | (bits >= _TC)  # quadrants b, d
        src = (src << 1) | sbit
        dst = (dst << 1) | dbit
    return src, dst


def _rmat(cfg: dict, device, chunk: int, buckets: int) -> Graph:
    n = cfg["num_nodes"]
    scale = cfg["rmat_scale"]
    seed = cfg["graph_seed"]
    draws = cfg["draws"]
    sym = cfg["symmetric"]
    perm = permutation(seed, _STREAM_PERM, n, device=device)
    bucket_keys = [[] for _ in range(buckets)]
    rows_per_bucket = (n + buckets - 1) // buckets
    for start in range(0, draws, chunk):
        e = torch.arange(start, min(draws, start + chunk), dtype=torch.int64, device=device)
        src, dst = _rmat_chunk(seed, scale, e)
        keep = (src != dst)
        if n < (1 << scale):
            keep &= (src < n) & (dst < n)
        src = perm[src[keep]]
        dst = perm[dst[keep]]
        del e, keep
        keys = (dst << 32) | src                       # row = destination
        if sym:
            keys = torch.cat([keys, (src << 32) | dst])
        del src, dst
        if buckets == 1:
            bucket_keys[0].append(keys)
        else:
            b = (keys >> 32) // rows_per_bucket
            for j in range(buckets):
                bucket_keys[j].append(keys[b == j])
            del b
        del keys
    deg_parts, idx_parts = [], []
    for j in range(buckets):
        k = torch.cat(bucket_keys[j])
        bucket_keys[j] = None
        k = torch.unique(k)
        lo = j * rows_per_bucket
        hi = min(n, lo + rows_per_bucket)
        deg_parts.append(torch.bincount((k >> 32) - lo, minlength=hi - lo))
        idx_parts.append((k & 0xFFFFFFFF).to(torch.int32))
        del k
    deg = torch.cat(deg_parts)
    indices = torch.cat(idx_parts)
    del deg_parts, idx_parts
    indptr = torch.zeros(n + 1, dtype=torch.int64, device=device)
    torch.cumsum(deg, 0, out=indptr[1:])
    return Graph(n, int(indices.numel()), indptr, indices)


def build_graph(cfg: dict, device="cpu") -> Graph:
    """Build the config's graph; tensors live on `device`."""
    if cfg["kind"] == "chunglu":
        return _chunglu(cfg).to(device)
    if cfg["kind"] == "rmat":
        dev = torch.device(device)
        draws = cfg["draws"]
        chunk = 1 << 26 if dev.type == "cuda" else 1 << 22
        buckets = 1
        while draws * (2 if cfg["symmetric"] else 1) // buckets > (1 << 28):
            buckets *= 2
        return _rmat(cfg, dev, chunk, buckets)
    raise ValueError(cfg["kind"])
