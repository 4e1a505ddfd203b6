"""Seeded feature matrices.

* ``hash``   - every element is a pure integer function of (seed, row, column) mapped to a
  finite float with |x| in [2^-7, 2): identical bits on CPU and CUDA, and any subset of rows
  can be re-evaluated without materialising the matrix (`feature_rows`).
* ``normal`` - N(0,1) by Box-Muller in float64 on the host, rounded to fp32 once; the
  resulting bytes are uploaded, so both sides read the same matrix.
* ``bow``    - binary bag-of-words-like rows: 1.0 with probability 18/feat_dim, else 0.0.
"""
from __future__ import annotations

import math

import torch

from .hashing import hash_u64, lsr

_STREAM_FEAT = 3


def _torch_dtype(cfg):
    return torch.float32 if cfg["feat_dtype"] == "f32" else torch.bfloat16


def _hash_rows(cfg: dict, rows: torch.Tensor) -> torch.Tensor:
    """Feature rows for node ids `rows` (int64, any device), 'hash' kind."""
    d = cfg["feat_dim"]
    seed = cfg["graph_seed"]
    if cfg["feat_dtype"] == "bf16":
        per = 4                                     # four 16-bit draws per hash
        nh = (d + per - 1) // per
        col = torch.arange(nh, dtype=torch.int64, device=rows.device)
        h = hash_u64(seed, _STREAM_FEAT, rows[:, None] * nh + col[None, :])
        parts = [(h >> (16 * j)) & 0xFFFF for j in range(per)]
        r = torch.stack(parts, dim=2).reshape(rows.numel(), nh * per)[:, :d]
        # sign(1) | exponent 120..127 (3 random bits) | mantissa(7)
        bits = ((r & 0x8000) | ((120 + ((r >> 7) & 7)) << 7) | (r & 0x7F))
        bits = torch.where(bits >= 0x8000, bits - 0x10000, bits).to(torch.int16)
        return bits.view(torch.bfloat16)
    per = 2
    nh = (d + per - 1) // per
    col = torch.arange(nh, dtype=torch.int64, device=rows.device)
    h = hash_u64(seed, _STREAM_FEAT, rows[:, None] * nh + col[None, :])
    parts = [(h >> (32 * j)) & 0xFFFFFFFF for j in range(per)]
    r = torch.stack(parts, dim=2).reshape(rows.numel(), nh * per)[:, :d]
    bits = (r & 0x80000000) | ((120 + ((r >> 23) & 7)) << 23) | (r & 0x7FFFFF)
    bits = torch.where(bits >= 0x80000000, bits - 0x100000000, bits).to(torch.int32)
    return bits.view(torch.float32)


def feature_rows(cfg: dict, ids: torch.Tensor) -> torch.Tensor:
    """Re-evaluate feature rows of a 'hash' matrix for the given node ids."""
    if cfg["feat_kind"] != "hash":
        raise ValueError("feature_rows needs a 'hash' feature matrix")
    return _hash_rows(cfg, ids.to(torch.int64))


def build_features(cfg: dict, device="cpu", rows_per_chunk: int = 1 << 19, row_range=None) -> torch.Tensor:
    """The [num_nodes, feat_dim] feature matrix on `device` (row-major, contiguous), or its rows
    [row_range[0], row_range[1]) - a shard."""
    n, d = cfg["num_nodes"], cfg["feat_dim"]
    seed = cfg["graph_seed"]
    kind = cfg["feat_kind"]
    first, last = row_range if row_range is not None else (0, n)
    if kind == "hash":
        out = torch.empty((last - first, d), dtype=_torch_dtype(cfg), device=device)
        for lo in range(first, last, rows_per_chunk):
            hi = min(last, lo + rows_per_chunk)
            out[lo - first:hi - first] = _hash_rows(cfg, torch.arange(lo, hi, dtype=torch.int64, device=device))
        return out
    if row_range is not None:
        return build_features(cfg, "cpu", rows_per_chunk)[first:last].contiguous().to(device)
    idx = torch.arange(n * d, dtype=torch.int64)
    if kind == "normal":
        u1 = (lsr(hash_u64(seed, _STREAM_FEAT, 2 * idx), 11).to(torch.float64) + 1.0) * (1.0 / (1 << 53))
        u2 = lsr(hash_u64(seed, _STREAM_FEAT, 2 * idx + 1), 11).to(torch.float64) * (1.0 / (1 << 53))
        z = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos(2.0 * math.pi * u2)
        return z.to(_torch_dtype(cfg)).reshape(n, d).contiguous().to(device)
    if kind == "bow":
        h = lsr(hash_u64(seed, _STREAM_FEAT, idx), 32)
        thr = int((18.0 / d) * (1 << 32))
        return (h < thr).to(_torch_dtype(cfg)).reshape(n, d).contiguous().to(device)
    raise ValueError(kind)
