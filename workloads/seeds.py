"""Seed batches: consecutive windows of one seeded node permutation (distinct within a batch)."""
from __future__ import annotations

import torch

from .hashing import permutation

_STREAM_SEEDS = 4


def seed_permutation(cfg: dict, device="cpu") -> torch.Tensor:
    return permutation(cfg["graph_seed"], _STREAM_SEEDS, cfg["num_nodes"], device=device).to(torch.int32)


def batch_seeds(perm: torch.Tensor, batch_index: int, batch_size: int, rank: int = 0, world: int = 1) -> torch.Tensor:
    """Batch `batch_index` of rank `rank`: ranks take interleaved windows, so no two ranks
    ever train on the same window and one rank with world=1 sees every window."""
    n = perm.numel()
    if batch_size > n:
        raise ValueError("batch larger than the graph")
    w = batch_index * world + rank
    start = (w * batch_size) % n
    if start + batch_size <= n:
        return perm[start:start + batch_size].contiguous()
    # wrap-around window; entries stay distinct because batch_size <= n
    return torch.cat([perm[start:], perm[: start + batch_size - n]]).contiguous()
