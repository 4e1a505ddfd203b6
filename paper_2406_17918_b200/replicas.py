"""Multi-GPU plumbing: independent replicas, one process per GPU.

Mini-batch GNN training is data parallel: every rank holds the whole graph, its own cache and
samples its own seed windows, so the sampling path has no exchange step and needs no
collective.  The only communication is the benchmark's: a barrier around the timed region, the
maximum of the ranks' device times and the sum of the units they processed.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_rank():
    """(rank, local_rank, world_size) from the launcher's environment (1 process if unset)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str, device=None):
    """Join the job's process group when there is more than one rank."""
    rank, local_rank, world = env_rank()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        kw = {}
        if backend == "nccl" and device is not None:
            kw["device_id"] = device
        dist.init_process_group(backend=backend, rank=rank, world_size=world, **kw)
    return rank, local_rank, world


def barrier():
    if dist.is_initialized():
        dist.barrier()


def aggregate(ms_local: float, units_local, device="cpu", reduce="sum"):
    """(max over ranks of ms, elementwise sum - or, with reduce="max", maximum - over ranks of units)."""
    units = [float(u) for u in units_local]
    if not dist.is_initialized():
        return float(ms_local), units
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    u = torch.tensor(units, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.MAX if reduce == "max" else dist.ReduceOp.SUM)
    return float(t.item()), [float(x) for x in u.tolist()]


def shutdown():
    if dist.is_initialized():
        dist.destroy_process_group()
