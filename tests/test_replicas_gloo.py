"""The multi-GPU plumbing (independent replicas, no data-path collective) on CPU with gloo."""
import os
import socket

import torch
import torch.multiprocessing as mp

from workloads import batch_seeds, get_config, seed_permutation


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2406_17918_b200 import replicas

    r, lr, w = replicas.init("gloo")
    assert (r, lr, w) == (rank, rank, world)
    replicas.barrier()
    # rank r took 10*(r+1) ms and processed (r+1)*100 edges, (r+1) rows
    ms, units = replicas.aggregate(10.0 * (rank + 1), [100 * (rank + 1), rank + 1])
    cfg = get_config("tiny")
    perm = seed_permutation(cfg)
    mine = [batch_seeds(perm, b, 64, rank, world) for b in range(3)]
    torch.save({"ms": ms, "units": units, "seeds": mine}, os.path.join(out_dir, "r%d.pt" % rank))
    replicas.barrier()
    replicas.shutdown()


def test_two_ranks_aggregate_and_shard(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    res = [torch.load(os.path.join(tmp_path, "r%d.pt" % r)) for r in range(world)]
    for r in res:
        assert r["ms"] == 20.0                      # max over ranks
        assert r["units"] == [300.0, 3.0]           # sum over ranks
    # the ranks' seed windows are disjoint and together are the one-rank sequence
    cfg = get_config("tiny")
    perm = seed_permutation(cfg)
    flat = [w for b in range(3) for r in range(world) for w in [res[r]["seeds"][b]]]
    for i, w in enumerate(flat):
        assert torch.equal(w, batch_seeds(perm, i, 64))


def test_single_process_is_identity():
    from paper_2406_17918_b200 import replicas

    assert replicas.aggregate(3.5, [7, 8]) == (3.5, [7.0, 8.0])
    assert replicas.env_rank()[2] >= 1
