"""The node-sharded driver (one process per rank, all_to_all_single) on CPU with gloo, world sizes 2 and 3,
with the oracle's per-node primitives standing in for the kernels; plus the oracle-level facts the
sharded design rests on."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

import oracle
from workloads import batch_seeds, build_graph, get_config, seed_permutation

THETA, SEED = 12, 5


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _features(n, d=6):
    return (torch.arange(n * d, dtype=torch.float32).reshape(n, d) * 0.5).contiguous()


def _worker(rank, world, port, out_dir, capacity=None):
    import torch.distributed as dist

    import fake_shard_ops as ops
    from paper_2406_17918_b200 import sharded

    dist.init_process_group("gloo", rank=rank, world_size=world, init_method="tcp://127.0.0.1:%d" % port)
    cfg = get_config("tiny")
    g = build_graph(cfg)
    perm = seed_permutation(cfg)
    X = _features(cfg["num_nodes"])
    ip, idx = sharded.shard_csr(g.indptr, g.indices, rank, world)
    lo, hi = sharded.shard_range(cfg["num_nodes"], rank, world)
    me = sharded.ShardRank(ops, rank, world, ip, idx, X[lo:hi].contiguous(), cfg["fanouts"], cfg["cache_width"], SEED,
                           cfg["shared"], THETA, max_seeds=cfg["batch"], max_requests=cfg["num_nodes"])
    if capacity:            # fixed-capacity exchanges: no size is read on the host inside a batch
        me.set_capacities([abs(capacity)] * (len(cfg["fanouts"]) + 1), merge=capacity > 0)
    out = []
    t = 1
    for mode, rate in [(ops.GS_MODE_OTF, 0.25), (ops.GS_MODE_OTF, 0.25), (ops.GS_MODE_FCR, 0.0), (ops.GS_MODE_OTF_FETCH, 0.5),
                       (ops.GS_MODE_FBL, 0.0)]:
        seeds = batch_seeds(perm, t, cfg["batch"], rank, world)
        blocks, frontier, n, m, feats = sharded.sample_batch(me, seeds, mode, rate, t)
        L = len(cfg["fanouts"])
        out.append({"n": n, "m": m, "frontier": frontier[: n[L]].clone(), "feats": feats.clone(),
                    "indptr": [blocks[l].indptr(n[L - 1 - l]).clone() for l in range(L)],
                    "indices": [blocks[l].indices(m[l]).clone() for l in range(L)]})
        t += 1
    torch.save(out, os.path.join(out_dir, "r%d.pt" % rank))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world,capacity", [(2, None), (3, None), (2, 1500), (3, 920), (3, -920), (4, 680)])
def test_ranks_equal_one_sampler_taking_the_batches_in_turn(tmp_path, world, capacity):
    """World size 3 gives uneven shards (2,708 nodes: 903 + 903 + 902).  With a capacity the exchanges have a
    fixed pitch (segments of that many ids per pair of ranks) and the driver reads no size inside a batch; the owners
    merge the requesters' lists and sample every distinct node once (negative: they serve the lists one by one)."""
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path), capacity), nprocs=world, join=True)
    res = [torch.load(os.path.join(tmp_path, "r%d.pt" % r)) for r in range(world)]
    cfg = get_config("tiny")
    g = build_graph(cfg)
    perm = seed_permutation(cfg)
    X = _features(cfg["num_nodes"])
    O = oracle.Sampler(g.indptr.numpy(), g.indices.numpy(), cfg["fanouts"], cfg["cache_width"], SEED, cfg["shared"])
    O.set_theta(THETA)
    L = len(cfg["fanouts"])
    modes = [(oracle.MODE_OTF, 0.25), (oracle.MODE_OTF, 0.25), (oracle.MODE_FCR, 0.0), (oracle.MODE_OTF_FETCH, 0.5),
             (oracle.MODE_FBL, 0.0)]
    for i, (om, rate) in enumerate(modes):
        t = i + 1
        for r in range(world):
            fr, n, blocks = O.sample_batch(batch_seeds(perm, t, cfg["batch"], r, world).numpy(), om, rate, t)
            got = res[r][i]
            assert got["n"] == n and np.array_equal(got["frontier"].numpy(), fr)
            for l in range(L):
                assert np.array_equal(got["indptr"][l].numpy(), blocks[l].indptr)
                assert np.array_equal(got["indices"][l].numpy(), blocks[l].indices)
            assert torch.equal(got["feats"], X[torch.from_numpy(fr.astype(np.int64))])


def _failing_worker(rank, world, port, out_dir, capacity=None):
    import torch.distributed as dist

    import fake_shard_ops as ops
    from paper_2406_17918_b200 import sharded

    dist.init_process_group("gloo", rank=rank, world_size=world, init_method="tcp://127.0.0.1:%d" % port)
    cfg = get_config("tiny")
    g = build_graph(cfg)
    perm = seed_permutation(cfg)
    X = _features(cfg["num_nodes"])
    ip, idx = sharded.shard_csr(g.indptr, g.indices, rank, world)
    lo, hi = sharded.shard_range(cfg["num_nodes"], rank, world)
    # the last rank can serve three nodes per list only: its first hop fails on the owner side
    cap = 3 if rank == world - 1 and not capacity else cfg["num_nodes"]
    me = sharded.ShardRank(ops, rank, world, ip, idx, X[lo:hi].contiguous(), cfg["fanouts"], cfg["cache_width"], SEED,
                           cfg["shared"], THETA, max_seeds=cfg["batch"], max_requests=cap)
    if capacity:            # negative: the last rank is given other segment sizes than the rest
        me.set_capacities([abs(capacity) + (7 if capacity < 0 and rank == world - 1 else 0)] * (len(cfg["fanouts"]) + 1))
    seeds = batch_seeds(perm, 1, cfg["batch"], rank, world)
    outcome = "returned"
    try:
        sharded.sample_batch(me, seeds, ops.GS_MODE_OTF, 0.25, 1)
    except sharded.ShardedBatchError as e:
        outcome = "raised %d" % e.code
    with open(os.path.join(out_dir, "f%d.txt" % rank), "w") as fh:
        fh.write(outcome)
    dist.barrier()            # every rank is still alive and in step
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_a_failure_on_one_rank_ends_the_batch_on_every_rank(tmp_path, world):
    """An owner that cannot serve a list must not leave the others inside a collective: all ranks raise."""
    mp.spawn(_failing_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    for r in range(world):
        assert open(os.path.join(tmp_path, "f%d.txt" % r)).read() == "raised 2"


@pytest.mark.parametrize("world", [2, 3])
def test_a_group_that_outgrows_its_segment_ends_the_batch_on_every_rank(tmp_path, world):
    """Fixed-capacity exchanges: segments of 40 ids cannot hold the second hop's groups; nothing overruns, every
    exchange of the batch still takes place, and all ranks raise (a requester-side error: code 1)."""
    mp.spawn(_failing_worker, args=(world, _free_port(), str(tmp_path), 40), nprocs=world, join=True)
    for r in range(world):
        assert open(os.path.join(tmp_path, "f%d.txt" % r)).read() == "raised 1"


def test_ranks_with_different_capacities_are_told_before_any_exchange(tmp_path):
    """Equal-split exchanges of unequal buffers would hang or corrupt: the first batch compares the capacities."""
    mp.spawn(_failing_worker, args=(3, _free_port(), str(tmp_path), -920), nprocs=3, join=True)
    for r in range(3):
        assert open(os.path.join(tmp_path, "f%d.txt" % r)).read() == "raised 1"


@pytest.mark.parametrize("capacity,merge", [(None, None), (920, True), (920, False)])
def test_all_ranks_in_one_process_equal_one_sampler(capacity, merge):
    """The phase-by-phase driver (sharded.sample_batch_local, what a one-GPU check of a multi-rank run uses) with the
    oracle's primitives standing in for the kernels: exact-size and fixed-capacity exchanges, owners serving list by
    list and merged."""
    import fake_shard_ops as ops
    from paper_2406_17918_b200 import sharded

    cfg = get_config("tiny")
    g = build_graph(cfg)
    perm = seed_permutation(cfg)
    X = _features(cfg["num_nodes"])
    world, L = 3, len(cfg["fanouts"])
    ranks = []
    for r in range(world):
        ip, idx = sharded.shard_csr(g.indptr, g.indices, r, world)
        lo, hi = sharded.shard_range(cfg["num_nodes"], r, world)
        ranks.append(sharded.ShardRank(ops, r, world, ip, idx, X[lo:hi].contiguous(), cfg["fanouts"], cfg["cache_width"], SEED,
                                       cfg["shared"], THETA, max_seeds=cfg["batch"], max_requests=cfg["num_nodes"]))
        if capacity:
            ranks[-1].set_capacities([capacity] * (L + 1), merge=merge)
    O = oracle.Sampler(g.indptr.numpy(), g.indices.numpy(), cfg["fanouts"], cfg["cache_width"], SEED, cfg["shared"])
    O.set_theta(THETA)
    for t, (gm, om, rate) in enumerate([(ops.GS_MODE_OTF, oracle.MODE_OTF, 0.25), (ops.GS_MODE_FCR, oracle.MODE_FCR, 0.0),
                                        (ops.GS_MODE_OTF_FETCH, oracle.MODE_OTF_FETCH, 0.5)], start=1):
        seeds = [batch_seeds(perm, t, cfg["batch"], r, world) for r in range(world)]
        res = sharded.sample_batch_local(ranks, seeds, gm, rate, t)
        for r in range(world):
            blocks, frontier, n, m, feats = res[r]
            fr, n_o, blocks_o = O.sample_batch(seeds[r].numpy(), om, rate, t)
            assert n == n_o and np.array_equal(frontier[: n[L]].numpy(), fr)
            for l in range(L):
                assert np.array_equal(blocks[l].indptr(n[L - 1 - l]).numpy(), blocks_o[l].indptr)
                assert np.array_equal(blocks[l].indices(m[l]).numpy(), blocks_o[l].indices)
            assert torch.equal(feats, X[torch.from_numpy(fr.astype(np.int64))])


def test_refreshing_a_row_twice_in_one_step_equals_once():
    """Two ranks may ask an owner for the same node in the same step."""
    cfg = get_config("tiny")
    g = build_graph(cfg)
    indptr, indices = g.indptr.numpy(), g.indices.numpy()
    deg = indptr[1:] - indptr[:-1]
    W = cfg["cache_width"]
    a = oracle.Sampler(indptr, indices, cfg["fanouts"], W, 3)
    b = oracle.Sampler(indptr, indices, cfg["fanouts"], W, 3)
    nodes = np.nonzero(deg > W)[0][:200]
    for step, r in [(1, 3), (2, W), (3, 1), (4, 5)]:
        for v in nodes:
            a.refresh_node(0, v, step, r)
            b.refresh_node(0, v, step, r)
            b.refresh_node(0, v, step, r)
        assert np.array_equal(a.cache_rows(0, nodes), b.cache_rows(0, nodes))


def test_a_shard_gives_its_nodes_the_rows_of_the_whole_graph():
    """Keys use global node ids and a row's offsets, so an owner that holds only its CSR rows
    computes for them what a sampler over the whole graph computes."""
    from paper_2406_17918_b200 import sharded

    cfg = get_config("tiny")
    g = build_graph(cfg)
    W, N = cfg["cache_width"], cfg["num_nodes"]
    whole = oracle.Sampler(g.indptr.numpy(), g.indices.numpy(), cfg["fanouts"], W, 9)
    deg = (g.indptr[1:] - g.indptr[:-1]).numpy()
    world = 3
    for rank in range(world):
        ip, idx = sharded.shard_csr(g.indptr, g.indices, rank, world)
        lo, hi = sharded.shard_range(N, rank, world)
        d = (ip[1:] - ip[:-1]).numpy()
        assert (d[lo:hi] == deg[lo:hi]).all() and d[:lo].sum() == 0 and d[hi:].sum() == 0
        part = oracle.Sampler(ip.numpy(), idx.numpy(), cfg["fanouts"], W, 9)
        mine = np.arange(lo, hi)[deg[lo:hi] > W][:60]
        for v in mine:
            for s_ in (whole, part):
                s_.refresh_node(1, v, 4, 3)
            assert list(whole.pick_node(1, v, 4)) == list(part.pick_node(1, v, 4))
            assert list(whole.fbl_node(0, v, 2)) == list(part.fbl_node(0, v, 2))
        assert np.array_equal(whole.cache_rows(1, mine), part.cache_rows(1, mine))
    assert sharded.shard_range(10, 3, 4) == (9, 10) and sharded.rows_per_shard(10, 4) == 3
