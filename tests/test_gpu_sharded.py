"""Node-sharded sampling on one GPU (all ranks in one process, run phase by phase) vs the CPU oracle.

A sharded run must equal ONE sampler with the shards' dense/sparse split that takes the ranks'
batches of a step one after the other: every choice is keyed by (seed, node, item, step)."""
import numpy as np
import pytest
import torch

import oracle
from workloads import batch_seeds, build_features, build_graph, get_config, seed_permutation

pytestmark = pytest.mark.gpu

MODES = {"fcr": (0, oracle.MODE_FCR), "otf": (1, oracle.MODE_OTF), "fbl": (2, oracle.MODE_FBL),
         "fetch": (3, oracle.MODE_OTF_FETCH)}


class Setup:
    def __init__(self, name, world, theta, seed=5, B=None, fixed=False):
        import paper_2406_17918_b200 as gs
        from paper_2406_17918_b200 import sharded
        self.gs, self.sharded = gs, sharded
        cfg = self.cfg = get_config(name)
        g = build_graph(cfg)
        self.indptr, self.indices = g.indptr.numpy(), g.indices.numpy()
        self.deg = self.indptr[1:] - self.indptr[:-1]
        self.X = build_features(cfg)
        self.perm = seed_permutation(cfg)
        self.world, self.theta = world, theta
        self.B = B or cfg["batch"]
        N = cfg["num_nodes"]
        self.ranks = []
        for r in range(world):
            ip, idx = sharded.shard_csr(g.indptr, g.indices, r, world)
            lo, hi = sharded.shard_range(N, r, world)
            self.ranks.append(sharded.ShardRank(gs, r, world, ip.cuda(), idx.cuda(), self.X[lo:hi].cuda().contiguous(),
                                                cfg["fanouts"], cfg["cache_width"], seed, cfg["shared"], theta,
                                                max_seeds=self.B, max_requests=min(N, self.B * 400)))
        if fixed:   # fixed-capacity exchanges; a group holds distinct nodes of one owner, so a shard's size always suffices
            for r in self.ranks:    # owners merge the requesters' lists unless fixed == "lists"
                r.set_capacities([sharded.rows_per_shard(N, world)] * (len(cfg["fanouts"]) + 1), merge=fixed != "lists")   # merged serving also with one rank, for coverage
        self.O = oracle.Sampler(self.indptr, self.indices, cfg["fanouts"], cfg["cache_width"], seed, cfg["shared"])
        self.O.set_theta(theta)

    def step(self, mode, rate, t, features=True):
        gm, om = MODES[mode]
        L = len(self.cfg["fanouts"])
        seeds = [batch_seeds(self.perm, t, self.B, r, self.world) for r in range(self.world)]
        res = self.sharded.sample_batch_local(self.ranks, [s.cuda() for s in seeds], gm, rate, t, features=features)
        for r in range(self.world):
            blocks, frontier, n, m, feats = res[r]
            fr_o, n_o, blocks_o = self.O.sample_batch(seeds[r].numpy(), om, rate, t)
            assert n == n_o, (r, n, n_o)
            assert np.array_equal(frontier[: n[L]].cpu().numpy(), fr_o)
            for layer in range(L):
                k = L - 1 - layer
                assert m[layer] == blocks_o[layer].num_edges
                assert np.array_equal(blocks[layer].indptr(n[k]).cpu().numpy(), blocks_o[layer].indptr)
                assert np.array_equal(blocks[layer].indices(m[layer]).cpu().numpy(), blocks_o[layer].indices)
            if features:
                want = self.X[torch.from_numpy(fr_o.astype(np.int64))]
                assert torch.equal(feats.cpu().view(torch.int32 if want.element_size() == 4 else torch.int16),
                                   want.view(torch.int32 if want.element_size() == 4 else torch.int16))
        return res

    def check_rows(self, sample=None):
        """Cache rows of the dense nodes, read from their owners."""
        N = self.cfg["num_nodes"]
        nodes = np.nonzero(self.deg > self.theta)[0].astype(np.int32)
        if sample and len(nodes) > sample:
            nodes = np.sort(np.random.default_rng(1).choice(nodes, sample, replace=False))
        S = self.sharded.rows_per_shard(N, self.world)
        for layer in range(1 if self.cfg["shared"] else len(self.cfg["fanouts"])):
            want = self.O.cache_rows(layer, nodes)
            for r in range(self.world):
                mine = nodes[(nodes // S) == r]
                if len(mine) == 0:
                    continue
                got = self.gs.gs_cache_read_rows(self.ranks[r].cache, layer, torch.from_numpy(mine).cuda()).cpu().numpy()
                assert np.array_equal(got, want[(nodes // S) == r]), (layer, r)


@pytest.mark.parametrize("fixed", [False, True, "lists"])
@pytest.mark.parametrize("world", [1, 2, 3])
def test_sharded_tiny_all_modes(world, fixed):
    s = Setup("tiny", world, theta=12, fixed=fixed)
    t = 1
    for mode, rate in [("otf", 0.25), ("otf", 0.25), ("fcr", 0.0), ("fetch", 0.5), ("fbl", 0.0), ("otf", 0.0), ("otf", 1.0)]:
        s.step(mode, rate, t)
        t += 1
    s.check_rows()
    s.step("otf", 0.25, t, features="peer")     # the feature rows pulled from their owners by one kernel


def test_sharded_mid_and_shared_cache():
    s = Setup("mid", 4, theta=24, B=512)
    for t in (1, 2):
        s.step("otf", 0.3, t, features="peer" if t == 2 else True)
    s.step("fcr", 0.0, 3, features=False)
    s.check_rows(sample=4000)
    s = Setup("shared", 2, theta=32, B=1024)
    for t in (1, 2):
        s.step("otf", 0.3, t)
    s.check_rows(sample=4000)


def test_sharded_mid_fixed_capacity_exchanges():
    """Segments sized from an exact-size batch (the largest group seen, plus a margin), as a deployment would do."""
    s = Setup("mid", 3, theta=24, B=512)
    s.step("otf", 0.3, 1)
    seen = np.max([r.largest_groups() for r in s.ranks], axis=0)      # one entry per exchange: L hops + features
    caps = [int(c * 1.3) + 8 for c in seen]
    for r in s.ranks:
        r.set_capacities(caps)
    for t in (2, 3):
        s.step("otf", 0.3, t, features="peer" if t == 3 else True)
    s.step("fetch", 0.5, 4)
    s.check_rows(sample=4000)
    # segments that cannot hold the groups: the batch is reported as failed and nothing overruns
    for r in s.ranks:
        r.set_capacities([64] * len(caps))
    seeds = [batch_seeds(s.perm, 5, s.B, r, s.world).cuda() for r in range(s.world)]
    with pytest.raises(RuntimeError):
        s.sharded.sample_batch_local(s.ranks, seeds, 1, 0.3, 5)
    torch.cuda.synchronize()


def test_fixed_pitch_primitives():
    import paper_2406_17918_b200 as gs
    rng = np.random.default_rng(11)
    N, world, cap = 100003, 5, 13000
    S = (N + world - 1) // world
    full = torch.from_numpy(rng.choice(N, 60000, replace=False).astype(np.int32)).cuda()
    count = torch.tensor(41234, dtype=torch.int32, device="cuda")
    for cnt in (None, count):
        n = full.numel() if cnt is None else int(cnt.item())
        sorted_ids, slot, counts = gs.gs_shard_bucket(full, N, world, count=cnt, capacity=cap)
        v = full.cpu().numpy()[:n]
        c, so, sl = counts.cpu().numpy(), sorted_ids.cpu().numpy(), slot.cpu().numpy()[:n]
        owner = v // S
        assert sorted_ids.numel() == world * cap and c[2 * world] == 0
        assert np.array_equal(c[:world], np.bincount(owner, minlength=world))
        assert np.array_equal(sl // cap, owner) and (sl % cap < c[owner]).all()        # each id inside its owner's segment
        assert np.array_equal(so[sl], v) and len(np.unique(sl)) == n
    # a group larger than its segment: flagged, the surplus gets slot -1, nothing is written beyond the segment
    small = 7000
    out = (torch.full((world * small + 64,), -5, dtype=torch.int32, device="cuda"), torch.empty_like(full),
           torch.empty(2 * world + 1, dtype=torch.int32, device="cuda"))
    sorted_ids, slot, counts = gs.gs_shard_bucket(full, N, world, capacity=small, out=out)
    c, sl = counts.cpu().numpy(), slot.cpu().numpy()
    owner = full.cpu().numpy() // S
    assert c[2 * world] == 4 and (c[:world] > small).any()                                 # GS_ERR_WORKSPACE
    assert bool((sorted_ids[world * small:] == -5).all())
    for o in range(world):
        mine = sl[owner == o]
        assert (mine >= 0).sum() == min(small, c[o]) and ((mine < 0) | (mine // small == o)).all()
    # a device length above the bound: flagged as well
    long = torch.tensor(full.numel() + 1, dtype=torch.int32, device="cuda")
    assert gs.gs_shard_bucket(full, N, world, count=long, capacity=cap)[2].cpu().numpy()[2 * world] == 4
    assert gs.gs_shard_bucket(full, N, world, count=long)[2].cpu().numpy()[2 * world] == 4
    with pytest.raises(gs.GsError):
        gs.gs_shard_bucket(full, N, world, capacity=0)
    # owner side with the list's length on the device: the first *count rows equal the exact-size call, the rest is untouched
    s = Setup("tiny", 1, theta=12)
    me = s.ranks[0]
    nodes = torch.from_numpy(np.random.default_rng(2).choice(s.cfg["num_nodes"], 300, replace=False).astype(np.int32)).cuda()
    f = me.fanouts[0]
    want = gs.gs_shard_sample_rows(me.cache, nodes[:211].contiguous(), 0, gs.GS_MODE_FBL, 0.0, 3, me.ws_owner)
    got = torch.full((300, f), -9, dtype=torch.int32, device="cuda")
    gs.gs_shard_sample_rows(me.cache, nodes, 0, gs.GS_MODE_FBL, 0.0, 3, me.ws_owner, picks=got,
                            count=torch.tensor([211], dtype=torch.int32, device="cuda"))
    gs.gs_shard_status(me.cache)
    assert torch.equal(got[:211], want) and bool((got[211:] == -9).all())
    gs.gs_shard_sample_rows(me.cache, nodes, 0, gs.GS_MODE_FBL, 0.0, 3, me.ws_owner, picks=got,
                            count=torch.tensor([0], dtype=torch.int32, device="cuda"))       # an empty list
    gs.gs_shard_status(me.cache)
    assert torch.equal(got[:211], want)


def test_bucket_and_gather_rows_primitives():
    import paper_2406_17918_b200 as gs
    rng = np.random.default_rng(3)
    N, world = 100003, 7
    nodes = torch.from_numpy(rng.choice(N, 50001, replace=False).astype(np.int32)).cuda()
    sorted_ids, slot, counts = gs.gs_shard_bucket(nodes, N, world)
    S = (N + world - 1) // world
    c = counts.cpu().numpy()
    owner = (nodes.cpu().numpy() // S)
    assert c[2 * world] == 0 and np.array_equal(c[:world], np.bincount(owner, minlength=world))
    so = sorted_ids.cpu().numpy()
    assert np.array_equal(so // S, np.sort(owner))                              # grouped by owner
    assert np.array_equal(so[slot.cpu().numpy()], nodes.cpu().numpy())          # slot ties each id to its place
    assert len(np.unique(slot.cpu().numpy())) == nodes.numel()
    bad = nodes.clone()
    bad[17] = N + 5 * S
    assert gs.gs_shard_bucket(bad, N, world)[2].cpu().numpy()[2 * world] == 3   # GS_ERR_RANGE
    # rows of a shard addressed by global ids
    X = torch.randn(1000, 24, device="cuda").to(torch.bfloat16)
    ids = torch.from_numpy(rng.integers(400, 700, 333).astype(np.int32)).cuda()
    out = torch.empty((333, 24), dtype=torch.bfloat16, device="cuda")
    gs.gs_gather_rows(X[400:700], ids, out, first_row=400)
    assert torch.equal(out, X[ids.long()])
    # ids outside the rows the source holds are skipped
    ids2 = ids.clone()
    ids2[3], ids2[4], ids2[5] = 399, 700, -2
    out2 = torch.full((333, 24), 9, dtype=torch.bfloat16, device="cuda")
    gs.gs_gather_rows(X[400:700], ids2, out2, first_row=400)
    keep = torch.ones(333, dtype=torch.bool, device="cuda")
    keep[3:6] = False
    assert torch.equal(out2[keep], X[ids2[keep].long()]) and bool((out2[~keep] == 9).all())
    # the same matrix as three shards of ceil(1000/3) rows, each at its own address
    parts = [X[0:334].clone(), X[334:668].clone(), X[668:1000].clone()]
    ids = torch.from_numpy(rng.integers(0, 1000, 4001).astype(np.int32)).cuda()
    ids[5] = -1
    ids[6] = 1000
    out = torch.full((4001, 24), 7, dtype=torch.bfloat16, device="cuda")
    gs.gs_gather_rows_peer([p.data_ptr() for p in parts], 1000, torch.bfloat16, 24, 24, ids, out)
    ok = (ids >= 0) & (ids < 1000)
    assert torch.equal(out[ok], X[ids[ok].long()]) and bool((out[~ok] == 7).all())
    with pytest.raises(gs.GsError):
        gs.gs_gather_rows_peer([parts[0].data_ptr(), 0, parts[2].data_ptr()], 1000, torch.bfloat16, 24, 24, ids, out)


def test_merge_and_fan_out_primitives():
    import paper_2406_17918_b200 as gs
    rng = np.random.default_rng(21)
    world, C, first, owned, f = 4, 5000, 70000, 30011, 7
    lists = torch.full((world * C,), -3, dtype=torch.int32)
    cnt = [4100, 0, 5000, 777]
    hot = rng.choice(owned, 600, replace=False) + first                       # nodes every requester asks for
    for r in range(world):
        rest = rng.choice(owned, cnt[r], replace=False) + first
        v = np.unique(np.concatenate([hot[: min(600, cnt[r])], rest]))[: cnt[r]] if cnt[r] else rest
        lists[r * C: r * C + cnt[r]] = torch.from_numpy(rng.permutation(v).astype(np.int32))
    lists_d, counts = lists.cuda(), torch.tensor(cnt, dtype=torch.int32, device="cuda")
    index = torch.full((owned,), -1, dtype=torch.int32, device="cuda")
    D = min(world * C, owned)
    distinct = torch.empty(D, dtype=torch.int32, device="cuda")
    num = torch.zeros(2, dtype=torch.int32, device="cuda")
    gs.gs_shard_merge(lists_d, counts, world, first, index, distinct, num)
    asked = np.unique(np.concatenate([lists.numpy()[r * C: r * C + cnt[r]] for r in range(world)]))
    n = int(num[0].item())
    got = distinct[:n].cpu().numpy()
    assert int(num[1].item()) == 0 and n == len(asked) and np.array_equal(np.sort(got), asked)
    idx = index.cpu().numpy()
    assert np.array_equal(idx[got - first], np.arange(n)) and (np.delete(idx, asked - first) == -1).all()
    rows = torch.from_numpy(rng.integers(0, 1 << 30, (D, f)).astype(np.int32)).cuda()
    out = torch.full((world * C, f), -8, dtype=torch.int32, device="cuda")
    gs.gs_shard_fan_out(lists_d, counts, world, first, index, distinct, num, rows, out)
    want = np.full((world * C, f), -8, dtype=np.int32)
    rows_h = rows.cpu().numpy()
    for r in range(world):
        ids = lists.numpy()[r * C: r * C + cnt[r]]
        want[r * C: r * C + cnt[r]] = rows_h[idx[ids - first]]
    assert np.array_equal(out.cpu().numpy(), want)
    assert bool((index == -1).all())                                            # ready for the next hop
    # an id this shard does not own: reported, skipped, the others are placed
    bad = lists_d.clone()
    bad[3] = first + owned
    gs.gs_shard_merge(bad, counts, world, first, index, distinct, num)
    assert num.cpu().tolist() == [len(asked) - 1 if lists[3].item() not in np.concatenate(
        [lists.numpy()[r * C: r * C + cnt[r]] for r in range(1, world)] + [lists.numpy()[:3], lists.numpy()[4:cnt[0]]]) else len(asked), 3]
    gs.gs_shard_fan_out(bad, counts, world, first, index, distinct, num, rows, out)
    assert bool((index == -1).all())
    with pytest.raises(gs.GsError):
        gs.gs_shard_merge(lists_d[: 65 * 300], torch.zeros(65, dtype=torch.int32, device="cuda"), 65, first, index, distinct, num)


def test_sharded_entry_points_reject_bad_arguments():
    import paper_2406_17918_b200 as gs
    s = Setup("tiny", 2, theta=12)
    me = s.ranks[0]
    nodes = torch.arange(0, 8, dtype=torch.int32, device="cuda")
    picks_ws = me.ws_owner
    for bad in [dict(layer=5), dict(layer=-1), dict(mode=9), dict(rate=1.5, mode=gs.GS_MODE_OTF), dict(step=0)]:
        kw = dict(layer=0, mode=gs.GS_MODE_OTF, rate=0.25, step=1)
        kw.update(bad)
        with pytest.raises(gs.GsError):
            gs.gs_shard_sample_rows(me.cache, nodes, kw["layer"], kw["mode"], kw["rate"], kw["step"], picks_ws)
    with pytest.raises(gs.GsError) as e:
        gs.gs_shard_sample_rows(me.cache, nodes, 0, gs.GS_MODE_OTF, 0.25, 1, picks_ws[:256])
    assert e.value.status == 4                                           # GS_ERR_WORKSPACE
    assert gs.gs_shard_sample_rows(me.cache, nodes[:0], 0, gs.GS_MODE_OTF, 0.25, 1, picks_ws).shape == (0, me.fanouts[0])
    # a node id that is not a node: reported by the status call, nothing else breaks
    bad_nodes = torch.tensor([1, 2, s.cfg["num_nodes"] + 7], dtype=torch.int32, device="cuda")
    gs.gs_shard_sample_rows(me.cache, bad_nodes, 0, gs.GS_MODE_OTF, 0.25, 1, picks_ws)
    with pytest.raises(gs.GsError) as e:
        gs.gs_shard_status(me.cache)
    assert e.value.status == 3                                           # GS_ERR_RANGE
    gs.gs_shard_sample_rows(me.cache, nodes, 0, gs.GS_MODE_OTF, 0.25, 1, picks_ws)
    gs.gs_shard_status(me.cache)                                         # the next call starts clean
    # requester side: hops in order, starting at 0
    reply = torch.full((8, me.fanouts[-1]), -1, dtype=torch.int32, device="cuda")
    slot = torch.arange(8, dtype=torch.int32, device="cuda")
    fresh = Setup("tiny", 1, theta=12).ranks[0]
    with pytest.raises(gs.GsError):
        gs.gs_shard_extend(fresh.cache, 1, None, reply, slot, fresh.ws)          # hop 1 before hop 0
    with pytest.raises(gs.GsError):
        gs.gs_shard_extend(fresh.cache, 0, None, reply, slot, fresh.ws)          # hop 0 without seeds
    with pytest.raises(gs.GsError):
        gs.gs_shard_extend(fresh.cache, 7, nodes, reply, slot, fresh.ws)
    # all rows empty: every block is empty, the frontier is the seeds
    block, frontier = gs.gs_shard_extend(fresh.cache, 0, nodes, reply, slot, fresh.ws)
    n, m = gs.gs_batch_counts(fresh.cache)
    assert n[:2] == [8, 8] and m[-1] == 0 and torch.equal(frontier[:8], nodes)
    # a slot that is not a row of the reply, a pick that is not a node: reported, nothing is read or written out of bounds
    for bad_slot, bad_pick in ((True, False), (False, True)):
        other = Setup("tiny", 1, theta=12).ranks[0]
        sl, rp = slot.clone(), reply.clone()
        if bad_slot:
            sl[2] = 8
        if bad_pick:
            rp[3, 0] = s.cfg["num_nodes"]
        gs.gs_shard_extend(other.cache, 0, nodes, rp, sl, other.ws)
        with pytest.raises(gs.GsError) as e:
            gs.gs_batch_counts(other.cache)
        assert e.value.status == 3
    with pytest.raises(gs.GsError):
        gs.gs_shard_bucket(nodes, 100, 65)
    with pytest.raises(gs.GsError):
        X = torch.zeros((4, 8), device="cuda")
        gs.gs_gather_rows(X, nodes, torch.zeros((8, 4), device="cuda"))              # output rows narrower than the source rows


@pytest.mark.parametrize("case", range(16))
def test_randomised_sharded_runs(case):
    """Seeded random graphs, world sizes, shapes, modes and rates; every rank's batch against one oracle sampler."""
    import paper_2406_17918_b200 as gs
    from paper_2406_17918_b200 import sharded
    from test_gpu_parity import _random_graph

    rng = np.random.default_rng(5000 + case)
    indptr, indices = _random_graph(rng)
    n = len(indptr) - 1
    world = int(rng.integers(1, 6))
    L = int(rng.integers(1, 4))
    W = int(rng.choice([2, 8, 20, 32]))
    fanouts = [int(rng.integers(1, W + 1)) for _ in range(L)]
    shared = bool(rng.random() < 0.3)
    theta = int(rng.integers(W, 129))
    seed = int(rng.integers(1, 2**63))
    ip_t, ix_t = torch.from_numpy(indptr), torch.from_numpy(indices)
    X = torch.arange(n, dtype=torch.float32).reshape(n, 1).repeat(1, 4).contiguous()
    B = int(rng.integers(1, min(n // world, 100) + 1))
    ranks = []
    for r in range(world):
        ip, idx = sharded.shard_csr(ip_t, ix_t, r, world)
        lo, hi = sharded.shard_range(n, r, world)
        ranks.append(sharded.ShardRank(gs, r, world, ip.cuda(), idx.cuda(), X[lo:hi].cuda().contiguous(), fanouts, W, seed,
                                       shared, theta, max_seeds=B, max_requests=n))
        if case % 2:            # odd cases: fixed-capacity exchanges (a shard's size always holds a group)
            ranks[-1].set_capacities([sharded.rows_per_shard(n, world)] * (L + 1), merge=case % 4 == 1)
        # the requester's dedup + relabel with each way of finding first occurrences
        gs.gs_cache_set_dedup(ranks[-1].cache, [gs.GS_DEDUP_AUTO, gs.GS_DEDUP_HASH, gs.GS_DEDUP_SORT, gs.GS_DEDUP_DIRECT][(case // 2) % 4])
    O = oracle.Sampler(indptr, indices, fanouts, W, seed, shared)
    O.set_theta(theta)
    step = int(rng.integers(1, 2**32 - 10))
    for b in range(3):
        mode = str(rng.choice(["otf", "otf", "fcr", "fetch", "fbl"]))
        rate = float(rng.choice([0.0, 0.1, 0.25, 0.5, 1.0]))
        gm, om = MODES[mode]
        pool = rng.permutation(n)[: world * B].astype(np.int32)                 # the ranks' seeds may not overlap within a rank
        seeds = [torch.from_numpy(pool[r * B:(r + 1) * B].copy()) for r in range(world)]
        res = sharded.sample_batch_local(ranks, [s_.cuda() for s_ in seeds], gm, rate, step + b,
                                         features="peer" if rng.random() < 0.5 else True)
        for r in range(world):
            blocks, frontier, nn, m, feats = res[r]
            fr_o, n_o, blocks_o = O.sample_batch(seeds[r].numpy(), om, rate, step + b)
            assert nn == n_o and np.array_equal(frontier[: nn[L]].cpu().numpy(), fr_o)
            for layer in range(L):
                k = L - 1 - layer
                assert np.array_equal(blocks[layer].indptr(nn[k]).cpu().numpy(), blocks_o[layer].indptr)
                assert np.array_equal(blocks[layer].indices(m[layer]).cpu().numpy(), blocks_o[layer].indices)
            assert torch.equal(feats[:, 0].cpu(), torch.from_numpy(fr_o.astype(np.float32)))
    # the owners' rows, dense part
    deg = np.diff(indptr)
    dense = np.nonzero(deg > theta)[0].astype(np.int32)
    S = sharded.rows_per_shard(n, world)
    for layer in range(1 if shared else L):
        want = O.cache_rows(layer, dense)
        for r in range(world):
            sel = (dense // S) == r
            if sel.any():
                got = gs.gs_cache_read_rows(ranks[r].cache, layer, torch.from_numpy(dense[sel]).cuda()).cpu().numpy()
                assert np.array_equal(got, want[sel])
