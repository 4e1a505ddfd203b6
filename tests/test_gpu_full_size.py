"""Parity at the full sizes of the two large workloads, in the launch configuration the benchmark
times (needs a B200).  `large` is compared element by element on one whole batch; `scale`
(2^26 nodes, 2.1 G edges) on sampled nodes the oracle recomputes one by one, plus properties that
hold at any size."""
import numpy as np
import pytest
import torch

import oracle
from workloads import batch_seeds, build_features, build_graph, feature_rows, get_config, seed_permutation

pytestmark = pytest.mark.gpu


def test_large_one_whole_batch():
    from parity import Pair

    pair = Pair(get_config("large"), features=False)
    C, ws, O = pair.samplers(pair.cfg["batch"])
    rng = np.random.default_rng(3)
    hubs = np.argsort(-pair.deg)[:64]
    pair.check_rows(C, O, np.concatenate([hubs, rng.integers(0, pair.cfg["num_nodes"], 2000)]).astype(np.int32))
    seeds = batch_seeds(pair.perm, 0, pair.cfg["batch"])
    # the whole batch element by element; cache rows of 3,000 sampled frontier nodes, every layer
    pair.check_batch(C, ws, O, seeds, "otf", 0.2, 1, features=False, rows=3000)


def test_large_split_cache_whole_batch_then_whole_cache_refresh():
    """Dense/sparse split (theta = 32) at full size: one whole batch element by element, then the
    whole-cache refresh checked on sampled nodes the oracle refreshes one by one."""
    import paper_2406_17918_b200 as gs
    from parity import Pair

    pair = Pair(get_config("large"), features=False)
    theta = 32
    C, ws, O = pair.samplers(pair.cfg["batch"], theta=theta)
    full = gs.gs_cache_bytes(pair.G, pair.L, pair.W, False)
    assert C.storage.numel() < 0.6 * full
    seeds = batch_seeds(pair.perm, 0, pair.cfg["batch"])
    pair.check_batch(C, ws, O, seeds, "otf", 0.2, 1, features=False, rows=2000)
    rng = np.random.default_rng(11)
    dense = np.nonzero(pair.deg > theta)[0]
    nodes = np.concatenate([np.argsort(-pair.deg)[:16], rng.choice(dense, 1500, replace=False)]).astype(np.int32)
    for mode, gamma, step in (("otf", 0.2, 2), ("fcr", 0.0, 3)):
        gm, om = {"otf": (gs.GS_MODE_OTF, oracle.MODE_OTF), "fcr": (gs.GS_MODE_FCR, oracle.MODE_FCR)}[mode]
        gs.gs_cache_refresh_all(C, gm, gamma, step)
        gs.gs_sync_status(C)
        r = oracle.refresh_count(om, gamma, pair.W)
        for layer in range(pair.L):
            for v in nodes:
                O.refresh_node(layer, int(v), step, r)
        pair.check_rows(C, O, nodes)
    # a sparse node has no row, before and after
    sparse = np.nonzero(pair.deg <= theta)[0][:100].astype(np.int32)
    assert (gs.gs_cache_read_rows(C, 0, torch.from_numpy(sparse).cuda()).cpu().numpy() == -1).all()


def test_large_two_shards_two_steps():
    """Node-sharded sampling at full size: two ranks run phase by phase on this GPU; each rank's whole
    batch must equal what one sampler (theta = 32) gives when it takes the two batches in turn."""
    import paper_2406_17918_b200 as gs
    from paper_2406_17918_b200 import sharded

    cfg = get_config("large")
    g = build_graph(cfg)
    perm = seed_permutation(cfg)
    N, B, L, theta, seed, world = cfg["num_nodes"], cfg["batch"], len(cfg["fanouts"]), 32, 7, 2
    X = torch.arange(N, dtype=torch.float32).reshape(N, 1).repeat(1, 4).contiguous()    # row v holds v: cheap to check
    ranks = []
    for r in range(world):
        ip, idx = sharded.shard_csr(g.indptr, g.indices, r, world)
        lo, hi = sharded.shard_range(N, r, world)
        ranks.append(sharded.ShardRank(gs, r, world, ip.cuda(), idx.cuda(), X[lo:hi].cuda().contiguous(), cfg["fanouts"],
                                       cfg["cache_width"], seed, False, theta, max_seeds=B, max_requests=B * 6 * 11))
    O = oracle.Sampler(g.indptr.numpy(), g.indices.numpy(), cfg["fanouts"], cfg["cache_width"], seed, False)
    O.set_theta(theta)
    for step in (1, 2):
        if step == 2:
            # the second step with fixed-capacity exchanges sized from the first one, the owners merging the two
            # requesters' lists, and rank 1 finding first occurrences with the hash table
            seen = np.max([r.largest_groups() for r in ranks], axis=0)
            for r in ranks:
                r.set_capacities([int(c * 1.3) + 64 for c in seen], merge=True)
            gs.gs_cache_set_dedup(ranks[1].cache, gs.GS_DEDUP_HASH)
        seeds = [batch_seeds(perm, step, B, r, world) for r in range(world)]
        res = sharded.sample_batch_local(ranks, [s.cuda() for s in seeds], gs.GS_MODE_OTF, 0.2, step)
        for r in range(world):
            blocks, frontier, n, m, feats = res[r]
            fr_o, n_o, blocks_o = O.sample_batch(seeds[r].numpy(), oracle.MODE_OTF, 0.2, step)
            assert n == n_o
            assert np.array_equal(frontier[: n[L]].cpu().numpy(), fr_o)
            for layer in range(L):
                k = L - 1 - layer
                assert np.array_equal(blocks[layer].indptr(n[k]).cpu().numpy(), blocks_o[layer].indptr)
                assert np.array_equal(blocks[layer].indices(m[layer]).cpu().numpy(), blocks_o[layer].indices)
            assert torch.equal(feats[:, 0].cpu(), torch.from_numpy(fr_o.astype(np.float32)))


def _is_neighbour(indptr, indices, dst, src):
    """Vectorised binary search of src in the sorted CSR row of dst (all on the GPU)."""
    lo = indptr[dst]
    hi = indptr[dst + 1]
    for _ in range(32):
        mid = (lo + hi) // 2
        active = lo < hi
        val = indices[mid.clamp(max=indices.numel() - 1)]
        go_right = active & (val < src)
        hi = torch.where(active & ~go_right, mid, hi)
        lo = torch.where(go_right, mid + 1, lo)
    ok = lo < indptr[dst + 1]
    return ok & (indices[lo.clamp(max=indices.numel() - 1)] == src)


def test_scale_sampled_nodes_and_properties():
    import paper_2406_17918_b200 as gs

    cfg = get_config("scale")
    g = build_graph(cfg, device="cuda")
    X = build_features(cfg, device="cuda")
    perm = seed_permutation(cfg, device="cuda")
    fan, W, B, L = cfg["fanouts"], cfg["cache_width"], cfg["batch"], len(cfg["fanouts"])
    gamma = 0.1
    G = gs.gs_graph_create(g.indptr, g.indices, X)
    seed = 0x6A09E667F3BCC908
    C = gs.gs_cache_init(G, fan, W, seed, False)
    ws = torch.empty(gs.gs_workspace_bytes(G, fan, B), dtype=torch.uint8, device="cuda")
    deg = g.degrees()
    all_pre = {}
    rng = np.random.default_rng(5)

    # ---- S0 on sampled nodes (before any batch touches the cache)
    indptr_h, indices_h = g.indptr.cpu().numpy(), g.indices.cpu().numpy()
    O = oracle.Sampler(indptr_h, indices_h, fan, W, seed, False)
    cand = torch.nonzero((deg > W) & (deg < 20000)).flatten()
    pick = cand[torch.from_numpy(rng.integers(0, cand.numel(), 300)).cuda()]
    low = torch.from_numpy(rng.integers(0, cfg["num_nodes"], 300)).cuda()
    big = torch.topk(deg, 3).indices
    nodes = torch.cat([pick, low, big]).to(torch.int32)
    for l in range(L):
        got = gs.gs_cache_read_rows(C, l, nodes).cpu().numpy()
        assert np.array_equal(got, O.cache_rows(l, nodes.cpu().numpy()))

    # ---- one full-size batch on the GPU
    seeds = batch_seeds(perm, 0, B)
    blocks, input_nodes, cnt = gs.gs_sample_batch(C, seeds, gs.GS_MODE_OTF, gamma, 1, ws)
    n, m = gs.gs_batch_counts(C)
    r = oracle.refresh_count(oracle.MODE_OTF, gamma, W)
    frontier = input_nodes[: n[L]]
    fl = frontier.long()

    # properties that hold at any size
    assert torch.equal(frontier[:B], seeds)
    assert torch.unique(fl).numel() == n[L]                                # frontier ids are distinct
    for layer in range(L):
        k = L - 1 - layer
        ip = blocks[layer].indptr(n[k]).long()
        ix = blocks[layer].indices(m[layer]).long()
        assert int(ip[0]) == 0 and int(ip[-1]) == m[layer]
        assert torch.equal(ip[1:] - ip[:-1], torch.minimum(deg[fl[: n[k]]], torch.tensor(fan[layer], device="cuda")))
        assert int(ix.min()) >= 0 and int(ix.max()) < n[k + 1]
        # relabel: a new id's first appearance positions increase with its local id, and all new ids appear
        e = torch.arange(m[layer], device="cuda")
        first = torch.full((n[k + 1],), m[layer], dtype=torch.int64, device="cuda")
        first.scatter_reduce_(0, ix, e, reduce="amin")
        new_first = first[n[k]:]
        assert bool((new_first < m[layer]).all()) and bool((new_first[1:] > new_first[:-1]).all())
        # every block edge exists in the graph, and no neighbour repeats within a row (sampled edges)
        sel = torch.from_numpy(rng.integers(0, m[layer], 200000)).cuda()
        dst_pos = torch.searchsorted(ip, sel, right=True) - 1
        assert bool(_is_neighbour(g.indptr, g.indices, fl[dst_pos], fl[ix[sel]].to(torch.int32)).all())
    # sampled nodes, recomputed one by one by the oracle from the pre-sampled state
    for layer in range(L):
        k = L - 1 - layer
        ip = blocks[layer].indptr(n[k]).cpu().numpy()
        ix = blocks[layer].indices(m[layer]).cpu().numpy()
        fr = frontier.cpu().numpy()
        d = deg[fl[: n[k]]].cpu().numpy()
        ok = np.nonzero(d < 30000)[0]
        ps = np.concatenate([ok[rng.integers(0, len(ok), 250)], np.argsort(-d)[:2]])
        vs = fr[ps]
        rows_gpu = gs.gs_cache_read_rows(C, layer, torch.from_numpy(vs).cuda()).cpu().numpy()
        for p, v, row_gpu in zip(ps, vs, rows_gpu):
            O.refresh_node(layer, int(v), 1, r)
            assert np.array_equal(O.cache_row(layer, int(v)), row_gpu), (layer, int(v))
            assert np.array_equal(O.pick_node(layer, int(v), 1), fr[ix[ip[p]:ip[p + 1]]]), (layer, int(v))

    # S5 at full size: sampled rows against the feature function, the rest by checksum of a second gather
    out = torch.empty((n[L], cfg["feat_dim"]), dtype=X.dtype, device="cuda")
    gs.gs_gather_features(G, input_nodes, cnt, out)
    sel = torch.from_numpy(rng.integers(0, n[L], 5000)).cuda()
    want = feature_rows(cfg, fl[sel].cpu())
    got = out[sel].cpu()
    assert np.array_equal(got.view(torch.int16).numpy(), oracle.gather(want.view(torch.int16).numpy(), np.arange(5000, dtype=np.int32)))
    assert torch.equal(out.view(torch.int16), X[fl].view(torch.int16))


def test_scale_whole_batch_against_the_oracle():
    """A whole batch of the benchmarked configuration (8,192 seeds, OTF gamma = 0.1; the oracle needs about
    three minutes on one core), every output array element by element: the 2.0 M input nodes, block offsets
    and the 5.1 M block indices of all hops, the cache rows of 3,000 sampled frontier nodes at every layer,
    and the gathered feature rows of all input nodes."""
    import paper_2406_17918_b200 as gs
    from parity import Pair

    cfg = get_config("scale")
    g = build_graph(cfg, device="cuda")
    X = build_features(cfg, device="cuda")
    perm = seed_permutation(cfg, device="cuda")
    fan, W, L = cfg["fanouts"], cfg["cache_width"], len(cfg["fanouts"])
    B = cfg["batch"]
    seed = 0x6A09E667F3BCC908
    pair = Pair.__new__(Pair)
    pair.cfg, pair.L, pair.W, pair.shared, pair.X, pair.theta = cfg, L, W, False, None, None
    pair.G = gs.gs_graph_create(g.indptr, g.indices, X)
    C = gs.gs_cache_init(pair.G, fan, W, seed, False)
    ws = torch.empty(gs.gs_workspace_bytes(pair.G, fan, B), dtype=torch.uint8, device="cuda")
    O = oracle.Sampler(g.indptr.cpu().numpy(), g.indices.cpu().numpy(), fan, W, seed, False)
    seeds = batch_seeds(perm, 5, cfg["batch"])[:B]
    n, m = pair.check_batch(C, ws, O, seeds, "otf", 0.1, 1, features=False, rows=3000)
    assert n[L] > 1000000 and sum(m) > 4000000 and int(g.degrees().max()) > 500000
    # S5: every input node's row against the feature function, copied by the oracle's gather
    input_nodes = pair.last_input_nodes
    out = torch.empty((n[L], cfg["feat_dim"]), dtype=X.dtype, device="cuda")
    gs.gs_gather_features(pair.G, input_nodes, None, out)
    ids = input_nodes[: n[L]].cpu()
    want = feature_rows(cfg, ids.long()).view(torch.int16).numpy()
    assert np.array_equal(out.cpu().view(torch.int16).numpy(), oracle.gather(want, np.arange(n[L], dtype=np.int32)))
