"""A CPU stand-in for the binding's sharded entry points, built from the oracle's per-node
primitives: lets the multi-rank drivers of `paper_2406_17918_b200.sharded` run under gloo
without a GPU.  Test infrastructure only."""
import numpy as np
import torch

import oracle

GS_MODE_FCR, GS_MODE_OTF, GS_MODE_FBL, GS_MODE_OTF_FETCH = 0, 1, 2, 3
_OM = {0: oracle.MODE_FCR, 1: oracle.MODE_OTF, 2: oracle.MODE_FBL, 3: oracle.MODE_OTF_FETCH}


class _Graph:
    def __init__(self, indptr, indices):
        self.indptr, self.indices = indptr.numpy().copy(), indices.numpy().copy()
        self.deg = self.indptr[1:] - self.indptr[:-1]


class _Block:
    def __init__(self, indptr, indices, num_src=0):
        self._indptr, self._indices = indptr, indices
        self._counts = (len(indptr) - 1, num_src, len(indices))

    def counts_device(self):
        return tuple(torch.tensor(c, dtype=torch.int32) for c in self._counts)

    def indptr(self, n):
        return torch.from_numpy(self._indptr[: n + 1])

    def indices(self, m):
        return torch.from_numpy(self._indices[:m])


class _Cache:
    pass


def gs_graph_create(indptr, indices, features):
    return _Graph(indptr, indices)


def gs_cache_init_split(graph, fanouts, W, seed, shared, theta):
    c = _Cache()
    c.graph, c.fanouts, c.W, c.theta = graph, list(fanouts), W, theta
    c.O = oracle.Sampler(graph.indptr, graph.indices, fanouts, W, seed, shared)
    c.O.set_theta(theta)
    return c


def gs_workspace_bytes(graph, fanouts, max_seeds):
    return 256


def gs_shard_workspace_bytes(graph, fanout, max_nodes):
    return 256


def gs_shard_bucket(nodes, num_nodes, world, count=None, capacity=None, out=None):
    v = nodes.numpy() if count is None else nodes.numpy()[: int(count)]
    S = (num_nodes + world - 1) // world
    owner = v // S
    order = np.argsort(owner, kind="stable")
    counts = np.zeros(2 * world + 1, dtype=np.int32)
    counts[:world] = np.bincount(owner, minlength=world)
    slot = np.zeros(nodes.numel(), dtype=np.int32)
    if capacity is None:
        slot[order] = np.arange(len(v), dtype=np.int32)
        sorted_ids = np.zeros(nodes.numel(), dtype=np.int32)
        sorted_ids[: len(v)] = v[order]
    else:                                   # every owner's group in a segment of `capacity` ids; the surplus is dropped
        sorted_ids = np.full(world * capacity, -7, dtype=np.int32)
        starts = np.concatenate([[0], np.cumsum(counts[:world])])
        rank_in_group = np.arange(len(v)) - starts[owner[order]]
        pos = np.where(rank_in_group < capacity, owner[order] * capacity + rank_in_group, -1).astype(np.int32)
        slot[order] = pos
        sorted_ids[pos[pos >= 0]] = v[order][pos >= 0]
        if (pos < 0).any():
            counts[2 * world] = 4          # GS_ERR_WORKSPACE
    res = (torch.from_numpy(sorted_ids), torch.from_numpy(slot), torch.from_numpy(counts))
    if out is not None:
        for dst, src in zip(out, res):
            dst[: src.numel()].copy_(src)
        return out
    return res


def gs_shard_sample_rows(cache, nodes, layer, mode, rate, step, ws, picks=None, count=None):
    f = cache.fanouts[layer]
    ids = nodes.numpy() if count is None else nodes.numpy()[: int(count)]
    out = np.full((len(ids), f), -1, dtype=np.int32)
    O, om = cache.O, _OM[mode]
    for i, v in enumerate(ids.tolist()):
        if om == oracle.MODE_FBL or cache.graph.deg[v] <= cache.theta:
            row = O.fbl_node(layer, v, step)
        elif om == oracle.MODE_OTF_FETCH:
            row = O.fetch_node(layer, v, step, oracle.fetch_count(rate, f))
        else:
            O.refresh_node(layer, v, step, oracle.refresh_count(om, rate, cache.W))
            row = O.pick_node(layer, v, step)
        out[i, : len(row)] = row
    if picks is not None:                   # only the list's rows are written
        picks[: len(ids)].copy_(torch.from_numpy(out))
        return picks
    return torch.from_numpy(out)


def gs_shard_merge(lists, counts, world, first_row, index, distinct, num_distinct):
    C = lists.numel() // world
    L, cnt, idx = lists.numpy(), counts.numpy(), index.numpy()
    assert (idx == -1).all()
    n, bad = 0, 0
    for r in range(world):
        for v in L[r * C: r * C + min(int(cnt[r]), C)].tolist():
            loc = v - first_row
            if loc < 0 or loc >= len(idx):
                bad = 3
            elif idx[loc] < 0:
                idx[loc] = n
                distinct[n] = v
                n += 1
    num_distinct[0], num_distinct[1] = n, bad
    return distinct, num_distinct


def gs_shard_fan_out(lists, counts, world, first_row, index, distinct, num_distinct, rows, out):
    C = lists.numel() // world
    L, cnt, idx = lists.numpy(), counts.numpy(), index.numpy()
    for r in range(world):
        for i in range(min(int(cnt[r]), C)):
            loc = L[r * C + i] - first_row
            if 0 <= loc < len(idx):
                out[r * C + i] = rows[idx[loc]]
    for v in distinct[: int(num_distinct[0])].tolist():
        idx[v - first_row] = -1
    return out


def gs_shard_status(cache):
    pass


def gs_shard_extend(cache, k, seeds, reply, slot, ws, reply_rows=None):
    L = len(cache.fanouts)
    if k == 0:
        cache.frontier = seeds.numpy().tolist()
        cache.pos = {v: i for i, v in enumerate(cache.frontier)}
        cache.n, cache.m = [len(cache.frontier)], [0] * L
    rows, sl = reply.numpy(), slot.numpy()
    n_k = cache.n[k]
    indptr, local = [0], []
    for p in range(n_k):
        if sl[p] < 0:                       # dropped by a full segment: no picks (the batch is reported as failed)
            indptr.append(len(local))
            continue
        for u in rows[sl[p]]:
            if u < 0:
                break
            if u not in cache.pos:
                cache.pos[int(u)] = len(cache.frontier)
                cache.frontier.append(int(u))
            local.append(cache.pos[int(u)])
        indptr.append(len(local))
    cache.n.append(len(cache.frontier))
    cache.m[L - 1 - k] = len(local)
    return _Block(np.array(indptr, dtype=np.int32), np.array(local, dtype=np.int32), len(cache.frontier)), \
        torch.tensor(cache.frontier, dtype=torch.int32)


def gs_batch_counts(cache):
    return list(cache.n), list(cache.m)


def gs_gather_rows(src, ids, out, first_row=0, count=None):
    n = min(out.shape[0], ids.numel()) if count is None else min(int(count), out.shape[0], ids.numel())
    idx = ids[:n].long() - first_row
    ok = (idx >= 0) & (idx < src.shape[0])  # an id outside the source leaves its output row as it is
    out[:n][ok] = src[idx[ok]]
    return out
