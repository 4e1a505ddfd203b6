"""Node-sharded sampling over several GPUs: one exchange per hop.

Nodes are partitioned by id range; rank o owns the CSR rows, cache rows and feature rows of
``[o*S, (o+1)*S)``, ``S = ceil(N / world)``.  Every random choice of the sampler is keyed by
(seed, node, item, step), so the picks an owner computes for a node are the picks a single
device would compute, and a sharded run equals one sampler (with the dense/sparse split the
shards' caches use) that takes the ranks' batches of a step one after the other.

One hop of a rank's batch (sampling step k, layer L-1-k):

    bucket frontier_k by owner  ->  all-to-all(v) ids  ->  owners refresh + pick
                                <-  all-to-all(v) rows of f picks  <-
    dedup + relabel + block CSR

and after the last hop one more round trip for the feature rows (or one kernel that pulls them from the
owners' memory).  The exchanges come in two forms: packed groups whose sizes the host reads back for the
all-to-all (one host sync per hop), or segments of a fixed capacity per pair of ranks whose sizes travel
as a device array (:meth:`ShardRank.set_capacities`: no host read inside a batch; owners then merge the
requesters' lists and sample every distinct node once).  The per-rank phases live in
:class:`ShardRank`; two drivers run them: :func:`sample_batch` (one process per GPU, the
exchange is ``torch.distributed.all_to_all_single`` over NCCL / NVLink) and
:func:`sample_batch_local` (all ranks in one process, the exchange is a copy; used to check a
multi-rank run on one GPU - the ranks' kernels run one after the other, nothing waits).
This module only moves arguments: every step of the path runs in the library's kernels
(``ops`` is the binding; tests may pass a stand-in with the same functions).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def rows_per_shard(num_nodes: int, world: int) -> int:
    return (num_nodes + world - 1) // world


def shard_range(num_nodes: int, rank: int, world: int):
    s = rows_per_shard(num_nodes, world)
    return min(num_nodes, rank * s), min(num_nodes, (rank + 1) * s)


def shard_csr(indptr: torch.Tensor, indices: torch.Tensor, rank: int, world: int):
    """The shard's CSR: full-length indptr in which only the owned rows are non-empty, and the
    owned rows' neighbour ids (global)."""
    n = indptr.numel() - 1
    lo, hi = shard_range(n, rank, world)
    e0, e1 = int(indptr[lo].item()), int(indptr[hi].item())
    ip = torch.empty_like(indptr)
    ip[: lo + 1] = 0
    ip[lo:hi + 1] = indptr[lo:hi + 1] - e0
    ip[hi + 1:] = e1 - e0
    return ip.contiguous(), indices[e0:e1].contiguous()


class ShardRank:
    """One rank of a sharded run: its shard's graph, split cache, feature rows and workspaces."""

    def __init__(self, ops, rank, world, indptr_shard, indices_shard, features_shard, fanouts, cache_width, seed,
                 shared, theta, max_seeds, max_requests):
        self.ops, self.rank, self.world = ops, rank, world
        self.num_nodes = indptr_shard.numel() - 1
        self.first_row = shard_range(self.num_nodes, rank, world)[0]
        self.fanouts, self.L = list(fanouts), len(fanouts)
        self.features = features_shard
        self.graph = ops.gs_graph_create(indptr_shard, indices_shard, None)
        self.cache = ops.gs_cache_init_split(self.graph, fanouts, cache_width, seed, shared, theta)
        dev = indptr_shard.device
        self.ws = torch.empty(ops.gs_workspace_bytes(self.graph, fanouts, max_seeds), dtype=torch.uint8, device=dev)
        self.max_requests = max_requests
        self.ws_owner = torch.empty(ops.gs_shard_workspace_bytes(self.graph, max(fanouts), max_requests),
                                    dtype=torch.uint8, device=dev)
        self.blocks = [None] * self.L
        self.n = []
        self.caps = None                           # fixed-capacity exchanges: see set_capacities
        self.merge_exact = world > 1               # exact-size exchanges: owners merge the requesters' lists too
        self.exact_index = None                    # one word per owned row, -1 between hops (allocated on first use)
        self.exact_merge_status = []

    # ---- requester side
    # The host learns the size of a frontier only from the group sizes it has to read back for the exchange
    # anyway (one host sync per hop): the bucket kernel takes the frontier's length from the device, the
    # batch's counts and device status are read once, at the end of the batch.
    def begin(self, seeds):
        self.seeds = seeds
        self.frontier, self.n = seeds, [seeds.numel()]
        self.count_dev = None                      # device scalar with the current frontier's length
        self.blocks = [None] * self.L
        self.m = [0] * self.L
        self.seen = []                             # exact-size mode: the largest group of every exchange so far
        self.feat_bound = None

    def requests(self, nodes, count=None):
        """Bucket `nodes` (all of it, or its first *count ids) by owner -> (ids grouped by owner, group sizes
        as a list); remembers the slots."""
        if count is None:
            sorted_ids, self.slot, counts = self.ops.gs_shard_bucket(nodes, self.num_nodes, self.world)
        else:
            sorted_ids, self.slot, counts = self.ops.gs_shard_bucket(nodes, self.num_nodes, self.world, count=count)
        c = counts.cpu().tolist()                      # the all-to-all needs the sizes on the host
        if c[2 * self.world] != 0:
            raise ValueError("a node id is outside [0, num_nodes)" if c[2 * self.world] == 3 else
                             "the frontier is longer than the bound it was bucketed with")
        total = sum(c[: self.world])
        self.seen.append(max(c[: self.world]))     # largest group of this exchange: what a fixed capacity has to hold
        return sorted_ids[:total], c[: self.world]

    def _frontier_bound(self, k):
        """Upper bound of n_k from the last size the host knows."""
        if k == 0:
            return self.n[0]
        layer_before = self.L - k              # fan-out of sampling step k - 1
        return min(self.num_nodes, self.n[k - 1] * (1 + self.fanouts[layer_before]))

    def hop_requests(self, k):
        bound = self._frontier_bound(k)
        ids, counts = self.requests(self.frontier[:bound], self.count_dev)
        if k > 0:
            self.n.append(sum(counts))             # n_k
        return ids, counts

    def hop_finish(self, k, reply):
        """`reply`: [n_k, f] rows of picks in the order the requests were sent."""
        block, frontier = self.ops.gs_shard_extend(self.cache, k, self.seeds if k == 0 else None, reply, self.slot, self.ws)
        self.blocks[self.L - 1 - k] = block
        self.frontier = frontier
        self.count_dev = block.counts_device()[1]  # n_{k+1}, on the device

    def feature_requests(self):
        ids, counts = self.requests(self.frontier[: self._frontier_bound(self.L)], self.count_dev)
        self.n.append(sum(counts))                 # n_L
        return ids, counts

    def finish_batch(self):
        """Counts and device status of the batch, read once (synchronises)."""
        n, m = self.ops.gs_batch_counts(self.cache)
        self.n, self.m = list(n), list(m)
        self.ops.gs_shard_status(self.cache)       # the lists this rank served
        merged, self.exact_merge_status = self.exact_merge_status, []
        if merged and any(int(w[1]) for w in merged):
            raise ValueError("a requested node id is not a row of this shard")

    def feature_pull(self, shard_bases, bound=None):
        """The feature step as one kernel: every input node's row is read straight from its owner's
        memory (`shard_bases[o]`: device address of rank o's feature rows, peer-mapped where o is another GPU).
        `bound`: rows to allocate for when the host does not know the last hop's size."""
        if bound is None:
            bound = self._frontier_bound(self.L) if self.caps is None else self._product_bound(self.L)
        out = torch.empty((bound, self.features.shape[1]), dtype=self.features.dtype, device=self.features.device)
        self.feat_bound = bound
        return self.ops.gs_gather_rows_peer(shard_bases, self.num_nodes, self.features.dtype, self.features.shape[1],
                                            self.features.stride(0), self.frontier[:bound], out, count=self.count_dev)

    def feature_finish(self, rows):
        out = torch.empty((self.n[self.L], rows.shape[1]), dtype=rows.dtype, device=rows.device)
        return self.ops.gs_gather_rows(rows, self.slot[: self.n[self.L]], out)

    # ---- the same phases with fixed-capacity exchanges: no size ever goes through the host
    # Every (requester, owner) pair gets a segment of caps[k] ids at hop k (caps[L]: the feature request), the
    # group sizes travel as a device array beside the ids, owners take each list's length from there, and the
    # replies come back at the same pitch.  The exchanges are equal-split all-to-alls of pre-allocated buffers,
    # so a batch has no host synchronisation before finish_batch.  A group that outgrows its segment is a
    # device-detected error of the batch (reported by finish_batch), never an overrun.
    def set_capacities(self, caps, merge=None):
        """caps[0..L-1]: ids per (requester, owner) pair at each hop; caps[L]: at the feature request (omit or 0
        when features are pulled from peer memory).  Every rank must use the same values.
        merge: the owner merges the requesters' lists of a hop and samples every distinct node once (a hub sits
        in every requester's frontier) instead of serving the lists one by one; same rows either way.  Default: with
        more than one rank (with one there is nothing to merge, only the cost of doing it)."""
        if merge is None:
            merge = self.world > 1
        self.caps_agreed = False                   # checked against the other ranks by the first batch
        caps = [int(c) for c in caps] + [0] * (self.L + 1 - len(caps))
        if len(caps) != self.L + 1 or min(caps[: self.L]) < 1:
            raise ValueError("one positive capacity per hop (and optionally one for the features) expected")
        R, dev = self.world, self.features.device
        self.caps = caps
        need = min(self.num_nodes, max(caps[: self.L]))
        if need > self.max_requests:
            self.max_requests = need
            self.ws_owner = torch.empty(self.ops.gs_shard_workspace_bytes(self.graph, max(self.fanouts), need),
                                        dtype=torch.uint8, device=dev)
        i32 = dict(dtype=torch.int32, device=dev)
        lo, hi = shard_range(self.num_nodes, self.rank, self.world)
        self.merge = bool(merge) and hi > lo
        if self.merge:
            D = min(R * max(caps[: self.L]), hi - lo)          # distinct nodes a hop can ask this owner for
            if D > self.max_requests:
                self.max_requests = D
                self.ws_owner = torch.empty(self.ops.gs_shard_workspace_bytes(self.graph, max(self.fanouts), D),
                                            dtype=torch.uint8, device=dev)
            self.merge_index = torch.full((hi - lo,), -1, **i32)
            self.merge_distinct = torch.empty(D, **i32)
            self.merge_rows = torch.empty(D * max(self.fanouts), **i32)
            self.merge_num = torch.zeros((self.L, 2), **i32)   # per hop: distinct nodes, status word
            self.merge_host = torch.zeros((self.L, 2), dtype=torch.int32, pin_memory=dev.type == "cuda")
        self.counts_all = torch.zeros((self.L + 1, 2 * R + 1), **i32)
        self.counts_host = torch.zeros((self.L + 1, 2 * R + 1), dtype=torch.int32, pin_memory=dev.type == "cuda")
        self.fx = []
        for k in range(self.L + 1):
            C = caps[k]
            b = {"sorted": torch.empty(R * C, **i32), "recv": torch.empty(R * C, **i32), "recv_counts": torch.empty(R, **i32)}
            if k < self.L:
                f = self.fanouts[self.L - 1 - k]
                b["out"], b["reply"] = torch.empty((R * C, f), **i32), torch.empty((R * C, f), **i32)
            else:
                D = self.features.shape[1]
                b["out"] = torch.empty((R * C, D), dtype=self.features.dtype, device=dev)
                b["reply"] = torch.empty((R * C, D), dtype=self.features.dtype, device=dev)
            self.fx.append(b)
        self.fx_slot = None

    def largest_groups(self):
        """After an exact-size batch: the largest group of each of its exchanges (L hops, then the feature request;
        when the rows were pulled instead, the share of the input nodes a rank would get).  The maximum of this over
        some batches and all ranks, plus a margin, is what set_capacities needs."""
        got = list(self.seen)
        if len(got) == self.L:
            got.append((self.n[self.L] + self.world - 1) // self.world)
        return got

    def _product_bound(self, k):
        bound = self.n[0]
        for j in range(k):
            bound = min(self.num_nodes, bound * (1 + self.fanouts[self.L - 1 - j]))
        return bound

    def _bound_fixed(self, k):
        """Upper bound of n_k that needs no host knowledge of the batch: the fan-out product, the node count, and
        what the segments can hold at all."""
        bound = self._product_bound(k)
        # the slots of a hop are read for every frontier node, so they cover the whole bound; the feature
        # request needs no more than the segments can hold (a longer frontier is reported by the bucket call)
        return min(bound, self.world * self.caps[k]) if k == self.L and self.caps[k] > 0 else bound

    def requests_fixed(self, k):
        """-> (ids [world * caps[k]] at fixed pitch, group sizes as a device tensor [world])."""
        bound = self._bound_fixed(k)
        if self.fx_slot is None or self.fx_slot.numel() < bound:
            self.fx_slot = torch.empty(max(bound, 1), dtype=torch.int32, device=self.features.device)
        b = self.fx[k]
        _, self.slot, counts = self.ops.gs_shard_bucket(self.frontier[:bound], self.num_nodes, self.world,
                                                        count=self.count_dev, capacity=self.caps[k],
                                                        out=(b["sorted"], self.fx_slot[:bound], self.counts_all[k]))
        return b["sorted"], counts[: self.world]

    def hop_finish_fixed(self, k, reply):
        block, frontier = self.ops.gs_shard_extend(self.cache, k, self.seeds if k == 0 else None, reply, self.slot, self.ws,
                                                   reply_rows=self.world * self.caps[k])
        self.blocks[self.L - 1 - k] = block
        self.frontier = frontier
        self.count_dev = block.counts_device()[1]

    def hop_serve_fixed(self, layer, recv, recv_counts, mode, rate, step, out):
        """recv [world * C] ids, requester r's list in segment r, its length recv_counts[r] -> out [world * C, f]."""
        C = recv.numel() // self.world
        if self.merge:
            f = self.fanouts[layer]
            D = min(recv.numel(), self.merge_index.numel())
            distinct, num = self.merge_distinct[:D], self.merge_num[self.L - 1 - layer]
            rows = self.merge_rows[: D * f].view(D, f)
            self.ops.gs_shard_merge(recv, recv_counts, self.world, self.first_row, self.merge_index, distinct, num)
            try:
                self.ops.gs_shard_sample_rows(self.cache, distinct, layer, mode, rate, step, self.ws_owner, picks=rows,
                                              count=num[0:1])
            finally:    # the fan-out also clears the index: it must run even when the sampling call was refused
                self.ops.gs_shard_fan_out(recv, recv_counts, self.world, self.first_row, self.merge_index, distinct, num,
                                          rows, out)
            return out
        for r in range(self.world):
            self.ops.gs_shard_sample_rows(self.cache, recv[r * C:(r + 1) * C], layer, mode, rate, step, self.ws_owner,
                                          picks=out[r * C:(r + 1) * C], count=recv_counts[r:r + 1])
        return out

    def feature_serve_fixed(self, recv, recv_counts, out):
        C = recv.numel() // self.world
        for r in range(self.world):
            self.ops.gs_gather_rows(self.features, recv[r * C:(r + 1) * C], out[r * C:(r + 1) * C], first_row=self.first_row,
                                    count=recv_counts[r:r + 1])
        return out

    def feature_finish_fixed(self, rows):
        bound = self._bound_fixed(self.L)
        out = torch.empty((bound, rows.shape[1]), dtype=rows.dtype, device=rows.device)
        return self.ops.gs_gather_rows(rows, self.slot[:bound], out, count=self.count_dev)

    def finish_batch_fixed(self):
        """Counts, device status and the bucket calls' error words of the batch, read once (synchronises)."""
        self.counts_host.copy_(self.counts_all, non_blocking=True)
        if self.merge:
            self.merge_host.copy_(self.merge_num, non_blocking=True)
        self.finish_batch()                        # synchronises the stream the copies above are on
        if self.merge and any(self.merge_host[:, 1].tolist()):
            raise ValueError("a requested node id is not a row of this shard")
        if self.feat_bound is not None and self.n[self.L] > self.feat_bound:
            raise RuntimeError("%d input nodes, feature rows were allocated for %d" % (self.n[self.L], self.feat_bound))
        words = self.counts_host[:, 2 * self.world].tolist()
        if any(w == 3 for w in words):             # GS_ERR_RANGE
            raise ValueError("a node id is outside [0, num_nodes)")
        if any(words):
            k = [i for i, w in enumerate(words) if w][0]
            raise RuntimeError("the requests of %s outgrew their segment of %d ids (groups: %s)"
                               % ("hop %d" % k if k < self.L else "the feature step", self.caps[k],
                                  self.counts_host[k, : self.world].tolist()))

    # ---- owner side
    def hop_serve(self, layer, lists, mode, rate, step):
        """One list of distinct nodes per requester -> one [len, f] tensor of picks each.  With several requesters
        the packed lists are merged like the fixed-pitch ones (one list with repeats, one requester): every
        distinct node is sampled once and its row copied to every place that asked for it."""
        sizes = [nodes.numel() for nodes in lists]
        for n in sizes:
            if n > self.max_requests:
                raise ValueError("a request list of %d nodes exceeds max_requests %d" % (n, self.max_requests))
        total = sum(sizes)
        lo, hi = shard_range(self.num_nodes, self.rank, self.world)
        # the distinct nodes must fit the owner's workspace like any single list
        if len(lists) > 1 and total > 0 and hi > lo and self.merge_exact and min(total, hi - lo) <= self.max_requests:
            dev, f = self.features.device, self.fanouts[layer]
            i32 = dict(dtype=torch.int32, device=dev)
            if self.exact_index is None:
                self.exact_index = torch.full((hi - lo,), -1, **i32)
            packed = torch.cat([nodes.contiguous() for nodes in lists])
            count = torch.tensor([total], **i32)
            D = min(total, hi - lo)
            distinct, num = torch.empty(D, **i32), torch.zeros(2, **i32)
            rows, out = torch.empty((distinct.numel(), f), **i32), torch.empty((total, f), **i32)
            self.ops.gs_shard_merge(packed, count, 1, self.first_row, self.exact_index, distinct, num)
            try:
                self.ops.gs_shard_sample_rows(self.cache, distinct, layer, mode, rate, step, self.ws_owner, picks=rows,
                                              count=num[0:1])
            finally:    # the fan-out also clears the index
                self.ops.gs_shard_fan_out(packed, count, 1, self.first_row, self.exact_index, distinct, num, rows, out)
            self.exact_merge_status.append(num)
            return list(torch.split(out, sizes))
        out = []
        for nodes in lists:
            out.append(self.ops.gs_shard_sample_rows(self.cache, nodes.contiguous(), layer, mode, rate, step, self.ws_owner))
        return out                                 # device-detected problems are read once, in finish_batch

    def feature_serve(self, lists):
        out = []
        for nodes in lists:
            rows = torch.empty((nodes.numel(), self.features.shape[1]), dtype=self.features.dtype, device=self.features.device)
            out.append(self.ops.gs_gather_rows(self.features, nodes.contiguous(), rows, first_row=self.first_row))
        return out


def _split(t, counts):
    return list(torch.split(t, counts)) if t.numel() else [t[:0] for _ in counts]


# --------------------------------------------------------------------------- all ranks in one process
def sample_batch_local(ranks, seeds_per_rank, mode, rate, step, features=True):
    """Runs one batch per rank, phase by phase; the exchange is a local copy.  Returns, per rank,
    (blocks by layer, frontier tensor, n list, m list, feature rows or None)."""
    R = len(ranks)
    L = ranks[0].L
    for r, seeds in zip(ranks, seeds_per_rank):
        r.begin(seeds)
    if ranks[0].caps is not None:
        return _sample_batch_local_fixed(ranks, mode, rate, step, features)

    def round_trip(req, serve):
        sent = [_split(ids, counts) for ids, counts in req]                 # sent[r][o]
        served = [serve(ranks[o], [sent[r][o] for r in range(R)]) for o in range(R)]   # served[o][r]
        return [torch.cat([served[o][r] for o in range(R)]) for r in range(R)]

    for k in range(L):
        layer = L - 1 - k
        replies = round_trip([r.hop_requests(k) for r in ranks],
                             lambda owner, lists: owner.hop_serve(layer, lists, mode, rate, step))
        for r, reply in zip(ranks, replies):
            r.hop_finish(k, reply.contiguous())
    feats = [None] * R
    if features == "peer":     # all shards live in this process: their addresses are the "peer" mappings
        bases = [r.features.data_ptr() for r in ranks]
        feats = [r.feature_pull(bases) for r in ranks]
    elif features:
        rows = round_trip([r.feature_requests() for r in ranks], lambda owner, lists: owner.feature_serve(lists))
        feats = [r.feature_finish(x.contiguous()) for r, x in zip(ranks, rows)]
    for r in ranks:
        r.finish_batch()
    feats = [f if f is None else f[: r.n[L]] for r, f in zip(ranks, feats)]
    return [(r.blocks, r.frontier, r.n, r.m, f) for r, f in zip(ranks, feats)]


def _sample_batch_local_fixed(ranks, mode, rate, step, features):
    """sample_batch_local with fixed-capacity exchanges (ShardRank.set_capacities): the copies below stand for the
    equal-split all-to-alls; the host reads nothing before the end of the batch."""
    R, L = len(ranks), ranks[0].L

    def round_trip(k, req, serve):
        C = ranks[0].caps[k]
        for o, owner in enumerate(ranks):                        # what the ranks send to owner o, one copy per owner
            b = owner.fx[k]
            torch.stack([req[r][0].view(R, C)[o] for r in range(R)], out=b["recv"].view(R, C))
            torch.stack([req[r][1][o] for r in range(R)], out=b["recv_counts"])
            serve(owner, b["recv"], b["recv_counts"], b["out"])
        replies = [r.fx[k]["reply"] for r in ranks]
        for r in range(R):                                       # and what comes back, one copy per requester
            width = replies[r].shape[1]
            torch.stack([ranks[o].fx[k]["out"].view(R, C, width)[r] for o in range(R)], out=replies[r].view(R, C, width))
        return replies

    for k in range(L):
        layer = L - 1 - k
        replies = round_trip(k, [r.requests_fixed(k) for r in ranks],
                             lambda owner, recv, rc, out: owner.hop_serve_fixed(layer, recv, rc, mode, rate, step, out))
        for r, reply in zip(ranks, replies):
            r.hop_finish_fixed(k, reply)
    feats = [None] * R
    if features == "peer":
        bases = [r.features.data_ptr() for r in ranks]
        feats = [r.feature_pull(bases, bound=r._bound_fixed(L) if r.caps[L] else None) for r in ranks]
    elif features:
        rows = round_trip(L, [r.requests_fixed(L) for r in ranks],
                          lambda owner, recv, rc, out: owner.feature_serve_fixed(recv, rc, out))
        feats = [r.feature_finish_fixed(x) for r, x in zip(ranks, rows)]
    for r in ranks:
        r.finish_batch_fixed()
    feats = [f if f is None else f[: r.n[L]] for r, f in zip(ranks, feats)]
    return [(r.blocks, r.frontier, r.n, r.m, f) for r, f in zip(ranks, feats)]


# --------------------------------------------------------------------------- one process per rank
def _all_to_all_v(send, send_counts, width, group):
    """send: [sum(send_counts), *width] grouped by destination -> (received tensor, receive counts)."""
    dev = send.device
    sc = torch.tensor(send_counts, dtype=torch.int64, device=dev)
    rc = torch.empty_like(sc)
    dist.all_to_all_single(rc, sc, group=group)
    recv_counts = rc.cpu().tolist()
    recv = torch.empty((sum(recv_counts),) + tuple(width), dtype=send.dtype, device=dev)
    dist.all_to_all_single(recv, send.contiguous(), recv_counts, send_counts, group=group)
    return recv, recv_counts


class ShardedBatchError(RuntimeError):
    """Raised by EVERY rank of a sharded batch when any rank met an error inside a hop."""

    def __init__(self, code, local_message):
        what = {1: "a rank could not build its requests (a node id outside the graph)",
                2: "an owner could not serve a request list (longer than max_requests, or a device-detected error)"}
        super().__init__("sharded batch abandoned: %s%s" % (what.get(code, "error %d" % code),
                                                            "; on this rank: " + local_message if local_message else ""))
        self.code = code


def sample_batch(rank_state: ShardRank, seeds, mode, rate, step, features=True, group=None, feature_bases=None):
    """This rank's part of a sharded batch (every rank of `group` calls it with the same mode, rate
    and step).  Returns (blocks by layer, frontier tensor, n list, m list, feature rows or None).
    `feature_bases`: device addresses of every rank's feature rows as mapped into this process (CUDA
    IPC, symmetric memory, ...); when given, the feature step is one kernel of peer loads instead of an
    all-to-all round trip.

    Failures are collective: a rank that cannot build its requests or serve a list still takes part in
    every exchange of the batch (with no requests / placeholder rows), an error word is reduced over the
    group after the last exchange, and then every rank raises :class:`ShardedBatchError` - no rank is
    left waiting inside a collective for one that has gone."""
    me = rank_state
    L = me.L
    me.begin(seeds)
    dev = seeds.device
    state = {"err": 0, "msg": ""}

    def fail(code, e):
        if not state["err"]:
            state["err"], state["msg"] = code, str(e)

    if me.caps is not None:
        return _sample_batch_fixed(me, mode, rate, step, features, group, feature_bases, state, fail)

    def round_trip(make_requests, serve, width, dtype):
        ids, counts = torch.empty(0, dtype=torch.int32, device=dev), [0] * me.world
        if state["err"] != 1:                      # a rank whose own batch is broken asks for nothing more
            try:
                ids, counts = make_requests()
            except (ValueError, RuntimeError) as e:
                fail(1, e)
                ids, counts = torch.empty(0, dtype=torch.int32, device=dev), [0] * me.world
        recv, recv_counts = _all_to_all_v(ids, counts, (), group)
        back = None
        try:
            served = serve(_split(recv, recv_counts))
            back = torch.cat(served) if served else torch.empty((0,) + width, dtype=dtype, device=dev)
        except (ValueError, RuntimeError) as e:
            fail(2, e)
        if back is None or back.shape[0] != sum(recv_counts):
            back = torch.zeros((sum(recv_counts),) + width, dtype=dtype, device=dev)   # placeholder rows keep the exchange whole
        reply = torch.empty((ids.numel(),) + width, dtype=dtype, device=dev)
        dist.all_to_all_single(reply, back.contiguous(), counts, recv_counts, group=group)
        return reply

    for k in range(L):
        layer = L - 1 - k
        reply = round_trip(lambda: me.hop_requests(k), lambda lists: me.hop_serve(layer, lists, mode, rate, step),
                           (me.fanouts[layer],), torch.int32)
        if state["err"] != 1:
            me.hop_finish(k, reply)
    feats = None
    if features and feature_bases is not None:
        if state["err"] != 1:
            feats = me.feature_pull(feature_bases)
    elif features:
        rows = round_trip(me.feature_requests, me.feature_serve, (me.features.shape[1],), me.features.dtype)
        if state["err"] != 1:
            feats = me.feature_finish(rows)
    if state["err"] != 1:
        try:
            me.finish_batch()
        except (ValueError, RuntimeError) as e:
            fail(2, e)
    word = torch.tensor([state["err"]], dtype=torch.int32, device=dev)
    dist.all_reduce(word, op=dist.ReduceOp.MAX, group=group)
    code = int(word.item())
    if code:
        raise ShardedBatchError(code, state["msg"])
    if feats is not None:
        feats = feats[: me.n[L]]
    return me.blocks, me.frontier, me.n, me.m, feats


def _sample_batch_fixed(me, mode, rate, step, features, group, feature_bases, state, fail):
    """sample_batch with fixed-capacity exchanges (ShardRank.set_capacities): three equal-split all-to-alls per hop
    (group sizes, ids, rows) on pre-allocated buffers, no host synchronisation before the end of the batch.  Every
    rank always takes part in every exchange, whatever it has met; errors (host- or device-detected, a group that
    outgrew its segment included) are reduced once, after the last exchange."""
    L, dev = me.L, me.features.device
    if not me.caps_agreed:
        # equal-split exchanges need the same segment sizes everywhere: compare once, and fail on every rank if not
        lo = torch.tensor(me.caps, dtype=torch.int64, device=dev)
        hi = lo.clone()
        dist.all_reduce(lo, op=dist.ReduceOp.MIN, group=group)
        dist.all_reduce(hi, op=dist.ReduceOp.MAX, group=group)
        if not torch.equal(lo, hi):
            raise ShardedBatchError(1, "the ranks were given different capacities: %s here" % me.caps)
        me.caps_agreed = True

    def round_trip(k, serve):
        b = me.fx[k]
        ids, counts = b["sorted"], me.counts_all[k, : me.world]
        if state["err"] != 1:
            try:
                ids, counts = me.requests_fixed(k)
            except (ValueError, RuntimeError) as e:
                fail(1, e)
        if state["err"] == 1:
            counts = torch.zeros(me.world, dtype=torch.int32, device=dev)      # this rank asks for nothing more
        dist.all_to_all_single(b["recv_counts"], counts, group=group)
        dist.all_to_all_single(b["recv"], ids, group=group)
        try:
            serve(b["recv"], b["recv_counts"], b["out"])
        except (ValueError, RuntimeError) as e:
            fail(2, e)
        dist.all_to_all_single(b["reply"], b["out"], group=group)
        return b["reply"]

    for k in range(L):
        layer = L - 1 - k
        reply = round_trip(k, lambda recv, rc, out: me.hop_serve_fixed(layer, recv, rc, mode, rate, step, out))
        if state["err"] != 1:
            try:
                me.hop_finish_fixed(k, reply)
            except (ValueError, RuntimeError) as e:
                fail(1, e)
    feats = None
    if features and feature_bases is not None:
        if state["err"] != 1:
            feats = me.feature_pull(feature_bases, bound=me._bound_fixed(L) if me.caps[L] else None)
    elif features:
        rows = round_trip(L, me.feature_serve_fixed)
        if state["err"] != 1:
            feats = me.feature_finish_fixed(rows)
    if state["err"] != 1:
        try:
            me.finish_batch_fixed()
        except (ValueError, RuntimeError) as e:
            fail(2 if "requested node" in str(e) else 1, e)
    word = torch.tensor([state["err"]], dtype=torch.int32, device=dev)
    dist.all_reduce(word, op=dist.ReduceOp.MAX, group=group)
    code = int(word.item())
    if code:
        raise ShardedBatchError(code, state["msg"])
    if feats is not None:
        feats = feats[: me.n[L]]
    return me.blocks, me.frontier, me.n, me.m, feats
