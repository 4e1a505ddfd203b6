"""Runs the CUDA library and the CPU oracle on the same seeded inputs and compares every output
bit for bit (tolerance 0: ids, offsets and copied feature bits are integers)."""
import numpy as np
import torch

import oracle
import paper_2406_17918_b200 as gs
from workloads import batch_seeds, build_features, build_graph, seed_permutation

MODES = {"fcr": (gs.GS_MODE_FCR, oracle.MODE_FCR), "otf": (gs.GS_MODE_OTF, oracle.MODE_OTF),
         "fbl": (gs.GS_MODE_FBL, oracle.MODE_FBL), "fetch": (gs.GS_MODE_OTF_FETCH, oracle.MODE_OTF_FETCH)}


def bits(t: torch.Tensor) -> np.ndarray:
    """Feature tensor -> integer bit patterns (numpy has no bfloat16)."""
    t = t.detach().cpu().contiguous()
    return t.view(torch.int32 if t.dtype == torch.float32 else torch.int16).numpy()


class Pair:
    """One graph resident on the GPU (library) and on the host (oracle), same bytes."""

    def __init__(self, cfg, seed=0x1234ABCD5678EF01, gen_device="cuda", features=True):
        self.cfg = cfg
        g = build_graph(cfg, device=gen_device if cfg["kind"] == "rmat" else "cpu")
        self.g_dev = g.to("cuda")
        self.indptr = g.indptr.cpu().numpy()
        self.indices = g.indices.cpu().numpy()
        self.deg = self.indptr[1:] - self.indptr[:-1]
        self.X = build_features(cfg, device="cuda" if cfg["feat_kind"] == "hash" else "cpu").to("cuda") if features else None
        self.perm = seed_permutation(cfg)
        self.L, self.W, self.shared = len(cfg["fanouts"]), cfg["cache_width"], cfg["shared"]
        self.G = gs.gs_graph_create(self.g_dev.indptr, self.g_dev.indices, self.X)
        self.seed = seed

    @classmethod
    def from_csr(cls, indptr, indices, fanouts, cache_width, shared=False, seed=0x1234ABCD5678EF01):
        """A hand-made graph (numpy CSR) instead of a named workload; no features, seeds = node order."""
        self = cls.__new__(cls)
        n = len(indptr) - 1
        self.cfg = dict(name="custom", num_nodes=n, fanouts=list(fanouts), cache_width=cache_width, shared=shared, batch=n)
        self.indptr, self.indices = np.asarray(indptr, dtype=np.int64), np.asarray(indices, dtype=np.int32)
        self.deg = self.indptr[1:] - self.indptr[:-1]
        from workloads.graphs import Graph
        self.g_dev = Graph(n, len(self.indices), torch.from_numpy(self.indptr).cuda(), torch.from_numpy(self.indices).cuda())
        self.X = None
        self.perm = torch.arange(n, dtype=torch.int32)
        self.L, self.W, self.shared = len(fanouts), cache_width, shared
        self.G = gs.gs_graph_create(self.g_dev.indptr, self.g_dev.indices, None)
        self.seed = seed
        return self

    def samplers(self, max_seeds, tuning=None, theta=None):
        self.theta = theta
        if theta is None:
            C = gs.gs_cache_init(self.G, self.cfg["fanouts"], self.W, self.seed, self.shared)
        else:
            C = gs.gs_cache_init_split(self.G, self.cfg["fanouts"], self.W, self.seed, self.shared, theta)
        if tuning:
            gs.gs_cache_set_tuning(C, **tuning)
        if getattr(self, "dedup", 0):
            gs.gs_cache_set_dedup(C, self.dedup)
        ws = torch.empty(gs.gs_workspace_bytes(self.G, self.cfg["fanouts"], max_seeds), dtype=torch.uint8, device="cuda")
        O = oracle.Sampler(self.indptr, self.indices, self.cfg["fanouts"], self.W, self.seed, self.shared)
        if theta is not None:
            O.set_theta(theta)
        return C, ws, O

    def check_rows(self, C, O, nodes):
        nodes = np.asarray(nodes, dtype=np.int32)
        if getattr(self, "theta", None) is not None:      # a split cache has rows for the dense part only
            sparse = nodes[self.deg[nodes] <= self.theta]
            nodes = nodes[self.deg[nodes] > self.theta]
            if len(sparse):
                got = gs.gs_cache_read_rows(C, 0, torch.from_numpy(sparse).cuda()).cpu().numpy()
                assert (got == -1).all()
        for layer in range(1 if self.shared else self.L):
            got = gs.gs_cache_read_rows(C, layer, torch.from_numpy(nodes).cuda()).cpu().numpy()
            want = O.cache_rows(layer, nodes)
            assert np.array_equal(got, want), "cache rows differ at layer %d" % layer

    def check_batch(self, C, ws, O, seeds, mode, gamma, step, features=True, rows=True, host_api=False):
        gm, om = MODES[mode]
        if host_api:
            blocks, input_nodes, n, m = gs.gs_sample_batch_host(C, seeds.cpu(), gm, gamma, step, ws)
            cnt = None
        else:
            blocks, input_nodes, cnt = gs.gs_sample_batch(C, seeds.cuda(), gm, gamma, step, ws)
            n, m = gs.gs_batch_counts(C)
        self.last_input_nodes = input_nodes      # aliases the workspace: valid until the next batch on it
        frontier, n_o, blocks_o = O.sample_batch(seeds.cpu().numpy(), om, gamma, step)
        assert n == n_o, (n, n_o)
        got_frontier = input_nodes[: n[self.L]].cpu().numpy()
        assert np.array_equal(got_frontier, frontier)
        for layer in range(self.L):
            k = self.L - 1 - layer
            bo = blocks_o[layer]
            assert m[layer] == bo.num_edges
            assert blocks[layer].max_dst >= n[k] and blocks[layer].max_src >= n[k + 1] and blocks[layer].max_edges >= m[layer]
            assert np.array_equal(blocks[layer].indptr(n[k]).cpu().numpy(), bo.indptr)
            assert np.array_equal(blocks[layer].indices(m[layer]).cpu().numpy(), bo.indices)
            d = [int(x) for x in blocks[layer].counts_device()]
            assert d == [n[k], n[k + 1], m[layer]]
        if rows is True:
            self.check_rows(C, O, frontier)
        elif rows:   # an int: that many sampled frontier nodes
            pickrng = np.random.default_rng(step)
            self.check_rows(C, O, frontier[pickrng.choice(len(frontier), min(int(rows), len(frontier)), replace=False)])
        if features and self.X is not None:
            out = torch.full((n[self.L] + 3, self.X.shape[1]), 7, dtype=self.X.dtype, device="cuda")
            gs.gs_gather_features(self.G, input_nodes, cnt, out)
            Xh = bits(self.X)
            assert np.array_equal(bits(out[: n[self.L]]), oracle.gather(Xh, frontier))
            if cnt is not None:   # rows past the device count stay untouched
                assert bool((out[n[self.L]:] == 7).all())
        return n, m

    def run_periodic(self, mode, gamma, T, batches, batch_size=None, tuning=None, theta=None, **kw):
        """Algorithms 2/3 as written: every T-th batch refreshes the whole cache, all batches only pick."""
        B = batch_size or self.cfg["batch"]
        C, ws, O = self.samplers(B, tuning, theta)
        gm, om = MODES[mode]
        all_nodes = np.arange(self.cfg["num_nodes"], dtype=np.int32)
        for t in range(1, batches + 1):
            if t % T == 0:
                gs.gs_cache_refresh_all(C, gm, gamma, t)
                O.refresh_all(om, gamma, t)
                gs.gs_sync_status(C)
                self.check_rows(C, O, all_nodes)
            self.check_batch(C, ws, O, batch_seeds(self.perm, t, B), "otf", 0.0, t, **kw)
        self.check_rows(C, O, all_nodes)
        return C, ws, O

    def run(self, mode, gamma, batches, batch_size=None, tuning=None, first_step=1, theta=None, **kw):
        B = batch_size or self.cfg["batch"]
        C, ws, O = self.samplers(B, tuning, theta)
        out = []
        for b in range(batches):
            seeds = batch_seeds(self.perm, b, B)
            out.append(self.check_batch(C, ws, O, seeds, mode, gamma, first_step + b, **kw))
        return C, ws, O, out
