#!/usr/bin/env python
"""Benchmark of the cached neighbour sampling hot path.

One step = one mini-batch through the whole path: gs_sample_batch (refresh + pick + relabel +
block CSR for every hop) followed by gs_gather_features for the input nodes, on fresh seeds and
the next step number (the cache evolves as in training).  The headline leg runs every batch start
to end on one stream; a second leg (skipped with --no-overlap) runs each batch's gather on a second
stream beside the first hops of the next batch and is reported beside it under "pipelined".

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload scale|large|shared|mid|tiny]
                    [--mode otf|fcr|fbl|fetch] [--rate R] [--fanouts a,b,c] [--cache-width W] [--shared-cache 0|1]
                    [--theta T]        dense/sparse split cache
                    [--period T]       whole-cache refresh every T-th batch, pick-only batches
                    [--sharded]        node-sharded run (one all-to-all round trip per hop)
    python bench.py --impl reference ...        # times the CPU oracle on a bounded sample

Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from workloads import batch_seeds, build_features, build_graph, get_config, seed_permutation  # noqa: E402

METRIC = "sampled edges/s + feature GB/s per batch (OTF), fraction of HBM roofline"
FALLBACK_HBM_GBS = 6650.0
SAMPLER_SEED = 0x6A09E667F3BCC908
# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one captured launch, from ncu captures of the same
# kernels on small workloads (scaled to a launch of the benchmarked workload by the units it processes).
#   k_scan, workload large, sampling step 2 of a batch: 5,612,800 B read + 12,544 B written for 16.38 M Philox
#     blocks in 45 K work items.  The traffic is the items' descriptors, so it follows the number of items; larger
#     rows mean fewer items per block, which makes the per-block scaling an upper estimate for the scale workload.
#   k_gather with 256-byte bf16 rows, all 736,389 rows of workload shared once each in random order (--gather-only):
#     191,698,944 B read by the bulk-copy kernel (260 B per row: the row and its id, no over-fetch; the load/store
#     kernel: 191,470,592 B); 141 MB of the 188.5 MB written reached
#     DRAM inside the launch, the rest was still in L2 when it ended, so the written bytes are counted as the
#     algorithmic 256 B per row.
NCU_SCAN_BYTES_PER_BLOCK = (5612800 + 12544) / 16380004
NCU_GATHER_READ_BYTES_PER_256B_ROW = 191698944 / 736389


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.samples = []
        self.proc = None
        try:
            uuid = "GPU-" + str(torch.cuda.get_device_properties(device_index).uuid)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", uuid, "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append((time.time(), line.strip()))

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self, t0: float, t1: float):
        rows = [s for (t, s) in self.samples if t0 <= t <= t1] or [s for (_, s) in self.samples]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            f = [x.strip() for x in r.split(",")]
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except Exception:
                continue
            for name, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------- workload
def run_spec(cfg):
    """(mode, gamma) the metric is quoted on: the config's OTF run."""
    for mode, gamma in cfg["runs"]:
        if mode == "otf":
            return mode, gamma
    return cfg["runs"][0]


def algorithmic_bytes(cfg, n, m_by_step, refreshed_by_step, r):
    """Bytes the method itself must move for one batch (sector over-fetch excluded).

    Per step k: two int64 row bounds and one cache row per frontier node, r neighbour ids read and
    r slots written per refreshed node, picked ids written and re-read, one 8-byte relabel-table
    entry per frontier node and per pick plus one written per new id, local ids and block offsets
    written, new frontier ids written.  The key scan of a refreshed row moves no bytes: keys depend
    on (node, offset, step), not on neighbour ids.  Features: id read, row read, row written."""
    W = cfg["cache_width"]
    L = len(cfg["fanouts"])
    total = 0
    for k in range(L):
        nk, mk, uk = n[k], m_by_step[k], n[k + 1] - n[k]
        total += 16 * nk + 4 * W * nk + 8 * r * refreshed_by_step[k]
        total += 4 * mk + 8 * (nk + mk) + 8 * uk + 8 * mk + 4 * (nk + 1) + 4 * uk
    s = 4 if cfg["feat_dtype"] == "f32" else 2
    feat = n[L] * (4 + 2 * cfg["feat_dim"] * s)
    return total + feat, feat


def cpu_oracle_baseline(cfg, indptr_h, indices_h, perm, mode, gamma, budget_s=32.0, reps=1, first_seeds=None,
                        theta=None):
    """Times the CPU oracle, as it stands, on the first `s` seeds of batch 0 (s grown until one
    batch takes a few seconds).  Returns (edges/s, feature GB/s, description, seconds per batch)."""
    import numpy as np

    import oracle
    from workloads import feature_rows

    O = oracle.Sampler(indptr_h, indices_h, cfg["fanouts"], cfg["cache_width"], SAMPLER_SEED, cfg["shared"])
    if theta is not None:
        O.set_theta(theta)
    om = {"otf": oracle.MODE_OTF, "fcr": oracle.MODE_FCR, "fbl": oracle.MODE_FBL, "fetch": oracle.MODE_OTF_FETCH}[mode]
    B = cfg["batch"]
    s = first_seeds or max(1, min(B, 16))
    step = 1
    esize = 4 if cfg["feat_dtype"] == "f32" else 2
    best = None
    while True:
        seeds = batch_seeds(perm, 0, B)[:s].numpy()
        t0 = time.perf_counter()
        frontier, n, blocks = O.sample_batch(seeds, om, gamma, step)
        t_sample = time.perf_counter() - t0
        # feature rows of the sampled nodes, re-evaluated or sliced on the host, then gathered row by row
        ids = torch.from_numpy(frontier.astype("int64"))
        if cfg["feat_kind"] == "hash":
            Xs = feature_rows(cfg, ids)
        else:
            Xs = cpu_oracle_baseline.features[ids]
        Xb = Xs.view(torch.int32 if esize == 4 else torch.int16).numpy()
        t1 = time.perf_counter()
        oracle.gather(Xb, np.arange(len(frontier), dtype=np.int32))
        t_gather = time.perf_counter() - t1
        dt = t_sample + t_gather
        edges = sum(b.num_edges for b in blocks)
        best = (edges / dt, len(frontier) * cfg["feat_dim"] * esize / dt / 1e9, s, dt)
        step += 1
        if dt >= budget_s / 4 or s >= B or first_seeds:
            break
        s = min(B, s * (4 if dt < budget_s / 16 else 2))
    desc = ("oracle sample_batch + row-by-row gather, first %d of %d seeds of batch 0, %s gamma=%g, %.2f s"
            % (best[2], B, mode, gamma, best[3]))
    O.close()
    return best[0], best[1], desc, best[3]


def verify_first_batch(gs, cfg, g, G, C, X, seeds, gm, mode, gamma, ws, theta, row_samples=4000):
    """One whole batch (step 1 on a fresh cache) on the GPU and through the CPU oracle, compared element by
    element.  Raises on the first difference; returns a summary for the result line."""
    import numpy as np

    import oracle
    from workloads import feature_rows

    L, W = len(cfg["fanouts"]), cfg["cache_width"]
    blocks, input_nodes, cnt = gs.gs_sample_batch(C, seeds, gm, gamma, 1, ws)
    n, m = gs.gs_batch_counts(C)
    got_frontier = input_nodes[: n[L]].cpu().numpy()
    got_blocks = [(blocks[l].indptr(n[L - 1 - l]).cpu().numpy(), blocks[l].indices(m[l]).cpu().numpy()) for l in range(L)]
    out = torch.empty((n[L], cfg["feat_dim"]), dtype=X.dtype, device=X.device)
    gs.gs_gather_features(G, input_nodes, cnt, out)
    got_feat = out.cpu().view(torch.int32 if X.dtype == torch.float32 else torch.int16).numpy()
    del out
    O = oracle.Sampler(g.indptr.cpu().numpy(), g.indices.cpu().numpy(), cfg["fanouts"], W, SAMPLER_SEED, cfg["shared"])
    if theta is not None:
        O.set_theta(theta)
    om = {"otf": oracle.MODE_OTF, "fcr": oracle.MODE_FCR, "fbl": oracle.MODE_FBL, "fetch": oracle.MODE_OTF_FETCH}[mode]
    t0 = time.perf_counter()
    frontier, n_o, blocks_o = O.sample_batch(seeds.cpu().numpy(), om, gamma, 1)
    t_oracle = time.perf_counter() - t0

    def same(a, b, what):
        if a.shape != b.shape or not np.array_equal(a, b):
            raise SystemExit("verify: %s differs from the oracle" % what)

    if list(n) != list(n_o):
        raise SystemExit("verify: frontier sizes %s differ from the oracle's %s" % (n, n_o))
    same(got_frontier, frontier, "the input-node list")
    for l in range(L):
        same(got_blocks[l][0], blocks_o[l].indptr, "block %d offsets" % l)
        same(got_blocks[l][1], blocks_o[l].indices, "block %d indices" % l)
    rng = np.random.default_rng(1)
    nodes = frontier[rng.choice(len(frontier), min(row_samples, len(frontier)), replace=False)]
    if theta is not None:
        deg = (g.indptr[1:] - g.indptr[:-1]).cpu().numpy()
        nodes = nodes[deg[nodes] > theta]
    for layer in range(1 if cfg["shared"] else L):
        rows = gs.gs_cache_read_rows(C, layer, torch.from_numpy(nodes).to(X.device)).cpu().numpy()
        same(rows, O.cache_rows(layer, nodes), "cache rows of layer %d" % layer)
    ids = torch.from_numpy(frontier.astype("int64"))
    Xs = feature_rows(cfg, ids) if cfg["feat_kind"] == "hash" else X.cpu()[ids]
    want = Xs.view(torch.int32 if X.dtype == torch.float32 else torch.int16).numpy()
    same(got_feat, oracle.gather(want, np.arange(len(frontier), dtype=np.int32)), "the gathered feature rows")
    O.close()
    return {"workload": cfg["name"], "batches": 1, "seeds": int(seeds.numel()), "input_nodes": int(n[L]),
            "edges": int(sum(m)), "cache_rows_compared": int(len(nodes)) * (1 if cfg["shared"] else L),
            "compared": "input nodes, block offsets and indices of every hop, sampled cache rows, all gathered feature rows: identical",
            "oracle_seconds": t_oracle}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="scale", choices=["tiny", "mid", "large", "shared", "scale"])
    ap.add_argument("--mode", default=None, choices=["otf", "fcr", "fbl", "fetch"],
                    help="sampling mode (default: the config's OTF run); fbl = no cache, the paper's baseline "
                         "sampler; fetch = OTF Fetch")
    ap.add_argument("--rate", type=float, default=None, help="gamma (otf) or delta (fetch); default: the config's")
    ap.add_argument("--fanouts", default=None, help="comma-separated fan-outs, input layer first (default: the workload's)")
    ap.add_argument("--cache-width", type=int, default=None, help="cache width W (default: the workload's)")
    ap.add_argument("--shared-cache", type=int, default=None, choices=[0, 1], help="one cache for all hops (default: the workload's)")
    ap.add_argument("--theta", type=int, default=None,
                    help="dense/sparse split: cache rows only for nodes with degree > theta (default: one row per node)")
    ap.add_argument("--period", type=int, default=None,
                    help="T: the schedule of Algorithms 2/3 as written - every T-th batch refreshes the whole cache "
                         "(--mode otf/fcr, --rate), every batch only samples from the cache; no CPU baseline "
                         "(the oracle's whole-cache refresh of this graph takes hours)")
    ap.add_argument("--sharded", action="store_true",
                    help="node-sharded run: rank o owns the CSR, cache and feature rows of an id range, one "
                         "all-to-all round trip per hop (needs --theta; default 32); at 1 GPU it measures the "
                         "protocol's overhead, the exchange being a local copy")
    ap.add_argument("--feature-exchange", default=None, choices=["peer", "roundtrip"],
                    help="with --sharded: how feature rows reach the requester (default: peer with one rank, roundtrip otherwise)")
    ap.add_argument("--local-ranks", type=int, default=1,
                    help="with --sharded on one GPU: run this many ranks of the sharded job in this process, phase by phase")
    ap.add_argument("--no-merge", action="store_true",
                    help="with --sharded: owners serve the requesters' lists one by one instead of merging them")
    ap.add_argument("--exact-sizes", action="store_true",
                    help="with --sharded: keep the exact-size exchanges (host reads the group sizes) for the timed batches")
    ap.add_argument("--no-overlap", action="store_true",
                    help="skip the second, pipelined leg (gather of a batch on a second stream, overlapping the "
                         "first, latency-bound hops of the next batch)")
    ap.add_argument("--gather-kernel", default="bulk", choices=["bulk", "loads"],
                    help="the gather on the one stream: rows staged through shared memory by bulk copies (default), or the "
                         "load/store kernel with 16 blocks per SM")
    ap.add_argument("--gather-grid", type=int, default=None,
                    help="blocks per SM in the gather's grid during the pipelined leg (default 1024 short blocks; "
                         "the one-stream leg always uses 16 long-lived ones)")
    ap.add_argument("--dedup", default=None, choices=["direct", "hash", "sort", "auto"],
                    help="how first occurrences are found for dedup + relabel (default: the library's choice)")
    ap.add_argument("--lambda-otf", type=float, default=None,
                    help="expected number of candidates the threshold scan keeps per row for a partial refresh "
                         "(selection tuning; never changes results)")
    ap.add_argument("--verify", action="store_true",
                    help="before anything is timed, run the first batch (full size, step 1) on the GPU and through "
                         "the CPU oracle and compare every output element by element: input nodes, every block's "
                         "offsets and indices, cache rows of sampled frontier nodes, gathered feature rows "
                         "(the oracle needs minutes on the largest workload)")
    ap.add_argument("--gather-only", type=int, default=None, metavar="ROWS",
                    help="time gs_gather_features alone on ROWS distinct, randomly ordered rows of the workload's feature matrix "
                         "(a small, self-contained launch for profiler captures of the gather kernel); prints its own line")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3

    rank, local_rank = int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0"))
    over = {}
    if args.fanouts:
        over["fanouts"] = [int(x) for x in args.fanouts.split(",")]
    if args.cache_width:
        over["cache_width"] = args.cache_width
    if args.shared_cache is not None:
        over["shared"] = bool(args.shared_cache)
    cfg = get_config(args.workload, **over)
    mode, gamma = run_spec(cfg)
    if args.mode and args.mode != mode:
        mode, gamma = args.mode, {"fcr": 1.0, "fbl": 0.0, "fetch": 0.5, "otf": gamma}[args.mode]
    if args.rate is not None:
        gamma = args.rate
    L = len(cfg["fanouts"])

    if args.impl == "reference":
        if rank != 0:
            return 0
        return reference_arm(args, cfg, mode, gamma)

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the sampler has no CPU fallback")
    import paper_2406_17918_b200 as gs
    from paper_2406_17918_b200 import replicas

    device = torch.device("cuda", local_rank)
    torch.cuda.set_device(device)
    rank, local_rank, world = replicas.init("nccl", device)
    if world != args.gpus:
        print("warning: --gpus %d but WORLD_SIZE=%d" % (args.gpus, world), file=sys.stderr)
    if args.sharded:
        return sharded_arm(args, cfg, mode, gamma, rank, local_rank, world, device)
    if args.gather_only:
        return gather_arm(args, cfg, device)

    # ---- inputs, resident in HBM before anything is timed
    t_setup = time.time()
    g = build_graph(cfg, device=device)
    X = build_features(cfg, device=device if cfg["feat_kind"] == "hash" else "cpu").to(device)
    perm = seed_permutation(cfg, device=device)
    torch.cuda.synchronize()
    t_graph = time.time() - t_setup
    G = gs.gs_graph_create(g.indptr, g.indices, X)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    L_hops = len(cfg["fanouts"])
    if args.theta is None:
        storage = torch.empty(gs.gs_cache_bytes(G, L_hops, cfg["cache_width"], cfg["shared"]), dtype=torch.uint8, device=device)
        ev0.record()
        C = gs.gs_cache_init(G, cfg["fanouts"], cfg["cache_width"], SAMPLER_SEED, cfg["shared"], storage=storage)
    else:
        dense_rows = gs.gs_graph_count_dense(G, args.theta)
        storage = torch.empty(gs.gs_cache_bytes_split(G, L_hops, cfg["cache_width"], cfg["shared"], dense_rows),
                              dtype=torch.uint8, device=device)
        ev0.record()
        C = gs.gs_cache_init_split(G, cfg["fanouts"], cfg["cache_width"], SAMPLER_SEED, cfg["shared"], args.theta,
                                   dense_rows, storage=storage)
    ev1.record()
    torch.cuda.synchronize()
    presample_ms = ev0.elapsed_time(ev1)
    if args.lambda_otf:
        gs.gs_cache_set_tuning(C, lambda_otf=args.lambda_otf)
    if args.dedup:
        gs.gs_cache_set_dedup(C, {"direct": gs.GS_DEDUP_DIRECT, "hash": gs.GS_DEDUP_HASH, "sort": gs.GS_DEDUP_SORT, "auto": gs.GS_DEDUP_AUTO}[args.dedup])
    B = cfg["batch"]
    ws = torch.empty(gs.gs_workspace_bytes(G, cfg["fanouts"], B), dtype=torch.uint8, device=device)
    gm = {"otf": gs.GS_MODE_OTF, "fcr": gs.GS_MODE_FCR, "fbl": gs.GS_MODE_FBL, "fetch": gs.GS_MODE_OTF_FETCH}[mode]
    r = {"otf": int(gamma * cfg["cache_width"] + 0.5), "fcr": cfg["cache_width"], "fbl": 0, "fetch": 0}[mode]
    hdr = C.storage[:512].view(torch.int32)
    stat0 = gs.gs_stats_word_offset()

    if args.period:
        if mode not in ("otf", "fcr"):
            raise SystemExit("--period needs --mode otf or fcr")
        args.no_cpu_baseline = True
        refresh_mode, refresh_gamma = gm, gamma
        gm, gamma, r = gs.GS_MODE_OTF, 0.0, 0

    K, Wm = args.steps, args.warmup
    seeds_all = [batch_seeds(perm, b, B, rank, world) for b in range(Wm + 3 * K)]
    verified = None
    if args.verify and args.period:
        raise SystemExit("--verify checks a batch with its own refresh; it does not combine with --period")
    if args.verify and rank == 0:
        verified = verify_first_batch(gs, cfg, g, G, C, X, seeds_all[0], gm, mode, gamma, ws, args.theta)
    alone_grid = 16 if args.gather_kernel == "loads" else -1
    gs.gs_graph_set_gather_grid(G, alone_grid)     # the gather with the GPU to itself: bulk copies where the rows allow it (-1), or loads/stores with a few long-lived blocks (16)
    s_main = torch.cuda.Stream(device=device, priority=-1)
    out_rows = None
    refresh_events = []

    def one_step(b, step, workspace):
        if args.period and step % args.period == 0:
            ra, rb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ra.record()
            gs.gs_cache_refresh_all(C, refresh_mode, refresh_gamma, step)
            rb.record()
            refresh_events.append((ra, rb))
        return gs.gs_sample_batch(C, seeds_all[b], gm, gamma, step, workspace)

    # ---- leg 1 (the headline): every batch start to end on ONE stream - gs_sample_batch, then gs_gather_features
    torch.cuda.synchronize()
    with torch.cuda.stream(s_main):
        for b in range(Wm):
            blocks, input_nodes, cnt = one_step(b, b + 1, ws)
            if out_rows is None:
                out_rows = torch.empty((blocks[0].max_src, cfg["feat_dim"]), dtype=X.dtype, device=device)
            gs.gs_gather_features(G, input_nodes, cnt, out_rows)
        gs.gs_sync_status(C)
        torch.cuda.synchronize()

        pinned_counts = torch.zeros((K, 128), dtype=torch.int32).pin_memory()
        events = [torch.cuda.Event(enable_timing=True) for _ in range(K + 1)]
        clocks = ClockSampler(local_rank) if rank == 0 else None
        time.sleep(0.3)
        replicas.barrier()
        torch.cuda.synchronize()
        launches0 = gs.gs_kernel_launches()
        wall0 = time.time()
        for i in range(K):
            b = Wm + i
            events[i].record()                                  # nothing but the batch boundaries is timed here
            blocks, input_nodes, cnt = one_step(b, b + 1, ws)
            gs.gs_gather_features(G, input_nodes, cnt, out_rows)
            pinned_counts[i].copy_(hdr, non_blocking=True)      # the batch's counts, read after the run
        events[K].record()
        torch.cuda.synchronize()
        replicas.barrier()
        wall1 = time.time()
        launches = gs.gs_kernel_launches() - launches0
        total_ms = events[0].elapsed_time(events[K])
        gs.gs_sync_status(C)

        # ---- leg 1b: where a batch's time goes.  The same loop with CUDA events around the kernel groups (inside the
        # library, on the launching stream) and around sample_batch / gather_features; the events sit between kernels
        # that otherwise follow each other without a gap, so this leg is a little slower than the headline and only
        # its shares and per-kernel rates are used.
        Kb = min(K, 200)
        pinned_b = torch.zeros((Kb, 128), dtype=torch.int32).pin_memory()
        ev_b = [torch.cuda.Event(enable_timing=True) for _ in range(3 * Kb + 1)]
        gs.gs_cache_profile_begin(C, Kb)
        for i in range(Kb):
            b = Wm + i
            ev_b[3 * i].record()
            blocks, input_nodes, cnt = one_step(b, Wm + K + 1 + i, ws)
            ev_b[3 * i + 1].record()
            pinned_b[i].copy_(hdr, non_blocking=True)
            ev_b[3 * i + 2].record()
            gs.gs_gather_features(G, input_nodes, cnt, out_rows)
        ev_b[3 * Kb].record()
        torch.cuda.synchronize()
        group_ms, _ = gs.gs_cache_profile_end(C)
        gs.gs_sync_status(C)
    batch_ms = sorted(events[i].elapsed_time(events[i + 1]) for i in range(K))
    median_ms = batch_ms[K // 2]
    sample_ms = sum(ev_b[3 * i].elapsed_time(ev_b[3 * i + 1]) for i in range(Kb))
    gather_ms = sum(ev_b[3 * i + 2].elapsed_time(ev_b[3 * i + 3]) for i in range(Kb))
    breakdown_total_ms = ev_b[0].elapsed_time(ev_b[3 * Kb])

    # word positions of the counts inside the cache's state header, by sampling step
    n_words = [blocks[L - 1 - k].count_words()[0] for k in range(L)] + [blocks[0].count_words()[1]]
    m_words = [blocks[L - 1 - k].count_words()[2] for k in range(L)]
    counts = pinned_counts.numpy().copy()
    edges = 0
    feat_rows = 0
    # refreshed nodes per step, from the last timed batch's frontier (outside the timed region)
    deg = g.degrees()
    n_last = [int(counts[K - 1][w]) for w in n_words]
    fr = input_nodes[: n_last[L]].long()
    over = (deg[fr] > (cfg["cache_width"] if args.theta is None else args.theta))
    listed = (deg[fr] > max(128, cfg["cache_width"]))     # rows whose refill reads a candidate list of the scan
    refreshed_frac, listed_frac = [], []
    for k in range(L):
        lo = n_last[k - 1] if (cfg["shared"] and k > 0) else 0
        refreshed_frac.append(float(over[lo:n_last[k]].sum().item()) / max(1, n_last[k]))
        listed_frac.append(float(listed[lo:n_last[k]].sum().item()) / max(1, n_last[k]) if r > 0 else 0.0)
    alg_total, alg_feat = 0, 0
    philox_blocks = sum(int(counts[i][stat0 + 3]) & 0xFFFFFFFF for i in range(K))
    philox_blocks_b = sum(int(pinned_b[i][stat0 + 3]) & 0xFFFFFFFF for i in range(Kb))   # of the breakdown leg's batches
    slow_refills = sum(int(counts[i][stat0]) for i in range(K))
    for i in range(K):
        n = [int(counts[i][w]) for w in n_words]
        m = [int(counts[i][w]) for w in m_words]
        edges += sum(m)
        feat_rows += n[L]
        # rows refreshed in this batch, all steps together (counted on the device by the row-count kernel)
        refreshed_rows = int(counts[i][stat0 + 2]) & 0xFFFFFFFF
        a, f = algorithmic_bytes(cfg, n, m, [refreshed_rows] + [0] * (L - 1), r)
        alg_total += a
        alg_feat += f

    # the gather alone (nothing else on the GPU, L2 flushed), on the last batch's input nodes: the kernel's own rate
    iso = []
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)    # larger than L2: no row survives between launches
    with torch.cuda.stream(s_main):
        for _ in range(8):
            flush.zero_()
            ia, ib = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ia.record()
            gs.gs_gather_features(G, input_nodes, cnt, out_rows)
            ib.record()
            iso.append((ia, ib))
    torch.cuda.synchronize()
    gather_alone_ms = sorted(a.elapsed_time(b) for a, b in iso[2:])[len(iso[2:]) // 2]
    del flush

    # ---- leg 2 (reported beside it): batches are independent once sampled, so the gather of batch t runs on a
    # second, lower-priority stream while the sampling stream already works on the first hops of batch t+1 (small,
    # latency-bound kernels).  Two workspaces / output buffers alternate; the batch's row count is copied out of the
    # state header before the next batch clears it.  The gather uses many short blocks here so that the next batch's
    # kernels find free block slots at once.
    pipelined = None
    if not args.no_overlap:
        gs.gs_graph_set_gather_grid(G, args.gather_grid if args.gather_grid else 1024)
        ws_list = [ws, torch.empty_like(ws)]
        out_list = [out_rows, torch.empty_like(out_rows)]
        cnt_copy = [torch.zeros((), dtype=torch.int32, device=device) for _ in range(2)]
        s_gather = torch.cuda.Stream(device=device, priority=0)
        ready = [torch.cuda.Event() for _ in range(2)]
        done = [torch.cuda.Event() for _ in range(2)]
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        replicas.barrier()
        torch.cuda.synchronize()
        with torch.cuda.stream(s_main):
            for i in range(K + 3):                       # three untimed batches fill the pipeline
                if i == 3:
                    p0.record()
                j = i % 2
                s_main.wait_event(done[j])               # the gather that last read this workspace has finished
                blocks, input_nodes, cnt = one_step(Wm + K + (i % K), Wm + K + 1 + i, ws_list[j])
                cnt_copy[j].copy_(cnt)
                ready[j].record()
                s_gather.wait_event(ready[j])
                gs.gs_gather_features(G, input_nodes, cnt_copy[j], out_list[j], stream=s_gather)
                done[j].record(s_gather)
            for j in range(2):
                s_main.wait_event(done[j])
            p1.record()
        torch.cuda.synchronize()
        replicas.barrier()
        p_ms, _ = replicas.aggregate(p0.elapsed_time(p1), [0], device)
        pipelined = {"ms_per_step": p_ms / K, "what": "gather of batch t on a second stream beside the first hops of batch t+1; "
                     "same batches' worth of work, %d steps" % K,
                     "gather_grid_blocks_per_sm": args.gather_grid if args.gather_grid else 1024}
        gs.gs_graph_set_gather_grid(G, alone_grid)
        del ws_list, out_list
    if clocks:
        time.sleep(0.1)
        clocks.stop()

    # ---- end-to-end: seeds in pinned host memory go in, the batch's counts come back, every step (one stream)
    e2e = None
    if not args.no_e2e:
        host_seeds = [seeds_all[Wm + 2 * K + i].cpu().pin_memory() for i in range(K)]
        step0 = Wm + 2 * K + 8
        replicas.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e_edges = 0
        seeds_dev = torch.empty(B, dtype=torch.int32, device=device)
        with torch.cuda.stream(s_main):
            e0.record()
            for i in range(K):
                step = step0 + i
                if args.period and step % args.period == 0:
                    gs.gs_cache_refresh_all(C, refresh_mode, refresh_gamma, step)
                # seeds from pinned host memory, sampling and gather queued behind the copy, then the batch's counts
                # read back (synchronises the stream): the host never holds the GPU up between the two calls
                seeds_dev.copy_(host_seeds[i], non_blocking=True)
                blocks, input_nodes, cnt = gs.gs_sample_batch(C, seeds_dev, gm, gamma, step, ws)
                gs.gs_gather_features(G, input_nodes, cnt, out_rows)
                n, m = gs.gs_batch_counts(C)
                e_edges += sum(m)
            e1.record()
        torch.cuda.synchronize()
        replicas.barrier()
        e_ms, (e_edges_all,) = replicas.aggregate(e0.elapsed_time(e1), [e_edges], device)
        e2e = {"value": e_edges_all / (e_ms * 1e-3), "unit": "edges/s", "h2d_bytes_per_step": B * 4,
               "d2h_bytes_per_step": gs.COUNTS_READBACK_BYTES,
               "ms_per_step": e_ms / K}

    gs.gs_gather_status()     # raises if a bulk-copy gather ever ran out of patience (it never should)

    # ---- measured integer-ALU ceilings (nothing but the arithmetic, same process, same clocks)
    ceil = None
    if rank == 0:
        with torch.cuda.stream(s_main):
            ceil = {"philox_blocks_per_s": gs.gs_alu_ceiling(0, 30), "wide_multiplies_per_s": gs.gs_alu_ceiling(1, 30),
                    "logic_ops_per_s": gs.gs_alu_ceiling(2, 30)}

    t_ms, (edges_all, feat_rows_all, alg_all, alg_feat_all, gather_ms_max, philox_all) = replicas.aggregate(
        total_ms, [edges, feat_rows, alg_total, alg_feat, gather_ms, philox_blocks], device)
    if rank != 0:
        replicas.shutdown()
        return 0

    esize = 4 if cfg["feat_dtype"] == "f32" else 2
    peak, peak_kind = measured_peak()
    secs = t_ms * 1e-3
    sms = torch.cuda.get_device_properties(device).multi_processor_count
    clk = clocks.summary(wall0, wall1) if clocks else None
    sm_hz = (clk["sm_mhz"] or 1965.0) * 1e6 if clk else 1965.0e6
    gather_bytes_per_launch = alg_feat / K
    gather_ms_per_launch = gather_ms / Kb
    achieved = gather_bytes_per_launch / (gather_ms_per_launch * 1e-3) / 1e9
    last_rows = int(counts[K - 1][n_words[L]])
    alone_gbs = last_rows * (4 + 2 * cfg["feat_dim"] * esize) / (gather_alone_ms * 1e-3) / 1e9
    row_bytes = cfg["feat_dim"] * esize
    gather_traffic = None   # only the 256-byte-row capture scales cleanly by rows (no sector over-fetch)
    if row_bytes == 256:
        gather_traffic = (feat_rows / K) * (NCU_GATHER_READ_BYTES_PER_256B_ROW + row_bytes)
    roof_gather = {"kernel": "k_gather (feature rows), 1 launch per step", "bound": "hbm", "achieved": achieved,
                   "peak": peak, "peak_kind": "of " + peak_kind, "unit": "GB/s", "frac": achieved / peak,
                   "ms_per_launch": gather_ms_per_launch, "traffic": gather_traffic,
                   "alone": {"achieved": alone_gbs, "frac": alone_gbs / peak, "ms_per_launch": gather_alone_ms,
                             "what": "the same rows with nothing else running, L2 flushed before each launch, median of 6"},
                   "traffic_note": "bytes per launch; read bytes scaled by rows from an ncu capture of the same kernel on "
                                   "256-byte rows, written bytes algorithmic" if gather_traffic else
                                   "no capture with this row size scales by rows"}
    # the threshold scan (k_scan, one launch per sampling step) is bound by integer ALU work: Philox blocks
    scan_launches = Kb * L
    roof_scan = None
    if group_ms["scan"] > 0 and philox_blocks_b > 0:
        a_scan = philox_blocks_b / (group_ms["scan"] * 1e-3) / 1e9
        # derived peak: a Philox4x32-10 block is 20 wide multiplies and 20 three-input logic operations.  Integer
        # multiplies and logic operations share one datapath (the profiler shows its two pipes' active cycles adding up
        # to the elapsed ones, and a multiply + xor pair runs at half the rate of a lone logic operation), so the block
        # costs 40 integer instructions at the measured integer rate (rounded to a power of two lanes per SM and clock).
        int_lanes = ceil["logic_ops_per_s"] / (sms * sm_hz)
        lanes = 2 ** round(__import__("math").log2(max(int_lanes, 1.0)))
        p_scan = sms * lanes * sm_hz / 40.0 / 1e9
        roof_scan = {"kernel": "k_scan (Philox threshold scan), %d launches per step" % L, "bound": "alu",
                     "achieved": a_scan, "peak": p_scan,
                     "peak_kind": "derived: %d SMs x %d integer lanes per SM and clock x %.0f MHz / 40 integer instructions per "
                                  "block (measured: %.1f logic lanes, %.1f multiply + xor pairs per SM and clock)"
                                  % (sms, lanes, sm_hz / 1e6, int_lanes, ceil["wide_multiplies_per_s"] / (sms * sm_hz)),
                     "unit": "G Philox4x32-10 blocks/s", "frac": a_scan / p_scan,
                     "peak_measured": ceil["philox_blocks_per_s"] / 1e9,
                     "frac_of_measured": a_scan / (ceil["philox_blocks_per_s"] / 1e9),
                     "peak_measured_kind": "a kernel of nothing but the scan's Philox blocks and threshold test, same run",
                     "ms_per_launch": group_ms["scan"] / scan_launches,
                     "traffic": NCU_SCAN_BYTES_PER_BLOCK * philox_blocks_b / scan_launches,
                     "traffic_note": "DRAM bytes per launch, scaled by Philox blocks from an ncu capture of the same kernel "
                                     "on the large workload (an upper estimate: the traffic follows work items, and larger "
                                     "rows have fewer items per block); the scan reads no CSR bytes"}
    # the kernel group with the largest time on the one stream (nothing overlaps there)
    groups = dict(group_ms)
    groups["gather"] = gather_ms
    dominant = max(groups, key=groups.get)
    med_s = median_ms * 1e-3
    alg_b, phil_b = alg_total / K, philox_blocks / K
    result = {
        "metric": METRIC,
        "value": edges_all / secs,
        "unit": "edges/s",
        "feature_gbs": feat_rows_all * cfg["feat_dim"] * esize / secs / 1e9,
        "ms_per_step_median": median_ms,
        "hbm_frac_batch": (alg_b / med_s / 1e9) / peak,
        "hbm_frac_batch_incl_scanned_csr": ((alg_b + 16.0 * phil_b) / med_s / 1e9) / peak,
        "hbm_frac_batch_incl_scanned_csr_of_nominal_8tbs": ((alg_b + 16.0 * phil_b) / med_s / 1e9) / 8000.0,
        "hbm_frac_note": "per batch, from the median batch time of this rank on one stream; the second figure also charges "
                         "4 bytes per scanned edge offset, which this design evaluates keys for but never reads",
        "n_gpus": world,
        "steps": K,
        "warmup": Wm,
        "ms_per_step": t_ms / K,
        "higher_is_better": True,
        "scaling": "weak",
        "vs_baseline": None,
        "dtype": "int32 ids + %s feature copy" % cfg["feat_dtype"],
        "data": "synthetic",
        "config": {"workload": cfg["name"], "num_nodes": g.num_nodes, "num_edges": g.num_edges,
                   "fanouts": cfg["fanouts"], "cache_width": cfg["cache_width"], "mode": mode, "gamma": gamma,
                   "batch": B, "shared_cache": cfg["shared"], "feat_dim": cfg["feat_dim"],
                   "theta": args.theta, "period": args.period, "dedup": args.dedup or "default",
                   "refresh": ({"mode": mode, "gamma": refresh_gamma} if args.period else "per batch, frontier rows"), "cache_bytes": C.storage.numel(),
                   "parallelism": "replicas x%d" % world, "l2": "inputs_larger_than_L2",
                   "streams": "one: sample_batch then gather_features, batch after batch",
                   "gather_kernel": "bulk copies through shared memory where the rows allow it (128 - 512 bytes on 64-byte boundaries), else "
                                    "loads / stores with 16 blocks per SM" if alone_grid < 0 else "loads / stores, 16 blocks per SM",
                   "sampled_edges_per_batch": edges / K, "input_nodes_per_batch": feat_rows / K},
        "breakdown_ms_per_step": {"sample_batch": sample_ms / Kb, "gather_features": gather_ms / Kb,
                                  "kernel_groups": {k: v / Kb for k, v in groups.items()}, "dominant": dominant,
                                  "ms_per_step_with_these_events": breakdown_total_ms / Kb, "steps": Kb,
                                  "what": "a second pass over the same batches with CUDA events around the kernel "
                                          "groups; the headline pass above records batch boundaries only"},
        "frontier_shares_last_batch": {"refreshed": refreshed_frac, "refill_from_scan_list": listed_frac,
                                       "n_by_step": n_last},
        "pipelined": pipelined,
        "verified": verified,
        "alu_ceiling": ceil,
        "philox_blocks_per_batch": philox_blocks / K,
        "slow_refills_per_batch": slow_refills / K,
        "presample_ms": presample_ms,
        "whole_cache_refresh_ms": ([a.elapsed_time(b) for a, b in refresh_events] if args.period else None),
        "setup_s": {"graph_and_features": t_graph},
        "roofline": roof_scan if (dominant == "scan" and roof_scan) else roof_gather,
        "roofline_gather": roof_gather,
        "roofline_scan": roof_scan,
        "algorithmic_bytes_per_batch": alg_total / K,
        "gpu_launches": launches,
        "clocks": clk,
    }
    if pipelined:
        pipelined["value"] = result["value"] * result["ms_per_step"] / pipelined["ms_per_step"]
    if e2e:
        result["e2e"] = e2e
    if not args.no_cpu_baseline and world == 1:
        indptr_h, indices_h = g.indptr.cpu().numpy(), g.indices.cpu().numpy()
        if cfg["feat_kind"] != "hash":
            cpu_oracle_baseline.features = X.cpu()
        v, fg, desc, _ = cpu_oracle_baseline(cfg, indptr_h, indices_h, perm.cpu(), mode, gamma, theta=args.theta)
        result["cpu_baseline"] = {"value": v, "unit": "edges/s", "feature_gbs": fg, "cores": 1,
                                  "host_cores": os.cpu_count(), "kind": "oracle", "sample": desc}
    print(json.dumps(result))
    replicas.shutdown()
    return 0


def gather_arm(args, cfg, device):
    """gs_gather_features alone: ROWS distinct rows of the workload's feature matrix in a seeded random order."""
    import paper_2406_17918_b200 as gs
    from workloads.hashing import splitmix64

    N, rows = cfg["num_nodes"], args.gather_only
    X = build_features(cfg, device=device if cfg["feat_kind"] == "hash" else "cpu").to(device)
    rows = min(rows, N)
    # distinct rows in a seeded random order: every row is read from DRAM once, none is served twice from L2
    ids = torch.argsort(splitmix64(torch.arange(N, dtype=torch.int64, device=device) + 0x5EED))[:rows].to(torch.int32)
    indptr = torch.zeros(N + 1, dtype=torch.int64, device=device)
    G = gs.gs_graph_create(indptr, torch.zeros(1, dtype=torch.int32, device=device), X)
    gs.gs_graph_set_gather_grid(G, 16 if args.gather_kernel == "loads" else -1)
    out = torch.empty((rows, cfg["feat_dim"]), dtype=X.dtype, device=device)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
    times = []
    for i in range(args.warmup + args.steps):
        flush.zero_()                       # larger than L2: no row survives between launches
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        gs.gs_gather_features(G, ids, None, out)
        b.record()
        torch.cuda.synchronize()
        if i >= args.warmup:
            times.append(a.elapsed_time(b))
    times.sort()
    ms = times[len(times) // 2]
    esize = 4 if cfg["feat_dtype"] == "f32" else 2
    nbytes = rows * (4 + 2 * cfg["feat_dim"] * esize)
    peak, peak_kind = measured_peak()
    assert torch.equal(out.view(torch.int16 if esize == 2 else torch.int32), X[ids.long()].view(torch.int16 if esize == 2 else torch.int32))
    print(json.dumps({"gather_only": {"workload": cfg["name"], "rows": rows, "row_bytes": cfg["feat_dim"] * esize,
                                      "ms_per_launch_median": ms, "algorithmic_bytes": nbytes,
                                      "achieved_gbs": nbytes / (ms * 1e-3) / 1e9, "peak_gbs": peak, "peak_kind": "of " + peak_kind,
                                      "frac": nbytes / (ms * 1e-3) / 1e9 / peak, "gpu_launches": args.warmup + args.steps}}))
    return 0


def sharded_arm(args, cfg, mode, gamma, rank, local_rank, world, device):
    """Node-sharded sampling: every rank samples its own batch per step; frontier nodes are served by
    their owners.  Same metric, whole-job edges/s; host syncs of the exchange are inside the timed region."""
    import paper_2406_17918_b200 as gs
    from paper_2406_17918_b200 import replicas, sharded

    theta = 32 if args.theta is None else args.theta
    # With one process, --local-ranks R runs R ranks of a sharded job on this GPU, phase by phase (nothing waits
    # on anything): what the protocol and the owners' merged serving cost and save can be measured without R GPUs.
    R = max(1, args.local_ranks) if world == 1 else 1
    vworld = world * R
    g = build_graph(cfg, device=device)
    N = cfg["num_nodes"]
    num_edges = g.num_edges
    perm = seed_permutation(cfg, device=device)
    B, L = cfg["batch"], len(cfg["fanouts"])
    bound = B
    for k in range(L - 1):
        bound = min(N, bound * (1 + cfg["fanouts"][L - 1 - k]))
    shards = [sharded.shard_csr(g.indptr, g.indices, rank * R + j, vworld) for j in range(R)]
    del g
    mine = []
    for j, (ip, idx) in enumerate(shards):
        X = build_features(cfg, device=device, row_range=sharded.shard_range(N, rank * R + j, vworld))
        mine.append(sharded.ShardRank(gs, rank * R + j, vworld, ip, idx, X, cfg["fanouts"], cfg["cache_width"], SAMPLER_SEED,
                                      cfg["shared"], theta, max_seeds=B, max_requests=bound))
    del shards
    me = mine[0]
    gm = {"otf": gs.GS_MODE_OTF, "fcr": gs.GS_MODE_FCR, "fbl": gs.GS_MODE_FBL, "fetch": gs.GS_MODE_OTF_FETCH}[mode]
    K, Wm = args.steps, args.warmup

    # The feature step: a round trip like a hop (ids out, rows back, reordered), or one kernel that loads every
    # row straight from its owner's memory.  The latter needs the peers' feature shards mapped into this
    # process; with one process every "peer" is this GPU.
    feat = args.feature_exchange or ("peer" if world == 1 else "roundtrip")
    if feat == "peer" and world > 1:
        raise SystemExit("--feature-exchange peer needs the peers' feature shards mapped into every process: not set up by this script")

    def one(step):
        """-> (edges, input rows) of this process's batches of the step"""
        if world > 1:
            blocks, frontier, n, m, feats = sharded.sample_batch(me, batch_seeds(perm, step, B, rank, world), gm, gamma, step)
            return sum(m), n[L]
        res = sharded.sample_batch_local(mine, [batch_seeds(perm, step, B, j, R) for j in range(R)], gm, gamma, step,
                                         features="peer" if feat == "peer" else True)
        return sum(sum(r[3]) for r in res), sum(r[2][L] for r in res)

    def largest_groups(seen):
        for r in mine:
            seen = [max(a, b) for a, b in zip(seen, r.largest_groups())]
        return seen

    # Warm-up with exact-size exchanges (the host reads the group sizes of every exchange): the largest group
    # seen sizes the segments of the fixed-capacity exchanges the timed batches use (+25 %, the same on every rank).
    seen = [0] * (L + 1)
    for t in range(1, Wm + 1):
        one(t)
        seen = largest_groups(seen)
    exact_ms = None
    if not args.exact_sizes:
        torch.cuda.synchronize()
        x0, x1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        x0.record()
        for t in range(Wm + 1, Wm + 1 + max(3, K // 4)):
            one(t)
            seen = largest_groups(seen)
        x1.record()
        torch.cuda.synchronize()
        exact_ms = replicas.aggregate(x0.elapsed_time(x1) / max(3, K // 4), [0], device)[0]
        _, seen = replicas.aggregate(0.0, seen, device, reduce="max")
        caps = [(int(c * 1.25) + 255) // 256 * 256 for c in seen]
        for r in mine:
            r.set_capacities(caps, merge=False if args.no_merge else None)
        for t in range(1, 4):
            one(Wm + K + t)
    clocks = ClockSampler(local_rank) if rank == 0 else None
    time.sleep(0.3)
    replicas.barrier()
    torch.cuda.synchronize()
    launches0 = gs.gs_kernel_launches()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    wall0 = time.time()
    edges = rows = 0
    e0.record()
    for t in range(2 * Wm + K + 4, 2 * Wm + 2 * K + 4):
        em, rn = one(t)
        edges += em
        rows += rn
    e1.record()
    torch.cuda.synchronize()
    replicas.barrier()
    wall1 = time.time()
    launches = gs.gs_kernel_launches() - launches0
    t_ms, (edges_all, rows_all) = replicas.aggregate(e0.elapsed_time(e1), [edges, rows], device)
    if clocks:
        clocks.stop()
    if rank == 0:
        esize = 4 if cfg["feat_dtype"] == "f32" else 2
        print(json.dumps({
            "metric": METRIC, "value": edges_all / (t_ms * 1e-3), "unit": "edges/s",
            "feature_gbs": rows_all * cfg["feat_dim"] * esize / (t_ms * 1e-3) / 1e9,
            "n_gpus": world, "steps": K, "warmup": Wm, "ms_per_step": t_ms / K, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int32 ids + %s feature copy" % cfg["feat_dtype"],
            "data": "synthetic",
            "config": {"workload": cfg["name"], "num_nodes": N, "num_edges": num_edges, "fanouts": cfg["fanouts"],
                       "cache_width": cfg["cache_width"], "mode": mode, "gamma": gamma, "batch": B, "theta": theta,
                       "shared_cache": cfg["shared"], "feat_dim": cfg["feat_dim"],
                       "parallelism": "node-sharded x%d (one all-to-all round trip per hop%s)"
                                      % (vworld, "" if world > 1 else "; %d rank(s) in one process on one GPU, phase by phase: "
                                                                        "the exchange is a local copy" % R),
                       "ms_per_batch": t_ms / K / R,
                       "owner_serving": None if me.caps is None else
                                        ("requesters' lists merged, distinct nodes sampled once" if me.merge else "list by list"),
                       "exchange": "exact sizes (one host read per exchange)" if me.caps is None else
                                   "fixed capacity per pair of ranks %s, no host read inside a batch" % me.caps,
                       "ms_per_step_exact_sizes": exact_ms,
                       "feature_step": "one kernel of loads from the owners' memory" if feat == "peer" else
                                       "all-to-all round trip (ids out, rows back, reorder)",
                       "l2": "inputs_larger_than_L2", "cache_bytes_per_rank": me.cache.storage.numel()},
            "roofline": None, "e2e": None, "gpu_launches": launches,
            "clocks": clocks.summary(wall0, wall1) if clocks else None}))
    replicas.shutdown()
    return 0


def reference_arm(args, cfg, mode, gamma):
    """The CPU oracle, as it stands, on bounded samples of the same workload (one sample per step)."""
    dev = "cuda" if (torch.cuda.is_available() and cfg["kind"] == "rmat") else "cpu"
    g = build_graph(cfg, device=dev)
    indptr_h, indices_h = g.indptr.cpu().numpy(), g.indices.cpu().numpy()
    perm = seed_permutation(cfg)
    if cfg["feat_kind"] != "hash":
        cpu_oracle_baseline.features = build_features(cfg)
    # size the per-step sample once, then time warm-up + K steps at that size
    v, fg, desc, dt = cpu_oracle_baseline(cfg, indptr_h, indices_h, perm, mode, gamma, budget_s=8.0, theta=args.theta)
    s = int(desc.split("first ")[1].split(" ")[0])
    per_step_budget = max(1, min(args.steps, int(120.0 / max(dt, 1e-3))))
    K = per_step_budget
    tot_edges, tot_t, fgs = 0.0, 0.0, []
    for i in range(min(args.warmup, 1) + K):
        vv, ff, _, tt = cpu_oracle_baseline(cfg, indptr_h, indices_h, perm, mode, gamma, first_seeds=s, theta=args.theta)
        if i >= min(args.warmup, 1):
            tot_edges += vv * tt
            tot_t += tt
            fgs.append(ff)
    value = tot_edges / tot_t
    sample = "each step: " + desc.split(", %.2f" % dt)[0] + "; %d timed steps" % K
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "edges/s", "n_gpus": args.gpus,
        "steps": K, "warmup": min(args.warmup, 1), "ms_per_step": tot_t / K * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int32 ids + %s feature copy" % cfg["feat_dtype"],
        "data": "synthetic",
        "config": {"workload": cfg["name"], "num_nodes": g.num_nodes, "num_edges": g.num_edges,
                   "fanouts": cfg["fanouts"], "cache_width": cfg["cache_width"], "mode": mode, "gamma": gamma,
                   "batch": cfg["batch"], "shared_cache": cfg["shared"], "feat_dim": cfg["feat_dim"]},
        "cpu_baseline": {"value": value, "unit": "edges/s", "cores": 1, "host_cores": os.cpu_count(),
                         "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "edges/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


if __name__ == "__main__":
    sys.exit(main())
