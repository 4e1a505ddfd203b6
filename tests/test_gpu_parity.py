"""CUDA library vs CPU oracle, element by element, through the C ABI (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle
from workloads import batch_seeds, get_config

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tiny():
    from parity import Pair
    return Pair(get_config("tiny"))


@pytest.fixture(scope="module")
def mid():
    from parity import Pair
    return Pair(get_config("mid"))


@pytest.fixture(scope="module")
def shared_cfg():
    from parity import Pair
    return Pair(get_config("shared"))


def test_presample_all_rows_tiny_mid(tiny, mid):
    for pair in (tiny, mid):
        C, ws, O = pair.samplers(8)
        pair.check_rows(C, O, np.arange(pair.cfg["num_nodes"], dtype=np.int32))


def test_tiny_otf_20_batches(tiny):
    tiny.run("otf", 0.25, 20)


def test_tiny_fcr_and_gamma_edges(tiny):
    tiny.run("fcr", 0.0, 4)
    tiny.run("otf", 0.0, 3)
    tiny.run("otf", 1.0, 3)


def test_tiny_host_seed_entry_point(tiny):
    tiny.run("otf", 0.25, 3, host_api=True)


@pytest.mark.parametrize("mode,gamma", [("fcr", 1.0), ("otf", 0.1), ("otf", 0.3), ("otf", 0.5)])
def test_mid_runs(mid, mode, gamma):
    mid.run(mode, gamma, 4)


@pytest.mark.parametrize("tuning", [
    dict(lambda_otf=0.5, lambda_full=1.0),          # thresholds too tight: retry and exact paths decide
    dict(lambda_otf=1e6, lambda_full=1e6),          # thresholds too loose: buffer overflow -> exact path
    dict(hub_degree=40),                            # almost every refreshed node takes the block kernel
    dict(lambda_otf=0.5, lambda_full=1.0, hub_degree=40),
    dict(lambda_otf=1e6, lambda_full=1e6, hub_degree=40),
])
def test_mid_internal_paths_agree(mid, tuning):
    mid.run("otf", 0.3, 2, tuning=tuning)
    mid.run("fcr", 1.0, 1, tuning=tuning)


def test_full_batch_load_mode(tiny, mid, shared_cfg):
    # no cache: every hop samples the CSR rows directly; cache rows must stay as pre-sampled
    tiny.run("fbl", 0.0, 5)
    mid.run("fbl", 0.0, 2)
    mid.run("fbl", 0.0, 1, tuning=dict(hub_degree=40))
    mid.run("fbl", 0.0, 1, tuning=dict(lambda_full=1.0))
    shared_cfg.run("fbl", 0.0, 1)


@pytest.mark.parametrize("delta", [0.0, 0.04, 0.3, 0.5, 1.0])
def test_otf_fetch_mode(tiny, mid, delta):
    # part of every sample comes straight from the graph; the cache rows must stay as pre-sampled
    tiny.run("fetch", delta, 3)
    mid.run("fetch", delta, 2)


def test_otf_fetch_mode_internal_paths_and_shared(mid, shared_cfg):
    mid.run("fetch", 0.4, 1, tuning=dict(lambda_otf=0.5, lambda_full=1.0))
    mid.run("fetch", 0.4, 1, tuning=dict(lambda_otf=1e6, lambda_full=1e6))
    shared_cfg.run("fetch", 0.3, 2)
    # modes can be mixed on one cache from batch to batch
    C, ws, O = mid.samplers(mid.cfg["batch"])
    for b, (mode, rate) in enumerate([("otf", 0.3), ("fetch", 0.5), ("fbl", 0.0), ("fcr", 0.0), ("fetch", 0.2), ("otf", 0.1)]):
        mid.check_batch(C, ws, O, batch_seeds(mid.perm, b, mid.cfg["batch"]), mode, rate, b + 1)


@pytest.mark.parametrize("theta", [10, 16, 128])
def test_dense_sparse_split_tiny(tiny, theta):
    C, ws, O, _ = tiny.run("otf", 0.25, 4, theta=theta)
    tiny.check_rows(C, O, np.arange(tiny.cfg["num_nodes"], dtype=np.int32))
    tiny.run("fcr", 0.0, 2, theta=theta)


def test_dense_sparse_split_other_modes_and_graphs(mid, shared_cfg):
    import paper_2406_17918_b200 as gs
    mid.run("otf", 0.3, 3, theta=20)
    mid.run("otf", 0.0, 1, theta=64)
    mid.run("fetch", 0.4, 2, theta=48)
    mid.run("fbl", 0.0, 1, theta=48)
    mid.run("fcr", 1.0, 1, theta=128, tuning=dict(lambda_full=1.0))
    shared_cfg.run("otf", 0.3, 2, theta=32)
    # the split cache is much smaller: rows only for the dense part
    G = mid.G
    dense = int((mid.deg > 20).sum())
    full = gs.gs_cache_bytes(G, 3, 20, False)
    split = gs.gs_cache_bytes_split(G, 3, 20, False, dense)
    assert split < 0.25 * full
    with pytest.raises(gs.GsError) as e:
        gs.gs_cache_init_split(G, [15, 10, 5], 20, 1, False, 20, dense_rows=dense + 1)
    assert e.value.status == 1 and "dense_rows" in str(e.value)
    with pytest.raises(gs.GsError):
        gs.gs_cache_init_split(G, [15, 10, 5], 20, 1, False, 129)


def test_periodic_whole_cache_refresh(tiny, mid, shared_cfg):
    import paper_2406_17918_b200 as gs
    tiny.run_periodic("otf", 0.3, 2, 6)
    tiny.run_periodic("fcr", 0.0, 3, 6)
    tiny.run_periodic("otf", 0.5, 2, 4, theta=16)
    mid.run_periodic("otf", 0.25, 2, 4, rows=64, features=False)
    mid.run_periodic("fcr", 0.0, 2, 2, rows=64, features=False, tuning=dict(hub_degree=64))
    C, ws, O = shared_cfg.run_periodic("otf", 0.3, 2, 2, rows=64, features=False)
    # a whole-cache refresh followed by per-batch refreshes keeps working (stamps restart cleanly)
    shared_cfg.check_batch(C, ws, O, batch_seeds(shared_cfg.perm, 7, shared_cfg.cfg["batch"]), "otf", 0.3, 3, rows=64)
    for bad in [(gs.GS_MODE_FBL, 0.0, 1), (gs.GS_MODE_OTF_FETCH, 0.5, 1), (gs.GS_MODE_OTF, 1.5, 1), (gs.GS_MODE_FCR, 0.0, 0)]:
        with pytest.raises(gs.GsError):
            gs.gs_cache_refresh_all(C, *bad)


def test_shared_cache_mode(shared_cfg):
    shared_cfg.run("otf", 0.3, 3)
    shared_cfg.run("fcr", 0.0, 1)


def test_shared_presample_sample(shared_cfg):
    C, ws, O = shared_cfg.samplers(8)
    rng = np.random.default_rng(1)
    hubs = np.argsort(-shared_cfg.deg)[:200]
    nodes = np.concatenate([hubs, rng.integers(0, shared_cfg.cfg["num_nodes"], 3000)]).astype(np.int32)
    shared_cfg.check_rows(C, O, nodes)


def test_batch_stats_and_event_profile(mid):
    """The diagnostics counters agree with the oracle's own count of refreshed rows, and the optional
    event timing returns one positive figure per kernel group."""
    import paper_2406_17918_b200 as gs
    B = mid.cfg["batch"]
    C, ws, O = mid.samplers(B)
    gs.gs_cache_profile_begin(C, 2)
    for b in range(3):                                  # the third batch is beyond max_batches: not timed
        seeds = batch_seeds(mid.perm, b, B)
        n, m = mid.check_batch(C, ws, O, seeds, "otf", 0.3, b + 1, features=False, rows=False)
        st = gs.gs_batch_stats(C)
        refreshed, scanned = O.stats()
        assert st["refreshed_nodes"] == refreshed
        assert 0 <= st["slow_refills"] <= refreshed and st["queued_rescans"] <= st["slow_refills"]
        assert 0 < st["philox_blocks"] <= (scanned + 3 * refreshed) // 4 + refreshed
    ms, batches = gs.gs_cache_profile_end(C)
    assert batches == 2 and set(ms) == {"row_counts", "scan", "finish", "relabel"}
    assert all(v > 0 for v in ms.values())
    with pytest.raises(gs.GsError):
        gs.gs_cache_profile_end(C)                      # not on any more
    assert gs.gs_stats_word_offset() > 0


def test_ragged_batch_sizes(tiny):
    for B in (1, 2, 31, 33, 1000):
        tiny.run("otf", 0.25, 2, batch_size=B)


def test_whole_graph_as_seeds(tiny):
    # every node is a seed: later frontiers cannot grow, dedup sees only known ids
    C, ws, O, out = tiny.run("otf", 0.25, 1, batch_size=tiny.cfg["num_nodes"])
    n, m = out[0]
    assert n[0] == n[-1] == tiny.cfg["num_nodes"]


@pytest.mark.parametrize("fanouts,W", [([1], 1), ([32], 32), ([3], 32), ([2] * 8, 4), ([5, 5], 5), ([1, 32, 1], 32)])
def test_extreme_shapes(fanouts, W):
    """One hop and the maximum of eight, cache width 1 and the maximum 32, fan-out equal to the width."""
    from parity import Pair
    pair = Pair(get_config("tiny", fanouts=fanouts, cache_width=W), features=False)
    for mode, gamma in (("otf", 0.3), ("fcr", 0.0), ("fetch", 0.5), ("fbl", 0.0)):
        pair.run(mode, gamma, 2, batch_size=48, features=False)


def test_otf_fetch_with_every_sample_fetched_and_fanout_equal_to_width():
    """delta = 1 with f = W: as many neighbours are fetched as the row has slots, and the row must stay as it is."""
    from parity import Pair
    pair = Pair(get_config("tiny", fanouts=[10, 10], cache_width=10), features=False)
    pair.run("fetch", 1.0, 3, features=False)
    pair = Pair(get_config("mid", fanouts=[20, 20], cache_width=20), features=False)
    pair.run("fetch", 1.0, 2, batch_size=256, features=False, rows=500)
    pair.run("fetch", 1.0, 1, batch_size=256, features=False, rows=500, tuning=dict(lambda_full=1.0, hub_degree=64))
    pair.run("fetch", 0.97, 1, batch_size=256, features=False, rows=500, tuning=dict(lambda_otf=1.0))


def test_hand_made_graphs_hub_isolated_and_chain():
    """A hub far above every chunking threshold next to isolated nodes; seeds without neighbours."""
    from helpers import csr_from_rows
    from parity import Pair
    hub_deg = 150_000
    n = hub_deg + 40
    rows = [[] for _ in range(n)]
    rows[0] = list(range(40, n))                    # the hub: every node from 40 on points to node 0
    rows[1] = list(range(40, 40 + 9000))            # above the degree at which a row is split over warps
    rows[2] = list(range(40, 40 + 129))             # just above the in-register limit
    rows[3] = list(range(40, 40 + 128))             # at the in-register limit
    rows[4] = list(range(40, 40 + 33))
    rows[5] = list(range(40, 40 + 32))              # holds its whole adjacency
    for v in range(40, 60):
        rows[v] = [0, 1, 2, 3, 4, 5]                # so that later hops reach the hub rows again
    indptr, indices = csr_from_rows(rows)
    pair = Pair.from_csr(indptr, indices, [7, 10], 32)
    C, ws, O = pair.samplers(64)
    pair.check_rows(C, O, np.arange(64))
    seeds = torch.arange(0, 64, dtype=torch.int32)                          # rows 6..39 are isolated
    for step, (mode, gamma) in enumerate([("otf", 0.1), ("otf", 0.5), ("fcr", 0.0), ("fetch", 0.3), ("fbl", 0.0)], 1):
        pair.check_batch(C, ws, O, seeds, mode, gamma, step, features=False)
    # only isolated seeds: every block is empty and the frontier is the seeds
    iso = torch.arange(6, 40, dtype=torch.int32)
    n_, m_ = pair.check_batch(C, ws, O, iso, "otf", 0.3, 9, features=False)
    assert n_ == [34, 34, 34] and m_ == [0, 0]
    # the same graph with a split cache and a whole-cache refresh
    C2, ws2, O2 = pair.samplers(64, theta=64)
    pair.check_batch(C2, ws2, O2, seeds, "otf", 0.25, 1, features=False)
    import paper_2406_17918_b200 as gs
    gs.gs_cache_refresh_all(C2, gs.GS_MODE_OTF, 0.5, 2)
    O2.refresh_all(oracle.MODE_OTF, 0.5, 2)
    pair.check_rows(C2, O2, np.arange(64))


@pytest.mark.parametrize("shared", [False, True])
def test_degrees_at_every_internal_threshold(shared):
    """Rows whose degree sits on and next to each switch inside the kernels (cache width, the in-register
    limit, the candidate-pop switch, the scan chunk, the degree from which a row is split over warps), with the
    default thresholds and with thresholds that make the first attempt fail."""
    from helpers import csr_from_rows
    from parity import Pair
    degs = [0, 1, 31, 32, 33, 63, 64, 65, 127, 128, 129, 1023, 1024, 1025, 4095, 4096, 4097, 4100, 8191, 8192, 8193, 12289, 20000]
    base = 64
    n = base + max(degs)
    rows = [[] for _ in range(n)]
    for v, d in enumerate(degs):
        rows[v] = list(range(base, base + d))
    for v in range(base, base + 40):
        rows[v] = list(range(0, len(degs)))          # the next hop comes back to the rows above
    indptr, indices = csr_from_rows(rows)
    pair = Pair.from_csr(indptr, indices, [9, 32], 32, shared=shared)
    seeds = torch.arange(0, len(degs), dtype=torch.int32)
    runs = [("otf", 0.1), ("otf", 0.5), ("fcr", 0.0), ("fetch", 0.3), ("fetch", 1.0), ("fbl", 0.0), ("otf", 0.97)]
    for tuning in (None, dict(lambda_otf=1.0, lambda_full=4.0), dict(lambda_otf=60.0, lambda_full=200.0), dict(hub_degree=64)):
        C, ws, O = pair.samplers(len(degs), tuning=tuning)
        pair.check_rows(C, O, np.arange(len(degs)))
        for i, (mode, gamma) in enumerate(runs):
            step = 0xFFFFFFFF - i if tuning is None else i + 1           # the largest step numbers as well
            pair.check_batch(C, ws, O, seeds, mode, gamma, step, features=False)


def _random_graph(rng):
    n = int(rng.integers(200, 2500)) if rng.random() < 0.75 else int(rng.integers(9000, 12000))
    kind = rng.random(n)
    deg = np.where(kind < 0.15, 0, np.where(kind < 0.75, rng.integers(1, 40, n), rng.integers(40, 400, n)))
    for v in rng.choice(n, size=int(rng.integers(0, 4)), replace=False):      # a few rows far above the chunk sizes
        deg[v] = int(rng.integers(1500, min(n - 1, 20000) + 1)) if n > 1501 else n - 1
    deg = np.minimum(deg, n - 1)
    indptr = np.zeros(n + 1, dtype=np.int64)
    indptr[1:] = np.cumsum(deg)
    indices = np.empty(int(indptr[-1]), dtype=np.int32)
    for v in range(n):
        if deg[v]:
            nb = rng.choice(n - 1, size=int(deg[v]), replace=False)
            nb = np.sort(np.where(nb >= v, nb + 1, nb))                        # no self loop, sorted, distinct
            indices[indptr[v]:indptr[v + 1]] = nb
    return indptr, indices


@pytest.mark.parametrize("case", range(64))
def test_randomised_configurations(case):
    """Seeded random graphs, shapes, modes, rates, splits and thresholds: everything compared with the oracle."""
    from parity import Pair
    rng = np.random.default_rng(1000 + case)
    indptr, indices = _random_graph(rng)
    n = len(indptr) - 1
    L = int(rng.integers(1, 5))
    W = int(rng.choice([1, 2, 5, 8, 16, 20, 31, 32]))
    fanouts = [int(rng.integers(1, W + 1)) for _ in range(L)]
    shared = bool(rng.random() < 0.3)
    theta = None if rng.random() < 0.6 else int(rng.integers(W, 129))
    tuning = None
    if rng.random() < 0.4:
        tuning = dict(lambda_otf=float(rng.choice([1.0, 4.0, 40.0])), lambda_full=float(rng.choice([2.0, 30.0, 150.0])),
                      hub_degree=int(rng.choice([64, 1000, 8192])))
    pair = Pair.from_csr(indptr, indices, fanouts, W, shared=shared, seed=int(rng.integers(1, 2**63)))
    B = int(rng.integers(1, min(n, 300) + 1))
    C, ws, O = pair.samplers(B, tuning=tuning, theta=theta)
    pair.check_rows(C, O, np.arange(n))
    step = int(rng.integers(1, 2**32 - 10))
    for b in range(4):
        mode = str(rng.choice(["otf", "otf", "fcr", "fetch", "fbl"]))
        rate = float(rng.choice([0.0, 0.1, 0.25, 0.5, 0.9, 1.0]))
        seeds = torch.from_numpy(rng.choice(n, size=int(rng.integers(1, B + 1)), replace=False).astype(np.int32))
        pair.check_batch(C, ws, O, seeds, mode, rate, step + b, features=False)
        if rng.random() < 0.25:
            import paper_2406_17918_b200 as gs
            which = str(rng.choice(["otf", "fcr"]))
            gs.gs_cache_refresh_all(C, {"otf": gs.GS_MODE_OTF, "fcr": gs.GS_MODE_FCR}[which], rate, step + b)
            O.refresh_all({"otf": oracle.MODE_OTF, "fcr": oracle.MODE_FCR}[which], rate, step + b)
    pair.check_rows(C, O, np.arange(n))


def test_graph_contract_check(tiny):
    import paper_2406_17918_b200 as gs
    assert gs.gs_graph_validate(tiny.G) == -1
    indptr, indices = torch.from_numpy(tiny.indptr), torch.from_numpy(tiny.indices)
    v = int(np.nonzero(tiny.deg >= 3)[0][5])
    a = int(tiny.indptr[v])

    def first_bad(ip, ix):
        G = gs.gs_graph_create(ip.cuda(), ix.cuda(), None)
        with pytest.raises(gs.GsError) as e:
            gs.gs_graph_validate(G)
        assert e.value.status == 1
        return int(str(e.value).split("CSR row ")[1].split(" ")[0])

    ix = indices.clone(); ix[a], ix[a + 1] = indices[a + 1], indices[a]          # not ascending
    assert first_bad(indptr, ix) == v
    ix = indices.clone(); ix[a + 1] = ix[a]                                        # duplicate neighbour
    assert first_bad(indptr, ix) == v
    ix = indices.clone(); ix[a + 2] = tiny.cfg["num_nodes"]                        # id out of range
    assert first_bad(indptr, ix) == v
    ix = indices.clone(); ix[a] = -4
    assert first_bad(indptr, ix) == v
    ip = indptr.clone(); ip[v + 1] = ip[v] - 1                                     # offsets decrease
    assert first_bad(ip, indices) == v
    ip = indptr.clone(); ip[-1] += 1                                               # last offset is not num_edges
    assert first_bad(ip, indices) == tiny.cfg["num_nodes"] - 1


def test_pipelined_batches_with_the_gather_on_a_second_stream(mid):
    """The launch pattern the benchmark times: batches enqueued back to back without a host sync, each batch's
    gather on a second stream overlapping the next batch, two workspaces and output buffers alternating."""
    import paper_2406_17918_b200 as gs
    B, K, L = 1024, 12, mid.L
    C, ws0, O = mid.samplers(B)
    ws = [ws0, torch.empty_like(ws0)]
    hdr = C.storage[:512].view(torch.int32)
    pinned = torch.zeros((K, 128), dtype=torch.int32).pin_memory()
    s_main, s_gather = torch.cuda.Stream(priority=-1), torch.cuda.Stream(priority=0)
    ready = [torch.cuda.Event() for _ in range(2)]
    done = [torch.cuda.Event() for _ in range(2)]
    cnt_copy = [torch.zeros((), dtype=torch.int32, device="cuda") for _ in range(2)]
    out, sums, fronts = [None, None], [], []
    gs.gs_graph_set_gather_grid(mid.G, 1024)
    torch.cuda.synchronize()
    with torch.cuda.stream(s_main):
        for i in range(K):
            j = i & 1
            s_main.wait_event(done[j])
            blocks, input_nodes, cnt = gs.gs_sample_batch(C, batch_seeds(mid.perm, i, B).cuda(), gs.GS_MODE_OTF, 0.3, i + 1, ws[j])
            if out[j] is None:
                out[j] = torch.zeros((blocks[0].max_src, mid.X.shape[1]), dtype=mid.X.dtype, device="cuda")
            pinned[i].copy_(hdr, non_blocking=True)
            cnt_copy[j].copy_(cnt)
            ready[j].record()
            s_gather.wait_event(ready[j])
            with torch.cuda.stream(s_gather):
                gs.gs_gather_features(mid.G, input_nodes, cnt_copy[j], out[j], stream=s_gather)
                # a device-side digest of this batch's rows and ids, taken before the buffers are reused
                sums.append((out[j].view(torch.int32).sum(dtype=torch.int64), input_nodes.clone()))
                done[j].record(s_gather)
        s_main.wait_event(done[0])
        s_main.wait_event(done[1])
    torch.cuda.synchronize()
    gs.gs_graph_set_gather_grid(mid.G, 0)
    gs.gs_sync_status(C)
    n_word = blocks[0].count_words()[1]
    Xb = mid.X.view(torch.int32)
    prev_rows = [0, 0]
    for i in range(K):
        fr, n, _ = O.sample_batch(batch_seeds(mid.perm, i, B).numpy(), oracle.MODE_OTF, 0.3, i + 1)
        assert int(pinned[i][n_word]) == n[L]
        ids = sums[i][1][: n[L]]
        assert np.array_equal(ids.cpu().numpy(), fr)
        # rows beyond this batch's count still hold the previous use of the buffer (or zeros)
        want = Xb[ids.long()].sum(dtype=torch.int64)
        j = i & 1
        if prev_rows[j] > n[L]:
            want = want + Xb[sums[i - 2][1][n[L]:prev_rows[j]].long()].sum(dtype=torch.int64)
        prev_rows[j] = max(prev_rows[j], n[L])
        assert int(sums[i][0]) == int(want), i
    mid.check_rows(C, O, np.arange(mid.cfg["num_nodes"]))


def test_resume_from_export(tiny):
    import paper_2406_17918_b200 as gs
    B = tiny.cfg["batch"]
    C, ws, O = tiny.samplers(B)
    for b in range(3):
        tiny.check_batch(C, ws, O, batch_seeds(tiny.perm, b, B), "otf", 0.25, b + 1)
    blob = gs.gs_cache_export(C)
    C2, ws2, _ = tiny.samplers(B)
    gs.gs_cache_import(C2, blob)
    for b in range(3, 6):
        tiny.check_batch(C2, ws2, O, batch_seeds(tiny.perm, b, B), "otf", 0.25, b + 1)


def test_device_detected_errors(tiny):
    import paper_2406_17918_b200 as gs
    B = 16
    C, ws, O = tiny.samplers(B)
    good = batch_seeds(tiny.perm, 0, B)
    bad = good.clone()
    bad[5] = tiny.cfg["num_nodes"] + 3
    gs.gs_sample_batch(C, bad.cuda(), gs.GS_MODE_OTF, 0.25, 1, ws)
    with pytest.raises(gs.GsError) as e:
        gs.gs_batch_counts(C)
    assert e.value.status == 3
    dup = good.clone()
    dup[7] = dup[2]
    gs.gs_sample_batch(C, dup.cuda(), gs.GS_MODE_OTF, 0.25, 1, ws)
    with pytest.raises(gs.GsError) as e:
        gs.gs_batch_counts(C)
    assert e.value.status == 5
    # the cache is untouched by the rejected batches and the handle still works
    tiny.check_batch(C, ws, O, good, "otf", 0.25, 1)


def test_gather_bulk_copy_variant():
    """gs_graph_set_gather_grid(G, -1): the rows go through shared memory by bulk copies; same result, bit for bit."""
    import paper_2406_17918_b200 as gs
    from parity import bits
    g = torch.Generator().manual_seed(4)
    N = 5000
    indptr = torch.zeros(N + 1, dtype=torch.int64, device="cuda")
    indices = torch.zeros(1, dtype=torch.int32, device="cuda")
    # eligible: rows of 128 .. 512 bytes on 64-byte boundaries (4 warps per block up to 384 bytes, 3 above); the others
    # take the load/store kernel through the same call
    for dtype, d, ld in ((torch.bfloat16, 128, 128), (torch.float32, 32, 48), (torch.bfloat16, 192, 192), (torch.float32, 112, 112),
                         (torch.bfloat16, 256, 256), (torch.float32, 100, 100), (torch.bfloat16, 8, 8), (torch.float32, 36, 40),
                         (torch.float32, 1433, 1433), (torch.bfloat16, 7, 7)):
        base = torch.randn((N, ld), generator=g).to(dtype).cuda()
        X = base[:, :d]
        G = gs.gs_graph_create(indptr, indices, X)
        gs.gs_graph_set_gather_grid(G, -1)
        for n in (1, 31, 32, 33, 1000, 40001):
            ids = torch.randint(0, N, (n,), generator=g).to(torch.int32).cuda()
            out = torch.full((n + 5, d), 3, dtype=dtype, device="cuda")
            cnt = torch.tensor(n, dtype=torch.int32, device="cuda")
            gs.gs_gather_features(G, ids, cnt if n % 2 else None, out[:n])
            assert np.array_equal(bits(out[:n]), oracle.gather(bits(X), ids.cpu().numpy())), (dtype, d, n)
            assert bool((out[n:] == 3).all())
        # a device count below the bound: the rows beyond it stay as they are
        ids = torch.randint(0, N, (500,), generator=g).to(torch.int32).cuda()
        out = torch.full((500, d), 3, dtype=dtype, device="cuda")
        gs.gs_gather_features(G, ids, torch.tensor(77, dtype=torch.int32, device="cuda"), out)
        assert np.array_equal(bits(out[:77]), oracle.gather(bits(X), ids[:77].cpu().numpy())) and bool((out[77:] == 3).all())
    # rows of a shard addressed by global ids: ids outside the shard are skipped
    Xs = torch.randn((300, 64), generator=g).to(torch.bfloat16).cuda()
    ids = torch.randint(380, 720, (999,), generator=g).to(torch.int32).cuda()
    out = torch.full((999, 64), 9, dtype=torch.bfloat16, device="cuda")
    ref = out.clone()
    gs.gs_gather_rows(Xs, ids, ref, first_row=400)
    inside = (ids >= 400) & (ids < 700)
    assert torch.equal(ref[inside], Xs[(ids[inside] - 400).long()]) and bool((ref[~inside] == 9).all())
    gs.gs_gather_status()


def test_gather_alignment_paths():
    import paper_2406_17918_b200 as gs
    from parity import bits
    g = torch.Generator().manual_seed(0)
    indptr = torch.zeros(101, dtype=torch.int64, device="cuda")
    indices = torch.zeros(1, dtype=torch.int32, device="cuda")
    ids = torch.randint(0, 100, (257,), generator=g).to(torch.int32).cuda()
    for dtype, d, ld in ((torch.float32, 100, 100), (torch.float32, 1433, 1433), (torch.bfloat16, 128, 128),
                         (torch.bfloat16, 7, 7), (torch.float32, 6, 8), (torch.bfloat16, 130, 136), (torch.float32, 3, 3)):
        base = torch.randn((100, ld), generator=g).to(dtype).cuda()
        X = base[:, :d]
        G = gs.gs_graph_create(indptr, indices, X)
        for out_ld, grid in ((d, 0), (d + 3, 0), (d, 16), (d + 3, 16)):     # default kernel choice, and the load/store kernel
            gs.gs_graph_set_gather_grid(G, grid)
            outb = torch.zeros((257, out_ld), dtype=dtype, device="cuda")
            out = outb[:, :d]
            gs.gs_gather_features(G, ids, None, out)
            assert np.array_equal(bits(out), oracle.gather(bits(X), ids.cpu().numpy()))
            assert bool((outb[:, d:] == 0).all())
    out = torch.zeros((0, 3), dtype=torch.float32, device="cuda")
    gs.gs_gather_features(G, ids, None, out)           # empty gather is a no-op
