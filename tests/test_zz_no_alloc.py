"""gs_sample_batch_noalloc against gs_sample_batch (needs a B200; collected last on purpose).

Some users of the sampler cannot allocate device memory at all - their process runs inside a
memory pool that owns the whole GPU, or under a host application with a fixed budget - so they
have no workspace to give to gs_sample_batch.  The no-allocation entry point keeps its scratch in
an array inside the library and writes the results into buffers the caller already has.  This test
drives both entry points through the C ABI with the same seeds on two caches built from the same
seed, two batches in a row (the second batch finds the previous batch's leftovers in the shared
scratch array), and requires identical results: tolerance 0, as everywhere else in this suite.
"""
import pytest
import torch

from workloads import batch_seeds, build_graph, get_config, seed_permutation

pytestmark = pytest.mark.gpu


def _bounds(num_nodes, fanouts, seeds):
    n, m = [min(seeds, num_nodes)], []
    for f in reversed(fanouts):
        m.append(n[-1] * f)
        n.append(min(num_nodes, n[-1] + m[-1]))
    return n, m


@pytest.mark.parametrize("mode,gamma", [("otf", 0.25), ("fcr", 0.0)])
def test_noalloc_matches_workspace_call_two_batches_in_a_row(mode, gamma):
    import paper_2406_17918_b200 as gs

    cfg = get_config("tiny")
    g = build_graph(cfg).to("cuda")
    perm = seed_permutation(cfg)
    G = gs.gs_graph_create(g.indptr, g.indices, None)
    fan, W, B, L = cfg["fanouts"], cfg["cache_width"], cfg["batch"], len(cfg["fanouts"])
    gm = gs.GS_MODE_OTF if mode == "otf" else gs.GS_MODE_FCR
    ref = gs.gs_cache_init(G, fan, W, 77, False)
    sut = gs.gs_cache_init(G, fan, W, 77, False)
    ws = torch.empty(gs.gs_workspace_bytes(G, fan, B), dtype=torch.uint8, device="cuda")
    assert ws.numel() <= gs.NOALLOC_SCRATCH_BYTES

    # everything the no-allocation call writes to is created before the first call
    nb, mb = _bounds(cfg["num_nodes"], fan, B)
    input_nodes = torch.full((nb[L],), -7, dtype=torch.int32, device="cuda")
    indptr_bufs = [torch.full((nb[L - 1 - l] + 1,), -7, dtype=torch.int32, device="cuda") for l in range(L)]
    indices_bufs = [torch.full((mb[L - 1 - l],), -7, dtype=torch.int32, device="cuda") for l in range(L)]
    all_nodes = torch.arange(cfg["num_nodes"], dtype=torch.int32, device="cuda")

    for b in range(2):
        seeds = batch_seeds(perm, b, B).cuda()
        blocks_r, in_r, _ = gs.gs_sample_batch(ref, seeds, gm, gamma, b + 1, ws)
        n_r, m_r = gs.gs_batch_counts(ref)
        blocks_s = gs.gs_sample_batch_noalloc(sut, seeds, gm, gamma, b + 1, input_nodes, indptr_bufs, indices_bufs)
        n_s, m_s = gs.gs_batch_counts(sut)
        assert (n_s, m_s) == (n_r, m_r)
        assert torch.equal(input_nodes[: n_s[L]], in_r[: n_r[L]])
        for l in range(L):
            k = L - 1 - l
            assert torch.equal(blocks_s[l].indptr(n_s[k]), blocks_r[l].indptr(n_r[k]))
            assert torch.equal(blocks_s[l].indices(m_s[l]), blocks_r[l].indices(m_r[l]))
            assert torch.equal(gs.gs_cache_read_rows(sut, l, all_nodes), gs.gs_cache_read_rows(ref, l, all_nodes))


def test_noalloc_rejects_what_does_not_fit():
    """Sizes beyond the built-in scratch, or beyond the caller's buffers, are refused on the host
    with GS_ERR_WORKSPACE before any kernel is launched."""
    import paper_2406_17918_b200 as gs

    cfg = get_config("mid")
    g = build_graph(cfg).to("cuda")
    G = gs.gs_graph_create(g.indptr, g.indices, None)
    fan, W, L = cfg["fanouts"], cfg["cache_width"], len(cfg["fanouts"])
    C = gs.gs_cache_init(G, fan, W, 1, False)
    perm = seed_permutation(cfg)
    gs.gs_sync_status(C)
    launches = gs.gs_kernel_launches()

    small = torch.zeros(8, dtype=torch.int32, device="cuda")
    with pytest.raises(gs.GsError) as e:                       # the caller's output buffers are too small
        gs.gs_sample_batch_noalloc(C, perm[:64].cuda(), gs.GS_MODE_OTF, 0.3, 1, small, [small] * L, [small] * L)
    assert e.value.status == 4

    B = 8192                                                   # this batch needs ~76 MB of scratch
    assert gs.gs_workspace_bytes(G, fan, B) > gs.NOALLOC_SCRATCH_BYTES
    nb, mb = _bounds(cfg["num_nodes"], fan, B)
    inp = torch.zeros(nb[L], dtype=torch.int32, device="cuda")
    ip = [torch.zeros(nb[L - 1 - l] + 1, dtype=torch.int32, device="cuda") for l in range(L)]
    ix = [torch.zeros(mb[L - 1 - l], dtype=torch.int32, device="cuda") for l in range(L)]
    with pytest.raises(gs.GsError) as e:
        gs.gs_sample_batch_noalloc(C, perm[:B].cuda(), gs.GS_MODE_OTF, 0.3, 1, inp, ip, ix)
    assert e.value.status == 4 and "built-in scratch" in str(e.value)
    assert gs.gs_kernel_launches() == launches                 # nothing ran

    # a batch that fits still works afterwards (mid graph, 1,024 seeds: ~31 MB of scratch)
    nb, mb = _bounds(cfg["num_nodes"], fan, 1024)
    gs.gs_sample_batch_noalloc(C, perm[:1024].cuda(), gs.GS_MODE_OTF, 0.3, 1, inp, ip, ix)
    n, m = gs.gs_batch_counts(C)
    assert n[0] == 1024 and n[L] <= nb[L] and all(x > 0 for x in m)


def test_noalloc_refuses_misaligned_output_buffers_before_any_launch():
    """A caller that packs its int32 arrays back to back can end up with a d_indices that is only
    4-byte aligned; the ids are stored 16 bytes at a time, so the call must refuse such a buffer
    on the host (GS_ERR_ALIGN) and launch nothing.  Only the refusal is exercised here."""
    import paper_2406_17918_b200 as gs

    cfg = get_config("tiny")
    g = build_graph(cfg).to("cuda")
    perm = seed_permutation(cfg)
    G = gs.gs_graph_create(g.indptr, g.indices, None)
    fan, W, B, L = cfg["fanouts"], cfg["cache_width"], cfg["batch"], len(cfg["fanouts"])
    C = gs.gs_cache_init(G, fan, W, 5, False)
    gs.gs_sync_status(C)
    nb, mb = _bounds(cfg["num_nodes"], fan, B)
    inp = torch.zeros(nb[L], dtype=torch.int32, device="cuda")
    ip = [torch.zeros(nb[L - 1 - l] + 1, dtype=torch.int32, device="cuda") for l in range(L)]
    ix_big = [torch.zeros(mb[L - 1 - l] + 4, dtype=torch.int32, device="cuda") for l in range(L)]
    seeds = batch_seeds(perm, 0, B).cuda()
    launches = gs.gs_kernel_launches()
    for shift in (1, 2, 3):
        ix = [t[shift:] for t in ix_big]            # 4-, 8- and 12-byte offsets from a 16-byte boundary
        assert ix[0].data_ptr() % 16 != 0
        with pytest.raises(gs.GsError) as e:
            gs.gs_sample_batch_noalloc(C, seeds, gs.GS_MODE_OTF, 0.25, 1, inp, ip, ix)
        assert e.value.status == 2 and "16-byte" in str(e.value)
    assert gs.gs_kernel_launches() == launches      # refused on the host: nothing ran
    # the same buffers at an aligned offset are accepted
    gs.gs_sample_batch_noalloc(C, seeds, gs.GS_MODE_OTF, 0.25, 1, inp, ip, [t[4:] for t in ix_big])
    n, m = gs.gs_batch_counts(C)
    assert n[0] == B


def test_noalloc_call_leaves_device_memory_unchanged():
    """The built-in scratch array is materialised when the cache is created (gs_cache_init looks its
    address up), so a batch through the no-allocation call must not change the free device memory."""
    import paper_2406_17918_b200 as gs

    cfg = get_config("tiny")
    g = build_graph(cfg).to("cuda")
    perm = seed_permutation(cfg)
    G = gs.gs_graph_create(g.indptr, g.indices, None)
    fan, W, B, L = cfg["fanouts"], cfg["cache_width"], cfg["batch"], len(cfg["fanouts"])
    C = gs.gs_cache_init(G, fan, W, 9, False)
    nb, mb = _bounds(cfg["num_nodes"], fan, B)
    inp = torch.zeros(nb[L], dtype=torch.int32, device="cuda")
    ip = [torch.zeros(nb[L - 1 - l] + 1, dtype=torch.int32, device="cuda") for l in range(L)]
    ix = [torch.zeros(mb[L - 1 - l], dtype=torch.int32, device="cuda") for l in range(L)]
    seeds = [batch_seeds(perm, b, B).cuda() for b in range(3)]
    # first batch: the CUDA runtime loads the kernels' code on first use, which is not the call's doing
    gs.gs_sample_batch_noalloc(C, seeds[2], gs.GS_MODE_OTF, 0.25, 1, inp, ip, ix)
    gs.gs_sync_status(C)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for b in range(2):
        gs.gs_sample_batch_noalloc(C, seeds[b], gs.GS_MODE_OTF, 0.25, b + 2, inp, ip, ix)
    gs.gs_sync_status(C)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
