"""The C-ABI library loads without a GPU, exports every declared symbol and rejects bad
arguments on the host before anything is launched."""
import ctypes

import pytest

import paper_2406_17918_b200 as gs


@pytest.fixture(scope="module")
def L():
    lib = ctypes.CDLL(gs.library_path())
    lib.gs_last_error.restype = ctypes.c_char_p
    return lib


def test_every_declared_symbol_is_exported(L):
    names = gs.exported_symbols()
    assert {"gs_graph_create", "gs_cache_init", "gs_sample_batch", "gs_gather_features"} <= set(names)
    for n in names:
        assert getattr(L, n) is not None


def _graph(L, n=10, e=20, indptr=0x1000, indices=0x2000, feats=0x4000, dtype=0, dim=4, ld=4):
    h = ctypes.c_void_p()
    rc = L.gs_graph_create(ctypes.c_int64(n), ctypes.c_int64(e), ctypes.c_void_p(indptr), ctypes.c_void_p(indices),
                           ctypes.c_void_p(feats), dtype, dim, ctypes.c_int64(ld), ctypes.byref(h))
    return rc, h


def test_graph_create_validation(L):
    assert _graph(L)[0] == 0                                   # pointers are only recorded, never dereferenced
    assert _graph(L, n=0)[0] == 1
    assert _graph(L, n=1 << 31)[0] == 1
    assert _graph(L, indptr=0)[0] == 1
    assert _graph(L, indptr=0x1004)[0] == 2                    # int64 array on a 4-byte boundary
    assert _graph(L, indices=0x2002)[0] == 2
    assert _graph(L, dtype=9)[0] == 1
    assert _graph(L, dim=8, ld=4)[0] == 1
    assert b"feat_ld" in L.gs_last_error()
    assert _graph(L, feats=0x4002, dtype=0)[0] == 2


def test_sizes_and_cache_init_validation(L):
    rc, g = _graph(L, n=1000)
    out = ctypes.c_size_t()
    assert L.gs_cache_bytes(g, 2, 10, 0, ctypes.byref(out)) == 0
    assert out.value >= 1000 * 8 + 2 * 1000 * 10 * 4
    shared = ctypes.c_size_t()
    assert L.gs_cache_bytes(g, 2, 10, 1, ctypes.byref(shared)) == 0 and shared.value < out.value
    assert L.gs_cache_bytes(g, 0, 10, 0, ctypes.byref(out)) == 1
    assert L.gs_cache_bytes(g, 9, 10, 0, ctypes.byref(out)) == 1
    assert L.gs_cache_bytes(g, 2, 33, 0, ctypes.byref(out)) == 1
    fo = (ctypes.c_int32 * 2)(5, 5)
    ws = ctypes.c_size_t()
    assert L.gs_workspace_bytes(g, 2, fo, 64, ctypes.byref(ws)) == 0
    # worst case: 64 seeds -> 320 picks -> 384 nodes -> 1920 picks; frontier is capped by the 1000 nodes
    assert ws.value >= 4 * (1000 + 320 + 1920)
    assert L.gs_workspace_bytes(g, 2, fo, 0, ctypes.byref(ws)) == 1
    bad = (ctypes.c_int32 * 2)(5, 0)
    assert L.gs_workspace_bytes(g, 2, bad, 64, ctypes.byref(ws)) == 1
    c = ctypes.c_void_p()
    wide = (ctypes.c_int32 * 2)(5, 11)
    args = lambda f, storage, nbytes: L.gs_cache_init(g, 2, f, 10, ctypes.c_uint64(1), 0, ctypes.c_void_p(storage),
                                                      ctypes.c_size_t(nbytes), None, ctypes.byref(c))
    assert args(wide, 0x10000, 1 << 30) == 1                   # fan-out above the cache width
    assert args(fo, 0, 1 << 30) == 1
    assert args(fo, 0x10010, 1 << 30) == 2                     # storage must be 256-byte aligned
    assert args(fo, 0x10000, 100) == 4                         # too small
    L.gs_graph_destroy(g)


def test_null_handles(L):
    assert L.gs_sample_batch(None, None, 0, 0, ctypes.c_double(0), 1, None, ctypes.c_size_t(0), None, None, None, None) == 1
    assert L.gs_gather_features(None, None, None, 0, None, ctypes.c_int64(0), None) == 1
    assert L.gs_sync_status(None, None) == 1
    assert L.gs_cache_read_rows(None, 0, None, 0, None, None) == 1
    L.gs_kernel_launches.restype = ctypes.c_int64
    assert L.gs_kernel_launches() == 0                         # nothing was launched by any of the above
