"""ctypes binding of ``libgs.so``: argument marshalling only.

Functions keep the names and argument order of ``include/gs.h``.  Device buffers are torch CUDA
tensors (torch is used for device memory and streams only); the binding passes their
``data_ptr()`` and keeps them alive on the small Python handle objects.
"""
from __future__ import annotations

import ctypes
import os
import re

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libgs.so")
_HEADER = os.path.join(os.path.dirname(_HERE), "include", "gs.h")

GS_MODE_FCR, GS_MODE_OTF, GS_MODE_FBL, GS_MODE_OTF_FETCH = 0, 1, 2, 3
GS_F32, GS_BF16 = 0, 1
GS_DEDUP_DIRECT, GS_DEDUP_HASH, GS_DEDUP_SORT, GS_DEDUP_AUTO = 0, 1, 2, 3
GS_MAX_HOPS = 8
COUNTS_READBACK_BYTES = 4 * (1 + (GS_MAX_HOPS + 1) + GS_MAX_HOPS)  # status + n_k + m_k, what gs_batch_counts copies

_STATUS_NAMES = {0: "GS_OK", 1: "GS_ERR_ARG", 2: "GS_ERR_ALIGN", 3: "GS_ERR_RANGE", 4: "GS_ERR_WORKSPACE",
                 5: "GS_ERR_DUP_SEED", 6: "GS_ERR_CUDA"}


class GsError(RuntimeError):
    def __init__(self, status, message):
        super().__init__("%s: %s" % (_STATUS_NAMES.get(status, status), message))
        self.status = status


class _CBlock(ctypes.Structure):
    _fields_ = [("max_dst", ctypes.c_int32), ("max_src", ctypes.c_int32), ("max_edges", ctypes.c_int32),
                ("d_num_dst", ctypes.c_void_p), ("d_num_src", ctypes.c_void_p), ("d_num_edges", ctypes.c_void_p),
                ("d_indptr", ctypes.c_void_p), ("d_indices", ctypes.c_void_p)]


class _CBlockBuffers(ctypes.Structure):
    _fields_ = [("d_indptr", ctypes.c_void_p), ("indptr_capacity", ctypes.c_int64),
                ("d_indices", ctypes.c_void_p), ("indices_capacity", ctypes.c_int64)]


NOALLOC_SCRATCH_BYTES = 64 << 20


def library_path() -> str:
    return _LIB_PATH


def exported_symbols():
    """Names of the functions ``include/gs.h`` declares."""
    text = open(_HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gs_[a-z_]+)\s*\(", text)))


def _load():
    if not os.path.exists(_LIB_PATH):
        raise ImportError("%s is missing: run `python -m paper_2406_17918_b200.build` "
                          "(there is no CPU fallback)" % _LIB_PATH)
    L = ctypes.CDLL(_LIB_PATH)
    vp, i32, i64, u32, u64, dbl, sz = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint32,
                                       ctypes.c_uint64, ctypes.c_double, ctypes.c_size_t)
    pvp = ctypes.POINTER(vp)
    psz = ctypes.POINTER(sz)
    sig = {
        "gs_graph_create": [i64, i64, vp, vp, vp, ctypes.c_int, i32, i64, pvp],
        "gs_graph_validate": [vp, vp, ctypes.POINTER(i64)],
        "gs_graph_set_gather_grid": [vp, i32],
        "gs_gather_status": [vp],
        "gs_cache_bytes": [vp, i32, i32, i32, psz],
        "gs_workspace_bytes": [vp, i32, vp, i32, psz],
        "gs_cache_init": [vp, i32, vp, i32, u64, i32, vp, sz, vp, pvp],
        "gs_cache_refresh_all": [vp, ctypes.c_int, ctypes.c_double, ctypes.c_uint32, vp],
        "gs_cache_bytes_split": [vp, i32, i32, i32, i64, psz],
        "gs_cache_init_split": [vp, i32, vp, i32, u64, i32, i32, i64, vp, sz, vp, pvp],
        "gs_sample_batch": [vp, vp, i32, ctypes.c_int, dbl, u32, vp, sz, vp, vp, pvp, pvp],
        "gs_sample_batch_host": [vp, vp, i32, ctypes.c_int, dbl, u32, vp, sz, vp, vp, pvp, vp, vp],
        "gs_sample_batch_noalloc": [vp, vp, i32, ctypes.c_int, dbl, u32, vp, i64, vp, vp, vp, pvp],
        "gs_batch_counts": [vp, vp, vp, vp],
        "gs_gather_features": [vp, vp, vp, i32, vp, i64, vp],
        "gs_cache_read_rows": [vp, i32, vp, i32, vp, vp],
        "gs_cache_export_bytes": [vp, psz],
        "gs_cache_export": [vp, vp, sz, vp],
        "gs_cache_import": [vp, vp, sz, vp],
        "gs_sync_status": [vp, vp],
        "gs_gather_rows": [vp, ctypes.c_int, i32, i64, i64, i64, vp, vp, i32, vp, i64, vp],
        "gs_gather_rows_peer": [vp, i32, i64, ctypes.c_int, i32, i64, vp, vp, i32, vp, i64, vp],
        "gs_shard_bucket": [vp, i32, i64, i32, vp, vp, vp, vp],
        "gs_shard_bucket_counted": [vp, vp, i32, i64, i32, vp, vp, vp, vp],
        "gs_shard_workspace_bytes": [vp, i32, i32, psz],
        "gs_shard_bucket_fixed": [vp, vp, i32, i64, i32, i32, vp, vp, vp, vp],
        "gs_shard_sample_rows": [vp, vp, i32, i32, ctypes.c_int, dbl, u32, vp, sz, vp, vp],
        "gs_shard_sample_rows_counted": [vp, vp, vp, i32, i32, ctypes.c_int, dbl, u32, vp, sz, vp, vp],
        "gs_shard_status": [vp, vp],
        "gs_shard_merge": [vp, vp, i32, i32, i64, i64, vp, vp, vp, vp],
        "gs_shard_fan_out": [vp, vp, i32, i32, i64, i64, vp, vp, vp, vp, i32, vp, vp],
        "gs_shard_extend": [vp, i32, vp, i32, vp, vp, vp, sz, vp, vp, pvp],
        "gs_shard_extend_fixed": [vp, i32, vp, i32, vp, i32, vp, vp, sz, vp, vp, pvp],
        "gs_batch_stats": [vp, vp, vp],
        "gs_cache_profile_begin": [vp, i32],
        "gs_cache_profile_end": [vp, vp, vp, vp],
        "gs_cache_set_tuning": [vp, dbl, dbl, i32],
        "gs_debug_set_grid_cap": [i32],
        "gs_alu_ceiling": [i32, i32, vp, ctypes.POINTER(dbl)],
        "gs_cache_set_dedup": [vp, i32],
        "gs_graph_count_dense": [vp, i32, vp, ctypes.POINTER(i64)],
    }
    for name, args in sig.items():
        fn = getattr(L, name)
        fn.argtypes = args
        fn.restype = ctypes.c_int
    L.gs_graph_destroy.argtypes = [vp]
    L.gs_graph_destroy.restype = None
    L.gs_cache_destroy.argtypes = [vp]
    L.gs_cache_destroy.restype = None
    L.gs_last_error.argtypes = []
    L.gs_last_error.restype = ctypes.c_char_p
    L.gs_stats_word_offset.argtypes = []
    L.gs_stats_word_offset.restype = ctypes.c_int32
    L.gs_kernel_launches.argtypes = []
    L.gs_kernel_launches.restype = ctypes.c_int64
    return L


_L = _load()


def gs_stats_word_offset() -> int:
    return int(_L.gs_stats_word_offset())


def gs_last_error() -> str:
    return _L.gs_last_error().decode()


def gs_kernel_launches() -> int:
    return int(_L.gs_kernel_launches())


def _check(status):
    if status != 0:
        raise GsError(status, gs_last_error())


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _i32_array(values):
    return (ctypes.c_int32 * len(values))(*[int(v) for v in values])


class Graph:
    """Handle of gs_graph plus references that keep the borrowed tensors alive."""

    def __init__(self, handle, indptr, indices, features, dtype, feat_dim):
        self.handle, self.indptr, self.indices, self.features = handle, indptr, indices, features
        self.dtype, self.feat_dim = dtype, feat_dim
        self.num_nodes = indptr.numel() - 1

    def close(self):
        if self.handle:
            _L.gs_graph_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Cache:
    def __init__(self, handle, graph, storage, fanouts, cache_width, shared):
        self.handle, self.graph, self.storage = handle, graph, storage
        self.fanouts, self.cache_width, self.shared = list(fanouts), cache_width, bool(shared)
        self.num_hops = len(self.fanouts)

    def close(self):
        if self.handle:
            _L.gs_cache_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Block:
    """Device view of one hop's block; tensors alias the workspace (no copies)."""

    def __init__(self, cb: _CBlock, workspace: torch.Tensor, header: torch.Tensor):
        self.max_dst, self.max_src, self.max_edges = cb.max_dst, cb.max_src, cb.max_edges
        self._ws, self._hdr = workspace, header
        self._indptr_off = cb.d_indptr - workspace.data_ptr()
        self._indices_off = cb.d_indices - workspace.data_ptr()
        hp = header.data_ptr()
        self._cnt = ((cb.d_num_dst - hp) // 4, (cb.d_num_src - hp) // 4, (cb.d_num_edges - hp) // 4)

    def count_words(self):
        """int32 word positions of (num_dst, num_src, num_edges) inside the cache storage."""
        return self._cnt

    def counts_device(self):
        """(num_dst, num_src, num_edges) as 0-d device tensors aliasing the cache's state header."""
        h = self._hdr.view(torch.int32)
        return tuple(h[i] for i in self._cnt)

    def indptr(self, num_dst: int) -> torch.Tensor:
        return self._ws[self._indptr_off:self._indptr_off + 4 * (num_dst + 1)].view(torch.int32)

    def indices(self, num_edges: int) -> torch.Tensor:
        return self._ws[self._indices_off:self._indices_off + 4 * num_edges].view(torch.int32)


def gs_graph_create(indptr: torch.Tensor, indices: torch.Tensor, features, dtype=None) -> Graph:
    if indptr.dtype != torch.int64 or indices.dtype != torch.int32:
        raise TypeError("indptr must be int64 and indices int32")
    if not (indptr.is_cuda and indices.is_cuda and indptr.is_contiguous() and indices.is_contiguous()):
        raise ValueError("indptr/indices must be contiguous CUDA tensors")
    feat_dim, feat_ld = 0, 0
    if features is not None:
        if not features.is_cuda or features.dim() != 2 or features.stride(1) != 1:
            raise ValueError("features must be a row-major 2-D CUDA tensor")
        dtype = {torch.float32: GS_F32, torch.bfloat16: GS_BF16}[features.dtype]
        feat_dim, feat_ld = features.shape[1], features.stride(0)
    elif dtype is None:
        dtype = GS_F32
    h = ctypes.c_void_p()
    _check(_L.gs_graph_create(indptr.numel() - 1, indices.numel(), _ptr(indptr), _ptr(indices), _ptr(features),
                              dtype, feat_dim, feat_ld, ctypes.byref(h)))
    return Graph(h, indptr, indices, features, dtype, feat_dim)


def gs_graph_set_gather_grid(graph: Graph, blocks_per_sm: int):
    _check(_L.gs_graph_set_gather_grid(graph.handle, int(blocks_per_sm)))


def gs_gather_status(stream=None):
    """Synchronises; raises if a bulk-copy gather ever gave up waiting."""
    _check(_L.gs_gather_status(_stream(stream)))


def gs_graph_validate(graph: Graph, stream=None) -> int:
    """Checks the CSR contract on the device; returns -1, or raises GsError naming the first bad row."""
    bad = ctypes.c_int64(-1)
    _check(_L.gs_graph_validate(graph.handle, _stream(stream), ctypes.byref(bad)))
    return int(bad.value)


def gs_cache_bytes(graph: Graph, num_hops: int, cache_width: int, shared: bool) -> int:
    out = ctypes.c_size_t()
    _check(_L.gs_cache_bytes(graph.handle, num_hops, cache_width, int(shared), ctypes.byref(out)))
    return out.value


def gs_workspace_bytes(graph: Graph, fanouts, max_seeds: int) -> int:
    out = ctypes.c_size_t()
    _check(_L.gs_workspace_bytes(graph.handle, len(fanouts), _i32_array(fanouts), max_seeds, ctypes.byref(out)))
    return out.value


def gs_cache_init(graph: Graph, fanouts, cache_width: int, seed: int, shared: bool, storage: torch.Tensor = None,
                  stream=None) -> Cache:
    if storage is None:
        storage = torch.empty(gs_cache_bytes(graph, len(fanouts), cache_width, shared), dtype=torch.uint8,
                              device=graph.indptr.device)
    h = ctypes.c_void_p()
    _check(_L.gs_cache_init(graph.handle, len(fanouts), _i32_array(fanouts), cache_width, ctypes.c_uint64(seed),
                            int(shared), _ptr(storage), storage.numel(), _stream(stream), ctypes.byref(h)))
    return Cache(h, graph, storage, fanouts, cache_width, shared)


def gs_cache_bytes_split(graph: Graph, num_hops: int, cache_width: int, shared: bool, dense_rows: int) -> int:
    out = ctypes.c_size_t()
    _check(_L.gs_cache_bytes_split(graph.handle, num_hops, cache_width, int(shared), dense_rows, ctypes.byref(out)))
    return out.value


def gs_graph_count_dense(graph: Graph, theta: int, stream=None) -> int:
    """Nodes with degree > theta, counted by the library (synchronises)."""
    out = ctypes.c_int64()
    _check(_L.gs_graph_count_dense(graph.handle, int(theta), _stream(stream), ctypes.byref(out)))
    return int(out.value)


def gs_cache_init_split(graph: Graph, fanouts, cache_width: int, seed: int, shared: bool, theta: int,
                        dense_rows: int = None, storage: torch.Tensor = None, stream=None) -> Cache:
    """Cache rows only for nodes with degree > theta; the others are sampled from the graph."""
    if dense_rows is None:
        dense_rows = gs_graph_count_dense(graph, theta, stream)
    if storage is None:
        storage = torch.empty(gs_cache_bytes_split(graph, len(fanouts), cache_width, shared, dense_rows),
                              dtype=torch.uint8, device=graph.indptr.device)
    h = ctypes.c_void_p()
    _check(_L.gs_cache_init_split(graph.handle, len(fanouts), _i32_array(fanouts), cache_width, ctypes.c_uint64(seed),
                                  int(shared), int(theta), int(dense_rows), _ptr(storage), storage.numel(),
                                  _stream(stream), ctypes.byref(h)))
    return Cache(h, graph, storage, fanouts, cache_width, shared)


def gs_cache_refresh_all(cache: Cache, mode: int, gamma: float, step: int, stream=None) -> None:
    """Refresh every cached row of every layer (the periodic-refresh branch of Algorithms 2 and 3)."""
    _check(_L.gs_cache_refresh_all(cache.handle, mode, float(gamma), step, _stream(stream)))


def _blocks_out(cache: Cache, cblocks, workspace):
    return [Block(cblocks[l], workspace, cache.storage) for l in range(cache.num_hops)]


def gs_sample_batch(cache: Cache, seeds: torch.Tensor, mode: int, gamma: float, step: int, workspace: torch.Tensor,
                    stream=None):
    """Returns (blocks by layer, input_nodes tensor of capacity max_src, device count tensor)."""
    if seeds.dtype != torch.int32 or not seeds.is_cuda or not seeds.is_contiguous():
        raise TypeError("seeds must be a contiguous int32 CUDA tensor")
    cblocks = (_CBlock * cache.num_hops)()
    d_in, d_cnt = ctypes.c_void_p(), ctypes.c_void_p()
    _check(_L.gs_sample_batch(cache.handle, _ptr(seeds), seeds.numel(), mode, float(gamma), step, _ptr(workspace),
                              workspace.numel(), _stream(stream), cblocks, ctypes.byref(d_in), ctypes.byref(d_cnt)))
    blocks = _blocks_out(cache, cblocks, workspace)
    off = d_in.value - workspace.data_ptr()
    input_nodes = workspace[off:off + 4 * blocks[0].max_src].view(torch.int32)
    cnt_index = (d_cnt.value - cache.storage.data_ptr()) // 4
    return blocks, input_nodes, cache.storage.view(torch.int32)[cnt_index]


def gs_sample_batch_host(cache: Cache, seeds_host: torch.Tensor, mode: int, gamma: float, step: int,
                         workspace: torch.Tensor, stream=None):
    """Seeds in (pinned) host memory; synchronises.  Returns (blocks, input_nodes, n list, m list)."""
    if seeds_host.dtype != torch.int32 or seeds_host.is_cuda or not seeds_host.is_contiguous():
        raise TypeError("seeds_host must be a contiguous int32 CPU tensor")
    cblocks = (_CBlock * cache.num_hops)()
    d_in = ctypes.c_void_p()
    n = (ctypes.c_int32 * (cache.num_hops + 1))()
    m = (ctypes.c_int32 * cache.num_hops)()
    _check(_L.gs_sample_batch_host(cache.handle, _ptr(seeds_host), seeds_host.numel(), mode, float(gamma), step,
                                   _ptr(workspace), workspace.numel(), _stream(stream), cblocks, ctypes.byref(d_in),
                                   n, m))
    blocks = _blocks_out(cache, cblocks, workspace)
    off = d_in.value - workspace.data_ptr()
    input_nodes = workspace[off:off + 4 * blocks[0].max_src].view(torch.int32)
    return blocks, input_nodes, list(n), list(m)


class OutBlock:
    """One hop's block as written by gs_sample_batch_noalloc into the caller's tensors."""

    def __init__(self, cb, indptr, indices):
        self.max_dst, self.max_src, self.max_edges = cb.max_dst, cb.max_src, cb.max_edges
        self._indptr, self._indices = indptr, indices

    def indptr(self, num_dst: int) -> torch.Tensor:
        return self._indptr[: num_dst + 1]

    def indices(self, num_edges: int) -> torch.Tensor:
        return self._indices[:num_edges]


def gs_sample_batch_noalloc(cache: Cache, seeds: torch.Tensor, mode: int, gamma: float, step: int,
                            input_nodes: torch.Tensor, indptr_bufs, indices_bufs, stream=None):
    """The batch call for callers that may not allocate device memory: scratch is the library's
    built-in array, results land in the int32 CUDA tensors passed here (`indptr_bufs[l]`,
    `indices_bufs[l]` by layer, and `input_nodes`).  Nothing is allocated by this function either.
    Returns the blocks (views of the caller's tensors), by layer."""
    if seeds.dtype != torch.int32 or not seeds.is_cuda or not seeds.is_contiguous():
        raise TypeError("seeds must be a contiguous int32 CUDA tensor")
    bufs = (_CBlockBuffers * cache.num_hops)()
    for l in range(cache.num_hops):
        for t in (indptr_bufs[l], indices_bufs[l]):
            if t.dtype != torch.int32 or not t.is_cuda or not t.is_contiguous():
                raise TypeError("block buffers must be contiguous int32 CUDA tensors")
        bufs[l].d_indptr, bufs[l].indptr_capacity = indptr_bufs[l].data_ptr(), indptr_bufs[l].numel()
        bufs[l].d_indices, bufs[l].indices_capacity = indices_bufs[l].data_ptr(), indices_bufs[l].numel()
    cblocks = (_CBlock * cache.num_hops)()
    d_cnt = ctypes.c_void_p()
    _check(_L.gs_sample_batch_noalloc(cache.handle, _ptr(seeds), seeds.numel(), mode, float(gamma), step,
                                      _ptr(input_nodes), input_nodes.numel(), bufs, _stream(stream), cblocks,
                                      ctypes.byref(d_cnt)))
    return [OutBlock(cblocks[l], indptr_bufs[l], indices_bufs[l]) for l in range(cache.num_hops)]


def gs_batch_counts(cache: Cache, stream=None):
    """Synchronises; returns ([n_0..n_L] by sampling step, [edges per block] by layer)."""
    n = (ctypes.c_int32 * (cache.num_hops + 1))()
    m = (ctypes.c_int32 * cache.num_hops)()
    _check(_L.gs_batch_counts(cache.handle, _stream(stream), n, m))
    return list(n), list(m)


def gs_gather_features(graph: Graph, ids: torch.Tensor, count, out: torch.Tensor, stream=None):
    """count: a 0-d int32 CUDA tensor (device scalar) or None to gather out.shape[0] rows."""
    if ids.dtype != torch.int32 or not ids.is_cuda:
        raise TypeError("ids must be an int32 CUDA tensor")
    if out.dim() != 2 or out.stride(1) != 1 or out.dtype != graph.features.dtype:
        raise TypeError("out must be a row-major 2-D tensor of the feature dtype")
    bound = min(out.shape[0], ids.numel())
    _check(_L.gs_gather_features(graph.handle, _ptr(ids), _ptr(count), bound, _ptr(out), out.stride(0),
                                 _stream(stream)))
    return out


def gs_gather_rows(src: torch.Tensor, ids: torch.Tensor, out: torch.Tensor, first_row: int = 0, count=None, stream=None):
    """out[i] = src[ids[i] - first_row] for a row-major 2-D f32 / bf16 CUDA tensor."""
    if src.dim() != 2 or src.stride(1) != 1 or out.dim() != 2 or out.stride(1) != 1 or out.dtype != src.dtype:
        raise TypeError("src and out must be row-major 2-D tensors of one dtype")
    if ids.dtype != torch.int32 or not ids.is_cuda:
        raise TypeError("ids must be an int32 CUDA tensor")
    dtype = {torch.float32: GS_F32, torch.bfloat16: GS_BF16}[src.dtype]
    bound = min(out.shape[0], ids.numel())
    _check(_L.gs_gather_rows(_ptr(src), dtype, src.shape[1], src.stride(0), int(first_row), src.shape[0], _ptr(ids), _ptr(count), bound,
                             _ptr(out), out.stride(0), _stream(stream)))
    return out


def gs_gather_rows_peer(shard_bases, num_rows: int, dtype: torch.dtype, row_elems: int, src_ld: int, ids: torch.Tensor,
                        out: torch.Tensor, count=None, stream=None):
    """out[i] = row ids[i] of a matrix split over len(shard_bases) row shards; `shard_bases` are device
    addresses (ints), local or peer-mapped.  One kernel: the rows are pulled straight from their owners."""
    if ids.dtype != torch.int32 or not ids.is_cuda:
        raise TypeError("ids must be an int32 CUDA tensor")
    if out.dim() != 2 or out.stride(1) != 1 or out.dtype != dtype:
        raise TypeError("out must be a row-major 2-D tensor of the given dtype")
    world = len(shard_bases)
    arr = (ctypes.c_void_p * world)(*[ctypes.c_void_p(int(b)) for b in shard_bases])
    bound = min(out.shape[0], ids.numel())
    _check(_L.gs_gather_rows_peer(arr, world, int(num_rows), {torch.float32: GS_F32, torch.bfloat16: GS_BF16}[dtype],
                                  int(row_elems), int(src_ld), _ptr(ids), _ptr(count), bound, _ptr(out), out.stride(0),
                                  _stream(stream)))
    return out


def gs_shard_bucket(nodes: torch.Tensor, num_nodes: int, world: int, stream=None, count=None, capacity=None, out=None):
    """Group node ids by owner.  Returns (sorted ids, slot of every input id, int32[2*world+1] device counts).
    `count`: a 0-d int32 CUDA tensor with the list's length when only the device knows it (`nodes` is then the bound).
    `capacity`: every owner's group gets a segment of that many ids (sorted ids: world*capacity entries) instead of
    the groups being packed.  `out`: (sorted, slot, counts) tensors to write into instead of new ones."""
    if nodes.dtype != torch.int32 or not nodes.is_cuda or not nodes.is_contiguous():
        raise TypeError("nodes must be a contiguous int32 CUDA tensor")
    if out is not None:
        sorted_ids, slot, counts = out
        need = nodes.numel() if capacity is None else world * int(capacity)
        if sorted_ids.numel() < need or slot.numel() < nodes.numel() or counts.numel() < 2 * world + 1:
            raise ValueError("an output tensor is too small")
        for t in out:
            if t.dtype != torch.int32 or not t.is_cuda or not t.is_contiguous():
                raise TypeError("outputs must be contiguous int32 CUDA tensors")
    else:
        sorted_ids = torch.empty_like(nodes) if capacity is None else torch.empty(world * int(capacity), dtype=torch.int32, device=nodes.device)
        slot = torch.empty_like(nodes)
        counts = torch.empty(2 * world + 1, dtype=torch.int32, device=nodes.device)
    if capacity is not None:
        _check(_L.gs_shard_bucket_fixed(_ptr(nodes), _ptr(count), nodes.numel(), int(num_nodes), int(world), int(capacity),
                                        _ptr(sorted_ids), _ptr(slot), _ptr(counts), _stream(stream)))
    elif count is None:
        _check(_L.gs_shard_bucket(_ptr(nodes), nodes.numel(), int(num_nodes), int(world), _ptr(sorted_ids), _ptr(slot),
                                  _ptr(counts), _stream(stream)))
    else:
        _check(_L.gs_shard_bucket_counted(_ptr(nodes), _ptr(count), nodes.numel(), int(num_nodes), int(world),
                                          _ptr(sorted_ids), _ptr(slot), _ptr(counts), _stream(stream)))
    return sorted_ids, slot, counts


def gs_shard_workspace_bytes(graph: Graph, fanout: int, max_nodes: int) -> int:
    out = ctypes.c_size_t()
    _check(_L.gs_shard_workspace_bytes(graph.handle, int(fanout), int(max_nodes), ctypes.byref(out)))
    return out.value


def gs_shard_sample_rows(cache: Cache, nodes: torch.Tensor, layer: int, mode: int, rate: float, step: int,
                         workspace: torch.Tensor, picks: torch.Tensor = None, stream=None, count=None) -> torch.Tensor:
    """Owner side of one hop: picks[n, fanout(layer)] (-1 padded) for n distinct nodes of this shard.
    `count`: a 0-d / 1-element int32 CUDA tensor with the list's length (`nodes` is then the bound; only that
    many rows of `picks` are written)."""
    if nodes.dtype != torch.int32 or not nodes.is_cuda or not nodes.is_contiguous():
        raise TypeError("nodes must be a contiguous int32 CUDA tensor")
    f = cache.fanouts[layer] if 0 <= layer < cache.num_hops else 1     # a bad layer is reported by the library
    if picks is None:
        picks = torch.empty((nodes.numel(), f), dtype=torch.int32, device=nodes.device)
    elif picks.dtype != torch.int32 or not picks.is_contiguous() or picks.numel() < nodes.numel() * f:
        raise TypeError("picks must be a contiguous int32 tensor of at least [len(nodes), fanout]")
    if count is None:
        _check(_L.gs_shard_sample_rows(cache.handle, _ptr(nodes), nodes.numel(), int(layer), mode, float(rate), step,
                                       _ptr(workspace), workspace.numel(), _stream(stream), _ptr(picks)))
    else:
        _check(_L.gs_shard_sample_rows_counted(cache.handle, _ptr(nodes), _ptr(count), nodes.numel(), int(layer), mode,
                                               float(rate), step, _ptr(workspace), workspace.numel(), _stream(stream),
                                               _ptr(picks)))
    return picks


def _i32_cuda(*tensors):
    for t in tensors:
        if t.dtype != torch.int32 or not t.is_cuda or not t.is_contiguous():
            raise TypeError("contiguous int32 CUDA tensors expected")


def gs_shard_merge(lists: torch.Tensor, counts: torch.Tensor, world: int, first_row: int, index: torch.Tensor,
                   distinct: torch.Tensor, num_distinct: torch.Tensor, stream=None):
    """Owner side: one place in `distinct` for every node any of the `world` fixed-pitch lists asks for.
    index: int32[rows owned], all -1 between batches; num_distinct: int32[2] (count, status word)."""
    _i32_cuda(lists, counts, index, distinct, num_distinct)
    capacity = lists.numel() // int(world)
    if lists.numel() != capacity * world or counts.numel() < world or num_distinct.numel() < 2 or \
            distinct.numel() < min(lists.numel(), index.numel()):
        raise ValueError("bad tensor sizes")
    _check(_L.gs_shard_merge(_ptr(lists), _ptr(counts), int(world), capacity, int(first_row), index.numel(), _ptr(index),
                             _ptr(distinct), _ptr(num_distinct), _stream(stream)))
    return distinct, num_distinct


def gs_shard_fan_out(lists: torch.Tensor, counts: torch.Tensor, world: int, first_row: int, index: torch.Tensor,
                     distinct: torch.Tensor, num_distinct: torch.Tensor, rows: torch.Tensor, out: torch.Tensor, stream=None):
    """out[e] = rows[place of lists[e]] for every entry of every list; puts `index` back to all -1."""
    _i32_cuda(lists, counts, index, distinct, num_distinct, rows, out)
    capacity = lists.numel() // int(world)
    f = rows.shape[1]
    if out.numel() < lists.numel() * f or rows.shape[0] < min(lists.numel(), index.numel()) or distinct.numel() < min(lists.numel(), index.numel()):
        raise ValueError("bad tensor sizes")
    _check(_L.gs_shard_fan_out(_ptr(lists), _ptr(counts), int(world), capacity, int(first_row), index.numel(), _ptr(index),
                               _ptr(distinct), _ptr(num_distinct), _ptr(rows), int(f), _ptr(out), _stream(stream)))
    return out


def gs_shard_status(cache: Cache, stream=None):
    _check(_L.gs_shard_status(cache.handle, _stream(stream)))


def gs_shard_extend(cache: Cache, k: int, seeds, reply: torch.Tensor, slot: torch.Tensor, workspace: torch.Tensor,
                    stream=None, reply_rows=None):
    """Requester side of hop k.  Returns (block of layer L-1-k, frontier array aliasing the workspace).
    `reply_rows`: rows of a fixed-pitch reply (world * capacity, see gs_shard_bucket)."""
    cb = _CBlock()
    d_fr = ctypes.c_void_p()
    if reply_rows is None:
        _check(_L.gs_shard_extend(cache.handle, int(k), _ptr(seeds), 0 if seeds is None else seeds.numel(), _ptr(reply),
                                  _ptr(slot), _ptr(workspace), workspace.numel(), _stream(stream), ctypes.byref(cb),
                                  ctypes.byref(d_fr)))
    else:
        if 0 <= k < cache.num_hops and reply.numel() < int(reply_rows) * cache.fanouts[cache.num_hops - 1 - k]:
            raise ValueError("reply holds fewer than reply_rows rows")
        _check(_L.gs_shard_extend_fixed(cache.handle, int(k), _ptr(seeds), 0 if seeds is None else seeds.numel(), _ptr(reply),
                                        int(reply_rows), _ptr(slot), _ptr(workspace), workspace.numel(), _stream(stream),
                                        ctypes.byref(cb), ctypes.byref(d_fr)))
    block = Block(cb, workspace, cache.storage)
    off = d_fr.value - workspace.data_ptr()
    return block, workspace[off:off + 4 * block.max_src].view(torch.int32)


def gs_cache_read_rows(cache: Cache, layer: int, nodes: torch.Tensor, stream=None) -> torch.Tensor:
    out = torch.empty((nodes.numel(), cache.cache_width), dtype=torch.int32, device=nodes.device)
    _check(_L.gs_cache_read_rows(cache.handle, layer, _ptr(nodes), nodes.numel(), _ptr(out), _stream(stream)))
    return out


def gs_cache_export(cache: Cache, stream=None) -> torch.Tensor:
    nbytes = ctypes.c_size_t()
    _check(_L.gs_cache_export_bytes(cache.handle, ctypes.byref(nbytes)))
    blob = torch.empty(nbytes.value, dtype=torch.uint8, device=cache.storage.device)
    _check(_L.gs_cache_export(cache.handle, _ptr(blob), blob.numel(), _stream(stream)))
    return blob


def gs_cache_import(cache: Cache, blob: torch.Tensor, stream=None):
    _check(_L.gs_cache_import(cache.handle, _ptr(blob), blob.numel(), _stream(stream)))


def gs_batch_stats(cache: Cache, stream=None):
    """Synchronises; {'slow_refills': ..., 'queued_rescans': ...} of the last batch."""
    out = (ctypes.c_int64 * 4)()
    _check(_L.gs_batch_stats(cache.handle, _stream(stream), out))
    return {"slow_refills": int(out[0]), "queued_rescans": int(out[1]), "refreshed_nodes": int(out[2]),
            "philox_blocks": int(out[3])}


def gs_cache_profile_begin(cache: Cache, max_batches: int):
    _check(_L.gs_cache_profile_begin(cache.handle, int(max_batches)))


def gs_cache_profile_end(cache: Cache, stream=None):
    """Synchronises; ({'row_counts': ms, 'scan': ms, 'finish': ms, 'relabel': ms}, batches timed)."""
    ms = (ctypes.c_double * 4)()
    nb = ctypes.c_int64()
    _check(_L.gs_cache_profile_end(cache.handle, _stream(stream), ms, ctypes.byref(nb)))
    return dict(zip(("row_counts", "scan", "finish", "relabel"), [float(x) for x in ms])), int(nb.value)


def gs_sync_status(cache: Cache, stream=None):
    _check(_L.gs_sync_status(cache.handle, _stream(stream)))


def gs_debug_set_grid_cap(max_blocks: int):
    """Process-wide test knob: cap every kernel's grid at max_blocks blocks (0 = designed grids)."""
    _check(_L.gs_debug_set_grid_cap(int(max_blocks)))


def gs_cache_set_tuning(cache: Cache, lambda_otf=0.0, lambda_full=0.0, hub_degree=0):
    _check(_L.gs_cache_set_tuning(cache.handle, float(lambda_otf), float(lambda_full), int(hub_degree)))


def gs_alu_ceiling(what: int, milliseconds: int = 20, stream=None) -> float:
    """Measured rate (units per second) of 0: Philox blocks with the threshold test, 1: wide multiplies, 2: logic ops."""
    out = ctypes.c_double()
    _check(_L.gs_alu_ceiling(int(what), int(milliseconds), _stream(stream), ctypes.byref(out)))
    return float(out.value)


def gs_cache_set_dedup(cache: Cache, method: int):
    """GS_DEDUP_DIRECT / GS_DEDUP_HASH / GS_DEDUP_SORT for the following batches on this cache."""
    _check(_L.gs_cache_set_dedup(cache.handle, int(method)))
