"""ctypes front-end of the CPU oracle (``gso.c``).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this package;
the CUDA library and its Python binding never do.  Arrays go in and out as numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gso.c")
_HDR = os.path.join(_HERE, "gso.h")
_LIB = os.path.join(_HERE, "libgso.so")

MODE_FCR, MODE_OTF, MODE_FBL, MODE_OTF_FETCH = 0, 1, 2, 3
FILL, EVICT, PICK, FETCH = 1, 2, 3, 4

KEY_FN = ctypes.CFUNCTYPE(ctypes.c_uint32, ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint32,
                          ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32)


def build(force: bool = False) -> str:
    """Compile gso.c with the host compiler (no CUDA involved)."""
    stale = (not os.path.exists(_LIB)) or any(os.path.getmtime(p) > os.path.getmtime(_LIB) for p in (_SRC, _HDR))
    if force or stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-Wall", "-Wextra", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        i32p = ctypes.POINTER(ctypes.c_int32)
        L.gso_philox4x32_10.argtypes = [ctypes.POINTER(ctypes.c_uint32)] * 3
        L.gso_philox4x32_10.restype = None
        L.gso_refresh_count.argtypes = [ctypes.c_int, ctypes.c_double, ctypes.c_int32]
        L.gso_refresh_count.restype = ctypes.c_int32
        L.gso_create.argtypes = [ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, i32p,
                                 ctypes.c_int32, ctypes.c_uint64, ctypes.c_int32]
        L.gso_create.restype = ctypes.c_void_p
        L.gso_destroy.argtypes = [ctypes.c_void_p]
        L.gso_destroy.restype = None
        L.gso_set_key_fn.argtypes = [ctypes.c_void_p, KEY_FN, ctypes.c_void_p]
        L.gso_set_key_fn.restype = None
        L.gso_set_theta.argtypes = [ctypes.c_void_p, ctypes.c_int64]
        L.gso_set_theta.restype = None
        L.gso_cache_row.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p]
        L.gso_cache_set_row.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p]
        L.gso_refresh_node.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_uint32, ctypes.c_int32]
        L.gso_pick_node.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_uint32,
                                    ctypes.c_void_p, ctypes.POINTER(ctypes.c_int32)]
        L.gso_fbl_node.argtypes = L.gso_pick_node.argtypes
        L.gso_fetch_node.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_uint32, ctypes.c_int32,
                                     ctypes.c_void_p, ctypes.POINTER(ctypes.c_int32)]
        L.gso_fetch_count.argtypes = [ctypes.c_double, ctypes.c_int32]
        L.gso_fetch_count.restype = ctypes.c_int32
        L.gso_refresh_all.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_double, ctypes.c_uint32]
        L.gso_sample_batch.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int,
                                       ctypes.c_double, ctypes.c_uint32]
        for name in ("gso_num_nodes", "gso_num_edges"):
            getattr(L, name).argtypes = [ctypes.c_void_p, ctypes.c_int32]
            getattr(L, name).restype = ctypes.c_int32
        L.gso_frontier.argtypes = [ctypes.c_void_p]
        L.gso_frontier.restype = i32p
        for name in ("gso_block_indptr", "gso_block_indices", "gso_block_picked"):
            getattr(L, name).argtypes = [ctypes.c_void_p, ctypes.c_int32]
            getattr(L, name).restype = i32p
        for name in ("gso_stat_refreshed", "gso_stat_scanned"):
            getattr(L, name).argtypes = [ctypes.c_void_p]
            getattr(L, name).restype = ctypes.c_int64
        L.gso_gather.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p, ctypes.c_int64,
                                 ctypes.c_void_p, ctypes.c_int64]
        L.gso_gather.restype = None
        _lib = L
    return _lib


def philox4x32_10(ctr, key):
    c = (ctypes.c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in ctr])
    k = (ctypes.c_uint32 * 2)(*[int(x) & 0xFFFFFFFF for x in key])
    o = (ctypes.c_uint32 * 4)()
    lib().gso_philox4x32_10(c, k, o)
    return [int(x) for x in o]


def fetch_count(delta: float, f: int) -> int:
    return int(lib().gso_fetch_count(delta, f))


def refresh_count(mode: int, gamma: float, W: int) -> int:
    return int(lib().gso_refresh_count(mode, gamma, W))


def _copy(ptr, n):
    if n == 0:
        return np.empty(0, dtype=np.int32)
    return np.ctypeslib.as_array(ptr, shape=(n,)).copy()


class Block:
    """One hop's message-flow graph: dst = frontier[:num_dst], src = frontier[:num_src]."""

    def __init__(self, num_dst, num_src, indptr, indices, picked):
        self.num_dst, self.num_src = num_dst, num_src
        self.num_edges = int(indices.shape[0])
        self.indptr, self.indices, self.picked = indptr, indices, picked


class Sampler:
    """The oracle sampler over a host CSR graph (numpy int64 indptr, int32 indices)."""

    def __init__(self, indptr, indices, fanouts, cache_width, seed, shared=False):
        self.indptr = np.ascontiguousarray(indptr, dtype=np.int64)
        self.indices = np.ascontiguousarray(indices, dtype=np.int32)
        self.num_nodes = self.indptr.shape[0] - 1
        self.fanouts = [int(f) for f in fanouts]
        self.L = len(self.fanouts)
        self.W = int(cache_width)
        self.shared = bool(shared)
        fo = (ctypes.c_int32 * self.L)(*self.fanouts)
        self._h = lib().gso_create(self.num_nodes, self.indptr.ctypes.data, self.indices.ctypes.data, self.L, fo,
                                   self.W, ctypes.c_uint64(int(seed)), int(self.shared))
        if not self._h:
            raise ValueError("gso_create rejected the arguments")
        self._key_cb = None

    def close(self):
        if self._h:
            lib().gso_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_theta(self, theta):
        """Dense/sparse split: nodes with degree <= theta are sampled straight from the graph."""
        lib().gso_set_theta(self._h, int(theta))

    def set_key_fn(self, fn):
        """fn(purpose, tag, v, step, i) -> uint32 replaces the Philox keys (None restores them)."""
        if fn is None:
            self._key_cb = ctypes.cast(None, KEY_FN)
        else:
            self._key_cb = KEY_FN(lambda ctx, purpose, tag, v, step, i: int(fn(purpose, tag, v, step, i)) & 0xFFFFFFFF)
        lib().gso_set_key_fn(self._h, self._key_cb, None)

    def cache_row(self, layer, v):
        out = np.empty(self.W, dtype=np.int32)
        if lib().gso_cache_row(self._h, layer, int(v), out.ctypes.data):
            raise ValueError("bad layer/node")
        return out

    def cache_rows(self, layer, nodes):
        return np.stack([self.cache_row(layer, v) for v in nodes]) if len(nodes) else np.empty((0, self.W), np.int32)

    def cache_set_row(self, layer, v, row):
        row = np.ascontiguousarray(row, dtype=np.int32)
        assert row.shape == (self.W,)
        if lib().gso_cache_set_row(self._h, layer, int(v), row.ctypes.data):
            raise ValueError("bad layer/node")

    def refresh_node(self, layer, v, step, r):
        if lib().gso_refresh_node(self._h, layer, int(v), step, r):
            raise ValueError("bad arguments")

    def refresh_all(self, mode, gamma, step):
        if lib().gso_refresh_all(self._h, mode, float(gamma), step):
            raise ValueError("bad arguments")

    def pick_node(self, layer, v, step):
        out = np.empty(self.W, dtype=np.int32)
        cnt = ctypes.c_int32(0)
        if lib().gso_pick_node(self._h, layer, int(v), step, out.ctypes.data, ctypes.byref(cnt)):
            raise ValueError("bad arguments")
        return out[: cnt.value].copy()

    def fetch_node(self, layer, v, step, n_fetch):
        out = np.empty(max(self.fanouts), dtype=np.int32)
        cnt = ctypes.c_int32(0)
        if lib().gso_fetch_node(self._h, layer, int(v), step, int(n_fetch), out.ctypes.data, ctypes.byref(cnt)):
            raise ValueError("bad arguments")
        return out[: cnt.value].copy()

    def fbl_node(self, layer, v, step):
        out = np.empty(max(self.fanouts), dtype=np.int32)
        cnt = ctypes.c_int32(0)
        if lib().gso_fbl_node(self._h, layer, int(v), step, out.ctypes.data, ctypes.byref(cnt)):
            raise ValueError("bad arguments")
        return out[: cnt.value].copy()

    def sample_batch(self, seeds, mode, gamma, step):
        """Returns (frontier [n_L] global ids, [n_0..n_L], blocks indexed by layer)."""
        seeds = np.ascontiguousarray(seeds, dtype=np.int32)
        rc = lib().gso_sample_batch(self._h, seeds.ctypes.data, seeds.shape[0], mode, float(gamma), step)
        if rc:
            raise ValueError("gso_sample_batch failed with code %d" % rc)
        L = lib()
        n = [L.gso_num_nodes(self._h, k) for k in range(self.L + 1)]
        frontier = _copy(L.gso_frontier(self._h), n[self.L])
        blocks = []
        for layer in range(self.L):
            k = self.L - 1 - layer
            m = L.gso_num_edges(self._h, layer)
            blocks.append(Block(n[k], n[k + 1], _copy(L.gso_block_indptr(self._h, layer), n[k] + 1),
                                _copy(L.gso_block_indices(self._h, layer), m),
                                _copy(L.gso_block_picked(self._h, layer), m)))
        return frontier, n, blocks

    def stats(self):
        return int(lib().gso_stat_refreshed(self._h)), int(lib().gso_stat_scanned(self._h))


def gather(X: np.ndarray, ids) -> np.ndarray:
    """out[p, :] = X[ids[p], :] for a C-contiguous 2-D array of any item size."""
    X = np.ascontiguousarray(X)
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    out = np.empty((ids.shape[0], X.shape[1]), dtype=X.dtype)
    row_bytes = X.shape[1] * X.dtype.itemsize
    lib().gso_gather(X.ctypes.data, row_bytes, row_bytes, ids.ctypes.data, ids.shape[0], out.ctypes.data, row_bytes)
    return out
