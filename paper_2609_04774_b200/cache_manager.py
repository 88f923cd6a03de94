"""ctypes binding of the library's prefix-cache bookkeeping (cpcache.h): the same names as the C entry
points, argument marshalling only.  Host-only calls; they need the built libcpattn.so but no GPU."""
from __future__ import annotations

import ctypes

import numpy as np

from . import binding
from .binding import _check

EXPORTS = ["cp_prefill_time", "cp_prefer_degree", "cp_trie_create", "cp_trie_destroy", "cp_trie_set_worker",
           "cp_trie_add_replica", "cp_trie_drop_replica", "cp_trie_match", "cp_trie_reused", "cp_trie_reused_all", "cp_trie_replica_count",
           "cp_trie_stats", "cp_trie_size", "cp_trie_update", "cp_trie_scan"]


class cp_prefill_model(ctypes.Structure):
    _fields_ = [(n, ctypes.c_double) for n in ("d", "a", "b", "c", "alpha")]


class cp_trie_candidate(ctypes.Structure):
    _fields_ = [("node", ctypes.c_int32), ("degree", ctypes.c_int32), ("replicas", ctypes.c_int32),
                ("footprint", ctypes.c_int32), ("score", ctypes.c_double)]


def _lib():
    lib = binding.load()
    if not getattr(lib, "_cpcache_ready", False):
        lib.cp_prefill_time.restype = ctypes.c_double
        lib.cp_prefill_time.argtypes = [ctypes.POINTER(cp_prefill_model), ctypes.c_int64, ctypes.c_int64, ctypes.c_int32]
        for name in EXPORTS[1:]:
            getattr(lib, name).restype = ctypes.c_int
        lib._cpcache_ready = True
    return lib


def _model(m) -> cp_prefill_model:
    return m if isinstance(m, cp_prefill_model) else cp_prefill_model(*[float(x) for x in m])


class Keys:
    """Block keys of one request, marshalled once and accepted by every Trie method in place of a sequence."""

    def __init__(self, blocks):
        self.array = np.ascontiguousarray(blocks, dtype=np.uint64).reshape(-1)
        self.ptr = self.array.ctypes.data_as(ctypes.c_void_p)
        self.n = ctypes.c_int32(self.array.size)


def _keys(blocks):
    k = blocks if isinstance(blocks, Keys) else Keys(blocks)
    return k.array, k.ptr, k.n


def cp_prefill_time(model, R, P, C) -> float:
    return float(_lib().cp_prefill_time(ctypes.byref(_model(model)), int(R), int(P), int(C)))


def cp_prefer_degree(model, L, degree, reused_len, beta=1.0, lam=0.0):
    """-> (index of the preferred worker, its degree)."""
    d = np.ascontiguousarray(degree, dtype=np.int32)
    p = np.ascontiguousarray(reused_len, dtype=np.int64)
    assert d.size == p.size
    w, c = ctypes.c_int32(), ctypes.c_int32()
    _check(_lib().cp_prefer_degree(ctypes.byref(_model(model)), ctypes.c_int64(L), ctypes.c_int32(d.size),
                                   d.ctypes.data_as(ctypes.c_void_p), p.ctypes.data_as(ctypes.c_void_p),
                                   ctypes.c_double(beta), ctypes.c_double(lam), ctypes.byref(w), ctypes.byref(c)))
    return w.value, c.value


class Trie:
    """cp_trie handle with one method per entry point."""

    def __init__(self, degrees, block_tokens=64):
        d = np.ascontiguousarray(degrees, dtype=np.int32)
        self._h = ctypes.c_void_p()
        _check(_lib().cp_trie_create(ctypes.byref(self._h), d.ctypes.data_as(ctypes.c_void_p), ctypes.c_int32(d.size),
                                     ctypes.c_int32(block_tokens)))

    def close(self):
        if self._h:
            _lib().cp_trie_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_worker(self, worker, degree):
        _check(_lib().cp_trie_set_worker(self._h, ctypes.c_int32(worker), ctypes.c_int32(degree)))

    def add_replica(self, blocks, worker) -> int:
        a, ptr, n = _keys(blocks)
        node = ctypes.c_int32()
        _check(_lib().cp_trie_add_replica(self._h, ptr, n, ctypes.c_int32(worker), ctypes.byref(node)))
        return node.value

    def drop_replica(self, node, worker):
        _check(_lib().cp_trie_drop_replica(self._h, ctypes.c_int32(node), ctypes.c_int32(worker)))

    def match(self, blocks):
        a, ptr, n = _keys(blocks)
        nodes = np.zeros(max(a.size, 1), dtype=np.int32)
        m = ctypes.c_int32()
        _check(_lib().cp_trie_match(self._h, ptr, n, nodes.ctypes.data_as(ctypes.c_void_p), ctypes.byref(m)))
        return nodes[:m.value].tolist()

    def reused(self, blocks, worker) -> int:
        a, ptr, n = _keys(blocks)
        m = ctypes.c_int32()
        _check(_lib().cp_trie_reused(self._h, ptr, n, ctypes.c_int32(worker), ctypes.byref(m)))
        return m.value

    def reused_all(self, blocks, workers):
        """Reused blocks of every worker in `workers` (int32 array) -> int32 array."""
        a, ptr, n = _keys(blocks)
        w = np.ascontiguousarray(workers, dtype=np.int32)
        out = np.zeros(w.size, dtype=np.int32)
        _check(_lib().cp_trie_reused_all(self._h, ptr, n, w.ctypes.data_as(ctypes.c_void_p), ctypes.c_int32(w.size),
                                         out.ctypes.data_as(ctypes.c_void_p)))
        return out

    def replica_count(self, node, degree) -> int:
        c = ctypes.c_int32()
        _check(_lib().cp_trie_replica_count(self._h, ctypes.c_int32(node), ctypes.c_int32(degree), ctypes.byref(c)))
        return c.value

    def stats(self, node, degree):
        a, m = ctypes.c_double(), ctypes.c_double()
        _check(_lib().cp_trie_stats(self._h, ctypes.c_int32(node), ctypes.c_int32(degree), ctypes.byref(a), ctypes.byref(m)))
        return a.value, m.value

    def size(self) -> int:
        n = ctypes.c_int32()
        _check(_lib().cp_trie_size(self._h, ctypes.byref(n)))
        return n.value

    def update(self, blocks, L, worker, pref_degree, model):
        a, ptr, n = _keys(blocks)
        _check(_lib().cp_trie_update(self._h, ptr, n, ctypes.c_int64(L), ctypes.c_int32(worker),
                                     ctypes.c_int32(pref_degree), ctypes.byref(_model(model))))

    def scan(self, theta_inter, theta_intra, theta_reclaim, decay, max_ops):
        """-> (inter, intra, reclaim, totals); candidates as tuples (node, degree, replicas, footprint, score)."""
        arrs = [(cp_trie_candidate * max(max_ops, 1))() for _ in range(3)]
        written, totals = (ctypes.c_int32 * 3)(), (ctypes.c_int32 * 3)()
        _check(_lib().cp_trie_scan(self._h, ctypes.c_double(theta_inter), ctypes.c_double(theta_intra),
                                   ctypes.c_double(theta_reclaim), ctypes.c_double(decay), ctypes.c_int32(max_ops),
                                   arrs[0], arrs[1], arrs[2], written, totals))
        lists = [[(c.node, c.degree, c.replicas, c.footprint, c.score) for c in arr[:written[k]]]
                 for k, arr in enumerate(arrs)]
        return lists[0], lists[1], lists[2], tuple(totals)
