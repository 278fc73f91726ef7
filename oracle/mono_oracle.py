"""ctypes front end of the CPU oracle (oracle/mono_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg.  Nothing here touches the CUDA library.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mono_oracle.cpp")
_LIB = os.path.join(_HERE, "libmono_oracle.so")

OK, ERR_ARG, ERR_TIME, ERR_FULL = 0, -1, -2, -3


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = f"{_LIB}.{os.getpid()}.tmp"
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fno-fast-math",
                               "-shared", "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        vp, u64, u32, i64, f32 = (ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint32,
                                  ctypes.c_int64, ctypes.c_float)
        L.oracle_create.restype = vp
        L.oracle_create.argtypes = [u64, u32, u32, u32, f32, f32, f32, f32, u64]
        L.oracle_enable_sketch.restype = ctypes.c_int
        L.oracle_enable_sketch.argtypes = [vp, u32, u64]
        L.oracle_sketch_index.restype = u64
        L.oracle_sketch_index.argtypes = [vp, u32, u64]
        L.oracle_destroy.restype = None
        L.oracle_destroy.argtypes = [vp]
        L.oracle_lookup_pool.restype = ctypes.c_int
        L.oracle_lookup_pool.argtypes = [vp, vp, i64, vp, i64, vp]
        L.oracle_apply_grads.restype = ctypes.c_int
        L.oracle_apply_grads.argtypes = [vp, vp, i64, vp, i64, vp, i64]
        L.oracle_expire.restype = i64
        L.oracle_expire.argtypes = [vp, i64]
        L.oracle_n_tracked.restype = i64
        L.oracle_n_tracked.argtypes = [vp]
        L.oracle_n_resident.restype = i64
        L.oracle_n_resident.argtypes = [vp]
        L.oracle_probe.restype = ctypes.c_int
        L.oracle_probe.argtypes = [vp, vp, i64, vp, vp, vp, vp, vp]
        L.oracle_export.restype = i64
        L.oracle_export.argtypes = [vp, vp, vp, vp, vp, vp, vp]
        L.oracle_n_touched.restype = i64
        L.oracle_n_touched.argtypes = [vp]
        L.oracle_export_touched.restype = i64
        L.oracle_export_touched.argtypes = [vp, vp, vp]
        L.oracle_import.restype = ctypes.c_int
        L.oracle_import.argtypes = [vp, vp, vp, vp, vp, vp, vp, i64]
        L.oracle_philox4x32_10.restype = None
        L.oracle_philox4x32_10.argtypes = [vp, vp, vp]
        L.oracle_init_value.restype = f32
        L.oracle_init_value.argtypes = [u64, u64, u32, f32]
        _lib = L
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


class OracleTable:
    """The plain map-based table: one entry per tracked ID."""

    def __init__(self, capacity: int, dim: int, filter_threshold: int, ttl: int, *, lr: float = 0.05,
                 eps: float = 1e-8, init_acc: float = 0.0, init_scale: float = 0.01, seed: int = 0,
                 sketch_depth: int = 0, sketch_width: int = 0):
        self.dim = int(dim)
        self.capacity = int(capacity)
        self.threshold = max(int(filter_threshold), 1)
        self.ttl = int(ttl)
        self._h = lib().oracle_create(capacity, dim, filter_threshold, ttl, lr, eps, init_acc,
                                      init_scale, seed)
        if not self._h:
            raise ValueError("oracle_create rejected its arguments")
        if sketch_depth:
            if lib().oracle_enable_sketch(self._h, sketch_depth, sketch_width) != OK:
                raise ValueError("sketch needs depth >= 1 and a power-of-two width")

    def close(self):
        if self._h:
            lib().oracle_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def sketch_index(self, r: int, id_: int) -> int:
        return int(lib().oracle_sketch_index(self._h, r, id_))

    def lookup_pool(self, ids, offsets) -> np.ndarray:
        ids, offsets = _c(ids, np.uint64), _c(offsets, np.int64)
        n_bags = offsets.size - 1
        out = np.empty((n_bags, self.dim), dtype=np.float32)
        rc = lib().oracle_lookup_pool(self._h, _p(ids), ids.size, _p(offsets), n_bags, _p(out))
        if rc != OK:
            raise RuntimeError(f"oracle_lookup_pool failed: {rc}")
        return out

    def apply_grads(self, ids, offsets, grad_pooled, now: int) -> int:
        ids, offsets = _c(ids, np.uint64), _c(offsets, np.int64)
        grad_pooled = _c(grad_pooled, np.float32)
        n_bags = offsets.size - 1
        assert grad_pooled.size == n_bags * self.dim
        return lib().oracle_apply_grads(self._h, _p(ids), ids.size, _p(offsets), n_bags,
                                        _p(grad_pooled), int(now))

    def expire(self, now: int) -> int:
        return int(lib().oracle_expire(self._h, int(now)))

    @property
    def n_tracked(self) -> int:
        return int(lib().oracle_n_tracked(self._h))

    @property
    def n_resident(self) -> int:
        return int(lib().oracle_n_resident(self._h))

    def probe(self, ids, rows: bool = True):
        ids = _c(ids, np.uint64)
        n = ids.size
        res = np.empty(n, np.uint8)
        cnt = np.empty(n, np.uint32)
        seen = np.empty(n, np.int64)
        w = np.empty((n, self.dim), np.float32) if rows else None
        acc = np.empty((n, self.dim), np.float32) if rows else None
        lib().oracle_probe(self._h, _p(ids), n, _p(res), _p(cnt), _p(seen), _p(w), _p(acc))
        return {"resident": res, "count": cnt, "last_seen": seen, "w": w, "acc": acc}

    def export(self):
        n = self.n_tracked
        ids = np.empty(n, np.uint64)
        res = np.empty(n, np.uint8)
        cnt = np.empty(n, np.uint32)
        seen = np.empty(n, np.int64)
        w = np.empty((n, self.dim), np.float32)
        acc = np.empty((n, self.dim), np.float32)
        m = lib().oracle_export(self._h, _p(ids), _p(cnt), _p(seen), _p(res), _p(w), _p(acc))
        assert m == n
        return {"ids": ids, "resident": res, "count": cnt, "last_seen": seen, "w": w, "acc": acc}

    def export_touched(self):
        """IDs trained since the last call (sorted) and their rows; empties the set."""
        n = int(lib().oracle_n_touched(self._h))
        ids = np.empty(n, np.uint64)
        w = np.empty((n, self.dim), np.float32)
        m = lib().oracle_export_touched(self._h, _p(ids), _p(w))
        assert m == n
        return {"ids": ids, "w": w}

    def import_entries(self, ids, count, last_seen, resident, w=None, acc=None) -> int:
        ids = _c(ids, np.uint64)
        count, last_seen, resident = _c(count, np.uint32), _c(last_seen, np.int64), _c(resident, np.uint8)
        w = None if w is None else _c(w, np.float32)
        acc = None if acc is None else _c(acc, np.float32)
        return lib().oracle_import(self._h, _p(ids), _p(count), _p(last_seen), _p(resident),
                                   _p(w), _p(acc), ids.size)


def philox4x32_10(ctr, key) -> np.ndarray:
    ctr, key = _c(ctr, np.uint32), _c(key, np.uint32)
    out = np.empty(4, np.uint32)
    lib().oracle_philox4x32_10(_p(ctr), _p(key), _p(out))
    return out


def init_value(seed: int, id_: int, col: int, scale: float) -> float:
    return float(lib().oracle_init_value(seed, id_, col, scale))
