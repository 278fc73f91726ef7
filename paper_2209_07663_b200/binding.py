"""ctypes binding of the C ABI in include/mono.h.

Marshals arguments only: tensors become raw pointers, options become the C
structs, return codes become exceptions.  Every step of the table's work runs in
the CUDA library.  There is no fallback: if libmono.so is missing, loading
raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

_PKG = os.path.dirname(os.path.abspath(__file__))
# MONO_LIBRARY=checked selects the build with device-side index checks (libmono_checked.so, see build.py);
# any other value is taken as the path of a build of the library
_WHICH = os.environ.get("MONO_LIBRARY", "")
LIB_PATH = (os.path.join(_PKG, "libmono_checked.so") if _WHICH == "checked" else
            os.path.abspath(_WHICH) if _WHICH else os.path.join(_PKG, "libmono.so"))

MONO_OK, MONO_ERR_ARG, MONO_ERR_TIME, MONO_ERR_CUDA, MONO_ERR_NOMEM, MONO_ERR_SIZE = 0, -1, -2, -3, -4, -5
MONO_ERR_LIMIT = -6
MONO_NOALLOC_MAX_IDS = 1 << 20
MONO_DEV_ROWS_FULL, MONO_DEV_KEYS_FULL, MONO_DEV_BAD_OFFSETS, MONO_DEV_IMPORT_DUP, MONO_DEV_INTERNAL = 1, 2, 4, 8, 16
MONO_RESERVED_ID = 0xFFFFFFFFFFFFFFFF
MONO_MAX_NOW = 0xFFFFFFFE

EXPORTS = [
    "mono_table_create", "mono_table_destroy", "mono_reserve", "mono_lookup_pool", "mono_apply_grads",
    "mono_expire", "mono_lookup_pool_host", "mono_apply_grads_host", "mono_status", "mono_clear_errors",
    "mono_probe", "mono_read_rows", "mono_export", "mono_import", "mono_audit", "mono_last_cuda_error",
    "mono_error_string", "mono_timing_enable", "mono_timing_read", "mono_lookup_pool_noalloc", "mono_export_touched", "mono_rehash", "mono_expire_slice", "mono_prepare_push", "mono_group_ahead",
    "mono_group_lookup_pool", "mono_group_apply_grads", "mono_group_prepare_push", "mono_fence", "mono_snapshot_save", "mono_snapshot_restore",
    "mono_snapshot_drop",
]


class MonoError(RuntimeError):
    def __init__(self, fn: str, code: int, detail: str = ""):
        self.code = code
        super().__init__(f"{fn} failed: {error_string(code)} ({code}){': ' + detail if detail else ''}")


class mono_opt(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("lr", ctypes.c_float), ("eps", ctypes.c_float),
                ("init_acc", ctypes.c_float), ("init_scale", ctypes.c_float), ("seed", ctypes.c_uint64),
                ("key_cells", ctypes.c_uint64), ("max_ids", ctypes.c_uint64), ("max_bags", ctypes.c_uint64),
                ("sketch_width", ctypes.c_uint64), ("sketch_depth", ctypes.c_uint32), ("pad_", ctypes.c_uint32)]


class mono_status_t(ctypes.Structure):
    _fields_ = [("error_bits", ctypes.c_uint32), ("dim", ctypes.c_uint32), ("capacity", ctypes.c_uint64),
                ("key_cells", ctypes.c_uint64), ("n_tracked", ctypes.c_uint64), ("n_resident", ctypes.c_uint64),
                ("n_admitted_total", ctypes.c_uint64), ("n_expired_total", ctypes.c_uint64),
                ("n_inserted_total", ctypes.c_uint64), ("n_rows_refused", ctypes.c_uint64),
                ("n_keys_dropped", ctypes.c_uint64), ("n_evictions_total", ctypes.c_uint64),
                ("max_chain", ctypes.c_uint32), ("stash_used", ctypes.c_uint32), ("sum_ids", ctypes.c_uint64),
                ("sum_unique", ctypes.c_uint64), ("sum_unique_resident", ctypes.c_uint64),
                ("sum_new", ctypes.c_uint64), ("sum_single_resident", ctypes.c_uint64),
                ("scratch_reallocs", ctypes.c_uint64)]


class mono_audit_t(ctypes.Structure):
    _fields_ = [("occupied_cells", ctypes.c_uint64), ("misplaced", ctypes.c_uint64),
                ("duplicate_keys", ctypes.c_uint64), ("resident_cells", ctypes.c_uint64),
                ("bad_rows", ctypes.c_uint64), ("shared_rows", ctypes.c_uint64), ("free_rows", ctypes.c_uint64),
                ("unaccounted_rows", ctypes.c_uint64), ("ok", ctypes.c_uint32), ("behind_records", ctypes.c_uint32)]


class mono_kernel_time_t(ctypes.Structure):
    _fields_ = [("name", ctypes.c_char * 32), ("launches", ctypes.c_uint64), ("ms", ctypes.c_double)]


class mono_timing_t(ctypes.Structure):
    _fields_ = [("n_kernels", ctypes.c_uint32), ("pad_", ctypes.c_uint32), ("launches_total", ctypes.c_uint64),
                ("kernel", mono_kernel_time_t * 24)]


def _struct_dict(s: ctypes.Structure) -> dict:
    return {name: getattr(s, name) for name, _ in s._fields_ if not name.startswith("pad")}


_lib = None


def load_library(path: Optional[str] = None):
    """Load libmono.so and declare its prototypes.  Raises if it is not there."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    path = path or LIB_PATH
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python -m paper_2209_07663_b200.build` "
                           "(there is no non-CUDA fallback)")
    L = ctypes.CDLL(path)
    vp, i64, u64, u32, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_int
    proto = {
        "mono_table_create": (ci, [ctypes.POINTER(vp), u64, u32, u32, u32, ctypes.POINTER(mono_opt), vp]),
        "mono_table_destroy": (ci, [vp]),
        "mono_reserve": (ci, [vp, i64, i64]),
        "mono_lookup_pool": (ci, [vp, vp, i64, vp, i64, vp]),
        "mono_apply_grads": (ci, [vp, vp, i64, vp, i64, vp, i64]),
        "mono_expire": (ci, [vp, i64]),
        "mono_prepare_push": (ci, [vp, vp, i64, vp, i64]),
        "mono_group_ahead": (ci, [vp, vp, i64, vp, i64]),
        "mono_expire_slice": (ci, [vp, i64, u32, u32]),
        "mono_group_prepare_push": (ci, [ctypes.c_int32, vp, vp, vp, vp, vp, vp]),
        "mono_group_lookup_pool": (ci, [ctypes.c_int32, vp, vp, vp, vp, vp, vp, vp]),
        "mono_group_apply_grads": (ci, [ctypes.c_int32, vp, vp, vp, vp, vp, vp, i64, vp]),
        "mono_lookup_pool_host": (ci, [vp, vp, i64, vp, i64, vp]),
        "mono_apply_grads_host": (ci, [vp, vp, i64, vp, i64, vp, i64]),
        "mono_status": (ci, [vp, ctypes.POINTER(mono_status_t)]),
        "mono_clear_errors": (ci, [vp]),
        "mono_probe": (ci, [vp, vp, i64, vp, vp, vp]),
        "mono_read_rows": (ci, [vp, vp, i64, vp, vp]),
        "mono_export": (ci, [vp, vp, vp, vp, vp, vp, vp, i64, ctypes.POINTER(i64)]),
        "mono_import": (ci, [vp, vp, vp, vp, vp, vp, vp, i64]),
        "mono_export_touched": (ci, [vp, vp, vp, i64, ctypes.POINTER(i64)]),
        "mono_rehash": (ci, [vp, u64, u64]),
        "mono_audit": (ci, [vp, ctypes.POINTER(mono_audit_t)]),
        "mono_last_cuda_error": (ctypes.c_char_p, [vp]),
        "mono_error_string": (ctypes.c_char_p, [ci]),
        "mono_lookup_pool_noalloc": (ci, [vp, vp, i64, vp, i64, vp]),
        "mono_fence": (ci, [vp]),
        "mono_snapshot_save": (ci, [vp]),
        "mono_snapshot_restore": (ci, [vp]),
        "mono_snapshot_drop": (ci, [vp]),
        "mono_timing_enable": (ci, [vp, ci]),
        "mono_timing_read": (ci, [vp, ctypes.POINTER(mono_timing_t), ci]),
    }
    for name, (res, args) in proto.items():
        fn = getattr(L, name)
        fn.restype, fn.argtypes = res, args
    _lib = L
    return L


def error_string(code: int) -> str:
    try:
        return load_library().mono_error_string(code).decode()
    except Exception:
        return str(code)


def _ptr(x):
    """Raw address of a torch tensor / numpy array / int / None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        if not x.is_contiguous():
            raise ValueError("tensors passed to the C ABI must be contiguous")
        return x.data_ptr()
    if hasattr(x, "ctypes"):
        if not x.flags["C_CONTIGUOUS"]:
            raise ValueError("arrays passed to the C ABI must be C-contiguous")
        return x.ctypes.data
    raise TypeError(f"cannot take the address of {type(x)!r}")


def _check(fn: str, rc: int, handle=None):
    if rc != MONO_OK:
        detail = ""
        if rc in (MONO_ERR_CUDA, MONO_ERR_NOMEM) and handle:
            detail = (load_library().mono_last_cuda_error(handle) or b"").decode()
        raise MonoError(fn, rc, detail)


# ---- functions with the names of the C ABI ---------------------------------

def mono_table_create(capacity: int, dim: int, filter_threshold: int, ttl: int, *, lr: float = 0.05,
                      eps: float = 1e-8, init_acc: float = 0.0, init_scale: float = 0.0, seed: int = 0,
                      key_cells: int = 0, max_ids: int = 0, max_bags: int = 0, stream: int = 0,
                      sketch_depth: int = 0, sketch_width: int = 0) -> int:
    """Returns the table handle (an integer address)."""
    opt = mono_opt(kind=1, lr=lr, eps=eps, init_acc=init_acc, init_scale=init_scale, seed=seed,
                   key_cells=key_cells, max_ids=max_ids, max_bags=max_bags, sketch_width=sketch_width,
                   sketch_depth=sketch_depth)
    h = ctypes.c_void_p()
    rc = load_library().mono_table_create(ctypes.byref(h), capacity, dim, filter_threshold, ttl,
                                          ctypes.byref(opt), stream or None)
    _check("mono_table_create", rc)
    return h.value


def mono_table_destroy(t: int) -> None:
    _check("mono_table_destroy", load_library().mono_table_destroy(t))


def mono_reserve(t: int, max_ids: int, max_bags: int) -> None:
    _check("mono_reserve", load_library().mono_reserve(t, max_ids, max_bags), t)


def mono_lookup_pool(t: int, ids, n_ids: int, slot_offsets, n_bags: int, out) -> None:
    _check("mono_lookup_pool", load_library().mono_lookup_pool(t, _ptr(ids), n_ids, _ptr(slot_offsets), n_bags,
                                                               _ptr(out)), t)


def mono_lookup_pool_noalloc(t: int, ids, n_ids: int, slot_offsets, n_bags: int, out) -> None:
    """mono_lookup_pool for callers that may not allocate device memory: the per-ID scratch
    lives in a fixed array inside the library, so at most MONO_NOALLOC_MAX_IDS IDs per call,
    and calls must not overlap on the GPU."""
    _check("mono_lookup_pool_noalloc", load_library().mono_lookup_pool_noalloc(t, _ptr(ids), n_ids, _ptr(slot_offsets),
                                                                               n_bags, _ptr(out)), t)


def mono_apply_grads(t: int, ids, n_ids: int, slot_offsets, n_bags: int, grad_pooled, now: int) -> None:
    _check("mono_apply_grads", load_library().mono_apply_grads(t, _ptr(ids), n_ids, _ptr(slot_offsets), n_bags,
                                                               _ptr(grad_pooled), now), t)


def mono_expire(t: int, now: int) -> None:
    _check("mono_expire", load_library().mono_expire(t, now), t)


def mono_group_ahead(t: int, ids, n_ids: int, slot_offsets, n_bags: int) -> None:
    _check("mono_group_ahead", load_library().mono_group_ahead(t, _ptr(ids), n_ids, _ptr(slot_offsets), n_bags), t)


def mono_prepare_push(t: int, ids, n_ids: int, slot_offsets, n_bags: int) -> None:
    _check("mono_prepare_push", load_library().mono_prepare_push(t, _ptr(ids), n_ids, _ptr(slot_offsets), n_bags), t)


def _group_args(handles, ids, slot_offsets, vectors):
    """Host arrays of the grouped calls: one entry per table."""
    n = len(handles)
    if not (len(ids) == len(slot_offsets) == len(vectors) == n):
        raise ValueError("grouped calls take one batch per table")
    ptrs = ctypes.c_void_p * n
    i64s = ctypes.c_int64 * n
    return (n, ptrs(*handles), ptrs(*[_ptr(x) for x in ids]), i64s(*[x.numel() for x in ids]),
            ptrs(*[_ptr(x) for x in slot_offsets]), i64s(*[x.numel() - 1 for x in slot_offsets]),
            ptrs(*[_ptr(x) for x in vectors]))


def mono_group_prepare_push(handles, ids, slot_offsets, group_stream: int = 0) -> None:
    """Announce every table's next batch (lists of device tensors, one per table)."""
    n, tp, ip, nip, op, nbp, _ = _group_args(handles, ids, slot_offsets, ids)
    code = load_library().mono_group_prepare_push(n, tp, ip, nip, op, nbp, group_stream or None)
    if code != 0:
        raise MonoError("mono_group_prepare_push", code)


def mono_group_lookup_pool(handles, ids, slot_offsets, outs, group_stream: int = 0) -> None:
    """ids / slot_offsets / outs: lists of device tensors, one per table."""
    n, tp, ip, nip, op, nbp, vp_ = _group_args(handles, ids, slot_offsets, outs)
    code = load_library().mono_group_lookup_pool(n, tp, ip, nip, op, nbp, vp_, group_stream or None)
    if code != 0:
        raise MonoError("mono_group_lookup_pool", code)


def mono_group_apply_grads(handles, ids, slot_offsets, grads, now: int, group_stream: int = 0) -> None:
    n, tp, ip, nip, op, nbp, vp_ = _group_args(handles, ids, slot_offsets, grads)
    code = load_library().mono_group_apply_grads(n, tp, ip, nip, op, nbp, vp_, now, group_stream or None)
    if code != 0:
        raise MonoError("mono_group_apply_grads", code)


def mono_expire_slice(t: int, now: int, slice_index: int, n_slices: int) -> None:
    _check("mono_expire_slice", load_library().mono_expire_slice(t, now, slice_index, n_slices), t)


def mono_fence(t: int) -> None:
    _check("mono_fence", load_library().mono_fence(t), t)


def mono_snapshot_save(t: int) -> None:
    _check("mono_snapshot_save", load_library().mono_snapshot_save(t), t)


def mono_snapshot_restore(t: int) -> None:
    _check("mono_snapshot_restore", load_library().mono_snapshot_restore(t), t)


def mono_snapshot_drop(t: int) -> None:
    _check("mono_snapshot_drop", load_library().mono_snapshot_drop(t), t)


def mono_lookup_pool_host(t: int, ids, n_ids: int, slot_offsets, n_bags: int, out) -> None:
    _check("mono_lookup_pool_host", load_library().mono_lookup_pool_host(t, _ptr(ids), n_ids, _ptr(slot_offsets),
                                                                         n_bags, _ptr(out)), t)


def mono_apply_grads_host(t: int, ids, n_ids: int, slot_offsets, n_bags: int, grad_pooled, now: int) -> None:
    _check("mono_apply_grads_host", load_library().mono_apply_grads_host(t, _ptr(ids), n_ids, _ptr(slot_offsets),
                                                                         n_bags, _ptr(grad_pooled), now), t)


def mono_status(t: int) -> dict:
    s = mono_status_t()
    _check("mono_status", load_library().mono_status(t, ctypes.byref(s)), t)
    return _struct_dict(s)


def mono_clear_errors(t: int) -> None:
    _check("mono_clear_errors", load_library().mono_clear_errors(t), t)


def mono_probe(t: int, ids, n: int, resident=None, count=None, last_seen=None) -> None:
    _check("mono_probe", load_library().mono_probe(t, _ptr(ids), n, _ptr(resident), _ptr(count), _ptr(last_seen)), t)


def mono_read_rows(t: int, ids, n: int, w=None, acc=None) -> None:
    _check("mono_read_rows", load_library().mono_read_rows(t, _ptr(ids), n, _ptr(w), _ptr(acc)), t)


def mono_export(t: int, ids, count, last_seen, resident, w, acc, max_n: int) -> int:
    n = ctypes.c_int64(0)
    rc = load_library().mono_export(t, _ptr(ids), _ptr(count), _ptr(last_seen), _ptr(resident), _ptr(w), _ptr(acc),
                                    max_n, ctypes.byref(n))
    if rc == MONO_ERR_SIZE:
        raise MonoError("mono_export", rc, f"{n.value} entries needed, {max_n} given")
    _check("mono_export", rc, t)
    return n.value


def mono_rehash(t: int, new_key_cells: int = 0, new_seed: int = 0) -> None:
    _check("mono_rehash", load_library().mono_rehash(t, new_key_cells, new_seed), t)


def mono_export_touched(t: int, ids, w, max_n: int) -> int:
    """Export and clear the touched set; returns how many touched IDs there were (if that is more
    than max_n only the first max_n were exported and the rest stay touched)."""
    n = ctypes.c_int64(0)
    rc = load_library().mono_export_touched(t, _ptr(ids), _ptr(w), max_n, ctypes.byref(n))
    if rc != MONO_ERR_SIZE:
        _check("mono_export_touched", rc, t)
    return n.value


def mono_import(t: int, ids, count, last_seen, resident, w, acc, n: int) -> None:
    _check("mono_import", load_library().mono_import(t, _ptr(ids), _ptr(count), _ptr(last_seen), _ptr(resident),
                                                     _ptr(w), _ptr(acc), n), t)


def mono_audit(t: int) -> dict:
    a = mono_audit_t()
    _check("mono_audit", load_library().mono_audit(t, ctypes.byref(a)), t)
    return _struct_dict(a)


def mono_timing_enable(t: int, on: bool) -> None:
    _check("mono_timing_enable", load_library().mono_timing_enable(t, 1 if on else 0), t)


def mono_timing_read(t: int, reset: bool = False) -> dict:
    """{'launches_total': n, 'kernels': {name: {'launches': n, 'ms': total device ms}}}"""
    tm = mono_timing_t()
    _check("mono_timing_read", load_library().mono_timing_read(t, ctypes.byref(tm), 1 if reset else 0), t)
    ks = {tm.kernel[i].name.decode(): {"launches": int(tm.kernel[i].launches), "ms": float(tm.kernel[i].ms)}
          for i in range(tm.n_kernels)}
    return {"launches_total": int(tm.launches_total), "kernels": ks}


# ---- a small convenience wrapper over torch tensors -------------------------

class MonoTable:
    """Owns one table handle and allocates outputs as torch CUDA tensors.

    ids are passed as int64 or uint64 tensors (the bit pattern is what counts).
    """

    def __init__(self, capacity: int, dim: int, filter_threshold: int, ttl: int, **opt):
        import torch
        self._torch = torch
        if not torch.cuda.is_available():
            raise RuntimeError("MonoTable needs a CUDA device (there is no CPU path)")
        self.dim, self.capacity = int(dim), int(capacity)
        self.threshold = max(int(filter_threshold), 1)
        opt.setdefault("stream", torch.cuda.current_stream().cuda_stream)
        self.handle = mono_table_create(capacity, dim, filter_threshold, ttl, **opt)

    def close(self):
        if getattr(self, "handle", None):
            mono_table_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _dev(self, x, dtype):
        torch = self._torch
        if not torch.is_tensor(x):
            import numpy as np
            a = np.ascontiguousarray(x)
            if a.dtype == np.uint64:
                a = a.view(np.int64)
            elif a.dtype == np.uint32:
                a = a.view(np.int32)
            x = torch.from_numpy(a)
        if x.dtype == torch.uint64:
            x = x.view(torch.int64)
        return x.to(device="cuda", dtype=dtype).contiguous()

    def lookup_pool(self, ids, offsets, out=None):
        torch = self._torch
        ids, offsets = self._dev(ids, torch.int64), self._dev(offsets, torch.int64)
        n_bags = offsets.numel() - 1
        if out is None:
            out = torch.empty((n_bags, self.dim), dtype=torch.float32, device="cuda")
        mono_lookup_pool(self.handle, ids, ids.numel(), offsets, n_bags, out)
        return out

    def apply_grads(self, ids, offsets, grad_pooled, now: int):
        torch = self._torch
        ids, offsets = self._dev(ids, torch.int64), self._dev(offsets, torch.int64)
        grad_pooled = self._dev(grad_pooled, torch.float32)
        n_bags = offsets.numel() - 1
        assert grad_pooled.numel() == n_bags * self.dim
        mono_apply_grads(self.handle, ids, ids.numel(), offsets, n_bags, grad_pooled, int(now))

    def expire(self, now: int):
        mono_expire(self.handle, int(now))

    def status(self) -> dict:
        return mono_status(self.handle)

    def audit(self) -> dict:
        return mono_audit(self.handle)

    def probe(self, ids, rows: bool = True) -> dict:
        torch = self._torch
        ids = self._dev(ids, torch.int64)
        n = ids.numel()
        res = torch.empty(n, dtype=torch.uint8, device="cuda")
        cnt = torch.empty(n, dtype=torch.int32, device="cuda")
        seen = torch.empty(n, dtype=torch.int64, device="cuda")
        mono_probe(self.handle, ids, n, res, cnt, seen)
        out = {"resident": res.cpu().numpy(), "count": cnt.cpu().numpy().view("uint32"),
               "last_seen": seen.cpu().numpy(), "w": None, "acc": None}
        if rows:
            w = torch.empty((n, self.dim), dtype=torch.float32, device="cuda")
            acc = torch.empty((n, self.dim), dtype=torch.float32, device="cuda")
            mono_read_rows(self.handle, ids, n, w, acc)
            out["w"], out["acc"] = w.cpu().numpy(), acc.cpu().numpy()
        return out

    def export(self, rows: bool = True) -> dict:
        """All tracked IDs, sorted by ID (numpy arrays on the host)."""
        torch = self._torch
        import numpy as np
        n = int(self.status()["n_tracked"]) + 8
        ids = torch.empty(n, dtype=torch.int64, device="cuda")
        cnt = torch.empty(n, dtype=torch.int32, device="cuda")
        seen = torch.empty(n, dtype=torch.int64, device="cuda")
        res = torch.empty(n, dtype=torch.uint8, device="cuda")
        w = torch.empty((n, self.dim), dtype=torch.float32, device="cuda") if rows else None
        acc = torch.empty((n, self.dim), dtype=torch.float32, device="cuda") if rows else None
        m = mono_export(self.handle, ids, cnt, seen, res, w, acc, n)
        ids_h = ids[:m].cpu().numpy().view(np.uint64)
        order = np.argsort(ids_h, kind="stable")
        out = {"ids": ids_h[order], "count": cnt[:m].cpu().numpy().view(np.uint32)[order],
               "last_seen": seen[:m].cpu().numpy()[order], "resident": res[:m].cpu().numpy()[order]}
        if rows:
            out["w"], out["acc"] = w[:m].cpu().numpy()[order], acc[:m].cpu().numpy()[order]
        return out

    def rehash(self, new_key_cells: int = 0, new_seed: int = 0):
        mono_rehash(self.handle, new_key_cells, new_seed)

    def export_touched(self, max_n=None) -> dict:
        """IDs trained since the last call and their rows, sorted by ID; clears the set."""
        torch = self._torch
        import numpy as np
        n = int(self.status()["n_resident"]) + 8 if max_n is None else int(max_n)
        ids = torch.empty(n, dtype=torch.int64, device="cuda")
        w = torch.empty((n, self.dim), dtype=torch.float32, device="cuda")
        found = mono_export_touched(self.handle, ids, w, n)
        m = min(found, n)
        ids_h = ids[:m].cpu().numpy().view(np.uint64)
        order = np.argsort(ids_h, kind="stable")
        return {"ids": ids_h[order], "w": w[:m].cpu().numpy()[order], "found": found}

    def import_entries(self, ids, count, last_seen, resident, w=None, acc=None):
        torch = self._torch
        ids = self._dev(ids, torch.int64)
        count = self._dev(count, torch.int32) if not (torch.is_tensor(count) and count.dtype == torch.int32) \
            else count.cuda()
        last_seen = self._dev(last_seen, torch.int64)
        resident = self._dev(resident, torch.uint8)
        w = None if w is None else self._dev(w, torch.float32)
        acc = None if acc is None else self._dev(acc, torch.float32)
        mono_import(self.handle, ids, count, last_seen, resident, w, acc, ids.numel())
