"""Shared helpers of the GPU parity tests: run the same seeded steps through the
CPU oracle and the CUDA library and compare the complete table state.

Integer state (tracked set, resident set, counts, last-seen times) must be
bit-exact.  Floating point is compared per vector (a pooled bag, a row, an
accumulator row):  max|gpu - oracle| <= TOL * max|oracle|, and an all-zero
oracle vector must be all-zero on the GPU.  TOL is the 1e-5 the table's
specification states for fp32 results.
"""
from __future__ import annotations

import numpy as np

TOL = 1e-5


def assert_vectors_close(got: np.ndarray, want: np.ndarray, what: str, tol: float = TOL):
    assert got.shape == want.shape, f"{what}: shape {got.shape} vs {want.shape}"
    if got.size == 0:
        return
    got64, want64 = got.astype(np.float64), want.astype(np.float64)
    err = np.abs(got64 - want64).reshape(got.shape[0], -1).max(axis=1)
    ref = np.abs(want64).reshape(got.shape[0], -1).max(axis=1)
    bad = err > tol * ref
    if bad.any():
        k = int(np.argmax(err - tol * ref))
        raise AssertionError(f"{what}: {int(bad.sum())} of {len(bad)} vectors off; worst vector {k}: "
                             f"err {err[k]:.3e} vs ref {ref[k]:.3e}\n got {got[k][:8]}\nwant {want[k][:8]}")


def assert_state_equal(gpu_table, oracle, what: str = "state", rows: bool = True):
    """Full-table comparison through mono_export / oracle export (both sorted by ID)."""
    g, o = gpu_table.export(rows=rows), oracle.export()
    assert len(g["ids"]) == len(o["ids"]), f"{what}: tracked {len(g['ids'])} vs oracle {len(o['ids'])}"
    assert (g["ids"] == o["ids"]).all(), f"{what}: tracked ID sets differ"
    assert (g["resident"] == o["resident"]).all(), f"{what}: resident sets differ"
    assert (g["count"] == o["count"]).all(), f"{what}: counts differ"
    assert (g["last_seen"] == o["last_seen"]).all(), f"{what}: last_seen differ"
    st = gpu_table.status()
    assert st["n_tracked"] == oracle.n_tracked and st["n_resident"] == oracle.n_resident
    if rows:
        assert_vectors_close(g["w"], o["w"], f"{what}: rows")
        assert_vectors_close(g["acc"], o["acc"], f"{what}: accumulators")


def assert_audit_ok(gpu_table, what: str = "audit"):
    a = gpu_table.audit()
    assert a["ok"] == 1, f"{what}: {a}"
    return a


def run_stream(gpu_table, oracle, stream, steps, *, sweep_every: int = 1, check_every: int = 1,
               time_scale: int = 1, check_forward: bool = True, prepare=False):
    """Feed steps [0, steps) of `stream` to both sides; compare as it goes.  With `prepare`
    every batch is announced with mono_prepare_push before its lookup, as a training loop
    that knows its batch ahead of the pull would do; with prepare="ahead" the next batch is also
    grouped with mono_group_ahead while the current one is being pulled and pushed."""
    import torch
    from paper_2209_07663_b200 import binding as mb

    def device_batch(s):
        ids = torch.from_numpy(s.ids.view(np.int64)).cuda()
        off = torch.from_numpy(s.offsets).cuda()
        return ids, off, torch.from_numpy(s.grad_pooled).cuda()

    ahead = prepare == "ahead"
    upcoming = None
    if ahead and steps > 0:
        upcoming = (stream.step(0),) + device_batch(stream.step(0))
        mb.mono_group_ahead(gpu_table.handle, upcoming[1], upcoming[1].numel(), upcoming[2], upcoming[2].numel() - 1)
    for t in range(steps):
        s = upcoming[0] if ahead else stream.step(t)
        now = t * time_scale
        if prepare:
            ids, off, grad = upcoming[1:] if ahead else device_batch(s)
            n_bags = off.numel() - 1
            mb.mono_prepare_push(gpu_table.handle, ids, ids.numel(), off, n_bags)
            if ahead and t + 1 < steps:
                nxt = stream.step(t + 1)
                upcoming = (nxt,) + device_batch(nxt)
                mb.mono_group_ahead(gpu_table.handle, upcoming[1], upcoming[1].numel(), upcoming[2], upcoming[2].numel() - 1)
            if check_forward:
                out = torch.empty((n_bags, gpu_table.dim), dtype=torch.float32, device="cuda")
                mb.mono_lookup_pool(gpu_table.handle, ids, ids.numel(), off, n_bags, out)
                assert_vectors_close(out.cpu().numpy(), oracle.lookup_pool(s.ids, s.offsets), f"step {t}: pooled output")
            mb.mono_apply_grads(gpu_table.handle, ids, ids.numel(), off, n_bags, grad, now)
        else:
            if check_forward:
                got = gpu_table.lookup_pool(s.ids, s.offsets).cpu().numpy()
                assert_vectors_close(got, oracle.lookup_pool(s.ids, s.offsets), f"step {t}: pooled output")
            gpu_table.apply_grads(s.ids, s.offsets, s.grad_pooled, now)
        assert oracle.apply_grads(s.ids, s.offsets, s.grad_pooled, now) == 0, "stream overflowed the oracle"
        if sweep_every and t % sweep_every == sweep_every - 1:
            gpu_table.expire(now)
            oracle.expire(now)
        if check_every and (t % check_every == check_every - 1 or t == steps - 1):
            assert_state_equal(gpu_table, oracle, f"step {t}")
            assert_audit_ok(gpu_table, f"step {t}")
    st = gpu_table.status()
    assert st["error_bits"] == 0, f"device error bits {st['error_bits']}"
    return st
