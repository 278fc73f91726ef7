"""mono_lookup_pool_noalloc: the forward call for callers that cannot allocate device
memory (a serving loop with a fixed memory budget, a process whose allocator owns the
whole device).  Its per-ID scratch is a fixed array inside the library, shared by every
call, so the test checks it against the allocating entry point on two calls in a row --
the second call finds the first call's leftovers in the array -- and checks that an
oversized batch is refused instead of overrunning the array.

Collected last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

from paper_2209_07663_b200 import binding as mb
from paper_2209_07663_b200 import workload as wl
from tests.parity import assert_vectors_close

pytestmark = pytest.mark.gpu


def _table_with_rows(cfg):
    t = mb.MonoTable(cfg.capacity, cfg.dim, 1, 0, key_cells=cfg.key_cells, init_scale=0.05, seed=cfg.seed)
    stream = wl.Stream(cfg)
    for step in range(3):                       # threshold 1: every ID of these batches gets a row
        s = stream.step(step)
        t.apply_grads(s.ids, s.offsets, s.grad_pooled, step)
    return t, stream


def test_noalloc_lookup_matches_the_allocating_entry_point_twice_in_a_row():
    cfg = wl.scaled(wl.CONFIGS["tiny"], n_examples=2048, dim=64)
    t, stream = _table_with_rows(cfg)
    for step in (1, 7):                         # 1: all IDs known; 7: a fresh batch, many IDs without a row
        s = stream.step(step)
        ids = torch.from_numpy(s.ids.view(np.int64)).cuda()
        off = torch.from_numpy(s.offsets).cuda()
        want = torch.empty((cfg.n_bags, cfg.dim), device="cuda")
        got = torch.full((cfg.n_bags, cfg.dim), float("nan"), device="cuda")
        mb.mono_lookup_pool(t.handle, ids, ids.numel(), off, cfg.n_bags, want)
        mb.mono_lookup_pool_noalloc(t.handle, ids, ids.numel(), off, cfg.n_bags, got)
        torch.cuda.synchronize()
        assert_vectors_close(got.cpu().numpy(), want.cpu().numpy(), f"no-alloc lookup, batch {step}")
        assert want.abs().sum().item() > 0
    assert t.status()["error_bits"] == 0


def test_noalloc_lookup_refuses_batches_beyond_its_fixed_scratch():
    cfg = wl.scaled(wl.CONFIGS["tiny"], n_examples=64, dim=8)
    t, _ = _table_with_rows(cfg)
    n = mb.MONO_NOALLOC_MAX_IDS + 1
    ids = torch.zeros(n, dtype=torch.int64, device="cuda")
    off = torch.tensor([0, n], dtype=torch.int64, device="cuda")
    out = torch.zeros((1, cfg.dim), device="cuda")
    with pytest.raises(mb.MonoError) as e:
        mb.mono_lookup_pool_noalloc(t.handle, ids, n, off, 1, out)
    assert e.value.code == mb.MONO_ERR_LIMIT
    # exactly at the limit it runs
    mb.mono_lookup_pool_noalloc(t.handle, ids, n - 1, torch.tensor([0, n - 1], dtype=torch.int64, device="cuda"), 1, out)
    torch.cuda.synchronize()
    assert out.abs().sum().item() == 0          # ID 0 has no row


def test_noalloc_lookup_on_a_table_that_never_sized_its_own_scratch():
    """A table filled through mono_import only, created without max_ids: no call has sized the
    table's own scratch yet, and the no-alloc lookup, called first, must not need it."""
    dim, n = 16, 3000
    rng = np.random.default_rng(4)
    ids = wl.splitmix64(np.arange(1, n + 1, dtype=np.uint64))
    w = rng.standard_normal((n, dim)).astype(np.float32)
    t = mb.MonoTable(1 << 12, dim, 1, 0, key_cells=1 << 14)
    t.import_entries(ids, np.ones(n, np.uint32), np.zeros(n, np.int64), np.ones(n, np.uint8), w, np.zeros_like(w))
    assert t.status()["scratch_reallocs"] == 0
    lists = [rng.choice(n, rng.integers(0, 7), replace=False) for _ in range(500)]
    off = np.zeros(len(lists) + 1, np.int64)
    off[1:] = np.cumsum([len(x) for x in lists])
    flat = np.concatenate(lists).astype(np.int64)
    want = np.stack([w[x].astype(np.float64).sum(axis=0) if len(x) else np.zeros(dim) for x in lists]).astype(np.float32)
    d_ids = torch.from_numpy(ids[flat].view(np.int64)).cuda()
    d_off = torch.from_numpy(off).cuda()
    got = torch.full((len(lists), dim), float("nan"), device="cuda")
    mb.mono_lookup_pool_noalloc(t.handle, d_ids, d_ids.numel(), d_off, len(lists), got)
    torch.cuda.synchronize()
    assert_vectors_close(got.cpu().numpy(), want, "no-alloc lookup on an imported table")
    st = t.status()
    assert st["error_bits"] == 0 and st["scratch_reallocs"] == 0
