"""GPU parity: the CUDA library against the CPU oracle on the same seeded inputs,
through the C ABI.  Every test here needs a CUDA device.
"""
import numpy as np
import pytest
import torch

from oracle import mono_oracle as mo
from paper_2209_07663_b200 import binding as mb
from paper_2209_07663_b200 import workload as wl
from tests.parity import assert_audit_ok, assert_state_equal, assert_vectors_close, run_stream

pytestmark = pytest.mark.gpu
f32 = np.float32


def make_pair(cfg, **over):
    kw = dict(lr=cfg.lr, eps=cfg.eps, init_acc=cfg.init_acc, init_scale=cfg.init_scale, seed=cfg.seed)
    kw.update(over)
    gpu = mb.MonoTable(cfg.capacity, cfg.dim, cfg.filter_threshold, cfg.ttl, key_cells=cfg.key_cells, **kw)
    cpu = mo.OracleTable(cfg.capacity, cfg.dim, cfg.filter_threshold, cfg.ttl, **kw)
    return gpu, cpu


def bags(lists):
    ids = np.array([i for b in lists for i in b], dtype=np.uint64)
    off = np.zeros(len(lists) + 1, np.int64)
    off[1:] = np.cumsum([len(b) for b in lists])
    return ids, off


# ---------------------------------------------------------------- configured streams

@pytest.mark.parametrize("prepare", [False, True, "ahead"])
def test_tiny_config_full_stream(prepare):
    cfg = wl.CONFIGS["tiny"]
    gpu, cpu = make_pair(cfg)
    st = run_stream(gpu, cpu, wl.Stream(cfg), cfg.steps, sweep_every=1, check_every=1, prepare=prepare)
    assert st["n_expired_total"] > 0 and st["n_admitted_total"] > 0
    assert st["n_tracked"] > st["n_resident"] > 0


def test_medium_config_prefix():
    cfg = wl.scaled(wl.CONFIGS["medium"], steps=8)
    gpu, cpu = make_pair(cfg)
    run_stream(gpu, cpu, wl.Stream(cfg), cfg.steps, sweep_every=4, check_every=4)


@pytest.mark.parametrize("prepare", [False, True, "ahead"])
def test_medium_config_short_ttl_churn(prepare):
    # the medium shape with a TTL short enough that rows are recycled many times
    cfg = wl.scaled(wl.CONFIGS["medium"], steps=10, ttl=2, n_examples=2048, capacity=1 << 18, key_cells=1 << 20)
    gpu, cpu = make_pair(cfg)
    st = run_stream(gpu, cpu, wl.Stream(cfg), cfg.steps, sweep_every=1, check_every=5, prepare=prepare)
    assert st["n_expired_total"] > 10000


@pytest.mark.parametrize("prepare", [False, True, "ahead"])
def test_drift_config_scaled_down(prepare):
    cfg = wl.scaled(wl.CONFIGS["drift"], n_examples=512, n_slots=10, n_distinct=1 << 18, capacity=1 << 16,
                    key_cells=1 << 18, ttl=6, drift_period=4, steps=16)
    gpu, cpu = make_pair(cfg)
    run_stream(gpu, cpu, wl.Stream(cfg), cfg.steps, sweep_every=2, check_every=4, prepare=prepare)


@pytest.mark.parametrize("prepare", [False, True, "ahead"])
@pytest.mark.parametrize("dim", [4, 8, 12, 16, 32, 48, 64, 128, 200, 256, 512, 1024])
def test_every_dim_variant(dim, prepare):
    # bags of 0 to 40 IDs: longer than the widest lane group, so a bag takes several rounds
    cfg = wl.scaled(wl.CONFIGS["tiny"], dim=dim, n_examples=160, n_slots=5, n_distinct=1 << 12, steps=6,
                    capacity=1 << 12, key_cells=1 << 13, bag_len=("uniform", 0, 40))
    gpu, cpu = make_pair(cfg)
    run_stream(gpu, cpu, wl.Stream(cfg), cfg.steps, sweep_every=2, check_every=3, prepare=prepare)


def test_multi_table_configs_scaled_down():
    for cfg in wl.multi_table_configs(n_examples=256, slots=3):
        cfg = wl.scaled(cfg, capacity=1 << 13, key_cells=1 << 15, n_distinct=1 << 14, steps=5, ttl=3)
        gpu, cpu = make_pair(cfg)
        run_stream(gpu, cpu, wl.Stream(cfg), cfg.steps, sweep_every=1, check_every=5)


@pytest.mark.parametrize("announce", [False, True])
@pytest.mark.parametrize("own_streams", [False, True])
def test_grouped_calls_match_one_oracle_per_table(own_streams, announce):
    """mono_group_prepare_push / _lookup_pool / _apply_grads: the eight tables of the mixed-dim
    configuration (scaled down) and a ninth with rows of 256 columns, one launch per kernel
    for all of them; every table's outputs and state are those of its own oracle.  With the
    tables on the group's stream or each on a stream of its own; with the batches announced
    or not, and once with one table's announcement missing.  Also: a table whose batch is
    empty, a table named twice and a null entry are refused, an empty group is fine."""
    cfgs = [wl.scaled(c, capacity=1 << 13, key_cells=1 << 15, n_distinct=1 << 14, steps=5, ttl=3)
            for c in wl.multi_table_configs(n_examples=256, slots=3)]
    cfgs.append(wl.scaled(cfgs[2], dim=256, seed=cfgs[2].seed + 1, name="wide"))
    streams = [torch.cuda.Stream() if own_streams else torch.cuda.current_stream() for _ in cfgs]
    pairs = []
    for c, st in zip(cfgs, streams):
        kw = dict(lr=c.lr, eps=c.eps, init_acc=c.init_acc, init_scale=c.init_scale, seed=c.seed)
        pairs.append((mb.MonoTable(c.capacity, c.dim, c.filter_threshold, c.ttl, key_cells=c.key_cells,
                                   stream=st.cuda_stream, **kw),
                      mo.OracleTable(c.capacity, c.dim, c.filter_threshold, c.ttl, **kw)))
    gens = [wl.Stream(c) for c in cfgs]
    handles = [g.handle for g, _ in pairs]
    group_stream = torch.cuda.current_stream().cuda_stream
    for t in range(6):
        steps = [g.step(t) for g in gens]
        if t == 3:                                               # table 1 sits this step out
            steps[1] = wl.Step(ids=steps[1].ids[:0], offsets=np.zeros(1, np.int64),
                               grad_pooled=steps[1].grad_pooled[:0], now=t)
        dev = [_dev_batch(s) for s in steps]
        outs = [torch.empty((s.offsets.size - 1, c.dim), dtype=torch.float32, device="cuda") for c, s in zip(cfgs, steps)]
        if announce:
            mb.mono_group_prepare_push(handles, [d[0] for d in dev], [d[1] for d in dev], group_stream)
            if t == 4:                                           # one announcement is replaced by another batch's
                o = _dev_batch(gens[5].step(77))
                mb.mono_prepare_push(handles[5], o[0], o[0].numel(), o[1], cfgs[5].n_bags)
        mb.mono_group_lookup_pool(handles, [d[0] for d in dev], [d[1] for d in dev], outs, group_stream)
        for (gpu, cpu), s, out in zip(pairs, steps, outs):       # `out` is read on the group's stream
            assert_vectors_close(out.cpu().numpy(), cpu.lookup_pool(s.ids, s.offsets), f"step {t}: pooled output")
        mb.mono_group_apply_grads(handles, [d[0] for d in dev], [d[1] for d in dev], [d[2] for d in dev], t, group_stream)
        for (gpu, cpu), s in zip(pairs, steps):
            assert cpu.apply_grads(s.ids, s.offsets, s.grad_pooled, t) == 0
            gpu.expire(t)
            cpu.expire(t)
            assert_state_equal(gpu, cpu, f"step {t}")
    mb.mono_group_lookup_pool([], [], [], [], group_stream)
    d0 = _dev_batch(gens[0].step(9))
    out0 = torch.empty((cfgs[0].n_bags, cfgs[0].dim), dtype=torch.float32, device="cuda")
    with pytest.raises(mb.MonoError):
        mb.mono_group_lookup_pool([handles[0], handles[0]], [d0[0]] * 2, [d0[1]] * 2, [out0] * 2, group_stream)
    with pytest.raises(mb.MonoError):
        mb.mono_group_lookup_pool([handles[0], None], [d0[0]] * 2, [d0[1]] * 2, [out0] * 2, group_stream)
    # the whole step of nine tables is a handful of launches, not nine times the single-table count
    n_launches = mb.mono_timing_read(handles[0], reset=True)["launches_total"]
    for gpu, _ in pairs:
        assert_audit_ok(gpu)
        assert gpu.status()["error_bits"] == 0
    per_step = 3 + 4 + 17                                      # announcement, lookup, push: the most any step can take
    assert n_launches <= 6 * per_step + 6 * 2 + 4              # grouped kernels + table 0's own sweeps (gpu.expire)


# ---------------------------------------------------------------- edge cases

def test_empty_inputs_and_padding():
    gpu = mb.MonoTable(64, 8, 1, 0, init_scale=0.1, seed=3)
    cpu = mo.OracleTable(64, 8, 1, 0, init_scale=0.1, seed=3)
    # no IDs at all, one empty bag
    ids, off = bags([[]])
    assert not gpu.lookup_pool(ids, off).cpu().numpy().any()
    gpu.apply_grads(ids, off, np.ones((1, 8), f32), 0)
    assert gpu.status()["n_tracked"] == 0
    # zero bags
    gpu.apply_grads(np.zeros(0, np.uint64), np.zeros(1, np.int64), np.zeros((0, 8), f32), 0)
    # padding IDs, empty bags in between, an ID repeated inside one bag
    lists = [[5, mb.MONO_RESERVED_ID, 5], [], [mb.MONO_RESERVED_ID], [6, 7, 5], []]
    ids, off = bags(lists)
    grad = np.arange(40, dtype=f32).reshape(5, 8) / 7
    for t in range(3):
        gpu.apply_grads(ids, off, grad, t)
        cpu.apply_grads(ids, off, grad, t)
        assert_vectors_close(gpu.lookup_pool(ids, off).cpu().numpy(), cpu.lookup_pool(ids, off), "padding pooled")
    assert_state_equal(gpu, cpu)
    assert gpu.status()["n_tracked"] == 3 and gpu.status()["sum_ids"] == 15


def test_offsets_that_skip_ids():
    # offsets may start after 0 and end before n_ids: IDs outside every bag are ignored
    gpu = mb.MonoTable(64, 4, 1, 0, init_scale=0.1)
    cpu = mo.OracleTable(64, 4, 1, 0, init_scale=0.1)
    ids = np.array([1, 2, 3, 4, 5, 6], np.uint64)
    off = np.array([1, 3, 5], np.int64)
    grad = np.ones((2, 4), f32)
    gpu.apply_grads(ids, off, grad, 0)
    cpu.apply_grads(ids, off, grad, 0)
    assert_state_equal(gpu, cpu)
    assert gpu.export()["ids"].tolist() == [2, 3, 4, 5]
    assert_vectors_close(gpu.lookup_pool(ids, off).cpu().numpy(), cpu.lookup_pool(ids, off), "pooled")


@pytest.mark.parametrize("prepare", [False, True])
@pytest.mark.parametrize("n_occ", [63, 64, 65, 255, 257, 1000, 4096, 4097, 4200, 70000])
def test_one_hot_id_long_segment(n_occ, prepare):
    # a single ID owning a whole batch: the segment is split into parts and recombined
    dim = 64
    rng = np.random.default_rng(n_occ)
    gpu = mb.MonoTable(64, dim, 3, 0, init_scale=0.05, seed=9)
    cpu = mo.OracleTable(64, dim, 3, 0, init_scale=0.05, seed=9)
    n_bags = max(n_occ // 3, 1)
    lens = np.full(n_bags, 3)
    lens[-1] += n_occ - lens.sum()
    off = np.zeros(n_bags + 1, np.int64)
    off[1:] = np.cumsum(lens)
    ids = np.full(n_occ, 0xABCDEF0123456789, np.uint64)
    ids[::97] = 77          # a second, cooler ID mixed in
    d_ids, d_off = torch.from_numpy(ids.view(np.int64)).cuda(), torch.from_numpy(off).cuda()
    for t in range(2):
        grad = (rng.standard_normal((n_bags, dim)) * 0.01).astype(f32)
        if prepare:
            # announced and pushed without a lookup in between: the push files the bags itself
            mb.mono_prepare_push(gpu.handle, d_ids, n_occ, d_off, n_bags)
            mb.mono_apply_grads(gpu.handle, d_ids, n_occ, d_off, n_bags, torch.from_numpy(grad).cuda(), t)
        else:
            gpu.apply_grads(ids, off, grad, t)
        cpu.apply_grads(ids, off, grad, t)
    assert_state_equal(gpu, cpu)
    assert_vectors_close(gpu.lookup_pool(ids[:7], np.array([0, 7], np.int64)).cpu().numpy(),
                         cpu.lookup_pool(ids[:7], np.array([0, 7], np.int64)), "pooled hot")


def test_forward_equals_torch_embedding_bag():
    rng = np.random.default_rng(5)
    V, d, B = 3000, 32, 5000
    W = rng.standard_normal((V, d)).astype(f32)
    id_of_row = wl.splitmix64(np.arange(V, dtype=np.uint64) + np.uint64(31337))
    gpu = mb.MonoTable(4096, d, 1, 0)
    gpu.import_entries(id_of_row, np.ones(V, np.uint32), np.zeros(V, np.int64), np.ones(V, np.uint8), W,
                       np.zeros((V, d), f32))
    lens = rng.integers(0, 9, B)
    off = np.zeros(B + 1, np.int64)
    off[1:] = np.cumsum(lens)
    rows = rng.integers(0, V, off[-1])
    got = gpu.lookup_pool(id_of_row[rows], off).cpu().numpy()
    ref = torch.nn.functional.embedding_bag(torch.from_numpy(rows), torch.from_numpy(W.astype(np.float64)),
                                            torch.from_numpy(off[:-1]), mode="sum").numpy()
    assert_vectors_close(got, ref.astype(f32), "embedding_bag")
    assert_audit_ok(gpu)


def test_host_buffer_calls_match_device_calls():
    """mono_lookup_pool_host / mono_apply_grads_host: pinned host buffers in, pooled rows back out, no
    synchronisation inside the calls.  Steps are issued back to back (the result of each is read after
    a fence); one push is given a batch other than the one its lookup staged, one follows a sweep."""
    cfg = wl.scaled(wl.CONFIGS["tiny"], n_examples=256, steps=6)
    a, cpu = make_pair(cfg)
    stream = wl.Stream(cfg)
    host, outs = [], []
    for t in range(cfg.steps):
        s = stream.step(t)
        host.append((torch.from_numpy(s.ids.view(np.int64)).pin_memory(), torch.from_numpy(s.offsets).pin_memory(),
                     torch.from_numpy(s.grad_pooled).pin_memory(), s))
        outs.append(torch.full((cfg.n_bags, cfg.dim), float("nan"), dtype=torch.float32).pin_memory())
    for t, (ids, off, grad, s) in enumerate(host):
        mb.mono_lookup_pool_host(a.handle, ids, ids.numel(), off, cfg.n_bags, outs[t])
        want = cpu.lookup_pool(s.ids, s.offsets)
        if t == 4:       # a sweep between the lookup and the push: the push groups and looks up its batch again
            a.expire(t - 1); cpu.expire(t - 1)
        if t == 3:       # the push of another batch than the one just looked up: it brings its own IDs in
            o_ids, o_off, o_grad, o = host[5]
            mb.mono_apply_grads_host(a.handle, o_ids, o_ids.numel(), o_off, cfg.n_bags, o_grad, t)
            cpu.apply_grads(o.ids, o.offsets, o.grad_pooled, t)
        else:
            mb.mono_apply_grads_host(a.handle, ids, ids.numel(), off, cfg.n_bags, grad, t)
            cpu.apply_grads(s.ids, s.offsets, s.grad_pooled, t)
        if t % 2:        # every other step the host reads the result before it goes on
            mb.mono_fence(a.handle)
            torch.cuda.synchronize()
            assert_vectors_close(outs[t].numpy(), want, f"host pooled {t}")
        host[t] = (ids, off, grad, want)
    mb.mono_fence(a.handle)
    torch.cuda.synchronize()
    for t in range(cfg.steps):
        assert_vectors_close(outs[t].numpy(), host[t][3], f"host pooled {t}, read at the end")
    assert_state_equal(a, cpu)
    assert_audit_ok(a)
    assert a.status()["error_bits"] == 0


# ---------------------------------------------------------------- expiry, recycling, import/export

def test_expiry_sets_and_row_recycling():
    cfg = wl.scaled(wl.CONFIGS["tiny"], n_examples=512, ttl=2, capacity=1 << 14, key_cells=1 << 16, steps=14,
                    filter_threshold=1, n_distinct=1 << 18)
    gpu, cpu = make_pair(cfg)
    st = run_stream(gpu, cpu, wl.Stream(cfg), cfg.steps, sweep_every=1, check_every=1)
    # more rows were handed out than exist: expired rows were reused, never shared
    assert st["n_admitted_total"] > cfg.capacity
    a = assert_audit_ok(gpu)
    assert a["resident_cells"] + a["free_rows"] == cfg.capacity


def _dev_batch(s):
    return (torch.from_numpy(s.ids.view(np.int64)).cuda(), torch.from_numpy(s.offsets).cuda(),
            torch.from_numpy(s.grad_pooled).cuda())


def test_prepared_push_gives_the_same_table_as_the_oracle():
    """mono_prepare_push before the lookup of the same batch: the grouping runs beside the
    lookup, and lookup outputs and table state stay those of the oracle, step by step.  Also
    the ways a preparation is dropped: a different batch is pushed, a second preparation
    replaces the first, the scratch grows in between, the prepared batch is never pushed."""
    cfg = wl.scaled(wl.CONFIGS["medium"], n_examples=1024, steps=12, ttl=3)
    gpu, cpu = make_pair(cfg)
    stream = wl.Stream(cfg)
    out = torch.empty((cfg.n_bags, cfg.dim), dtype=torch.float32, device="cuda")
    h = gpu.handle
    for t in range(cfg.steps):
        s = stream.step(t)
        ids, off, grad = _dev_batch(s)
        other = _dev_batch(stream.step(t + 100))
        if t % 4 == 1:                                   # prepared for another batch, then replaced
            mb.mono_prepare_push(h, other[0], other[0].numel(), other[1], cfg.n_bags)
        if t % 4 != 3:
            mb.mono_prepare_push(h, ids, ids.numel(), off, cfg.n_bags)
        else:                                            # the wrong batch stays prepared: the push must drop it
            mb.mono_prepare_push(h, other[0], other[0].numel(), other[1], cfg.n_bags)
        mb.mono_lookup_pool(h, ids, ids.numel(), off, cfg.n_bags, out)
        assert_vectors_close(out.cpu().numpy(), cpu.lookup_pool(s.ids, s.offsets), f"step {t}: pooled output")
        if t == 5:                                       # the scratch is reallocated under a prepared grouping
            mb.mono_reserve(h, 4 * ids.numel(), 4 * cfg.n_bags)
        mb.mono_apply_grads(h, ids, ids.numel(), off, cfg.n_bags, grad, t)
        assert cpu.apply_grads(s.ids, s.offsets, s.grad_pooled, t) == 0
        if t % 2:
            gpu.expire(t)
            cpu.expire(t)
        assert_state_equal(gpu, cpu, f"step {t}")
    s = stream.step(50)
    ids, off, grad = _dev_batch(s)
    mb.mono_prepare_push(h, ids, ids.numel(), off, cfg.n_bags)       # never pushed
    mb.mono_prepare_push(h, ids, 0, off[:1], 0)                      # an empty batch prepares nothing
    st = gpu.status()
    assert st["error_bits"] == 0 and st["sum_ids"] == cpu_sum_ids(stream, cfg.steps)
    assert_state_equal(gpu, cpu, "after an abandoned preparation")
    assert_audit_ok(gpu)
    gpu.apply_grads(s.ids, s.offsets, s.grad_pooled, cfg.steps)      # and the table still works
    cpu.apply_grads(s.ids, s.offsets, s.grad_pooled, cfg.steps)
    assert_state_equal(gpu, cpu, "push after an abandoned preparation")


def cpu_sum_ids(stream, steps):
    return sum(int((stream.step(t).ids != np.uint64(wl.RESERVED_ID)).sum()) for t in range(steps))


def test_grouping_ahead_in_every_order_gives_the_same_table_as_the_oracle():
    """mono_group_ahead beside the calls of other batches: taken over by the mono_prepare_push of its
    batch; left alone by a mono_prepare_push or an unannounced push of another batch and taken over
    later; replaced by a second mono_group_ahead; lost when the scratch grows; never used at all."""
    cfg = wl.scaled(wl.CONFIGS["tiny"], n_examples=512, steps=14)
    gpu, cpu = make_pair(cfg)
    h = gpu.handle
    stream = wl.Stream(cfg)
    batches = [stream.step(t) for t in range(cfg.steps + 1)]
    dev = [(torch.from_numpy(s.ids.view(np.int64)).cuda(), torch.from_numpy(s.offsets).cuda(),
            torch.from_numpy(s.grad_pooled).cuda()) for s in batches]
    ahead = lambda k: mb.mono_group_ahead(h, dev[k][0], dev[k][0].numel(), dev[k][1], cfg.n_bags)
    out = torch.empty((cfg.n_bags, cfg.dim), dtype=torch.float32, device="cuda")
    ahead(0)
    for t in range(cfg.steps):
        s, (ids, off, grad) = batches[t], dev[t]
        kind = t % 7
        if kind == 0:                                     # the plain pipeline
            mb.mono_prepare_push(h, ids, ids.numel(), off, cfg.n_bags)
            ahead(t + 1)
        elif kind == 1:                                   # grouped ahead twice: the first is forgotten
            mb.mono_prepare_push(h, ids, ids.numel(), off, cfg.n_bags)
            ahead(t)
            ahead(t + 1)
        elif kind == 2:                                   # another batch announced first: the grouping made ahead waits
            mb.mono_prepare_push(h, dev[t + 1][0], dev[t + 1][0].numel(), dev[t + 1][1], cfg.n_bags)
            mb.mono_prepare_push(h, ids, ids.numel(), off, cfg.n_bags)
            ahead(t + 1)
        elif kind == 3:                                   # pushed without an announcement; batch t's grouping is never used
            ahead(t + 1)
        elif kind == 4:                                   # the scratch grows under a grouping made ahead
            mb.mono_reserve(h, gpu.status()["sum_ids"] // (t + 1) * (3 + t), cfg.n_bags * 2)
            mb.mono_prepare_push(h, ids, ids.numel(), off, cfg.n_bags)
            ahead(t + 1)
        elif kind == 5:                                   # a sweep and an empty grouping in between
            gpu.expire(t - 1); cpu.expire(t - 1)
            mb.mono_prepare_push(h, ids, ids.numel(), off, cfg.n_bags)
            mb.mono_group_ahead(h, ids, 0, off[:1], 0)
        else:                                             # nothing grouped ahead for this one
            mb.mono_prepare_push(h, ids, ids.numel(), off, cfg.n_bags)
            ahead(t + 1)
        mb.mono_lookup_pool(h, ids, ids.numel(), off, cfg.n_bags, out)
        assert_vectors_close(out.cpu().numpy(), cpu.lookup_pool(s.ids, s.offsets), f"step {t}: pooled output")
        mb.mono_apply_grads(h, ids, ids.numel(), off, cfg.n_bags, grad, t)
        assert cpu.apply_grads(s.ids, s.offsets, s.grad_pooled, t) == 0
        assert_state_equal(gpu, cpu, f"step {t}")
        assert_audit_ok(gpu, f"step {t}")
    assert gpu.status()["error_bits"] == 0


def test_prepared_push_with_malformed_offsets_is_flagged():
    gpu = mb.MonoTable(1 << 10, 8, 1, 0)
    ids = torch.arange(1, 9, dtype=torch.int64, device="cuda")
    off = torch.tensor([0, 3, 2, 8], dtype=torch.int64, device="cuda")
    grad = torch.ones((3, 8), dtype=torch.float32, device="cuda")
    mb.mono_prepare_push(gpu.handle, ids, 8, off, 3)
    mb.mono_apply_grads(gpu.handle, ids, 8, off, 3, grad, 0)
    assert gpu.status()["error_bits"] & mb.MONO_DEV_BAD_OFFSETS
    assert_audit_ok(gpu)


@pytest.mark.parametrize("n_slices", [1, 3, 7, 64])
def test_sliced_sweep_equals_one_full_sweep(n_slices):
    cfg = wl.scaled(wl.CONFIGS["tiny"], n_examples=512, steps=8, ttl=2, key_cells=1 << 16)
    gpu, cpu = make_pair(cfg)
    stream = wl.Stream(cfg)
    for t in range(cfg.steps):
        s = stream.step(t)
        gpu.apply_grads(s.ids, s.offsets, s.grad_pooled, t)
        cpu.apply_grads(s.ids, s.offsets, s.grad_pooled, t)
        for k in range(n_slices):
            mb.mono_expire_slice(gpu.handle, t, k, n_slices)
        cpu.expire(t)
        assert_state_equal(gpu, cpu, f"step {t}")
    assert gpu.status()["n_expired_total"] > 0
    assert_audit_ok(gpu)
    with pytest.raises(mb.MonoError):
        mb.mono_expire_slice(gpu.handle, cfg.steps, 3, 3)


def test_interleaved_sweep_slices_evict_neither_early_nor_late():
    """One slice per training step, with the time advancing: which step visits an ID's cell
    depends on where the ID hashes, so the oracle cannot be swept the same way.  What is unique:
    an ID whose occurrences are never more than ttl + 1 steps apart (and which is recent at the
    end) cannot have been evicted, so its whole state equals that of an oracle that never
    sweeps; an ID not seen for ttl + n_slices steps or more has met a visit of its cell that
    evicts it, so it must be gone."""
    n_slices, ttl = 5, 3
    cfg = wl.scaled(wl.CONFIGS["tiny"], n_examples=512, steps=40, ttl=ttl, key_cells=1 << 16, capacity=1 << 15)
    gpu = mb.MonoTable(cfg.capacity, cfg.dim, cfg.filter_threshold, ttl, key_cells=cfg.key_cells, lr=cfg.lr,
                       eps=cfg.eps, init_acc=cfg.init_acc, init_scale=cfg.init_scale, seed=cfg.seed)
    cpu = mo.OracleTable(cfg.capacity, cfg.dim, cfg.filter_threshold, 0, lr=cfg.lr, eps=cfg.eps,
                         init_acc=cfg.init_acc, init_scale=cfg.init_scale, seed=cfg.seed)
    stream = wl.Stream(cfg)
    seen_at = {}
    for t in range(cfg.steps):
        s = stream.step(t)
        gpu.apply_grads(s.ids, s.offsets, s.grad_pooled, t)
        assert cpu.apply_grads(s.ids, s.offsets, s.grad_pooled, t) == 0
        mb.mono_expire_slice(gpu.handle, t, t % n_slices, n_slices)
        for i in np.unique(s.ids[s.ids != np.uint64(wl.RESERVED_ID)]).tolist():
            seen_at.setdefault(i, []).append(t)
    end = cfg.steps - 1
    g, o = gpu.export(), cpu.export()
    g_at = {int(i): k for k, i in enumerate(g["ids"].tolist())}
    o_at = {int(i): k for k, i in enumerate(o["ids"].tolist())}
    n_safe = n_gone = 0
    for i, times in seen_at.items():
        gaps = np.diff(times)
        if end - times[-1] >= ttl + n_slices:
            assert i not in g_at, f"ID {i} last seen at {times[-1]} is still tracked at {end}"
            n_gone += 1
        elif end - times[-1] <= ttl and (gaps.size == 0 or gaps.max() <= ttl + 1):
            assert i in g_at, f"ID {i} was evicted although it was never inactive for longer than ttl"
            a, b = g_at[i], o_at[i]
            assert g["count"][a] == o["count"][b] and g["last_seen"][a] == o["last_seen"][b]
            assert g["resident"][a] == o["resident"][b]
            if g["resident"][a]:
                assert_vectors_close(g["w"][a][None], o["w"][b][None], f"row of ID {i}")
                assert_vectors_close(g["acc"][a][None], o["acc"][b][None], f"accumulator of ID {i}")
            n_safe += 1
    assert n_safe > 100 and n_gone > 100, (n_safe, n_gone)
    for i in g_at:                                     # nothing tracked that was never fed
        assert i in seen_at
    assert_audit_ok(gpu)


def test_unswept_entries_survive_and_refresh():
    gpu = mb.MonoTable(64, 4, 1, 3, init_scale=0.1)
    cpu = mo.OracleTable(64, 4, 1, 3, init_scale=0.1)
    g = np.ones((1, 4), f32)
    for now, lists in [(0, [[1, 2]]), (10, [[1]]), (11, [[3]])]:
        ids, off = bags(lists)
        gpu.apply_grads(ids, off, g, now)
        cpu.apply_grads(ids, off, g, now)
    assert_state_equal(gpu, cpu, "before sweep")       # 2 is stale but still there
    gpu.expire(13); cpu.expire(13)
    assert_state_equal(gpu, cpu, "after sweep(13)")    # 2 gone; 1 (10) and 3 (11) stay
    gpu.expire(14); cpu.expire(14)
    assert_state_equal(gpu, cpu, "after sweep(14)")    # 14-10 > 3: 1 gone
    assert gpu.export()["ids"].tolist() == [3]


def test_export_import_roundtrip_into_a_differently_seeded_table():
    cfg = wl.scaled(wl.CONFIGS["tiny"], n_examples=512, steps=6)
    gpu, cpu = make_pair(cfg)
    run_stream(gpu, cpu, wl.Stream(cfg), cfg.steps, sweep_every=0, check_every=0, check_forward=False)
    snap = gpu.export()
    other = mb.MonoTable(cfg.capacity, cfg.dim, cfg.filter_threshold, cfg.ttl, key_cells=cfg.key_cells * 2,
                         lr=cfg.lr, eps=cfg.eps, init_scale=cfg.init_scale, seed=cfg.seed + 1)
    other.import_entries(snap["ids"], snap["count"], snap["last_seen"], snap["resident"], snap["w"], snap["acc"])
    assert_state_equal(other, cpu, "restored")
    assert_audit_ok(other)
    # importing the same IDs again changes nothing and is reported
    other.import_entries(snap["ids"][:10], snap["count"][:10], snap["last_seen"][:10], snap["resident"][:10],
                         snap["w"][:10], snap["acc"][:10])
    assert other.status()["error_bits"] & mb.MONO_DEV_IMPORT_DUP
    assert_state_equal(other, cpu, "after duplicate import")


@pytest.mark.parametrize("depth,width", [(1, 1), (2, 1 << 10), (3, 1 << 14), (4, 1 << 22)])
def test_probabilistic_filter_matches_the_sketch_oracle(depth, width):
    cfg = wl.scaled(wl.CONFIGS["tiny"], n_examples=512, steps=14, ttl=4, filter_threshold=3)
    kw = dict(sketch_depth=depth, sketch_width=width)
    gpu, cpu = make_pair(cfg, **kw)
    stream = wl.Stream(cfg)
    seen = []
    for t in range(cfg.steps):
        s = stream.step(t)
        seen.append(np.unique(s.ids))
        got = gpu.lookup_pool(s.ids, s.offsets).cpu().numpy()
        assert_vectors_close(got, cpu.lookup_pool(s.ids, s.offsets), f"step {t}: pooled output")
        gpu.apply_grads(s.ids, s.offsets, s.grad_pooled, t)
        assert cpu.apply_grads(s.ids, s.offsets, s.grad_pooled, t) == 0
        if t % 3 == 2:                                    # clears the sketch every other sweep (ttl 4)
            if depth == 2:                                # once in slices: slice 0 is the one that clears
                for k in range(5):
                    mb.mono_expire_slice(gpu.handle, t, k, 5)
            else:
                gpu.expire(t)
            cpu.expire(t)
        assert_state_equal(gpu, cpu, f"step {t}")         # only IDs with a row have entries
        ids = np.unique(np.concatenate(seen[-3:]))
        g, o = gpu.probe(ids, rows=False), cpu.probe(ids, rows=False)
        assert (g["count"] == o["count"]).all() and (g["resident"] == o["resident"]).all(), f"estimates at step {t}"
    st = gpu.status()
    assert st["error_bits"] == 0 and st["n_tracked"] == st["n_resident"] > 0
    assert_audit_ok(gpu)


def test_rehash_moves_keys_but_changes_no_state():
    cfg = wl.scaled(wl.CONFIGS["tiny"], n_examples=512, steps=12)
    gpu, cpu = make_pair(cfg)
    stream = wl.Stream(cfg)
    for t in range(cfg.steps):
        s = stream.step(t)
        gpu.apply_grads(s.ids, s.offsets, s.grad_pooled, t)
        cpu.apply_grads(s.ids, s.offsets, s.grad_pooled, t)
        if t == 3:
            gpu.rehash(new_seed=12345)                       # same size, new hash functions
        if t == 6:
            gpu.rehash(cfg.key_cells * 4, new_seed=7)        # grow
        if t == 9:
            gpu.rehash(cfg.key_cells // 2, new_seed=99)      # shrink (still fits)
        if t in (3, 6, 9):
            assert_state_equal(gpu, cpu, f"after rehash at step {t}")
            a = assert_audit_ok(gpu)
            assert gpu.status()["key_cells"] in (cfg.key_cells, cfg.key_cells * 4, cfg.key_cells // 2)
            assert_vectors_close(gpu.lookup_pool(s.ids, s.offsets).cpu().numpy(), cpu.lookup_pool(s.ids, s.offsets),
                                 "pooled after rehash")
        gpu.expire(t); cpu.expire(t)
    assert_state_equal(gpu, cpu)
    assert gpu.status()["error_bits"] == 0


def test_rehash_into_a_larger_store_empties_the_stash():
    # a 64-cell store pushed to its limit: entries end up in the stash; a larger store takes them all back
    gpu = mb.MonoTable(16, 4, 100, 0, key_cells=64, seed=5)
    cpu = mo.OracleTable(16, 4, 100, 0, seed=5)
    ids = wl.splitmix64(np.arange(150, dtype=np.uint64))
    off = np.arange(0, 151, dtype=np.int64)
    gpu.apply_grads(ids, off, np.zeros((150, 4), f32), 0)
    cpu.apply_grads(ids, off, np.zeros((150, 4), f32), 0)
    st = gpu.status()
    assert st["stash_used"] > 0 and st["n_keys_dropped"] == 0 and st["n_tracked"] == 150
    gpu.rehash(1024, new_seed=1)
    st = gpu.status()
    assert st["stash_used"] == 0 and st["n_tracked"] == 150 and st["key_cells"] == 1024
    assert_state_equal(gpu, cpu)
    assert_audit_ok(gpu)
    with pytest.raises(mb.MonoError):
        gpu.rehash(1000)                                     # not a power of two


def test_touched_key_export_matches_the_oracle():
    cfg = wl.scaled(wl.CONFIGS["tiny"], n_examples=512, steps=12, ttl=3)
    gpu, cpu = make_pair(cfg)
    stream = wl.Stream(cfg)
    for t in range(cfg.steps):
        s = stream.step(t)
        gpu.apply_grads(s.ids, s.offsets, s.grad_pooled, t)
        cpu.apply_grads(s.ids, s.offsets, s.grad_pooled, t)
        if t % 2 == 1:
            gpu.expire(t); cpu.expire(t)
        if t % 3 == 2:
            g, o = gpu.export_touched(), cpu.export_touched()
            assert g["found"] == o["ids"].size > 0 and (g["ids"] == o["ids"]).all()
            assert_vectors_close(g["w"], o["w"], f"touched rows at step {t}")
            assert gpu.export_touched()["found"] == 0               # the set is empty afterwards
    assert_state_equal(gpu, cpu)
    assert_audit_ok(gpu)
    # a buffer that is too small exports what fits and keeps the rest for the next call
    s = stream.step(cfg.steps)
    gpu.apply_grads(s.ids, s.offsets, s.grad_pooled, cfg.steps)
    cpu.apply_grads(s.ids, s.offsets, s.grad_pooled, cfg.steps)
    want = cpu.export_touched()
    first = gpu.export_touched(max_n=100)
    assert first["found"] == want["ids"].size and first["ids"].size == 100
    rest = gpu.export_touched()
    assert rest["found"] == want["ids"].size - 100
    both = np.sort(np.concatenate([first["ids"], rest["ids"]]))
    assert (both == want["ids"]).all()


# ---------------------------------------------------------------- cuckoo structure under load

def test_announced_batch_survives_reads_and_is_dropped_by_anything_that_changes_the_table():
    """Between mono_prepare_push and the push of that batch: a second lookup of the batch, a lookup
    of another batch and the read-only fixtures leave the announcement in force; a sweep, an import,
    a rehash or an incremental export make the push look everything up again.  Either way the
    table ends up as the oracle's."""
    cfg = wl.scaled(wl.CONFIGS["tiny"], n_examples=512, steps=14, ttl=2, key_cells=1 << 16)
    gpu, cpu = make_pair(cfg)
    stream = wl.Stream(cfg)
    h = gpu.handle
    out = torch.empty((cfg.n_bags, cfg.dim), dtype=torch.float32, device="cuda")
    for t in range(cfg.steps):
        s = stream.step(t)
        ids, off, grad = _dev_batch(s)
        mb.mono_prepare_push(h, ids, ids.numel(), off, cfg.n_bags)
        kind = t % 7
        if kind == 0:                       # two lookups of the announced batch
            mb.mono_lookup_pool(h, ids, ids.numel(), off, cfg.n_bags, out)
            mb.mono_lookup_pool(h, ids, ids.numel(), off, cfg.n_bags, out)
        elif kind == 1:                     # a lookup of another batch in between, then the announced one
            o = _dev_batch(stream.step(t + 50))
            got = gpu.lookup_pool(o[0], o[1]).cpu().numpy()
            assert_vectors_close(got, cpu.lookup_pool(stream.step(t + 50).ids, stream.step(t + 50).offsets), "other batch")
            mb.mono_lookup_pool(h, ids, ids.numel(), off, cfg.n_bags, out)
        elif kind == 2:                     # read-only fixtures
            gpu.status(); gpu.probe(s.ids[:50]); gpu.audit()
            mb.mono_lookup_pool(h, ids, ids.numel(), off, cfg.n_bags, out)
        elif kind == 3:                     # a sweep between the announcement and the lookup
            gpu.expire(t - 1); cpu.expire(t - 1)
            mb.mono_lookup_pool(h, ids, ids.numel(), off, cfg.n_bags, out)
        elif kind == 4:                     # ... and between the lookup and the push
            mb.mono_lookup_pool(h, ids, ids.numel(), off, cfg.n_bags, out)
            want = cpu.lookup_pool(s.ids, s.offsets)
            assert_vectors_close(out.cpu().numpy(), want, f"step {t}: pooled before the sweep")
            for k in range(3):
                mb.mono_expire_slice(h, t - 1, k, 3)
            cpu.expire(t - 1)
        elif kind == 5:                     # a rehash moves every key
            gpu.rehash(0, 1000 + t)
            mb.mono_lookup_pool(h, ids, ids.numel(), off, cfg.n_bags, out)
        else:                               # an incremental export rewrites metadata
            g, o = gpu.export_touched(), cpu.export_touched()
            assert (g["ids"] == o["ids"]).all()
            mb.mono_lookup_pool(h, ids, ids.numel(), off, cfg.n_bags, out)
        if kind != 4:
            assert_vectors_close(out.cpu().numpy(), cpu.lookup_pool(s.ids, s.offsets), f"step {t}: pooled output")
        mb.mono_apply_grads(h, ids, ids.numel(), off, cfg.n_bags, grad, t)
        assert cpu.apply_grads(s.ids, s.offsets, s.grad_pooled, t) == 0
        assert_state_equal(gpu, cpu, f"step {t}")
        assert_audit_ok(gpu, f"step {t}")
    st = gpu.status()
    assert st["error_bits"] == 0 and st["n_expired_total"] > 0


def test_snapshot_restore_returns_to_the_saved_state():
    cfg = wl.scaled(wl.CONFIGS["tiny"], n_examples=512, steps=9, ttl=3, key_cells=1 << 16)
    gpu, cpu = make_pair(cfg)
    stream = wl.Stream(cfg)
    with pytest.raises(mb.MonoError):
        mb.mono_snapshot_restore(gpu.handle)              # nothing saved yet
    run_stream(gpu, cpu, stream, 4, sweep_every=2, check_every=4)
    mb.mono_snapshot_save(gpu.handle)
    saved = gpu.export()
    for rep in range(2):                                  # the same five steps twice, from the same state
        twin = mo.OracleTable(cfg.capacity, cfg.dim, cfg.filter_threshold, cfg.ttl, lr=cfg.lr, eps=cfg.eps,
                              init_acc=cfg.init_acc, init_scale=cfg.init_scale, seed=cfg.seed)
        assert twin.import_entries(saved["ids"], saved["count"], saved["last_seen"], saved["resident"],
                                   saved["w"], saved["acc"]) == 0
        for t in range(4, 9):
            s = stream.step(t)
            ids, off, grad = _dev_batch(s)
            mb.mono_prepare_push(gpu.handle, ids, ids.numel(), off, cfg.n_bags)
            gpu_out = torch.empty((cfg.n_bags, cfg.dim), device="cuda")
            mb.mono_lookup_pool(gpu.handle, ids, ids.numel(), off, cfg.n_bags, gpu_out)
            assert_vectors_close(gpu_out.cpu().numpy(), twin.lookup_pool(s.ids, s.offsets), f"rep {rep} step {t}")
            mb.mono_apply_grads(gpu.handle, ids, ids.numel(), off, cfg.n_bags, grad, t)
            twin.apply_grads(s.ids, s.offsets, s.grad_pooled, t)
            gpu.expire(t); twin.expire(t)
        assert_state_equal(gpu, twin, f"rep {rep}")
        assert_audit_ok(gpu)
        mb.mono_snapshot_restore(gpu.handle)              # time goes back with the state
        g = gpu.export()
        assert (g["ids"] == saved["ids"]).all() and (g["last_seen"] == saved["last_seen"]).all()
        assert np.array_equal(g["w"], saved["w"]) and np.array_equal(g["acc"], saved["acc"])
    mb.mono_snapshot_drop(gpu.handle)
    with pytest.raises(mb.MonoError):
        mb.mono_snapshot_restore(gpu.handle)


def test_growing_scratch_inside_a_hot_call_is_counted():
    gpu = mb.MonoTable(1 << 10, 8, 1, 0, max_ids=2048, max_bags=2048)
    ids = np.arange(1, 5001, dtype=np.uint64)
    off = np.arange(0, 5001, dtype=np.int64)
    assert gpu.status()["scratch_reallocs"] == 0
    gpu.lookup_pool(ids[:2000], off[:2001])
    assert gpu.status()["scratch_reallocs"] == 0
    gpu.lookup_pool(ids, off)                             # 5000 IDs: larger than the scratch
    assert gpu.status()["scratch_reallocs"] == 1
    gpu.apply_grads(ids, off, np.zeros((5000, 8), f32), 0)
    assert gpu.status()["scratch_reallocs"] == 1


@pytest.mark.parametrize("load", [0.5, 0.8, 0.9])
@pytest.mark.parametrize("kind", ["random", "sequential", "high_bits", "stride_4096"])
def test_cuckoo_membership_at_load(load, kind):
    cells = 1 << 16
    n = int(cells * load)
    if kind == "random":
        ids = wl.splitmix64(np.arange(n, dtype=np.uint64) + np.uint64(12345))
    elif kind == "sequential":
        ids = np.arange(1, n + 1, dtype=np.uint64)
    elif kind == "high_bits":
        ids = np.arange(1, n + 1, dtype=np.uint64) << np.uint64(40)
    else:
        ids = np.arange(1, n + 1, dtype=np.uint64) * np.uint64(4096)
    gpu = mb.MonoTable(1024, 4, 3, 0, key_cells=cells, seed=17)
    half = n // 2
    for part in (ids[:half], ids[half:]):          # second call inserts into an already loaded table
        gpu.import_entries(part, np.ones(part.size, np.uint32), np.zeros(part.size, np.int64),
                           np.zeros(part.size, np.uint8))
    st = gpu.status()
    assert st["error_bits"] == 0 and st["n_tracked"] == n, st
    a = assert_audit_ok(gpu)
    assert a["occupied_cells"] == n
    absent = wl.splitmix64(np.arange(5000, dtype=np.uint64) + np.uint64(999_999_999))
    assert gpu.probe(ids, rows=False)["count"].min() == 1
    assert gpu.probe(absent, rows=False)["count"].max() == 0
    assert set(gpu.export(rows=False)["ids"].tolist()) == set(ids.tolist())


def test_apply_grads_inserts_at_high_load():
    # the batch path (not import) pushing a small key store to ~0.9 load in a few calls
    cells = 1 << 14
    gpu = mb.MonoTable(256, 4, 1000, 0, key_cells=cells, seed=2)
    cpu = mo.OracleTable(256, 4, 1000, 0, seed=2)
    per_call = int(cells * 0.09)
    for t in range(10):
        ids = wl.splitmix64(np.arange(t * per_call, (t + 1) * per_call, dtype=np.uint64))
        off = np.arange(0, per_call + 1, 2, dtype=np.int64)
        grad = np.zeros((off.size - 1, 4), f32)
        gpu.apply_grads(ids, off, grad, t)
        cpu.apply_grads(ids, off, grad, t)
    st = gpu.status()
    assert st["error_bits"] == 0 and st["n_tracked"] == 10 * (per_call // 2 * 2)
    assert_state_equal(gpu, cpu)
    assert_audit_ok(gpu)
    assert st["n_evictions_total"] > 0          # the displacement path really ran


def test_sweep_finds_old_entries_that_displacements_moved():
    """A key store kept near load 0.85 by steady churn: new IDs displace entries of every age into
    buckets whose other entries are younger, and the sweep, which opens only the buckets its
    per-bucket record of the oldest stamp points at, has to remove exactly what a sweep over
    every cell removes -- the oracle's set -- at every sweep, whole or in slices."""
    cells, ttl = 1 << 14, 9
    gpu = mb.MonoTable(256, 4, 1000, ttl, key_cells=cells, seed=5)
    cpu = mo.OracleTable(256, 4, 1000, ttl, seed=5)
    per_call = int(cells * 0.075) // 2 * 2               # eleven calls' worth of IDs stay alive (a tenth renewed): load 0.85
    rng = np.random.default_rng(3)
    evictions = 0
    for t in range(40):
        fresh = wl.splitmix64(np.arange(t * per_call, (t + 1) * per_call, dtype=np.uint64))
        # a tenth of the IDs of the last ten calls come back, which renews their stamps
        back = wl.splitmix64(rng.integers(max(0, t - 10) * per_call, max(1, t * per_call), per_call // 10 * 2).astype(np.uint64))
        ids = np.concatenate([fresh, back])
        off = np.arange(0, ids.size + 1, 2, dtype=np.int64)
        grad = np.zeros((off.size - 1, 4), f32)
        gpu.apply_grads(ids, off, grad, t)
        assert cpu.apply_grads(ids, off, grad, t) == 0
        if t % 3 == 0:
            gpu.expire(t)
        else:
            for k in range(7):
                mb.mono_expire_slice(gpu.handle, t, k, 7)
        cpu.expire(t)
        st = gpu.status()
        assert st["error_bits"] == 0 and st["n_keys_dropped"] == 0, f"step {t}: {st}"
        assert_state_equal(gpu, cpu, f"step {t}")
        a = assert_audit_ok(gpu, f"step {t}")
        assert a["behind_records"] == 0
    st = gpu.status()
    assert st["error_bits"] == 0 and st["n_keys_dropped"] == 0
    assert st["n_tracked"] > 0.8 * cells and st["n_expired_total"] > 2 * cells and st["n_evictions_total"] > 1000, st


def test_sweep_finds_imported_entries_older_than_their_buckets():
    """Entries imported with an old last_seen land in buckets whose record was set by recent ones."""
    ttl = 5
    gpu = mb.MonoTable(64, 4, 1000, ttl, key_cells=1 << 9, seed=1)
    cpu = mo.OracleTable(64, 4, 1000, ttl, seed=1)
    recent = wl.splitmix64(np.arange(0, 150, dtype=np.uint64))
    off = np.arange(0, recent.size + 1, 2, dtype=np.int64)
    grad = np.zeros((off.size - 1, 4), f32)
    gpu.apply_grads(recent, off, grad, 100)
    cpu.apply_grads(recent, off, grad, 100)
    gpu.expire(100); cpu.expire(100)                     # every occupied bucket's record is exact: 100
    old = wl.splitmix64(np.arange(1000, 1060, dtype=np.uint64))
    seen = np.arange(60, dtype=np.int64) + 60             # 60 .. 119: some stale at 103, some not
    for side in (gpu, cpu):
        side.import_entries(old, np.ones(60, np.uint32), seen, np.zeros(60, np.uint8), None, None)
    assert_audit_ok(gpu)
    gpu.expire(103); cpu.expire(103)
    assert_state_equal(gpu, cpu, "after the sweep")
    left = set(gpu.export(rows=False)["ids"].tolist())
    assert left == set(recent.tolist()) | set(old[seen >= 98].tolist())
    assert_audit_ok(gpu)


# ---------------------------------------------------------------- overflow conditions (flagged, never fatal)

def test_rows_full_is_flagged_and_table_stays_consistent():
    gpu = mb.MonoTable(16, 4, 1, 0, key_cells=1 << 10)
    ids = np.arange(1, 41, dtype=np.uint64)
    off = np.arange(0, 41, dtype=np.int64)
    gpu.apply_grads(ids, off, np.ones((40, 4), f32), 0)
    st = gpu.status()
    assert st["error_bits"] & mb.MONO_DEV_ROWS_FULL
    assert st["n_resident"] == 16 and st["n_tracked"] == 40 and st["n_rows_refused"] == 24
    assert_audit_ok(gpu)
    pr = gpu.probe(ids)
    assert pr["resident"].sum() == 16 and (pr["count"] == 1).all()
    # IDs without a row pool as zero, the others as their row
    pooled = gpu.lookup_pool(ids, off).cpu().numpy()
    assert ((np.abs(pooled).max(axis=1) > 0) == (pr["resident"] == 1)).all()


def test_key_store_full_is_flagged_without_duplicates():
    gpu = mb.MonoTable(16, 4, 100, 0, key_cells=64)        # 64 cells + the stash
    ids = wl.splitmix64(np.arange(2000, dtype=np.uint64))
    off = np.arange(0, 2001, dtype=np.int64)
    gpu.apply_grads(ids, off, np.zeros((2000, 4), f32), 0)
    st = gpu.status()
    assert st["error_bits"] & mb.MONO_DEV_KEYS_FULL
    assert st["n_tracked"] + st["n_keys_dropped"] == 2000
    a = gpu.audit()
    assert a["duplicate_keys"] == 0 and a["misplaced"] == 0 and a["occupied_cells"] == st["n_tracked"]
    kept = set(gpu.export(rows=False)["ids"].tolist())
    assert kept <= set(ids.tolist()) and len(kept) == st["n_tracked"]
    # the table keeps working: a later call on tracked IDs raises their counts
    sub = np.array(sorted(kept)[:32], np.uint64)
    gpu.apply_grads(sub, np.arange(0, 33, dtype=np.int64), np.zeros((32, 4), f32), 1)
    assert (gpu.probe(sub, rows=False)["count"] == 2).all()


def _well_formed_only(ids, off):
    """The batch an oracle sees when every malformed bag is emptied."""
    lists = []
    for b in range(len(off) - 1):
        lo, hi = int(off[b]), int(off[b + 1])
        lists.append(list(ids[lo:hi]) if 0 <= lo <= hi <= len(ids) else [])
    return bags(lists)


@pytest.mark.parametrize("prepared", [False, True, "ahead"])
def test_malformed_offsets_empty_the_offending_bags_in_both_directions(prepared):
    kw = dict(init_scale=0.1, seed=5)
    gpu, cpu = mb.MonoTable(64, 4, 1, 0, **kw), mo.OracleTable(64, 4, 1, 0, **kw)
    ids = np.arange(1, 9, dtype=np.uint64)
    rng = np.random.default_rng(3)
    # a well-formed call first, so that the per-occurrence scratch holds plausible left-overs
    good = np.array([0, 2, 4, 6, 8], np.int64)
    g0 = rng.standard_normal((4, 4)).astype(f32)
    gpu.apply_grads(ids, good, g0, 0)
    cpu.apply_grads(ids, good, g0, 0)
    fresh = np.arange(101, 109, dtype=np.uint64)           # IDs 103..105 occur only in malformed bags
    for t, off in enumerate([np.array([0, 2, -1, 5, 8], np.int64),      # bags 1 and 2 malformed
                             np.array([0, 4, 2, 100, 100], np.int64)], 1):   # decreasing, then past the end
        grad = rng.standard_normal((4, 4)).astype(f32)
        ids_t = torch.from_numpy(fresh.view(np.int64)).cuda()
        off_t = torch.from_numpy(off).cuda()
        grad_t = torch.from_numpy(grad).cuda()
        o_ids, o_off = _well_formed_only(fresh, off)
        out = torch.empty((4, 4), device="cuda")
        if prepared == "ahead":                             # grouped beside the table's work: nothing is flagged yet
            mb.mono_group_ahead(gpu.handle, ids_t, 8, off_t, 4)
            assert gpu.status()["error_bits"] == 0
        if prepared:
            mb.mono_prepare_push(gpu.handle, ids_t, 8, off_t, 4)
        mb.mono_lookup_pool(gpu.handle, ids_t, 8, off_t, 4, out)
        assert_vectors_close(out.cpu().numpy(), cpu.lookup_pool(o_ids, o_off), f"call {t}: pooled")
        mb.mono_apply_grads(gpu.handle, ids_t, 8, off_t, 4, grad_t, t)
        assert cpu.apply_grads(o_ids, o_off, grad, t) == 0
        assert gpu.status()["error_bits"] & mb.MONO_DEV_BAD_OFFSETS
        assert_state_equal(gpu, cpu, f"call {t}")
        assert_audit_ok(gpu)
        mb.mono_clear_errors(gpu.handle)
    tracked = set(gpu.export(rows=False)["ids"].tolist())
    assert tracked & set(range(101, 109)) == {101, 102, 103, 104, 106, 107, 108}   # 105: only ever in malformed bags
    # a well-formed call afterwards is not affected by the earlier flag
    gpu.apply_grads(ids, good, g0, 3)
    cpu.apply_grads(ids, good, g0, 3)
    assert_state_equal(gpu, cpu, "well-formed call after malformed ones")
    assert gpu.status()["error_bits"] == 0


def test_host_detected_errors():
    with pytest.raises(mb.MonoError) as e:
        mb.mono_table_create(64, 6, 1, 0)                 # dim not a multiple of 4
    assert e.value.code == mb.MONO_ERR_ARG
    with pytest.raises(mb.MonoError):
        mb.mono_table_create(64, 8, 1, 0, key_cells=1000)  # not a power of two
    with pytest.raises(mb.MonoError):
        mb.mono_table_create(0, 8, 1, 0)
    gpu = mb.MonoTable(64, 8, 1, 5)
    ids = torch.arange(1, 9, dtype=torch.int64, device="cuda")
    off = torch.tensor([0, 8], dtype=torch.int64, device="cuda")
    grad = torch.ones((1, 8), device="cuda")
    mb.mono_apply_grads(gpu.handle, ids, 8, off, 1, grad, 7)
    for bad_now in (6, -1, mb.MONO_MAX_NOW + 1):
        with pytest.raises(mb.MonoError) as e:
            mb.mono_apply_grads(gpu.handle, ids, 8, off, 1, grad, bad_now)
        assert e.value.code == mb.MONO_ERR_TIME
    with pytest.raises(mb.MonoError) as e:
        mb.mono_expire(gpu.handle, 3)
    assert e.value.code == mb.MONO_ERR_TIME
    with pytest.raises(mb.MonoError) as e:                 # misaligned output
        mb.mono_lookup_pool(gpu.handle, ids, 8, off, 1, grad.data_ptr() + 4)
    assert e.value.code == mb.MONO_ERR_ARG
    with pytest.raises(mb.MonoError):
        mb.mono_lookup_pool(gpu.handle, None, 8, off, 1, grad)
    with pytest.raises(mb.MonoError):
        mb.mono_lookup_pool(gpu.handle, ids, -1, off, 1, grad)
    assert gpu.status()["n_tracked"] == 8 and gpu.status()["error_bits"] == 0


def test_large_times_near_the_limit():
    gpu = mb.MonoTable(64, 4, 1, 10, init_scale=0.1)
    cpu = mo.OracleTable(64, 4, 1, 10, init_scale=0.1)
    base = mb.MONO_MAX_NOW - 30
    for k, lists in enumerate([[[1, 2]], [[2, 3]], [[3]]]):
        ids, off = bags(lists)
        gpu.apply_grads(ids, off, np.ones((1, 4), f32), base + 10 * k)
        cpu.apply_grads(ids, off, np.ones((1, 4), f32), base + 10 * k)
    gpu.expire(mb.MONO_MAX_NOW); cpu.expire(mb.MONO_MAX_NOW)
    assert_state_equal(gpu, cpu)
    assert gpu.export()["ids"].tolist() == [3]
