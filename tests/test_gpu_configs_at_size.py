"""Parity at the size and length the configurations name, in the launch configuration the
benchmark times (every batch announced with mono_prepare_push, then looked up, then pushed).

`medium` is small enough for the oracle to hold whole: all 200 steps, full state compared.
`drift` and the eight mixed-dim tables are run at full size on the GPU and checked on a sample,
the scheme of test_gpu_full_size.py: an ID's state depends only on its own history (the property
the per-ID replay pins for the oracle), so the oracle is given the bags that hold a sampled ID,
with every other ID replaced by the padding ID, and must agree with the GPU on the sampled IDs'
state and on the pooled output of the bags whose IDs are all in the sample.
"""
import collections
import concurrent.futures
import os

import numpy as np
import pytest
import torch

from oracle import mono_oracle as mo
from paper_2209_07663_b200 import binding as mb
from paper_2209_07663_b200 import workload as wl
from tests.parity import assert_audit_ok, assert_state_equal, assert_vectors_close

pytestmark = pytest.mark.gpu
f32 = np.float32
PAD = np.uint64(mb.MONO_RESERVED_ID)


def _kw(cfg):
    return dict(lr=cfg.lr, eps=cfg.eps, init_acc=cfg.init_acc, init_scale=cfg.init_scale, seed=cfg.seed)


def _steps_ahead(stream, first, last, prepare=None, depth=6):
    """stream.step(t) for t in [first, last), drawn a few steps ahead on worker threads (the generators
    spend their time in numpy, outside the interpreter lock); `prepare(step)` runs there too."""
    def make(t):
        s = stream.step(t)
        return (s, prepare(s)) if prepare else s
    with concurrent.futures.ThreadPoolExecutor(max_workers=min(depth, os.cpu_count() or 1)) as pool:
        queue = collections.deque()
        t_next = first
        for t in range(first, last):
            while t_next < last and len(queue) < depth:
                queue.append(pool.submit(make, t_next))
                t_next += 1
            yield queue.popleft().result()


def _dev(s):
    return (torch.from_numpy(s.ids.view(np.int64)).cuda(), torch.from_numpy(s.offsets).cuda(),
            torch.from_numpy(s.grad_pooled).cuda())


def test_medium_config_all_200_steps():
    """The whole `medium` stream: 200 steps, a sweep every 10 steps (so the TTL of 100 expires IDs from
    step 110 on), pooled outputs compared every 20th step, the complete table every 50 steps.  Every batch
    is grouped while the batch before it is pulled and pushed."""
    cfg = wl.CONFIGS["medium"]
    gpu = mb.MonoTable(cfg.capacity, cfg.dim, cfg.filter_threshold, cfg.ttl, key_cells=cfg.key_cells,
                       max_ids=cfg.n_bags * 8, max_bags=cfg.n_bags, **_kw(cfg))
    cpu = mo.OracleTable(cfg.capacity, cfg.dim, cfg.filter_threshold, cfg.ttl, **_kw(cfg))
    stream = wl.Stream(cfg)
    out = torch.empty((cfg.n_bags, cfg.dim), dtype=torch.float32, device="cuda")
    h = gpu.handle
    # as the benchmark runs it: every batch grouped one step ahead, announced, pulled, pushed
    steps = _steps_ahead(stream, 0, cfg.steps)
    upcoming = next(steps)
    upcoming = (upcoming,) + _dev(upcoming)
    mb.mono_group_ahead(h, upcoming[1], upcoming[1].numel(), upcoming[2], cfg.n_bags)
    for t in range(cfg.steps):
        s, ids, off, grad = upcoming
        mb.mono_prepare_push(h, ids, ids.numel(), off, cfg.n_bags)
        if t + 1 < cfg.steps:
            upcoming = next(steps)
            upcoming = (upcoming,) + _dev(upcoming)
            mb.mono_group_ahead(h, upcoming[1], upcoming[1].numel(), upcoming[2], cfg.n_bags)
        mb.mono_lookup_pool(h, ids, ids.numel(), off, cfg.n_bags, out)
        if t % 20 == 19:
            assert_vectors_close(out.cpu().numpy(), cpu.lookup_pool(s.ids, s.offsets), f"step {t}: pooled output")
        mb.mono_apply_grads(h, ids, ids.numel(), off, cfg.n_bags, grad, t)
        assert cpu.apply_grads(s.ids, s.offsets, s.grad_pooled, t) == 0
        if t % 10 == 9:
            gpu.expire(t)
            cpu.expire(t)
        if t % 50 == 49:
            assert_state_equal(gpu, cpu, f"step {t}")
            assert_audit_ok(gpu, f"step {t}")
    st = gpu.status()
    assert st["error_bits"] == 0 and st["scratch_reallocs"] == 0
    assert st["n_expired_total"] > 100000, "the TTL must have expired IDs by step 200"
    assert st["n_resident"] > 1000000


# ---------------------------------------------------------------- sampled parity at full size

def _hot_middle_tail(s, rng, n_tail):
    uniq, cnt = np.unique(s.ids, return_counts=True)
    order = np.argsort(-cnt)
    picks = [uniq[order[:30]], uniq[order[30:30000]][:: 30000 // 150]]
    once = uniq[cnt == 1]
    picks.append(rng.choice(once, min(n_tail, once.size), replace=False))
    return picks


def _sampled_view(s, sample_ids, dim):
    """The bags of step `s` that hold a sampled ID, other IDs padded out: (ids, offsets, grads, bag numbers,
    which of those bags hold sampled IDs only)."""
    hit = np.isin(s.ids, sample_ids)
    lens = np.diff(s.offsets)
    bag_of = np.repeat(np.arange(lens.size), lens)
    per_bag = np.bincount(bag_of[hit], minlength=lens.size)
    bags = np.nonzero(per_bag)[0]
    keep = np.isin(bag_of, bags)
    ids = np.where(hit[keep], s.ids[keep], PAD)
    off = np.zeros(bags.size + 1, np.int64)
    np.cumsum(lens[bags], out=off[1:])
    pure = per_bag[bags] == lens[bags]
    return ids, off, s.grad_pooled[bags], bags, pure


def test_drift_config_full_size_sampled_parity():
    """The concept-drift configuration at its full size, from an empty table, across five re-keyings of
    the ID universe and past one TTL, so that insertions, admissions and expiries all occur.  Two tables
    take the same stream: the configured one (2^26 rows, which this stream fills to a tenth) and the one
    sized for the stream (`drift_dense`: both stores near load 0.9, where insertions displace other
    keys).  What a table holds does not depend on its size, so one oracle checks both."""
    free, _ = torch.cuda.mem_get_info()
    if free < 40 * (1 << 30):
        pytest.skip("needs ~30 GB of free device memory")
    cfg, dense = wl.CONFIGS["drift"], wl.CONFIGS["drift_dense"]
    assert wl.scaled(dense, name=cfg.name, capacity=cfg.capacity, key_cells=cfg.key_cells) == cfg    # same stream
    n_steps, sweep_every = cfg.ttl + cfg.drift_period + 12, 20
    stream = wl.Stream(cfg)
    rng = np.random.default_rng(17)
    # the sample: IDs from the head, the middle and the tail of batches before and after re-keyings,
    # and every ID of a few hundred bags
    picks = []
    for t in (0, cfg.drift_period - 1, cfg.drift_period, 2 * cfg.drift_period + 3, cfg.ttl - 1, cfg.ttl + 5, n_steps - 1):
        s = stream.step(t, with_grad=False)
        picks += _hot_middle_tail(s, rng, 300)
        for b in rng.choice(cfg.n_bags, 60, replace=False):
            picks.append(s.ids[s.offsets[b]:s.offsets[b + 1]])
    sample_ids = np.unique(np.concatenate(picks))

    gpus = [mb.MonoTable(c.capacity, c.dim, c.filter_threshold, c.ttl, key_cells=c.key_cells,
                         max_ids=int(c.n_bags * 5.6), max_bags=c.n_bags, **_kw(c)) for c in (cfg, dense)]
    cpu = mo.OracleTable(cfg.capacity, cfg.dim, cfg.filter_threshold, cfg.ttl, **_kw(cfg))
    outs = [torch.empty((cfg.n_bags, cfg.dim), dtype=torch.float32, device="cuda") for _ in gpus]
    n_pure = 0
    for t, (s, view) in enumerate(_steps_ahead(stream, 0, n_steps, lambda s: _sampled_view(s, sample_ids, cfg.dim))):
        ids, off, grad = _dev(s)
        o_ids, o_off, o_grad, bags, pure = view
        for gpu, out in zip(gpus, outs):
            mb.mono_prepare_push(gpu.handle, ids, ids.numel(), off, cfg.n_bags)
            mb.mono_lookup_pool(gpu.handle, ids, ids.numel(), off, cfg.n_bags, out)
        if t % 10 == 0 or t >= n_steps - 3:
            want = cpu.lookup_pool(o_ids, o_off)[pure]
            for k, out in enumerate(outs):
                got = out[torch.from_numpy(bags[pure]).cuda()].cpu().numpy()
                assert_vectors_close(got, want, f"table {k} step {t}: pooled output of sampled bags")
            n_pure += int(pure.sum())
        for gpu in gpus:
            mb.mono_apply_grads(gpu.handle, ids, ids.numel(), off, cfg.n_bags, grad, t)
        assert cpu.apply_grads(o_ids, o_off, o_grad, t) == 0
        if t % sweep_every == sweep_every - 1:
            for gpu in gpus:
                gpu.expire(t)
            cpu.expire(t)
        if t % 60 == 59 or t == n_steps - 1:
            o = cpu.probe(sample_ids)
            for k, gpu in enumerate(gpus):
                g = gpu.probe(sample_ids)
                assert (g["resident"] == o["resident"]).all() and (g["count"] == o["count"]).all(), f"table {k} step {t}"
                assert (g["last_seen"] == o["last_seen"]).all(), f"table {k} step {t}"
                assert_vectors_close(g["w"], o["w"], f"table {k} step {t}: rows of sampled IDs")
                assert_vectors_close(g["acc"], o["acc"], f"table {k} step {t}: accumulators of sampled IDs")
        del ids, off, grad
    assert n_pure > 500
    o = cpu.probe(sample_ids, rows=False)
    assert (o["count"] == 0).sum() > 50 and o["resident"].sum() > 50        # some sampled IDs expired, some own a row
    stats = [gpu.status() for gpu in gpus]
    for k, (gpu, st) in enumerate(zip(gpus, stats)):
        assert st["error_bits"] == 0 and st["scratch_reallocs"] == 0, f"table {k}: {st}"
        # insertions, admissions and expiries all took place
        assert st["n_inserted_total"] > st["n_tracked"] > 1000000 and st["n_expired_total"] > 1000000
        assert st["n_admitted_total"] > st["n_resident"] > 0
        assert_audit_ok(gpu, f"table {k}")
    # the two tables hold the same IDs and rows ...
    for key in ("n_tracked", "n_resident", "n_inserted_total", "n_expired_total", "n_admitted_total"):
        assert stats[0][key] == stats[1][key], key
    # ... the small one under displacement: loads near 0.9, chains, no key lost
    st = stats[1]
    assert st["n_resident"] > 0.7 * dense.capacity and st["n_tracked"] > 0.8 * dense.key_cells
    assert st["max_chain"] > 0 and st["n_evictions_total"] > 1000000 and st["n_keys_dropped"] == 0
    assert stats[0]["n_evictions_total"] < st["n_evictions_total"]


def test_eight_tables_full_size_grouped_calls_sampled_parity():
    """The mixed-dim multi-table configuration at its full size, every table pre-filled to the state after
    TTL steps, three steps through mono_group_lookup_pool / mono_group_apply_grads with every batch
    announced first; each table checked on its own sample against its own oracle."""
    free, _ = torch.cuda.mem_get_info()
    if free < 130 * (1 << 30):
        pytest.skip("needs ~120 GB of free device memory")
    cfgs = wl.multi_table_configs()
    n_steps = 3
    rng = np.random.default_rng(23)
    dev = torch.device("cuda")
    streams = [torch.cuda.Stream() for _ in cfgs]
    tables, oracles, samples, steps_all = [], [], [], []
    for cfg, cs in zip(cfgs, streams):
        now0 = cfg.ttl - 1
        gen = wl.Stream(cfg)
        steps = [gen.step(now0 + 1 + t) for t in range(n_steps)]
        picks = []
        for s in steps:
            picks += _hot_middle_tail(s, rng, 200)
            for b in rng.choice(cfg.n_bags, 80, replace=False):
                picks.append(s.ids[s.offsets[b]:s.offsets[b + 1]])
        sample_ids = np.unique(np.concatenate(picks))
        sample_dev = torch.from_numpy(sample_ids.view(np.int64)).cuda()
        gpu = mb.MonoTable(cfg.capacity, cfg.dim, cfg.filter_threshold, cfg.ttl, key_cells=cfg.key_cells,
                           max_ids=int(max(s.ids.size for s in steps)), max_bags=cfg.n_bags, stream=cs.cuda_stream,
                           **_kw(cfg))
        cpu = mo.OracleTable(cfg.capacity, cfg.dim, cfg.filter_threshold, cfg.ttl, **_kw(cfg))
        keep = []
        for ids, cnt, seen in wl.steady_state_population_torch(cfg, now0, dev):
            res = (cnt >= cfg.filter_threshold).to(torch.uint8)
            torch.cuda.synchronize()
            mb.mono_import(gpu.handle, ids, cnt, seen, res, None, None, ids.numel())
            hit = torch.isin(ids, sample_dev)
            keep.append((ids[hit].cpu().numpy().view(np.uint64), cnt[hit].cpu().numpy(), seen[hit].cpu().numpy()))
            del ids, cnt, seen, res, hit
        assert gpu.status()["error_bits"] == 0
        p_ids = np.concatenate([k[0] for k in keep])
        p_cnt = np.concatenate([k[1] for k in keep]).astype(np.uint32)
        p_seen = np.concatenate([k[2] for k in keep])
        p_res = (p_cnt >= cfg.filter_threshold).astype(np.uint8)
        w0 = np.array([[mo.init_value(cfg.seed, int(i), c, cfg.init_scale) for c in range(cfg.dim)] for i in p_ids],
                      f32).reshape(-1, cfg.dim)
        assert cpu.import_entries(p_ids, p_cnt, p_seen, p_res, w0, np.full((p_ids.size, cfg.dim), cfg.init_acc, f32)) == 0
        tables.append(gpu); oracles.append(cpu); samples.append(sample_ids); steps_all.append(steps)

    handles = [t.handle for t in tables]
    outs = [torch.empty((c.n_bags, c.dim), dtype=torch.float32, device="cuda") for c in cfgs]
    gs = torch.cuda.current_stream().cuda_stream
    now0 = cfgs[0].ttl - 1
    for t in range(n_steps):
        batch = [_dev(steps_all[i][t]) for i in range(len(cfgs))]
        torch.cuda.synchronize()
        for i, tb in enumerate(tables):
            mb.mono_prepare_push(tb.handle, batch[i][0], batch[i][0].numel(), batch[i][1], cfgs[i].n_bags)
        mb.mono_group_lookup_pool(handles, [b[0] for b in batch], [b[1] for b in batch], outs, gs)
        torch.cuda.synchronize()
        views = []
        for i, cfg in enumerate(cfgs):
            v = _sampled_view(steps_all[i][t], samples[i], cfg.dim)
            views.append(v)
            want = oracles[i].lookup_pool(v[0], v[1])[v[4]]
            got = outs[i][torch.from_numpy(v[3][v[4]]).cuda()].cpu().numpy()
            assert_vectors_close(got, want, f"table {i} step {t}: pooled output of sampled bags")
            assert v[4].sum() > 20
        mb.mono_group_apply_grads(handles, [b[0] for b in batch], [b[1] for b in batch], [b[2] for b in batch],
                                  now0 + 1 + t, gs)
        torch.cuda.synchronize()
        for i in range(len(cfgs)):
            v = views[i]
            assert oracles[i].apply_grads(v[0], v[1], v[2], now0 + 1 + t) == 0
    for i, (gpu, cpu) in enumerate(zip(tables, oracles)):
        last = now0 + n_steps
        for k in range(32):
            mb.mono_expire_slice(gpu.handle, last, k, 32)
        cpu.expire(last)
        g, o = gpu.probe(samples[i]), cpu.probe(samples[i])
        assert (g["resident"] == o["resident"]).all() and (g["count"] == o["count"]).all(), f"table {i}"
        assert (g["last_seen"] == o["last_seen"]).all(), f"table {i}"
        assert_vectors_close(g["w"], o["w"], f"table {i}: rows of sampled IDs")
        assert_vectors_close(g["acc"], o["acc"], f"table {i}: accumulators of sampled IDs")
        assert o["resident"].sum() > 100
        st = gpu.status()
        assert st["error_bits"] == 0 and st["scratch_reallocs"] == 0
        gpu.close()
