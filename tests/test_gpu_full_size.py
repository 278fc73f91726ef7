"""Parity at the full size of the `large` configuration, in the launch configuration the
benchmark times: table pre-filled to the state after TTL steps of the stream (hundreds of millions of
tracked IDs, ~0.9 row load), whole batches of 1.6 M bags through mono_prepare_push, mono_lookup_pool and
mono_apply_grads, then the sweep in the 32 slices the benchmark spreads over its steps
(here all at one time, which makes them equal to one mono_expire).

The oracle cannot hold that table, so it is checked on a sample: a few hundred bags and
every ID they contain, plus IDs drawn from the head, the middle and the tail of the batch.
Every ID's state depends only on its own history (the property the per-ID replay pins for
the oracle), so the oracle is given the sampled IDs' pre-fill entries and the same batches
with all other IDs replaced by the padding ID, and must then agree with the GPU on the
sampled IDs' state and on the sampled bags' pooled outputs.
"""
import numpy as np
import pytest
import torch

from oracle import mono_oracle as mo
from paper_2209_07663_b200 import binding as mb
from paper_2209_07663_b200 import workload as wl
from tests.parity import assert_vectors_close

pytestmark = pytest.mark.gpu
f32 = np.float32


def _sample(steps, rng, n_bags_sampled=150, n_extra=400):
    """Sampled bags per step and the set of sampled IDs."""
    bags_per_step, ids = [], []
    for s in steps:
        bags = np.sort(rng.choice(s.offsets.size - 1, n_bags_sampled, replace=False))
        bags_per_step.append(bags)
        for b in bags:
            ids.append(s.ids[s.offsets[b]:s.offsets[b + 1]])
        uniq, cnt = np.unique(s.ids, return_counts=True)
        order = np.argsort(-cnt)
        ids.append(uniq[order[:40]])                                  # head: the hottest IDs (long segments)
        ids.append(uniq[order[40:40000]][:: 40000 // 200])            # middle
        ids.append(rng.choice(uniq[cnt == 1], n_extra, replace=False))  # tail: seen once in this batch
    return bags_per_step, np.unique(np.concatenate(ids))


def test_large_config_full_size_sampled_parity():
    free, _ = torch.cuda.mem_get_info()
    if free < 80 * (1 << 30):
        pytest.skip("needs ~70 GB of free device memory")
    cfg = wl.CONFIGS["large"]
    now0, n_steps = cfg.ttl - 1, 3
    stream = wl.Stream(cfg)
    steps = [stream.step(now0 + 1 + t) for t in range(n_steps)]
    rng = np.random.default_rng(11)
    bags_per_step, sample_ids = _sample(steps, rng)
    sample_dev = torch.from_numpy(sample_ids.view(np.int64)).cuda()

    kw = dict(lr=cfg.lr, eps=cfg.eps, init_acc=cfg.init_acc, init_scale=cfg.init_scale, seed=cfg.seed)
    gpu = mb.MonoTable(cfg.capacity, cfg.dim, cfg.filter_threshold, cfg.ttl, key_cells=cfg.key_cells,
                       max_ids=int(max(s.ids.size for s in steps)), max_bags=cfg.n_bags, **kw)
    cpu = mo.OracleTable(cfg.capacity, cfg.dim, cfg.filter_threshold, cfg.ttl, **kw)

    # pre-fill the GPU table; keep the entries of the sampled IDs for the oracle
    keep = []
    for ids, cnt, seen in wl.steady_state_population_torch(cfg, now0, torch.device("cuda")):
        res = (cnt >= cfg.filter_threshold).to(torch.uint8)
        mb.mono_import(gpu.handle, ids, cnt, seen, res, None, None, ids.numel())
        hit = torch.isin(ids, sample_dev)
        keep.append((ids[hit].cpu().numpy().view(np.uint64), cnt[hit].cpu().numpy(), seen[hit].cpu().numpy()))
        del ids, cnt, seen, res, hit
    st = gpu.status()
    assert st["error_bits"] == 0 and st["n_tracked"] > 4e8 and 0.8 < st["n_resident"] / cfg.capacity < 1.0
    p_ids = np.concatenate([k[0] for k in keep])
    p_cnt = np.concatenate([k[1] for k in keep]).astype(np.uint32)
    p_seen = np.concatenate([k[2] for k in keep])
    p_res = (p_cnt >= cfg.filter_threshold).astype(np.uint8)
    w0 = np.array([[mo.init_value(cfg.seed, int(i), c, cfg.init_scale) for c in range(cfg.dim)] for i in p_ids], f32)
    assert cpu.import_entries(p_ids, p_cnt, p_seen, p_res, w0.reshape(-1, cfg.dim),
                              np.full((p_ids.size, cfg.dim), cfg.init_acc, f32)) == 0
    assert 0 < p_ids.size < sample_ids.size                       # some sampled IDs are new to the table

    sample_set = set(sample_ids.tolist())
    out = torch.empty((cfg.n_bags, cfg.dim), dtype=torch.float32, device="cuda")
    def on_device(s):
        return (torch.from_numpy(s.ids.view(np.int64)).cuda(), torch.from_numpy(s.offsets).cuda(),
                torch.from_numpy(s.grad_pooled).cuda())

    upcoming = on_device(steps[0])
    for t, s in enumerate(steps):
        now = now0 + 1 + t
        ids, off, grad = upcoming
        # the oracle's view: same bags, IDs outside the sample become padding
        masked = np.where(np.isin(s.ids, sample_ids), s.ids, np.uint64(mb.MONO_RESERVED_ID))
        mb.mono_prepare_push(gpu.handle, ids, ids.numel(), off, cfg.n_bags)      # as the benchmark does ...
        if t + 1 < len(steps):                                                   # ... with the next batch grouped beside this one
            upcoming = on_device(steps[t + 1])
            mb.mono_group_ahead(gpu.handle, upcoming[0], upcoming[0].numel(), upcoming[1], cfg.n_bags)
        mb.mono_lookup_pool(gpu.handle, ids, ids.numel(), off, cfg.n_bags, out)
        want = cpu.lookup_pool(masked, s.offsets)
        bags = bags_per_step[t]
        for b in bags[:5]:
            assert all(int(i) in sample_set for i in s.ids[s.offsets[b]:s.offsets[b + 1]])
        got = out[torch.from_numpy(bags).cuda()].cpu().numpy()
        assert_vectors_close(got, want[bags], f"step {t}: pooled output of sampled bags")
        mb.mono_apply_grads(gpu.handle, ids, ids.numel(), off, cfg.n_bags, grad, now)
        assert cpu.apply_grads(masked, s.offsets, s.grad_pooled, now) == 0
        del ids, off, grad
    last = now0 + n_steps
    for k in range(32):
        mb.mono_expire_slice(gpu.handle, last, k, 32)
    cpu.expire(last)

    g, o = gpu.probe(sample_ids), cpu.probe(sample_ids)
    assert (g["resident"] == o["resident"]).all() and (g["count"] == o["count"]).all()
    assert (g["last_seen"] == o["last_seen"]).all()
    assert_vectors_close(g["w"], o["w"], "rows of sampled IDs")
    assert_vectors_close(g["acc"], o["acc"], "accumulators of sampled IDs")
    assert o["resident"].sum() > 300 and (o["resident"] == 0).sum() > 100 and (o["count"] == 0).sum() == 0
    st = gpu.status()
    assert st["error_bits"] == 0
    # properties that hold at any size: counters are consistent with what the calls reported
    assert st["n_resident"] <= cfg.capacity and st["n_tracked"] >= st["n_resident"]
    assert st["sum_ids"] == sum(int(s.ids.size) for s in steps)
    assert st["sum_unique"] == sum(int(np.unique(s.ids).size) for s in steps)
