"""The checked build of the library (-DMONO_DEBUG): every index the kernels compute for
themselves -- segment positions, places in the per-call lists, slots of the per-call set,
positions of the free-row stack -- is tested on the device, and one that falls outside its
array sets MONO_DEV_INTERNAL instead of being used.  The streams below go through every
kernel of the hot path (short and long segments, insertions, expiry, grouped calls, both the
announced and the unannounced path) and must leave that bit clear, with results still those of
the oracle.  Runs in a process of its own, because a process loads one build of the library.
"""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SCRIPT = r"""
import numpy as np, torch
from oracle import mono_oracle as mo
from paper_2209_07663_b200 import binding as mb, workload as wl
from tests.parity import run_stream, assert_state_equal
assert mb.LIB_PATH.endswith("libmono_checked.so")

def pair(cfg):
    kw = dict(lr=cfg.lr, eps=cfg.eps, init_acc=cfg.init_acc, init_scale=cfg.init_scale, seed=cfg.seed)
    return (mb.MonoTable(cfg.capacity, cfg.dim, cfg.filter_threshold, cfg.ttl, key_cells=cfg.key_cells, **kw),
            mo.OracleTable(cfg.capacity, cfg.dim, cfg.filter_threshold, cfg.ttl, **kw))

for prepare in (False, True, "ahead"):
    cfg = wl.scaled(wl.CONFIGS["tiny"], steps=12)
    g, c = pair(cfg)
    st = run_stream(g, c, wl.Stream(cfg), cfg.steps, sweep_every=1, check_every=4, prepare=prepare)
    assert st["error_bits"] == 0 and st["n_expired_total"] > 0
    cfg = wl.scaled(wl.CONFIGS["medium"], steps=6, ttl=2, n_examples=1024, capacity=1 << 17, key_cells=1 << 19)
    g, c = pair(cfg)
    assert run_stream(g, c, wl.Stream(cfg), cfg.steps, sweep_every=1, check_every=3, prepare=prepare)["error_bits"] == 0

# one ID owning a whole batch: parts, folds and the combine levels
g = mb.MonoTable(64, 64, 3, 0, init_scale=0.05, seed=9)
c = mo.OracleTable(64, 64, 3, 0, init_scale=0.05, seed=9)
n_occ, n_bags = 70000, 70000 // 3
lens = np.full(n_bags, 3); lens[-1] += n_occ - lens.sum()
off = np.zeros(n_bags + 1, np.int64); off[1:] = np.cumsum(lens)
ids = np.full(n_occ, 0xABCDEF0123456789, np.uint64); ids[::97] = 77
rng = np.random.default_rng(1)
for t in range(2):
    grad = (rng.standard_normal((n_bags, 64)) * 0.01).astype(np.float32)
    g.apply_grads(ids, off, grad, t); c.apply_grads(ids, off, grad, t)
assert_state_equal(g, c)
assert g.status()["error_bits"] == 0

# grouped calls over tables of four lane-group widths
cfgs = [wl.scaled(x, capacity=1 << 13, key_cells=1 << 15, n_distinct=1 << 14, steps=4, ttl=3)
        for x in wl.multi_table_configs(n_examples=256, slots=3)]
pairs = [pair(x) for x in cfgs]
gens = [wl.Stream(x) for x in cfgs]
hs = [p[0].handle for p in pairs]
for t in range(4):
    steps = [s.step(t) for s in gens]
    dev = [(torch.from_numpy(s.ids.view(np.int64)).cuda(), torch.from_numpy(s.offsets).cuda(),
            torch.from_numpy(s.grad_pooled).cuda()) for s in steps]
    outs = [torch.empty((x.n_bags, x.dim), device="cuda") for x in cfgs]
    if t % 2:
        mb.mono_group_prepare_push(hs, [d[0] for d in dev], [d[1] for d in dev])
    mb.mono_group_lookup_pool(hs, [d[0] for d in dev], [d[1] for d in dev], outs)
    mb.mono_group_apply_grads(hs, [d[0] for d in dev], [d[1] for d in dev], [d[2] for d in dev], t)
    for (gt, ct), s in zip(pairs, steps):
        ct.apply_grads(s.ids, s.offsets, s.grad_pooled, t)
        gt.expire(t); ct.expire(t)
for gt, ct in pairs:
    assert_state_equal(gt, ct)
    assert gt.status()["error_bits"] == 0
print("checked build: ok")
"""


def test_hot_path_under_the_checked_build_reports_no_bad_index():
    lib = os.path.join(ROOT, "paper_2209_07663_b200", "libmono_checked.so")
    if not os.path.exists(lib):
        from paper_2209_07663_b200 import build as mbuild
        mbuild.build(checked=True)
    env = dict(os.environ, MONO_LIBRARY="checked", PYTHONPATH=ROOT)
    r = subprocess.run([sys.executable, "-c", SCRIPT], cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0 and "checked build: ok" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]
