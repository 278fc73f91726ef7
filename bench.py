#!/usr/bin/env python
"""Benchmark of the collisionless embedding-table step on B200.

One "step" is one pass of the whole hot path over one fresh synthetic batch:
mono_lookup_pool (probe, gather, sum pooling) + mono_apply_grads (dedup,
count/stamp/admit, cuckoo insert, segmented gradient reduce, Adagrad), followed
by one slice of the expiry sweep (mono_expire_slice: 1/`sweep_slices` of the key
store per step, so every step carries the same share of the sweep).  Each batch is
announced with mono_prepare_push before its lookup, so its IDs are grouped and looked up
in the key store once, for the lookup and the push together.  The timed region is repeated
--reps times from the same restored state (median and min reported).
The table is pre-filled to the state the configured stream reaches after TTL steps
from an empty table, so the timed steps run at that load, not on an empty table.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload large]
    python bench.py --impl reference ...     # the CPU oracle, timed on the host

Prints one JSON line (rank 0).  With N > 1 (under torchrun) every rank owns an
independent table and its own batches (weak scaling, no data-path collective).
"""
from __future__ import annotations

import argparse
import concurrent.futures
import hashlib
import json
import os
import statistics
import subprocess
import sys
import tempfile
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2209_07663_b200 import workload as wl  # noqa: E402

METRIC = "feature IDs/sec (lookup+pool+update) on 1 B200; % of HBM roofline"
UNIT = "IDs/s"
FALLBACK_HBM_GBS = 6650.0


# --------------------------------------------------------------------------- helpers

def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


KERNEL_SOURCES = {
    "probe_rows": ("kernels_forward.cuh", "table_layout.cuh"),
    "gather_pool": ("kernels_forward.cuh", "kernels_dedup.cuh", "table_layout.cuh"),
    "fill_occ_bag": ("kernels_dedup.cuh", "table_layout.cuh"),
    "dedup_tile": ("kernels_dedup.cuh", "table_layout.cuh"),
    "table_lookup": ("kernels_table.cuh", "kernels_forward.cuh", "kernels_dedup.cuh", "table_layout.cuh"),
    "table_update": ("kernels_table.cuh", "kernels_forward.cuh", "kernels_dedup.cuh", "table_layout.cuh"),
    "table_insert": ("kernels_table.cuh", "kernels_dedup.cuh", "table_layout.cuh"),
    "update_singletons": ("kernels_adagrad.cuh", "kernels_dedup.cuh", "table_layout.cuh"),
    "file_segments": ("kernels_adagrad.cuh", "kernels_dedup.cuh", "table_layout.cuh"),
    "reduce_adagrad": ("kernels_adagrad.cuh", "kernels_dedup.cuh", "table_layout.cuh"),
    "reduce_parts": ("kernels_adagrad.cuh", "kernels_dedup.cuh", "table_layout.cuh"),
    "combine_adagrad": ("kernels_adagrad.cuh", "kernels_dedup.cuh", "table_layout.cuh"),
    "fold_partials": ("kernels_adagrad.cuh", "kernels_dedup.cuh", "table_layout.cuh"),
}


def kernel_source_digest(kernel: str) -> str:
    """Digest of the source files a kernel is compiled from (its own file and what it includes)."""
    h = hashlib.sha256()
    d = os.path.join(ROOT, "paper_2209_07663_b200", "csrc")
    for name in KERNEL_SOURCES.get(kernel, sorted(os.listdir(d))):
        with open(os.path.join(d, name), "rb") as f:
            h.update(name.encode())
            h.update(f.read())
    return h.hexdigest()[:16]


def recorded_traffic(kernel: str, workload: str):
    """DRAM bytes per launch from the committed ncu summary of this kernel, or None when
    there is none or the kernels have changed since it was taken."""
    path = os.path.join(ROOT, "profiles", f"traffic_{kernel}_{workload}.txt")
    if not os.path.exists(path):
        return None
    kv = {}
    for line in open(path):
        if "=" in line and not line.lstrip().startswith("#"):
            k, v = line.split("=", 1)
            kv[k.strip()] = v.strip()
    if kv.get("source_digest") != kernel_source_digest(kernel):
        return None
    try:
        return float(kv["dram_bytes_per_launch_scaled"])
    except Exception:
        return None


class ClockSampler:
    """SM clock and clock-event reasons of one GPU, read through NVML every few milliseconds by a
    thread while the timed region runs (the region lasts tens of milliseconds, too short for
    nvidia-smi's own loop); nvidia-smi in the background when NVML cannot be loaded."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    PERIOD_S = 0.004

    def __init__(self, gpu_index: int, uuid: str = ""):
        self.gpu_index = gpu_index
        self.uuid = uuid
        self.proc = None
        self.path = None
        self.thread = None
        self.halt = threading.Event()
        self.sm, self.reason_bits, self.power_w = [], 0, []
        self.sm_max = None
        self.source = None

    def _nvml_loop(self, nv, handle):
        while not self.halt.is_set():
            try:
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(handle, nv.NVML_CLOCK_SM)))
                self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(handle))
                self.power_w.append(nv.nvmlDeviceGetPowerUsage(handle) / 1000.0)
            except Exception:
                pass
            self.halt.wait(self.PERIOD_S)

    def start(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            handle = None
            if self.uuid:
                try:
                    handle = nv.nvmlDeviceGetHandleByUUID(("GPU-" + self.uuid).encode())
                except Exception:
                    handle = None
            if handle is None:
                handle = nv.nvmlDeviceGetHandleByIndex(self.gpu_index)
            self.sm_max = float(nv.nvmlDeviceGetMaxClockInfo(handle, nv.NVML_CLOCK_SM))
            self.nv = nv
            self.thread = threading.Thread(target=self._nvml_loop, args=(nv, handle), daemon=True)
            self.source = "nvml"
            self.thread.start()
            return
        except Exception:
            self.thread = None
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu_index)], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
            self.source = "nvidia-smi"
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "source": self.source}
        if self.thread is not None:
            self.halt.set()
            self.thread.join(timeout=2)
            nv = self.nv
            names = (("hw_slowdown", "nvmlClocksEventReasonHwSlowdown", "nvmlClocksThrottleReasonHwSlowdown"),
                     ("hw_thermal_slowdown", "nvmlClocksEventReasonHwThermalSlowdown", "nvmlClocksThrottleReasonHwThermalSlowdown"),
                     ("sw_thermal_slowdown", "nvmlClocksEventReasonSwThermalSlowdown", "nvmlClocksThrottleReasonSwThermalSlowdown"),
                     ("sw_power_cap", "nvmlClocksEventReasonSwPowerCap", "nvmlClocksThrottleReasonSwPowerCap"))
            reasons = []
            for label, a, b in names:
                bit = getattr(nv, a, None) or getattr(nv, b, 0)
                if bit and (self.reason_bits & bit):
                    reasons.append(label)
            if self.sm:
                out.update(sm_mhz=statistics.median(self.sm), sm_min_mhz=min(self.sm), sm_max_mhz=self.sm_max,
                           reasons=sorted(reasons), samples=len(self.sm),
                           power_w_max=max(self.power_w) if self.power_w else None)
            try:
                nv.nvmlShutdown()
            except Exception:
                pass
            return out
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1]))
                    smax.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                     f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(smax), reasons=sorted(reasons), samples=len(sm))
        return out


def gpu_uuid(index: int) -> str:
    """UUID of CUDA device `index` (what NVML knows it by, whatever CUDA_VISIBLE_DEVICES says)."""
    try:
        import torch
        return str(torch.cuda.get_device_properties(index).uuid)
    except Exception:
        return ""


def sample_of_step(step: wl.Step, n_bags: int) -> wl.Step:
    """The first n_bags bags of a step (a bounded sample for the CPU oracle)."""
    n_bags = min(n_bags, step.offsets.size - 1)
    n_ids = int(step.offsets[n_bags])
    return wl.Step(ids=step.ids[:n_ids], offsets=step.offsets[:n_bags + 1],
                   grad_pooled=step.grad_pooled[:n_bags], now=step.now)


def time_oracle(cfg: wl.Config, steps: int, warmup: int, sample_bags: int, first_step: int = 0):
    """lookup_pool + apply_grads of the CPU oracle on the first `sample_bags` bags of each
    step, from an empty table.  Returns (ids_per_second, ms_per_step, ids_per_step)."""
    from oracle import mono_oracle as mo
    o = mo.OracleTable(cfg.capacity, cfg.dim, cfg.filter_threshold, cfg.ttl, lr=cfg.lr, eps=cfg.eps,
                       init_acc=cfg.init_acc, init_scale=cfg.init_scale, seed=cfg.seed)
    stream = wl.Stream(cfg)
    batches = [sample_of_step(stream.step(first_step + t), sample_bags) for t in range(warmup + steps)]
    n_ids, elapsed = 0, 0.0
    for t, s in enumerate(batches):
        t0 = time.perf_counter()
        o.lookup_pool(s.ids, s.offsets)
        o.apply_grads(s.ids, s.offsets, s.grad_pooled, first_step + t)
        dt = time.perf_counter() - t0
        if t >= warmup:
            elapsed += dt
            n_ids += s.ids.size
    return n_ids / elapsed, 1e3 * elapsed / steps, n_ids / steps


# --------------------------------------------------------------------------- reference arm

def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = wl.CONFIGS[args.workload]
    sample_bags = max(cfg.n_bags // args.oracle_fraction, 1)
    ids_s, ms_step, ids_step = time_oracle(cfg, args.steps, args.warmup, sample_bags)
    sample = (f"first {sample_bags} of {cfg.n_bags} bags of each step (~{int(ids_step)} IDs), "
              f"lookup_pool + apply_grads, from an empty table")
    line = {
        "impl": "reference", "metric": METRIC, "value": ids_s, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": args.workload, "capacity": cfg.capacity, "dim": cfg.dim,
                   "bags_per_step": cfg.n_bags, "sample": sample},
        "cpu_baseline": {"value": ids_s, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": ids_s, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- our arm

def algorithmic_bytes(n, b, u, ur, ur1, unew, d, sweep_cells=0, prepared=True, expired=0):
    """Bytes the method itself must move per step, per kernel (each distinct datum once per
    phase; 32-byte sector as the smallest random access).  n occurrences, b bags, u distinct
    IDs, ur of them with a row, ur1 of those occurring once in the batch, unew new IDs.
    prepared: the batch was announced, so the key store is read once per distinct ID ahead of
    the lookup instead of once per occurrence inside it.  sweep_cells: key cells the step's slice
    of the expiry sweep covers, expired: entries it removes."""
    per_kernel = {
        "probe_rows": 0,
        # offsets, one 8-byte record per occurrence (the ID, or its place in the grouping), each distinct row once, out
        "gather_pool": 8 * (b + 1) + 8 * n + (0 if prepared else 32 * n) + 4 * d * ur + 4 * d * b,
        "fill_occ_bag": 8 * (b + 1),                         # offsets
        "dedup_tile": 8 * n + 24 * n,                        # ids + (key, index) pairs written and read
        "table_lookup": 32 * u if prepared else 0,           # one bucket sector per distinct ID
        "table_update": 64 * u,                              # count/stamp read-modify-write of that sector
        "table_insert": (16 + 8 * d) * unew,                 # key write + row/accumulator initialisation
        "sketch_add": 0,                                     # (probabilistic filter: counted with table_insert's new IDs)
        "update_singletons": 20 * d * ur1,                   # IDs seen once: gradient row, row and accumulator in and out
        # rows of repeated IDs + the gradient rows the singletons did not read, once (the two launches of
        # reduce_adagrad_kernel, short segments and the parts of long ones, share them; counted on the first)
        "reduce_adagrad": 16 * d * (ur - ur1) + 4 * d * max(b - ur1, 0), "reduce_parts": 0,
        "file_segments": 0, "clear_set": 0,
        "expand_parts": 0, "order_parts": 0, "fold_partials": 0, "combine_adagrad": 0, "finish_apply": 0,
        # the sweep's 4-byte record per 4-cell bucket in order; a removed entry's bucket read (64) and its cell cleared (32)
        "expire": sweep_cells + 96 * expired,
    }
    return per_kernel, sum(per_kernel.values())


KERNEL_GROUP = {
    "probe_rows": "lookup_pool", "gather_pool": "lookup_pool",
    "fill_occ_bag": "dedup", "dedup_tile": "dedup", "finish_apply": "dedup", "clear_set": "dedup",
    "table_lookup": "table", "table_update": "table", "sketch_add": "table", "table_insert": "table", "expand_parts": "table", "order_parts": "table",
    "update_singletons": "adagrad", "file_segments": "lookup_pool", "reduce_parts": "adagrad", "reduce_adagrad": "adagrad", "fold_partials": "adagrad",
    "combine_adagrad": "adagrad", "expire": "expire",
}


def rank_config(base: wl.Config, rank: int) -> wl.Config:
    """Every rank owns an independent table and draws its own stream (weak scaling)."""
    return wl.scaled(base, seed=base.seed + 7919 * rank)


def aggregate_over_ranks(times_ms, work_units, device="cpu"):
    """Job-level figures from per-rank ones: the slowest rank's time for each timed region
    (MAX), the work of all ranks together (SUM).  Works without a process group (N = 1)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    w = torch.tensor(list(work_units), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(w, op=dist.ReduceOp.SUM)
    return t.tolist(), w.tolist()


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2209_07663_b200 import binding as mb

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the table has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dev = torch.device("cuda", local_rank)
    if args.stream_priority == "high":
        torch.cuda.set_stream(torch.cuda.Stream(device=dev, priority=-1))

    base = wl.CONFIGS[args.workload]
    cfg = rank_config(base, rank)
    sketch = args.filter == "sketch"
    if sketch:
        # probabilistic admission filter: IDs without a row live in a count-min sketch, not in the key
        # store, which is therefore sized for the IDs that own rows only
        cfg = wl.scaled(cfg, key_cells=max(cfg.key_cells >> args.sketch_key_shrink_log2, 1 << 10))
    drift = cfg.drift_period > 0
    if drift:
        # The drift stream has no closed-form steady state to pre-fill: it starts from an empty
        # table and warms up for more than ttl steps (past the first full expiry horizon and a
        # re-keying), and the timed steps span at least one re-keying of the ID universe.
        args.prefill = False
        if args.warmup < cfg.ttl + cfg.drift_period + 10:
            args.warmup = cfg.ttl + cfg.drift_period + 10
        if args.steps < 2 * cfg.drift_period:
            args.steps = 2 * cfg.drift_period
    K, W, E = args.steps, args.warmup, args.e2e_steps
    KT = min(K, args.kernel_steps)            # steps of the per-kernel timing pass
    S = args.sweep_slices
    now0 = cfg.ttl - 1 if args.prefill else 0
    stream = wl.Stream(cfg)

    # ---- table, pre-filled to the state after ttl steps of the stream
    t_setup = time.time()
    table = mb.MonoTable(cfg.capacity, cfg.dim, cfg.filter_threshold, cfg.ttl, lr=cfg.lr, eps=cfg.eps,
                         init_acc=cfg.init_acc, init_scale=cfg.init_scale, seed=cfg.seed,
                         key_cells=cfg.key_cells, max_ids=int(cfg.n_bags * wl._mean_bag_len(cfg.bag_len) * 1.1),
                         max_bags=cfg.n_bags, sketch_depth=args.sketch_depth if sketch else 0,
                         sketch_width=(1 << args.sketch_width_log2) if sketch else 0)
    if args.prefill:
        for ids, cnt, seen in wl.steady_state_population_torch(cfg, now0, dev):
            if sketch:      # only IDs with a row have an entry; the sketch starts empty, as after one of its clearings
                keep = cnt >= cfg.filter_threshold
                ids, cnt, seen = ids[keep], cnt[keep], seen[keep]
            res = (cnt >= cfg.filter_threshold).to(torch.uint8)
            mb.mono_import(table.handle, ids, cnt, seen, res, None, None, ids.numel())
            del ids, cnt, seen, res
    st0 = table.status()
    if st0["error_bits"]:
        raise SystemExit(f"pre-fill overflowed the table: {st0}")

    # ---- batches: ids/offsets from the seeded host generator, gradients drawn on the device
    EW = 1 if E > 0 else 0                     # one untimed end-to-end step first: it allocates the staging buffers
    n_batches = W + K + KT + EW + E

    def make(i):
        return stream.step(now0 + 1 + i, with_grad=False)

    gg = torch.Generator(device=dev)
    gg.manual_seed(cfg.seed)
    # every step has its own ids and offsets; its gradients too, except in a long drift run, where
    # the steps take turns on a ring of gradient tensors that is still several times larger than L2
    # (and in any run of more than 48 steps: a ring of 48 gradient tensors, 20 GB on `large`, keeps long runs within
    # device memory; consecutive steps still never share one)
    n_grads = min(W + K + KT, 16) if drift else min(W + K + KT, 48)
    grads = [torch.randn((cfg.n_bags, cfg.dim), device=dev, generator=gg).mul_(cfg.grad_std) for _ in range(n_grads)]
    dev_batches, host_batches = [], {}
    with concurrent.futures.ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1)) as pool:
        for t, s in enumerate(pool.map(make, range(n_batches))):
            if t < W + K + KT:
                ids = torch.from_numpy(s.ids.view(np.int64)).to(dev)
                off = torch.from_numpy(s.offsets).to(dev)
                dev_batches.append((ids, off, grads[t % n_grads]))
            else:
                host_batches[t] = s            # the end-to-end steps start from host memory
    out = torch.empty((cfg.n_bags, cfg.dim), dtype=torch.float32, device=dev)
    torch.cuda.synchronize()
    setup_s = time.time() - t_setup

    def step(i, prepare=True):
        """Step i of the stream (time now0 + 1 + i) on its own fresh batch."""
        ids, off, grad = dev_batches[i]
        if prepare and args.prepare:
            mb.mono_prepare_push(table.handle, ids, ids.numel(), off, cfg.n_bags)
            if args.group_ahead and i + 1 < len(dev_batches):
                # the next step's batch is grouped by ID beside this step's lookup and push (issued here, it
                # measured 1.0 % of a step faster than without; issued after the lookup, 0.3 %)
                nxt = dev_batches[i + 1]
                mb.mono_group_ahead(table.handle, nxt[0], nxt[0].numel(), nxt[1], cfg.n_bags)
        mb.mono_lookup_pool(table.handle, ids, ids.numel(), off, cfg.n_bags, out)
        mb.mono_apply_grads(table.handle, ids, ids.numel(), off, cfg.n_bags, grad, now0 + 1 + i)
        if S > 0:
            mb.mono_expire_slice(table.handle, now0 + 1 + i, i % S, S)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- warm-up, then the timed region: R repetitions of the same K steps, each from the state the
    # warm-up left (a device-resident snapshot restored in between), so that the spread between
    # repetitions is measurement noise and nothing else
    R = max(args.reps, 1)
    for t in range(W):
        step(t)
    barrier()
    reps_note = None
    if R > 1:
        try:
            mb.mono_snapshot_save(table.handle)
        except mb.MonoError as e:          # no room for a second copy of the table: one repetition, and say so
            if e.code != mb.MONO_ERR_NOMEM:
                raise
            R, reps_note = 1, "no device memory for the snapshot the repetitions return to: one repetition only"
        if world > 1:                      # every rank repeats as often as the rank with the least room
            r_all = torch.tensor([R], dtype=torch.int64, device=dev)
            dist.all_reduce(r_all, op=dist.ReduceOp.MIN)
            if int(r_all.item()) < R:
                R, reps_note = 1, "another rank had no device memory for the snapshot: one repetition only"
                mb.mono_snapshot_drop(table.handle)
    sampler = ClockSampler(local_rank, gpu_uuid(local_rank))
    rep_ms, launches, n_ids_timed = [], 0, 0
    st_a = st_b = None
    for r in range(R):
        if r > 0:
            mb.mono_snapshot_restore(table.handle)
        barrier()
        st_a = table.status()
        mb.mono_timing_read(table.handle, reset=True)
        if r == 0:
            sampler.start()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        ev0.record()
        for t in range(K):
            step(W + t)
        mb.mono_fence(table.handle)            # the last step's sweep slice runs on a stream of the table's own
        ev1.record()
        barrier()
        rep_ms.append(ev0.elapsed_time(ev1))
        st_b = table.status()
        launches = mb.mono_timing_read(table.handle, reset=True)["launches_total"]
        n_ids_timed = st_b["sum_ids"] - st_a["sum_ids"]
    clocks = sampler.stop()
    if R > 1:
        mb.mono_snapshot_drop(table.handle)
    ms_total = statistics.median(rep_ms)

    # ---- the same steps on fresh batches with every kernel bracketed by CUDA events
    mb.mono_timing_enable(table.handle, True)
    for t in range(KT):
        step(W + K + t)                      # the same calls; the events keep every kernel alone on the device
    torch.cuda.synchronize()
    tim = mb.mono_timing_read(table.handle, reset=True)
    mb.mono_timing_enable(table.handle, False)
    st_c = table.status()

    # ---- end to end: host buffers in, pooled output back out, through the host-buffer calls
    e2e = None
    if E > 0:
        pinned = []
        for t in sorted(host_batches):
            s = host_batches[t]
            ids = torch.from_numpy(s.ids.view(np.int64)).pin_memory()
            off = torch.from_numpy(s.offsets).pin_memory()
            grad = torch.randn((cfg.n_bags, cfg.dim)).mul_(cfg.grad_std).pin_memory()
            pinned.append((ids, off, grad))
        out_h = torch.empty((cfg.n_bags, cfg.dim), dtype=torch.float32).pin_memory()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_e2e_ids, h2d, d2h = 0, 0, 0
        for t, (ids, off, grad) in enumerate(pinned):
            if t == EW:
                mb.mono_fence(table.handle)
                barrier()
                e0.record()
            now = now0 + 1 + W + K + KT + t
            mb.mono_lookup_pool_host(table.handle, ids, ids.numel(), off, cfg.n_bags, out_h)
            mb.mono_apply_grads_host(table.handle, ids, ids.numel(), off, cfg.n_bags, grad, now)
            if S > 0:
                mb.mono_expire_slice(table.handle, now, (W + K + KT + t) % S, S)
            if t < EW:
                continue
            n_e2e_ids += ids.numel()
            h2d += ids.numel() * 8 + off.numel() * 8 + grad.numel() * 4    # the push reuses the IDs its lookup staged
            d2h += out_h.numel() * 4
        mb.mono_fence(table.handle)              # the copies run on streams of the table's own
        e1.record()
        barrier()
        e2e_ms = e0.elapsed_time(e1)
        e2e = {"ids": n_e2e_ids, "ms": e2e_ms, "h2d": h2d // E, "d2h": d2h // E}
    st_end = table.status()

    # ---- aggregate over ranks: max time, summed work
    (ms_max, e2e_ms_max), (ids_all, e2e_ids_all) = aggregate_over_ranks(
        [ms_total, e2e["ms"] if e2e else 0.0], [float(n_ids_timed), float(e2e["ids"]) if e2e else 0.0], dev)

    if rank == 0:
        peak, peak_kind = measured_peaks()
        d = cfg.dim
        # per-step averages over the per-kernel pass (the steps the kernel times belong to)
        n = (st_c["sum_ids"] - st_b["sum_ids"]) / KT
        u = (st_c["sum_unique"] - st_b["sum_unique"]) / KT
        ur = (st_c["sum_unique_resident"] - st_b["sum_unique_resident"]) / KT
        unew = (st_c["sum_new"] - st_b["sum_new"]) / KT
        ur1 = (st_c["sum_single_resident"] - st_b["sum_single_resident"]) / KT
        gone = (st_c["n_expired_total"] - st_b["n_expired_total"]) / KT
        alg_kernel, alg_total = algorithmic_bytes(n, cfg.n_bags, u, ur, ur1, unew, d, cfg.key_cells // S if S > 0 else 0,
                                                  prepared=args.prepare, expired=gone)
        per_kernel = {}
        for name, v in tim["kernels"].items():
            if v["launches"] and name in KERNEL_GROUP:
                per_kernel[name] = {"ms_per_launch": v["ms"] / v["launches"], "launches": v["launches"]}
        group_bytes, group_ms = {}, {}
        for name, v in per_kernel.items():
            g = KERNEL_GROUP[name]
            group_ms[g] = group_ms.get(g, 0.0) + v["ms_per_launch"]
            group_bytes[g] = group_bytes.get(g, 0) + alg_kernel[name]
        # the kernel that takes the most device time (reduce_adagrad_kernel is launched twice per step, for the
        # short segments and for the parts of the long ones: its time is the two launches together)
        if "reduce_parts" in per_kernel and "reduce_adagrad" in per_kernel:
            per_kernel["reduce_adagrad"]["ms_short_segments"] = per_kernel["reduce_adagrad"]["ms_per_launch"]
            per_kernel["reduce_adagrad"]["ms_parts"] = per_kernel["reduce_parts"]["ms_per_launch"]
            per_kernel["reduce_adagrad"]["ms_per_launch"] += per_kernel.pop("reduce_parts")["ms_per_launch"]
        dom = max(per_kernel, key=lambda k: per_kernel[k]["ms_per_launch"])
        dom_bytes, dom_ms = alg_kernel[dom], per_kernel[dom]["ms_per_launch"]
        achieved = dom_bytes / (dom_ms * 1e-3) / 1e9
        step_ms = ms_max / K
        line = {
            "metric": METRIC, "value": ids_all / (ms_max * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": W, "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
            "reps": {"n": R, "what": f"the timed region ({K} steps) repeated from the same restored state; value and "
                                     "ms_per_step are the median repetition (slowest rank)",
                     "ms_per_step_median": statistics.median(rep_ms) / K, "ms_per_step_min": min(rep_ms) / K,
                     "ms_per_step_max": max(rep_ms) / K, "ms_per_step_all_rank0": [round(x / K, 5) for x in rep_ms],
                     **({"note": reps_note} if reps_note else {})},
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {
                "workload": args.workload, "capacity": cfg.capacity, "dim": d, "key_cells": cfg.key_cells,
                "bags_per_step": cfg.n_bags, "ids_per_step": n, "unique_per_step": u,
                "unique_resident_per_step": ur, "unique_resident_once_per_step": ur1, "new_per_step": unew, "zipf_s": cfg.zipf_s,
                "id_universe": cfg.n_distinct, "filter_threshold": cfg.filter_threshold, "ttl": cfg.ttl,
                "prefill": "the state after ttl steps of the stream from an empty table (Poisson model)" if args.prefill else "empty table",
                "rows_resident_at_start": st0["n_resident"], "ids_tracked_at_start": st0["n_tracked"],
                "row_load": st0["n_resident"] / cfg.capacity, "key_load": st0["n_tracked"] / cfg.key_cells,
                "sweep": (f"every step sweeps 1/{S} of the key store (a full sweep every {S} steps)" if S > 0
                          else "none"), "l2": "every step reads a fresh batch larger than L2",
                "parallelism": f"{world} independent table(s), one per GPU",
                "filter": ({"kind": "count-min sketch", "depth": args.sketch_depth, "width": 1 << args.sketch_width_log2,
                            "sketch_bytes": 4 * args.sketch_depth << args.sketch_width_log2,
                            "key_store_bytes": 16 * cfg.key_cells, "key_store_bytes_exact_filter": 16 * base.key_cells,
                            "state": "sketch empty at the start (as after one of its clearings), rows pre-filled",
                            "admitted_per_step": (st_b["n_admitted_total"] - st_a["n_admitted_total"]) / K,
                            "entered_key_store_per_step": (st_b["n_inserted_total"] - st_a["n_inserted_total"]) / K}
                           if sketch else
                           {"kind": "exact per-ID counters in the key store", "key_store_bytes": 16 * cfg.key_cells,
                            "admitted_per_step": (st_b["n_admitted_total"] - st_a["n_admitted_total"]) / K,
                            "entered_key_store_per_step": (st_b["n_inserted_total"] - st_a["n_inserted_total"]) / K}),
                "push_prepared": ("mono_prepare_push before each lookup: the batch is grouped and every distinct ID "
                                  "looked up once, for the lookup and the push together" if args.prepare else "no"),
                "grouped_ahead": ("mono_group_ahead: each step groups the next step's batch by ID on a stream of its own, "
                                  "beside its own lookup and push" if args.prepare and args.group_ahead else "no"),
            },
            "bags_per_s": world * cfg.n_bags * K / (ms_max * 1e-3),
            "gpu_launches": launches,
            "clocks": clocks,
            "roofline": {
                "bound": "hbm", "kernel": dom + "_kernel",
                "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "peak_kind": f"of {peak_kind}", "algorithmic_bytes_per_launch": dom_bytes,
                "ms_per_launch": dom_ms,
                "traffic": recorded_traffic(dom, args.workload),
                **({"launches_per_step": 2,
                    "note": "this kernel runs twice per step (short segments, then the parts of long ones); bytes, "
                            "time and traffic are those of the two launches together"}
                   if dom == "reduce_adagrad" and "ms_parts" in per_kernel[dom] else {}),
            },
            "whole_step": {
                "algorithmic_bytes": alg_total, "achieved_gbs": alg_total / (step_ms * 1e-3) / 1e9,
                "frac_of_measured_peak": alg_total / (step_ms * 1e-3) / 1e9 / peak,
                "frac_of_8tbs": alg_total / (step_ms * 1e-3) / 1e9 / 8000.0,
                "bytes_by_kernel": alg_kernel,
                "frac_by_kernel": {k: round(alg_kernel[k] / (v["ms_per_launch"] * 1e-3) / 1e9 / peak, 3)
                                   for k, v in per_kernel.items()},
                "frac_by_phase": {g: round(group_bytes[g] / (group_ms[g] * 1e-3) / 1e9 / peak, 3) for g in group_ms},
                "ms_by_kernel": {k: round(v["ms_per_launch"], 4) for k, v in per_kernel.items()},
                "reduce_adagrad_ms": {"short_segments": per_kernel.get("reduce_adagrad", {}).get("ms_short_segments"),
                                      "parts": per_kernel.get("reduce_adagrad", {}).get("ms_parts")},
                "expire_ms_per_launch": (tim["kernels"]["expire"]["ms"] / tim["kernels"]["expire"]["launches"]
                                         if tim["kernels"]["expire"]["launches"] else None),
            },
            "table_after": {"n_tracked": st_end["n_tracked"], "n_resident": st_end["n_resident"],
                            "error_bits": st_end["error_bits"], "max_chain": st_end["max_chain"],
                            "evictions": st_end["n_evictions_total"], "stash_used": st_end["stash_used"]},
            "setup_s": round(setup_s, 1),
        }
        if drift:
            sec = ms_max * 1e-3
            line["drift"] = {
                "re_keyed": f"{cfg.drift_new_frac:.0%} of a batch's occurrences get new identities every {cfg.drift_period} steps",
                "inserts_per_s": (st_b["n_inserted_total"] - st_a["n_inserted_total"]) / sec,
                "admissions_per_s": (st_b["n_admitted_total"] - st_a["n_admitted_total"]) / sec,
                "expired_per_s": (st_b["n_expired_total"] - st_a["n_expired_total"]) / sec,
                "displacements_per_s": (st_b["n_evictions_total"] - st_a["n_evictions_total"]) / sec,
                "row_load_start": st_a["n_resident"] / cfg.capacity, "row_load_end": st_b["n_resident"] / cfg.capacity,
                "key_load_start": st_a["n_tracked"] / cfg.key_cells, "key_load_end": st_b["n_tracked"] / cfg.key_cells,
                "max_chain": st_b["max_chain"], "rows_refused": st_b["n_rows_refused"],
                "keys_dropped": st_b["n_keys_dropped"],
            }
        if e2e:
            line["e2e"] = {"value": e2e_ids_all / (e2e_ms_max * 1e-3), "unit": UNIT,
                           "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                           "ms_per_step": e2e_ms_max / E, "steps": E}
        if world == 1 and args.oracle_steps > 0:
            sample_bags = max(cfg.n_bags // args.oracle_fraction, 1)
            ids_s, _, ids_step = time_oracle(cfg, args.oracle_steps, 1, sample_bags, first_step=now0 + 1)
            line["cpu_baseline"] = {
                "value": ids_s, "unit": UNIT, "cores": 1, "kind": "oracle",
                "sample": (f"{args.oracle_steps} steps of the first {sample_bags} of {cfg.n_bags} bags "
                           f"(~{int(ids_step)} IDs each), lookup_pool + apply_grads, from an empty table; "
                           f"host has {os.cpu_count()} cores, the oracle uses one thread")}
        print(json.dumps(line), flush=True)
    table.close()
    if world > 1:
        dist.destroy_process_group()


def run_multi(args):
    """The mixed-dim multi-table configuration: 8 tables of one process on one stream, every
    step through the grouped calls (one kernel launch per step of the path for all eight
    tables).  A step = prepare + lookup_pool + apply_grads on every table, and one slice of the
    expiry sweep per table.  The same steps through the single-table calls, table after
    table, are timed beside it."""
    import torch
    from paper_2209_07663_b200 import binding as mb
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the table has no CPU path")
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dev = torch.device("cuda", local_rank)
    K, W, S = args.steps, args.warmup, args.sweep_slices
    base_cfgs = wl.many_small_table_configs() if args.workload == "multi_small" else wl.multi_table_configs()
    cfgs = [rank_config(c, rank) for c in base_cfgs]
    own_streams = args.multi_mode == "streams"
    streams = [torch.cuda.Stream(device=dev) for _ in cfgs] if own_streams else []
    tables, now0 = [], []
    for ti, cfg in enumerate(cfgs):
        t = mb.MonoTable(cfg.capacity, cfg.dim, cfg.filter_threshold, cfg.ttl, lr=cfg.lr, eps=cfg.eps,
                         init_acc=cfg.init_acc, init_scale=cfg.init_scale, seed=cfg.seed, key_cells=cfg.key_cells,
                         max_ids=int(cfg.n_bags * wl._mean_bag_len(cfg.bag_len) * 1.1), max_bags=cfg.n_bags,
                         **({"stream": streams[ti].cuda_stream} if own_streams else {}))
        n0 = cfg.ttl - 1
        for ids, cnt, seen in wl.steady_state_population_torch(cfg, n0, dev):
            res = (cnt >= cfg.filter_threshold).to(torch.uint8)
            torch.cuda.synchronize()
            mb.mono_import(t.handle, ids, cnt, seen, res, None, None, ids.numel())
            del ids, cnt, seen, res
        s0 = t.status()
        if s0["error_bits"]:
            raise SystemExit(f"pre-fill overflowed table {cfg.name}: {s0}")
        tables.append(t)
        now0.append(n0)

    n_batches = W + 2 * K
    jobs = [(ti, i) for ti in range(len(cfgs)) for i in range(n_batches)]
    gens = [wl.Stream(c) for c in cfgs]
    with concurrent.futures.ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1)) as pool:
        host = list(pool.map(lambda j: gens[j[0]].step(now0[j[0]] + 1 + j[1], with_grad=False), jobs))
    gg = torch.Generator(device=dev)
    gg.manual_seed(cfgs[0].seed)
    batches = [[None] * n_batches for _ in cfgs]
    outs = []
    for (ti, i), st in zip(jobs, host):
        cfg = cfgs[ti]
        batches[ti][i] = (torch.from_numpy(st.ids.view(np.int64)).to(dev), torch.from_numpy(st.offsets).to(dev),
                          torch.randn((cfg.n_bags, cfg.dim), device=dev, generator=gg).mul_(cfg.grad_std))
    for cfg in cfgs:
        outs.append(torch.empty((cfg.n_bags, cfg.dim), dtype=torch.float32, device=dev))
    torch.cuda.synchronize()

    handles = [t.handle for t in tables]
    gs = torch.cuda.current_stream().cuda_stream
    assert len(set(now0)) == 1

    def step(i, grouped):
        now = now0[0] + 1 + i
        if grouped:
            ids, off, grad = [b[i][0] for b in batches], [b[i][1] for b in batches], [b[i][2] for b in batches]
            if args.prepare:
                mb.mono_group_prepare_push(handles, ids, off, gs)
            mb.mono_group_lookup_pool(handles, ids, off, outs, gs)
            mb.mono_group_apply_grads(handles, ids, off, grad, now, gs)
        else:
            for ti, (cfg, t) in enumerate(zip(cfgs, tables)):
                ids, off, grad = batches[ti][i]
                if args.prepare:
                    mb.mono_prepare_push(t.handle, ids, ids.numel(), off, cfg.n_bags)
                mb.mono_lookup_pool(t.handle, ids, ids.numel(), off, cfg.n_bags, outs[ti])
                mb.mono_apply_grads(t.handle, ids, ids.numel(), off, cfg.n_bags, grad, now)
        if S > 0:
            for t in tables:
                mb.mono_expire_slice(t.handle, now, i % S, S)

    def timed(first, grouped):
        torch.cuda.synchronize()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for st in streams:
            st.wait_event(ev0)
        for i in range(first, first + K):
            step(i, grouped)
        for t in tables:
            mb.mono_fence(t.handle)
        for st in streams:                       # tables on streams of their own: the stop event waits for all of them
            done = torch.cuda.Event()
            done.record(st)
            torch.cuda.current_stream().wait_event(done)
        ev1.record()
        torch.cuda.synchronize()
        return ev0.elapsed_time(ev1)

    def launches_now():
        return sum(mb.mono_timing_read(t.handle, reset=True)["launches_total"] for t in tables)

    first_mode = not own_streams                 # grouped calls first, unless the tables sit on streams of their own
    for i in range(W):
        step(i, first_mode)
    before = [t.status() for t in tables]
    launches_now()
    sampler = ClockSampler(local_rank, gpu_uuid(local_rank))
    sampler.start()
    ms = timed(W, first_mode)
    clocks = sampler.stop()
    launches = launches_now()
    mid = [t.status() for t in tables]
    ms_serial = timed(W + K, False)
    launches_serial = launches_now()
    after = [t.status() for t in tables]
    n_ids = sum(b["sum_ids"] - a["sum_ids"] for a, b in zip(before, mid))
    n_ids_serial = sum(b["sum_ids"] - a["sum_ids"] for a, b in zip(mid, after))
    (ms_max,), (ids_all,) = aggregate_over_ranks([ms], [float(n_ids)], dev)
    alg = 0
    for cfg, a, b in zip(cfgs, before, mid):
        n = b["sum_ids"] - a["sum_ids"]
        u, ur = b["sum_unique"] - a["sum_unique"], b["sum_unique_resident"] - a["sum_unique_resident"]
        ur1, unew = b["sum_single_resident"] - a["sum_single_resident"], b["sum_new"] - a["sum_new"]
        alg += algorithmic_bytes(n, cfg.n_bags * K, u, ur, ur1, unew, cfg.dim, K * cfg.key_cells // S if S > 0 else 0,
                                 prepared=args.prepare, expired=b["n_expired_total"] - a["n_expired_total"])[1]
    if rank == 0:
        peak, peak_kind = measured_peaks()
        achieved = alg / (ms * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": ids_all / (ms_max * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": ms_max / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": args.workload, "calls": ("single-table calls, every table on a CUDA stream of its own"
                                                            if own_streams else "grouped calls, all tables on one stream"),
                       "tables": [{"name": c.name, "capacity": c.capacity, "dim": c.dim,
                                                         "slots": c.n_slots, "zipf_s": c.zipf_s,
                                                         "row_load": s0["n_resident"] / c.capacity,
                                                         "key_load": s0["n_tracked"] / c.key_cells}
                                                        for c, s0 in zip(cfgs, before)],
                       "examples_per_step": cfgs[0].n_examples, "slots_total": sum(c.n_slots for c in cfgs),
                       "ids_per_step": n_ids / K, "prefill": "the state after ttl steps of each stream from an empty table (Poisson model)",
                       "sweep": f"every step sweeps 1/{S} of every key store" if S > 0 else "none",
                       "l2": "every step reads fresh batches larger than L2",
                       "parallelism": (f"{len(cfgs)} tables of one process on one GPU; " +
                                       ("single-table calls on one stream per table" if own_streams else
                                        "grouped calls: one launch per kernel for all tables"))},
            "launches_per_step": launches / K,
            "one_table_at_a_time": {"value": n_ids_serial / (ms_serial * 1e-3), "ms_per_step": ms_serial / K,
                                    "launches_per_step": launches_serial / K,
                                    "what": "the same steps through the single-table calls, table after table"},
            "gpu_launches": launches, "clocks": clocks,
            "roofline": {"bound": "hbm", "kernel": "all kernels of the 8 tables (whole step)", "achieved": achieved,
                         "peak": peak, "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                         "traffic": None},
            "error_bits": [s["error_bits"] for s in after],
        }
        print(json.dumps(line), flush=True)
    for t in tables:
        t.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=32)
    ap.add_argument("--warmup", type=int, default=4)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="large", choices=sorted(wl.CONFIGS) + ["multi", "multi_small"])
    ap.add_argument("--multi-mode", default="grouped", choices=["grouped", "streams"],
                    help="multi-table workloads: grouped calls on one stream (then, for comparison, the single-table "
                         "calls table after table), or single-table calls with every table on a stream of its own")
    ap.add_argument("--no-prepare", dest="prepare", action="store_false",
                    help="do not announce each batch with mono_prepare_push before its lookup")
    ap.add_argument("--stream-priority", default="default", choices=["default", "high"],
                    help="priority of the CUDA stream the table is created on (its internal streams have the lowest)")
    ap.add_argument("--no-group-ahead", dest="group_ahead", action="store_false",
                    help="do not group the next step's batch with mono_group_ahead beside the current step")
    ap.add_argument("--sweep-slices", type=int, default=32,
                    help="every step sweeps 1/S of the key store for expired IDs (0 = no sweep)")
    ap.add_argument("--filter", default="exact", choices=["exact", "sketch"],
                    help="admission filter: exact per-ID counters (default) or the count-min sketch")
    ap.add_argument("--sketch-depth", type=int, default=4)
    ap.add_argument("--sketch-width-log2", type=int, default=28, help="counters per sketch row = 2^this")
    ap.add_argument("--sketch-key-shrink-log2", type=int, default=3,
                    help="with --filter sketch the key store has 2^-this of the configured cells")
    ap.add_argument("--reps", type=int, default=5,
                    help="repetitions of the timed region, each from the same restored state (median reported)")
    ap.add_argument("--e2e-steps", type=int, default=6)
    ap.add_argument("--kernel-steps", type=int, default=8, help="steps of the per-kernel CUDA-event pass")
    ap.add_argument("--no-prefill", dest="prefill", action="store_false")
    ap.add_argument("--oracle-steps", type=int, default=4)
    ap.add_argument("--oracle-fraction", type=int, default=8, help="the oracle runs on 1/this of each step's bags")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        if args.workload in ("multi", "multi_small"):
            args.workload = "large"
        run_reference(args)
    elif args.workload in ("multi", "multi_small"):
        run_multi(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
