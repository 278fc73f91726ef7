"""Host-side pieces of the benchmark that need no GPU: the clock sampler (against a stand-in
for the NVML module) and the per-step byte count."""
import sys
import time
import types

import bench


def _fake_nvml(clocks, reason_bits):
    m = types.ModuleType("pynvml")
    m.NVML_CLOCK_SM = 1
    m.nvmlClocksEventReasonHwSlowdown = 0x8
    m.nvmlClocksEventReasonSwPowerCap = 0x4
    m.nvmlClocksEventReasonSwThermalSlowdown = 0x20
    m.nvmlClocksEventReasonHwThermalSlowdown = 0x40
    state = {"i": 0, "init": 0}
    m.nvmlInit = lambda: state.__setitem__("init", state["init"] + 1)
    m.nvmlShutdown = lambda: state.__setitem__("init", state["init"] - 1)
    m.nvmlDeviceGetHandleByUUID = lambda u: ("by-uuid", u)
    m.nvmlDeviceGetHandleByIndex = lambda i: ("by-index", i)
    m.nvmlDeviceGetMaxClockInfo = lambda h, which: 1965

    def clock(h, which):
        state["i"] += 1
        return clocks[state["i"] % len(clocks)]
    m.nvmlDeviceGetClockInfo = clock
    m.nvmlDeviceGetCurrentClocksEventReasons = lambda h: reason_bits
    m.nvmlDeviceGetPowerUsage = lambda h: 500_000
    m._state = state
    return m


def test_clock_sampler_reads_clocks_and_reasons_through_nvml(monkeypatch):
    fake = _fake_nvml([1900, 1950, 1965], reason_bits=0x4)
    monkeypatch.setitem(sys.modules, "pynvml", fake)
    s = bench.ClockSampler(0, "0123")
    s.start()
    time.sleep(0.05)
    out = s.stop()
    assert out["source"] == "nvml" and out["samples"] >= 3
    assert out["sm_max_mhz"] == 1965.0 and 1900.0 <= out["sm_mhz"] <= 1965.0 and out["sm_min_mhz"] == 1900.0
    assert out["reasons"] == ["sw_power_cap"]          # kept and noted; the slowdown reasons are absent
    assert out["power_w_max"] == 500.0
    assert fake._state["init"] == 0                     # initialised once, shut down once


def test_clock_sampler_reports_slowdowns(monkeypatch):
    monkeypatch.setitem(sys.modules, "pynvml", _fake_nvml([1200], reason_bits=0x8 | 0x40))
    s = bench.ClockSampler(0)
    s.start()
    time.sleep(0.02)
    out = s.stop()
    assert out["reasons"] == ["hw_slowdown", "hw_thermal_slowdown"] and out["sm_mhz"] == 1200.0


def test_algorithmic_bytes_adds_up():
    n, b, u, ur, ur1, unew, d = 1000, 600, 400, 300, 250, 50, 64
    per, total = bench.algorithmic_bytes(n, b, u, ur, ur1, unew, d, sweep_cells=1 << 10, expired=7)
    assert total == sum(per.values())
    assert per["dedup_tile"] == 32 * n and per["table_lookup"] == 32 * u and per["table_update"] == 64 * u
    assert per["gather_pool"] == 8 * (b + 1) + 8 * n + 4 * d * ur + 4 * d * b
    # a batch that was not announced pays one key-store sector per occurrence inside the lookup instead
    per_u, total_u = bench.algorithmic_bytes(n, b, u, ur, ur1, unew, d, sweep_cells=1 << 10, prepared=False, expired=7)
    assert per_u["table_lookup"] == 0 and per_u["gather_pool"] == per["gather_pool"] + 32 * n
    assert total_u - total == 32 * n - 32 * u
    # the Adagrad phase reads every gradient row once and reads and writes row + accumulator of every ID with a row
    assert per["update_singletons"] + per["reduce_adagrad"] == 16 * d * ur + 4 * d * b
    assert per["expire"] == 4 * (1 << 8) + 7 * (64 + 32)      # a record per 4-cell bucket, a bucket and a cell per removed entry
    assert set(bench.KERNEL_GROUP) <= set(per) | {"finish_apply"}
