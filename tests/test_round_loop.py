"""The round loop (`sharded.run_steps`) and the clock-sample filter of bench.py, on the CPU with a recording engine.

run_steps is the one sequencing of Algorithm 2's rounds in the product: per round H - 1 plain local steps, then the
step that ends the round (one fused launch on one GPU; partial sums, all-reduce, finish when sharded).  The benchmark
times it and the multi-process tests drive it, so its window rules are pinned here against the host schedule."""
import datetime
import os
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2310_14423_b200 import binding as B
from paper_2310_14423_b200 import sharded
from paper_2310_14423_b200 import workloads as W


class Recorder:
    def __init__(self, cfg):
        self.cfg, self.calls = cfg, []

    def qsr_round_length(self, t):
        return B.qsr_config_round_length(self.cfg, t)

    def qsr_local_step(self, t):
        self.calls.append(("step", t))

    def qsr_local_step_sync(self, t, t_next):
        self.calls.append(("step+mean", t, t_next))

    def qsr_local_step_partial(self, t, sums):
        self.calls.append(("step+sums", t))

    def qsr_sync_finish(self, sums, K_total, t_next):
        self.calls.append(("finish", K_total, t_next))


@pytest.mark.parametrize("name", ["c1", "c4p"])
@pytest.mark.parametrize("t_end", [1, 3, 4, 5, 37, 424, 425, 1000])
def test_window_of_steps_on_one_gpu(name, t_end):
    w = W.workload(name)
    cfg = B.make_config(w)
    st, H = B.qsr_config_schedule(cfg)
    ends = set((st + H).tolist())
    eng = Recorder(cfg)
    seen = []
    rounds = sharded.run_steps(eng, 0, t_end, None, lambda kind, t: seen.append((kind, t)))
    expect = [("step+mean", t, t + 1) if t + 1 in ends else ("step", t) for t in range(t_end)]
    assert eng.calls == expect
    assert seen == [("sync" if t + 1 in ends else "step", t) for t in range(t_end)]
    done = [(int(a), int(b)) for a, b in zip(st, H) if a + b <= t_end]
    assert rounds == done


def test_whole_rounds_run_past_the_window_and_resume_where_they_ended():
    w = W.workload("c1")
    cfg = B.make_config(w)
    st, H = B.qsr_config_schedule(cfg)
    eng = Recorder(cfg)
    all_reduced = []
    ex = sharded.Exchange("buffer", 12, all_reduced.append)
    first = sharded.run_steps(eng, 0, 425, ex, whole_rounds=True)          # 424 starts a round of 5: run to 429
    t_mid = first[-1][0] + first[-1][1]
    assert t_mid == 429 and first[-1] == (424, 5)
    rest = sharded.run_steps(eng, t_mid, w.T, ex, whole_rounds=True)
    assert [r[0] for r in first + rest] == st.tolist() and [r[1] for r in first + rest] == H.tolist()
    assert sharded.run_rounds(Recorder(cfg), "buffer", 12, 0, w.T, lambda b: None) == first + rest
    steps = [c for c in eng.calls if c[0] in ("step", "step+sums")]
    assert [c[1] for c in steps] == list(range(w.T))                        # every step exactly once, in order
    finishes = [c for c in eng.calls if c[0] == "finish"]
    assert [c[2] for c in finishes] == (st + H).tolist() and all(c[1] == 12 for c in finishes)
    assert all_reduced == ["buffer"] * len(st)                              # one exchange per round
    # a finish directly follows its step+sums
    for i, c in enumerate(eng.calls):
        if c[0] == "step+sums":
            assert eng.calls[i + 1][0] == "finish" and eng.calls[i + 1][2] == c[1] + 1


def test_shard_rejects_more_ranks_than_workers():
    with pytest.raises(ValueError):
        sharded.shard(3, 4, 0)
    with pytest.raises(ValueError):
        sharded.shard(8, 2, 2)


def test_clock_samples_are_filtered_by_their_time_stamps():
    import bench
    t0 = datetime.datetime(2025, 3, 1, 12, 0, 0).timestamp()

    def line(dt, sm, power, cap):
        stamp = datetime.datetime.fromtimestamp(t0 + dt).strftime("%Y/%m/%d %H:%M:%S.%f")[:-3]
        return f"{stamp}, {sm}, 1965, {power}, 0x0000000000000004, Not Active, Not Active, Not Active, {cap}\n"

    lines = [line(-0.20, 1965, 250.0, "Not Active"), line(0.02, 1700, 900.0, "Active"), line(0.07, 1500, 995.0, "Active"),
             line(0.12, 1480, 996.0, "Active"), line(0.30, 1965, 300.0, "Not Active"), "garbage\n", ""]
    rows = bench.ClockSampler.parse(lines, t0, t0 + 0.15)
    assert [r[0] for r in rows] == [1700.0, 1500.0, 1480.0]
    assert all(r[3] == {"sw_power_cap"} for r in rows)
    assert len(bench.ClockSampler.parse(lines)) == 5
    assert bench.ClockSampler.parse(lines, t0 + 0.2, t0 + 0.25) == []
    near = bench.ClockSampler.parse(lines, t0 + 0.2, t0 + 0.25, slack_s=0.06)
    assert [r[0] for r in near] == [1965.0]


def test_nvml_sampler_keeps_the_readings_inside_the_region(monkeypatch):
    """The in-process clock sampler against a stand-in for the NVML binding: readings every few milliseconds, only
    those stamped inside the timed region are kept, reasons come from the bit mask, and a region shorter than the
    period takes the nearest reading."""
    import time
    import types
    import bench
    calls = {"n": 0}
    fake = types.ModuleType("pynvml")
    fake.NVML_CLOCK_SM = 1
    fake.nvmlClocksEventReasonHwSlowdown, fake.nvmlClocksEventReasonHwThermalSlowdown = 0x8, 0x40
    fake.nvmlClocksEventReasonSwThermalSlowdown, fake.nvmlClocksEventReasonSwPowerCap = 0x20, 0x4
    fake.nvmlInit = lambda: None
    fake.nvmlShutdown = lambda: None
    fake.nvmlDeviceGetHandleByUUID = lambda uuid: ("handle", uuid)
    fake.nvmlDeviceGetMaxClockInfo = lambda h, which: 1965

    def clock(h, which):
        calls["n"] += 1
        return 1500 if calls["n"] > 3 else 1965

    fake.nvmlDeviceGetClockInfo = clock
    fake.nvmlDeviceGetPowerUsage = lambda h: 990000
    fake.nvmlDeviceGetCurrentClocksEventReasons = lambda h: 0x4 if calls["n"] > 3 else 0x1
    monkeypatch.setitem(sys.modules, "pynvml", fake)
    s = bench.NvmlSampler("GPU-00000000-0000-0000-0000-000000000000")
    time.sleep(0.03)
    t0 = time.time()
    time.sleep(0.08)
    t1 = time.time()
    time.sleep(0.02)
    out = s.stop(t0, t1)
    assert out["source"] == "nvml" and out["sm_max_mhz"] == 1965.0
    assert 3 <= out["samples"] <= 20 and out["sm_mhz"] == 1500.0 and out["reasons"] == ["sw_power_cap"]
    assert out["power_w_median"] == 990.0
    # a region between two readings
    s = bench.NvmlSampler("GPU-00000000-0000-0000-0000-000000000000")
    time.sleep(0.03)
    t0 = time.time()
    out = s.stop(t0, t0 + 1e-4)
    assert out["samples"] == 1 and "note" in out
