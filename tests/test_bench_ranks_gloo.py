"""bench.py's multi-rank flow on the CPU: two gloo ranks run `bench.run_ours` end to end -- the rank layout, the timed
loop (the product's `sharded.run_steps`), the exchange at every round end, the max-over-ranks reduction of the device
times, the end-to-end leg and the rule that only rank 0 reports -- with stand-ins for what needs a GPU: the context
(an engine that records the calls it gets), device events (a counter) and the clock sampler.  The round lengths come
from the library's host schedule, as in the real run."""
import argparse
import json
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2310_14423_b200 import binding as B          # noqa: E402
from paper_2310_14423_b200 import workloads as W        # noqa: E402


class CountingEvent:
    """A device event whose clock is the number of events recorded so far on this rank, times (rank + 1) ms: rank r
    'measures' every span (r + 1) times longer than rank 0, so the slowest rank is known exactly."""
    seq = 0

    def __init__(self, rank):
        self.rank, self.at = rank, None

    def record(self):
        CountingEvent.seq += 1
        self.at = CountingEvent.seq

    def elapsed_time(self, later):
        return float(later.at - self.at) * (self.rank + 1)


class RecordingEngine:
    """The methods of binding.Context that the benchmark calls; every call is logged."""

    def __init__(self, cfg, theta, log, rank, world):
        self.cfg, self.theta, self.log, self.rank, self.world = cfg, theta, log, rank, world
        self.launches = 0
        log.append(("init", int(cfg.K), int(cfg.worker_offset), int(cfg.P)))

    def qsr_round_length(self, t):
        return B.qsr_config_round_length(self.cfg, t)

    def qsr_sync_sum_floats(self):
        return (int(self.cfg.P) + 3) // 4 * 4

    def qsr_launch_count(self):
        return self.launches

    def qsr_set_params(self, theta0):
        self.log.append(("set_params",))

    def qsr_local_step(self, t):
        self.launches += 1
        self.log.append(("step", t))

    def qsr_sync_partial(self, sums):
        self.launches += 1
        sums.fill_(float(self.rank + 1))
        self.log.append(("partial",))

    def qsr_local_step_partial(self, t, sums):
        self.launches += 1
        sums.fill_(float(self.rank + 1))
        self.log.append(("step_partial", t))

    def qsr_sync_finish(self, sums, K_total, t_next):
        self.launches += 1
        # the buffer was summed over ranks in between: 1 + 2 + ... + world
        assert float(sums.min()) == float(sums.max()) == self.world * (self.world + 1) / 2
        self.log.append(("finish", int(K_total), t_next))

    def qsr_sync(self, t_next):
        raise AssertionError("the single-GPU synchronization must not run when the workers are sharded")

    qsr_local_step_sync = qsr_sync

    def close(self):
        pass


class FakeBackend:
    name = "fake"

    def __init__(self, rank, world, port, log):
        self.torch, self.rank, self.world, self.port, self.log = torch, rank, world, port, log

    def init_process_group(self):
        os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(self.port))
        dist.init_process_group("gloo", rank=self.rank, world_size=self.world)

    def zeros(self, *shape):
        return torch.zeros(*shape)

    def pinned(self, array=None, n=None):
        return torch.from_numpy(array) if array is not None else torch.zeros(n)

    def context(self, cfg, theta, s1, s2, lam, ths):
        return RecordingEngine(cfg, theta, self.log, self.rank, self.world)

    def train_host(self, *a, **k):
        raise AssertionError("qsr_train_host is the single-GPU end-to-end call")

    def event(self):
        return CountingEvent(self.rank)

    def synchronize(self):
        pass

    def release_cached_memory(self):
        pass

    def clock_sampler(self):
        class _Sampler:
            def stop(self, t0, t1):
                assert t1 >= t0
                return {"sm_mhz": 1500.0, "sm_max_mhz": 1965.0, "reasons": [], "samples": 3}
        return _Sampler()


def _rank_main(rank, world, port, steps, out_dir):
    import bench
    log = []
    args = argparse.Namespace(gpus=world, steps=steps, warmup=3, impl="ours", workload="c1", no_cpu_baseline=False,
                              no_e2e=False, packed_rows=False, sharded_path=False)
    try:
        out = bench.run_ours(args, FakeBackend(rank, world, port, log))
    finally:
        if dist.is_initialized():
            dist.destroy_process_group()
    with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
        json.dump({"out": out, "log": log}, f)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_rank_layout_is_weak_scaling():
    import bench
    base = W.workload("c4")
    for world in (1, 2, 8):
        for rank in range(world):
            assert bench.rank_layout(base, world, rank) == (16, 16 * world, 16 * rank)


def test_two_ranks_run_the_whole_benchmark_flow(tmp_path):
    world, steps = 2, 42
    mp.spawn(_rank_main, args=(world, _free_port(), steps, str(tmp_path)), nprocs=world, join=True)
    res = [json.load(open(tmp_path / f"rank{r}.json")) for r in range(world)]
    base = W.workload("c1")
    assert res[1]["out"] is None                                   # only rank 0 reports
    out = res[0]["out"]
    assert out["n_gpus"] == 2 and out["scaling"] == "weak" and out["steps"] == steps
    assert out["config"]["K_per_gpu"] == base.K and out["config"]["K_total"] == 2 * base.K
    assert out["config"]["parallelism"] == "replica-sharded dp2"
    # times: rank 1's events run twice as slow, and the job is as fast as its slowest rank
    assert out["ms_per_step"] == pytest.approx(2.0)
    assert out["value"] == pytest.approx(2 * base.K * base.P * steps / (2.0 * steps * 1e-3))
    assert out["e2e"]["api"] == "sharded.run_steps"
    assert out["e2e"]["value"] == pytest.approx(2 * base.K * base.P * out["e2e"]["steps"] / 2e-3)
    assert "cpu_baseline" not in out                               # a one-GPU leg only
    assert out["clocks"]["samples"] == 3 and out["sm_mhz_x_ms_per_step"] == pytest.approx(3000.0)
    # what each rank's engine was asked to do
    st, H = B.qsr_config_schedule(B.make_config(base))
    ends = (st + H).tolist()
    for r in range(world):
        log = [tuple(x) for x in res[r]["log"]]
        inits = [x for x in log if x[0] == "init"]
        assert inits and all(x == ("init", base.K, r * base.K, base.P) for x in inits)
        # the timed window is what follows the second init (the first context ran the warm-up)
        second = [i for i, x in enumerate(log) if x[0] == "init"][1]
        third = [i for i, x in enumerate(log) if x[0] == "init"][2]
        window = log[second + 1:third]
        expect = []
        for t in range(steps):
            if t + 1 in ends:
                expect += [("step_partial", t), ("finish", 2 * base.K, t + 1)]
            else:
                expect.append(("step", t))
        assert window == expect
        # the end-to-end leg runs whole rounds through the same loop and ends on a round end
        tail = log[third + 1:]
        assert tail[0] == ("set_params",) and tail[-1][0] == "finish" and tail[-1][2] == out["e2e"]["steps"]
        assert out["e2e"]["steps"] in ends and out["e2e"]["steps"] >= steps
    assert out["gpu_launches"] == steps + sum(1 for t in range(steps) if t + 1 in ends)
    assert out["config"]["syncs_in_window"] == sum(1 for t in range(steps) if t + 1 in ends)
