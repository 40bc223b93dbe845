#!/usr/bin/env python
"""Throughput of the Local-OPT / QSR hot path on B200, with its roofline and a CPU-oracle baseline.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload c4]

A "step" is one global iteration of Algorithm 2 over all workers: one fused local-step launch (every worker takes
its optimizer step on a gradient generated in registers), plus the replica-averaging launch wherever the Quadratic
Synchronization Rule ends a round inside the timed window.  The default workload is the ViT-B/16-shaped run
(16 workers per GPU, 86,415,592 parameters each, Local AdamW, warm-up 100 + cosine, alpha = 0.0175, H_base = 4);
the timed window covers global steps [0, K) of its 10,000-step schedule.

metric  replica param-updates per second = (workers x parameters x steps) / time, whole job, inputs resident in HBM.
e2e     the same through qsr_train_host: host buffers in, host buffer out, copies inside the timed region.
With N > 1 (torchrun, one rank per GPU) the workers are sharded over ranks (16 per GPU, weak scaling); a round ends
with its last step fused with the rank's row sums, one NCCL all-reduce of P floats and a finish kernel.  On one GPU
a round's last step carries the averaging itself (one launch, no extra HBM traffic).

`--impl reference` times the CPU oracle (test infrastructure; plain C, binary64) on the host cores instead.
"""
from __future__ import annotations

import argparse
import datetime
import hashlib
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "replica_param_updates_per_s"
UNIT = "param-updates/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
L2_BYTES = 126e6

# DRAM traffic of the dominant kernel from an ncu capture (dram__bytes_read.sum + dram__bytes_write.sum per launch,
# taken on the 2^23-parameter variants c4s / c3s and stated per element-update: the kernel streams every element
# once, so traffic grows in proportion to K*P).  Valid only for the kernel source it was taken from: the hash covers
# the noise generator, the optimizer update and local_step_kernel in csrc/kernels.cu.
NCU_TRAFFIC = {
    "step_source_sha256": "35dba2222a898a7788bd1c2f05f600bec42d82d5b343b3587c17e1079241782c",
    "bytes_per_update": {"adamw": 24.07, "sgdm": 16.07},
}

# Thread-instructions per element-update of resident_steps_kernel's step loop (ncu smsp__thread_inst_executed.sum of
# one launch / (K * P * steps in the launch), captured on c2 and c1): the "algorithmic work" of the ALU roofline, which
# is a bound on instruction issue.  The kernel uses packed fp32 instructions (two operations per lane each);
# "scalar_equivalent" is the count of the same arithmetic issued one operation per instruction.
NCU_RESIDENT_INSTR = {"source_sha256": "dbf5f9d72f3533f877a85fdd47f30eaa4c90e7f0f96090100f4c950e8d5f81a1", "adamw": 39.75, "sgdm": 40.73,
                      "scalar_equivalent": {"adamw": 51.50, "sgdm": 49.24}}
SM_COUNT, LANES_PER_SM_CLK = 148, 4 * 32      # 4 schedulers per SM, one warp instruction (32 lanes) each per clock


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="c4")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--packed-rows", action="store_true",
                    help="rows packed at P (rounded up to 4) instead of the stride qsr_row_stride_hint recommends")
    ap.add_argument("--resident-steps", type=int, default=0,
                    help="BENCHMARK-ONLY: up to N (<= 128) consecutive steps per launch with parameters and state held in "
                         "registers (possible only with the in-kernel synthetic gradient); one GPU; the roofline is ALU")
    ap.add_argument("--sharded-path", action="store_true",
                    help="on one GPU, still end rounds the multi-GPU way (partial sums, all-reduce of one rank, finish)")
    return ap.parse_args()


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def source_region_hash(begin: str, end: str):
    """sha256 of csrc/kernels.cu between two of its section markers (None if either is gone)."""
    with open(os.path.join(ROOT, "paper_2310_14423_b200", "csrc", "kernels.cu")) as f:
        text = f.read()
    bar = "// " + "-" * 94 + " "
    try:
        region = text[text.index(bar + begin if begin else ""):text.index(end)]
    except ValueError:
        return None
    return hashlib.sha256(region.encode()).hexdigest()


def step_source_hash():
    return source_region_hash("noise", "// Sum over rows of one 16-byte column")


def resident_source_hash():
    a = source_region_hash("noise", "// Weight-decay scalar for the column")
    b = source_region_hash("resident steps", "// " + "-" * 94 + " test hook")
    return None if a is None or b is None else hashlib.sha256((a + b).encode()).hexdigest()


class ClockSampler:
    """nvidia-smi clock / throttle samples of one GPU every 50 ms, each with its time stamp.  It is started before the
    warm-up launches (the tool needs a few hundred ms to come up) and `stop(t0, t1)` keeps the samples taken between
    the host times t0 and t1 that bracket the timed region, so that even a window of a tenth of a second carries
    readings taken under its own load."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    PERIOD_MS = 50

    def __init__(self, gpu_id: str):
        self.gpu_id = gpu_id
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", gpu_id, f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", str(self.PERIOD_MS)],
                                         stdout=self.tmp, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    @staticmethod
    def parse(lines, t0=None, t1=None, slack_s=0.0):
        """[(sm, sm_max, power, reasons)] of the samples stamped within [t0 - slack, t1 + slack] (all if t0 is None)."""
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        out = []
        for line in lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                stamp = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                sm, smax, power = float(parts[1]), float(parts[2]), float(parts[3])
            except ValueError:
                continue
            if t0 is not None and not (t0 - slack_s <= stamp <= t1 + slack_s):
                continue
            out.append((sm, smax, power, {n for n, v in zip(names, parts[5:9]) if v.lower().startswith("active")}))
        return out

    def stop(self, t0: float, t1: float):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "source": "nvidia-smi",
               "period_ms": self.PERIOD_MS}
        if self.proc is None:
            return out
        time.sleep(2e-3 * self.PERIOD_MS)          # let the sample that covers the end of the region be written
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        lines = self.tmp.readlines()
        self.tmp.close()
        os.unlink(self.tmp.name)
        rows = self.parse(lines, t0, t1)
        if not rows:
            # a region shorter than the sampling period can fall between two samples: take its nearest neighbours
            rows = self.parse(lines, t0, t1, slack_s=1e-3 * self.PERIOD_MS)
            if rows:
                out["note"] = f"the timed region fell between two samples; these are the ones within {self.PERIOD_MS} ms of it"
        if rows:
            reasons = set().union(*[r[3] for r in rows])
            out.update(sm_mhz=float(np.median([r[0] for r in rows])), sm_max_mhz=float(max(r[1] for r in rows)),
                       reasons=sorted(reasons), samples=len(rows), power_w_median=float(np.median([r[2] for r in rows])))
        return out


class NvmlSampler:
    """The same record from NVML inside this process: a thread reads the SM clock, the power draw and the clock event
    reasons every few milliseconds (read-only queries).  The timed loop only enqueues kernels and then waits in
    cudaDeviceSynchronize with the interpreter lock released, so the thread runs freely and even the 0.1 s of a
    20-step window gets a dozen readings taken under its own load.  `stop(t0, t1)` keeps those stamped inside the
    region.  Raises if NVML cannot be used; the caller then falls back to the nvidia-smi sampler."""
    PERIOD_S = 0.005

    def __init__(self, gpu_uuid: str):
        import threading
        import pynvml
        self.nv = pynvml
        pynvml.nvmlInit()
        self.h = pynvml.nvmlDeviceGetHandleByUUID(gpu_uuid.encode() if hasattr(gpu_uuid, "encode") else gpu_uuid)
        self.sm_max = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        self.rows = []
        self.halt = threading.Event()
        self._read()                                  # fail here, not in the thread, if a query is unsupported
        self.thread = threading.Thread(target=self._loop, daemon=True)
        self.thread.start()

    def _read(self):
        nv = self.nv
        mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
        names = {"hw_slowdown": nv.nvmlClocksEventReasonHwSlowdown,
                 "hw_thermal_slowdown": nv.nvmlClocksEventReasonHwThermalSlowdown,
                 "sw_thermal_slowdown": nv.nvmlClocksEventReasonSwThermalSlowdown,
                 "sw_power_cap": nv.nvmlClocksEventReasonSwPowerCap}
        return (time.time(), float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)),
                float(nv.nvmlDeviceGetPowerUsage(self.h)) / 1e3, {n for n, bit in names.items() if mask & bit})

    def _loop(self):
        while not self.halt.is_set():
            try:
                self.rows.append(self._read())
            except Exception:
                break
            self.halt.wait(self.PERIOD_S)

    def stop(self, t0: float, t1: float):
        self.halt.set()
        self.thread.join(timeout=2)
        out = {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": [], "samples": 0, "source": "nvml",
               "period_ms": 1e3 * self.PERIOD_S}
        rows = [r for r in self.rows if t0 <= r[0] <= t1]
        if not rows and self.rows:
            # a region shorter than the period can fall between two readings: take the nearest one
            nearest = min(self.rows, key=lambda r: min(abs(r[0] - t0), abs(r[0] - t1)))
            if min(abs(nearest[0] - t0), abs(nearest[0] - t1)) <= 4 * self.PERIOD_S:
                rows = [nearest]
                out["note"] = "the timed region fell between two readings; this is the nearest one"
        if rows:
            out.update(sm_mhz=float(np.median([r[1] for r in rows])), reasons=sorted(set().union(*[r[3] for r in rows])),
                       samples=len(rows), power_w_median=float(np.median([r[2] for r in rows])))
        try:
            self.nv.nvmlShutdown()
        except Exception:
            pass
        return out


def step_bytes_per_update(w) -> float:
    """Algorithmic HBM bytes per element-update of the fused step with the gradient generated in the kernel:
    read + write of theta and each state slab, plus lambda and theta* once per column of K workers."""
    n_slabs = 3 if w.opt == "adamw" else 2
    return n_slabs * 8.0 + 8.0 / w.K


def oracle_sample(w, n_coords, first_step, count):
    """Times the CPU oracle on `count` steps of the schedule (with its syncs) over a coordinate sample."""
    from oracle import qsr_oracle as O
    from paper_2310_14423_b200 import workloads as W
    idx = W.coordinate_subset(w.layout, n_coords, seed=1)
    lam, ths = W.draw_inputs_at(w.P, w.data_seed, idx)
    S = O.State(w, lam, ths, idx=idx)
    starts, H = O.schedule(w)
    ends = set((starts + H).tolist())

    def steps(t0, n):
        for t in range(t0, t0 + n):
            S.local_step(t)
            if t + 1 in ends:
                S.sync(t + 1)

    steps(0, first_step)
    if callable(count):
        t0 = time.perf_counter()
        steps(first_step, 5)
        count = count((time.perf_counter() - t0) / 5)
        first_step += 5
    t0 = time.perf_counter()
    steps(first_step, count)
    dt = time.perf_counter() - t0
    return w.K * idx.size * count / dt, idx.size, count, dt


def run_reference(args):
    """The CPU oracle as it stands, timed on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from paper_2310_14423_b200 import workloads as W
    w = W.workload(args.workload)
    value, n, count, dt = oracle_sample(w, 32768, args.warmup, args.steps)
    sample = (f"{n} of {w.P} coordinates x {w.K} workers x {count} steps of the {w.name} schedule, "
              f"binary64, OpenMP over coordinates")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / count, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{w.name}: K={w.K}, P={w.P}, {w.opt}, sampled coordinates"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def cpu_baseline(w, budget_s=12.0):
    value, n, count, dt = oracle_sample(
        w, 16384, 3, lambda per_step: int(max(10, min(w.T - 10, budget_s / max(per_step, 1e-6)))))
    return {"value": value, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
            "sample": f"{n} of {w.P} coordinates x {w.K} workers x {count} steps (with the schedule's syncs), "
                      f"binary64, {dt:.1f} s"}


class CudaBackend:
    """Everything of the measurement that touches a device, a stream or the process group.  The timed loop, the rank
    bookkeeping and the JSON line are written against this small surface, so that the CPU tests can run the whole
    multi-rank flow over gloo with stand-ins for the device parts."""
    name = "cuda"

    def __init__(self, rank: int, local_rank: int, world: int):
        import torch
        self.torch = torch
        self.rank, self.world = rank, world
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
        torch.cuda.set_device(local_rank)
        self.local_rank = local_rank
        self.dev = torch.device("cuda", local_rank)

    def init_process_group(self):
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=self.dev)

    def zeros(self, *shape):
        return self.torch.zeros(*shape, device=self.dev)

    def empty_bytes(self, n):
        return self.torch.empty(n, dtype=self.torch.uint8, device=self.dev)

    def pinned(self, array=None, n=None):
        t = self.torch.from_numpy(array) if array is not None else self.torch.zeros(n, dtype=self.torch.float32)
        return t.pin_memory()

    def stream(self) -> int:
        return self.torch.cuda.current_stream().cuda_stream

    def context(self, cfg, theta, s1, s2, lam, ths):
        from paper_2310_14423_b200 import binding as B
        return B.Context(cfg, theta, s1, s2, lam, ths, stream=self.stream())

    def train_host(self, cfg, theta0, lam, ths, out, ws, t_end):
        from paper_2310_14423_b200 import binding as B
        return B.qsr_train_host(cfg, theta0, lam, ths, out, ws, t_end=t_end, stream=self.stream())

    def event(self):
        return self.torch.cuda.Event(enable_timing=True)

    def synchronize(self):
        self.torch.cuda.synchronize()

    def release_cached_memory(self):
        self.torch.cuda.empty_cache()

    def clock_sampler(self):
        uuid = "GPU-" + str(self.torch.cuda.get_device_properties(self.local_rank).uuid).replace("GPU-", "")
        try:
            return NvmlSampler(uuid)
        except Exception:
            return ClockSampler(uuid)


def rank_layout(base, world: int, rank: int):
    """(workers held by this rank, workers in the whole job, global index of this rank's first worker): weak scaling,
    every GPU holds the configuration's K workers, rank r the workers r*K .. r*K + K - 1."""
    return base.K, base.K * world, rank * base.K


def max_over_ranks(ms: float, backend) -> float:
    """A time measured on each rank's own device -> the slowest rank's (the job is as fast as that)."""
    if backend.world == 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = backend.zeros(1).double()
    t += ms
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def run_ours(args, backend):
    """The measurement on this rank.  Returns the result (a dict) on rank 0 and None elsewhere."""
    import torch.distributed as dist
    from paper_2310_14423_b200 import binding as B
    from paper_2310_14423_b200 import sharded
    from paper_2310_14423_b200 import workloads as W

    B.lib()  # fail loudly if the CUDA library is missing
    world, rank = backend.world, backend.rank
    if world > 1:
        backend.init_process_group()

    base = W.workload(args.workload)
    K_local, K_total, worker_offset = rank_layout(base, world, rank)
    w = base.replace(worker_offset=worker_offset)
    steps, warmup = args.steps, max(args.warmup, 3)
    if steps > w.T:
        raise SystemExit(f"--steps must be <= {w.T}")

    lam_h, ths_h = W.draw_inputs(w.P, w.data_seed)
    P4 = (w.P + 3) // 4 * 4
    lam = backend.zeros(P4)
    ths = backend.zeros(P4)
    lam[:w.P].copy_(backend.torch.from_numpy(lam_h))
    ths[:w.P].copy_(backend.torch.from_numpy(ths_h))
    # rows on large power-of-two boundaries (see include/qsr.h) unless asked to pack them
    stride = P4 if args.packed_rows else B.qsr_row_stride_hint(w.P)
    theta = backend.zeros(K_local, stride)
    s1 = backend.zeros(K_local, stride)
    s2 = backend.zeros(K_local, stride) if w.opt == W.OPT_ADAMW else None
    cfg = B.make_config(w, K=K_local, row_stride=stride)
    sharded_path = world > 1 or args.sharded_path      # rounds end with partial sums + all-reduce + finish

    def all_reduce(buf):
        if world > 1:
            dist.all_reduce(buf)

    def fresh_context():
        theta.zero_()
        s1.zero_()
        if s2 is not None:
            s2.zero_()
        return backend.context(cfg, theta, s1, s2, lam, ths)

    def exchange_for(ctx):
        if not sharded_path:
            return None
        return sharded.Exchange(backend.zeros(ctx.qsr_sync_sum_floats()), K_total, all_reduce)

    # ---- clocks are sampled from before the warm-up on; the samples inside the timed region are kept
    sampler = backend.clock_sampler() if rank == 0 else None

    # ---- warm-up: a few steps and one synchronization, then start again from zero
    ctx = fresh_context()
    ex = exchange_for(ctx)
    for t in range(warmup):
        ctx.qsr_local_step(t)
    if ex is None:
        ctx.qsr_sync(warmup)
    else:
        ctx.qsr_sync_partial(ex.sums)
        ex.all_reduce(ex.sums)
        ctx.qsr_sync_finish(ex.sums, K_total, warmup)
    backend.synchronize()
    ctx.close()
    ctx = fresh_context()

    # ---- timed region: global steps [0, steps) with the round ends the schedule places in it, through the same
    #      loop (sharded.run_steps) that the multi-process tests drive
    ev = [backend.event() for _ in range(steps + 1)]
    kinds = []

    def on_launch(kind, t):
        ev[len(kinds) + 1].record()
        kinds.append(kind)

    if world > 1:
        dist.barrier()
    backend.synchronize()
    launches0 = ctx.qsr_launch_count()
    wall0 = time.time()
    ev[0].record()
    sharded.run_steps(ctx, 0, steps, ex, on_launch)
    backend.synchronize()
    wall1 = time.time()
    if world > 1:
        dist.barrier()
    launches = ctx.qsr_launch_count() - launches0
    assert len(kinds) == steps
    total_ms = ev[0].elapsed_time(ev[steps])
    clocks = sampler.stop(wall0, wall1) if sampler else None
    gaps = np.array([ev[i].elapsed_time(ev[i + 1]) for i in range(steps)])
    kinds = np.array(kinds)
    step_ms = float(gaps[kinds == "step"].mean()) if (kinds == "step").any() else None
    n_syncs = int((kinds == "sync").sum())
    sync_ms = float(gaps[kinds == "sync"].mean()) if n_syncs else None
    # the stand-alone averaging kernel, outside the timed window (the window's rounds end in the fused launch)
    sync_alone_ms = None
    if world == 1:
        for _ in range(3):
            ctx.qsr_sync(steps)
        sa0, sa1 = backend.event(), backend.event()
        sa0.record()
        for _ in range(20):
            ctx.qsr_sync(steps)
        sa1.record()
        backend.synchronize()
        sync_alone_ms = sa0.elapsed_time(sa1) / 20
    ctx.close()

    total_ms = max_over_ranks(total_ms, backend)
    value = K_total * w.P * steps / (total_ms * 1e-3)

    # ---- end to end from host memory
    e2e = None
    if not args.no_e2e:
        theta0_h = backend.pinned(n=w.P)
        lam_p = backend.pinned(lam_h)
        ths_p = backend.pinned(ths_h)
        out_h = backend.pinned(n=w.P)
        t_end = min(w.T, steps)
        e0, e1 = backend.event(), backend.event()
        if not sharded_path:
            # the slabs above are released first: qsr_train_host works in one caller-owned workspace
            theta = s1 = s2 = None
            backend.release_cached_memory()
            ws = backend.empty_bytes(B.qsr_workspace_bytes(cfg))
            backend.synchronize()
            e0.record()
            r_st, r_H, _ = backend.train_host(cfg, theta0_h, lam_p, ths_p, out_h, ws, t_end)
            e1.record()
            backend.synchronize()
            e2e_ms = e0.elapsed_time(e1)
            done = int(r_st[-1] + r_H[-1])      # whole rounds: stops at the first round end at or after t_end
        else:
            if world > 1:
                dist.barrier()
            backend.synchronize()
            e0.record()
            lam[:w.P].copy_(lam_p, non_blocking=True)
            ths[:w.P].copy_(ths_p, non_blocking=True)
            theta0_d = backend.zeros(P4)
            theta0_d[:w.P].copy_(theta0_h, non_blocking=True)
            s1.zero_()
            if s2 is not None:
                s2.zero_()
            ctx = backend.context(cfg, theta, s1, s2, lam, ths)
            ctx.qsr_set_params(theta0_d)
            rounds = sharded.run_steps(ctx, 0, t_end, ex, whole_rounds=True)
            out_h.copy_(theta[0, :w.P], non_blocking=True)
            e1.record()
            backend.synchronize()
            ctx.close()
            done = rounds[-1][0] + rounds[-1][1]
            if world > 1:
                dist.barrier()
            e2e_ms = max_over_ranks(e0.elapsed_time(e1), backend)
        e2e = {"value": K_total * w.P * done / (e2e_ms * 1e-3), "unit": UNIT, "steps": done,
               "note": "a whole number of rounds: the run stops at the first round end at or after --steps",
               "h2d_bytes_per_step": 3 * w.P * 4 / done, "d2h_bytes_per_step": w.P * 4 / done,
               "api": "sharded.run_steps" if sharded_path else "qsr_train_host"}

    if rank != 0:
        return None

    peak, peak_kind = measured_peak()
    n_slabs = 3 if w.opt == W.OPT_ADAMW else 2
    streams_from_hbm = n_slabs * K_local * P4 * 4 > 2 * L2_BYTES     # else the slabs stay in L2 and DRAM sees little
    kernels = {}
    roofline = None
    if step_ms is not None:
        step_bytes = step_bytes_per_update(w) * K_local * w.P
        step_gbs = step_bytes / (step_ms * 1e-3) / 1e9
        traffic = None
        if NCU_TRAFFIC["step_source_sha256"] == step_source_hash() and streams_from_hbm:
            traffic = NCU_TRAFFIC["bytes_per_update"][w.opt] * K_local * w.P
        roofline = {"bound": "hbm", "kernel": "local_step_kernel", "achieved": step_gbs, "peak": peak, "unit": "GB/s",
                    "frac": step_gbs / peak, "peak_kind": f"of {peak_kind}", "traffic": traffic,
                    "frac_of_nominal_8TBps": step_gbs / NOMINAL_HBM_GBS,
                    "algorithmic_bytes_per_launch": step_bytes, "avg_launch_ms": step_ms}
        kernels["local_step"] = {"launches": int((kinds == "step").sum()), "avg_ms": step_ms, "GBps": step_gbs,
                                 "frac_of_measured": step_gbs / peak}
        if sync_ms is not None and not sharded_path:
            # fused: the round's last step also averages; its traffic is that of a plain step
            fused_gbs = step_bytes / (sync_ms * 1e-3) / 1e9
            kernels["local_step_with_mean"] = {"launches": n_syncs, "avg_ms": sync_ms, "GBps": fused_gbs,
                                               "frac_of_measured": fused_gbs / peak,
                                               "note": "last step of a round + replica averaging in one launch"}
        if sync_ms is not None and sharded_path:
            # last step without the theta write-back, [P] sums out, then sums in and K rows written
            end_bytes = step_bytes - 4.0 * K_local * w.P + 8.0 * w.P + 4.0 * K_local * w.P
            end_gbs = end_bytes / (sync_ms * 1e-3) / 1e9
            kernels["sharded_round_end"] = {"launches": n_syncs, "avg_ms": sync_ms, "GBps": end_gbs,
                                            "frac_of_measured": end_gbs / peak,
                                            "note": "last step fused with row sums + NCCL all-reduce of P floats + finish kernel"}
    if sync_alone_ms is not None:
        sa_gbs = 8.0 * K_local * w.P / (sync_alone_ms * 1e-3) / 1e9
        kernels["sync"] = {"launches_outside_window": 20, "avg_ms": sync_alone_ms, "GBps": sa_gbs,
                           "frac_of_measured": sa_gbs / peak, "frac_of_nominal_8TBps": sa_gbs / NOMINAL_HBM_GBS,
                           "note": "stand-alone replica-mean kernel (used when the state is averaged or reset)"}

    slab_bytes = n_slabs * K_local * P4 * 4
    l2_note = ("inputs larger than L2 (every launch streams the whole slabs)" if streams_from_hbm else
               f"slabs of {slab_bytes / 2**20:.0f} MiB stay resident in the 126 MB L2 between launches and no flush is "
               "done: a launch-bound small case, no HBM roofline claim")
    label = {"c4": "c4: ViT-B/16-shaped parameter set, Local AdamW + QSR",
             "c3": "c3: ResNet-152-shaped parameter set, Local SGD + QSR"}.get(w.name, w.name)
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": total_ms / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": label, "K_per_gpu": K_local, "K_total": K_total, "P": w.P, "row_stride": stride, "opt": w.opt, "T": w.T,
                   "window": f"global steps [0,{steps}) of the schedule", "syncs_in_window": n_syncs,
                   "l2": l2_note,
                   "parallelism": f"replica-sharded dp{world}" if sharded_path else "1 GPU, replicas as slab rows"},
        "roofline": roofline, "kernels": kernels, "gpu_launches": int(launches), "clocks": clocks,
    }
    if clocks and clocks.get("sm_mhz"):
        # time x clock: equal products at different clocks mean the difference is the clock's (the power cap's)
        out["sm_mhz_x_ms_per_step"] = clocks["sm_mhz"] * total_ms / steps
    if e2e is not None:
        out["e2e"] = e2e
    if world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(base)
    return out


def run_resident(args, backend):
    """BENCHMARK-ONLY leg: the run's rounds as register-resident launches of up to N steps (qsr_set_resident_steps).
    Times whole rounds: global steps [0, end of the round that holds step --steps - 1)."""
    from paper_2310_14423_b200 import binding as B
    from paper_2310_14423_b200 import workloads as W

    B.lib()
    w = W.workload(args.workload)
    if args.steps > w.T:
        raise SystemExit(f"--steps must be <= {w.T}")
    lam_h, ths_h = W.draw_inputs(w.P, w.data_seed)
    P4 = (w.P + 3) // 4 * 4
    lam, ths = backend.zeros(P4), backend.zeros(P4)
    lam[:w.P].copy_(backend.torch.from_numpy(lam_h))
    ths[:w.P].copy_(backend.torch.from_numpy(ths_h))
    stride = P4 if args.packed_rows else B.qsr_row_stride_hint(w.P)
    theta, s1 = backend.zeros(w.K, stride), backend.zeros(w.K, stride)
    s2 = backend.zeros(w.K, stride) if w.opt == W.OPT_ADAMW else None
    cfg = B.make_config(w, row_stride=stride)

    def fresh_context():
        theta.zero_()
        s1.zero_()
        if s2 is not None:
            s2.zero_()
        ctx = backend.context(cfg, theta, s1, s2, lam, ths)
        ctx.qsr_set_resident_steps(args.resident_steps)
        return ctx

    sampler = backend.clock_sampler()
    reps = max(args.warmup, 3)
    ctx = fresh_context()
    for _ in range(reps):                                   # warm-up: the same window, untimed
        ctx.qsr_run(0, args.steps)
    backend.synchronize()
    ctx.close()
    ctx = fresh_context()
    e0, e1 = backend.event(), backend.event()
    backend.synchronize()
    wall0 = time.time()
    e0.record()
    st, H = ctx.qsr_run(0, args.steps)
    e1.record()
    backend.synchronize()
    wall1 = time.time()
    launches = ctx.qsr_launch_count()
    ctx.close()
    clocks = sampler.stop(wall0, wall1)
    total_ms = e0.elapsed_time(e1)
    done = int(st[-1] + H[-1])
    updates = w.K * w.P * done
    value = updates / (total_ms * 1e-3)
    sm_mhz = (clocks or {}).get("sm_mhz") or 1965.0
    peak = SM_COUNT * LANES_PER_SM_CLK * sm_mhz * 1e6 / 1e9            # G thread-instructions per second
    instr = NCU_RESIDENT_INSTR[w.opt] if NCU_RESIDENT_INSTR["source_sha256"] == resident_source_hash() else None
    achieved = instr * value / 1e9 if instr else None
    n_slabs = 3 if w.opt == W.OPT_ADAMW else 2
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": 1, "steps": done, "warmup": reps,
        "ms_per_step": total_ms / done, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic", "benchmark_only": True,
        "config": {"workload": f"{w.name}: K={w.K}, P={w.P}, {w.opt}", "K_per_gpu": w.K, "K_total": w.K, "P": w.P,
                   "row_stride": stride, "opt": w.opt, "T": w.T, "resident_steps_per_launch": args.resident_steps,
                   "window": f"global steps [0,{done}): the whole rounds that cover --steps {args.steps}",
                   "syncs_in_window": int(len(st)),
                   "l2": f"slabs of {n_slabs * w.K * P4 * 4 / 2**20:.0f} MiB are read once and written once per launch of up "
                         f"to {args.resident_steps} steps; the launch is bound by its instruction stream, not by memory",
                   "parallelism": "1 GPU, replicas as slab rows",
                   "note": "BENCHMARK-ONLY: parameters and state stay in registers across steps, which only the "
                           "in-kernel synthetic gradient allows; not the path a training loop takes"},
        "roofline": {"bound": "alu", "kernel": "resident_steps_kernel", "achieved": achieved, "peak": peak,
                     "unit": "G thread-instr/s", "frac": achieved / peak if achieved else None,
                     "peak_kind": f"{SM_COUNT} SMs x {LANES_PER_SM_CLK} lanes per clock x the median SM clock sampled "
                                  f"during the run ({sm_mhz:.0f} MHz)",
                     "thread_instr_per_update": instr,
                     "scalar_equivalent_ops_per_update": NCU_RESIDENT_INSTR["scalar_equivalent"][w.opt] if instr else None,
                     "avg_launch_ms": total_ms / launches, "traffic": None},
        "gpu_launches": int(launches), "clocks": clocks,
    }
    if clocks and clocks.get("sm_mhz"):
        out["sm_mhz_x_ms_per_step"] = clocks["sm_mhz"] * total_ms / done
    if not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(w)
    return out


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    world = int(os.environ.get("WORLD_SIZE", "1"))
    backend = CudaBackend(int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), world)
    if args.resident_steps > 0:
        if world > 1:
            raise SystemExit("--resident-steps is a one-GPU leg")
        out = run_resident(args, backend)
    else:
        out = run_ours(args, backend)
    if out is not None:
        print(json.dumps(out))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
