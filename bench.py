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
    "step_source_sha256": "6c2fa12f453d27aa841b9366d84720bff8d1390a3c74bc8ff30a60d58949601e",
    "bytes_per_update": {"adamw": 24.08, "sgdm": 16.07},
}


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
    ap.add_argument("--sharded-path", action="store_true",
                    help="on one GPU, still end rounds the multi-GPU way (partial sums, all-reduce of one rank, finish)")
    return ap.parse_args()


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def step_source_hash():
    with open(os.path.join(ROOT, "paper_2310_14423_b200", "csrc", "kernels.cu")) as f:
        text = f.read()
    bar = "// " + "-" * 94 + " "
    try:
        region = text[text.index(bar + "noise"):text.index("// Sum over rows of one 16-byte column")]
    except ValueError:
        return None
    return hashlib.sha256(region.encode()).hexdigest()


class ClockSampler:
    """nvidia-smi clock / throttle samples of one GPU every 200 ms while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.gpu_id = gpu_id
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", gpu_id, f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=self.tmp, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        lines = self.tmp.readlines()
        late = not lines
        if late:
            # the timed region ended before the first 200 ms sample: take one reading now
            try:
                lines = subprocess.run(["nvidia-smi", "-i", self.gpu_id, f"--query-gpu={self.FIELDS}",
                                        "--format=csv,noheader,nounits"], capture_output=True, text=True,
                                       timeout=20).stdout.splitlines()
            except Exception:
                lines = []
        sm, smax, power, reasons = [], [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.tmp.close()
        os.unlink(self.tmp.name)
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(smax)), reasons=sorted(reasons),
                       samples=len(sm), power_w_median=float(np.median(power)))
            if late:
                out["note"] = "one reading taken right after the timed region, which was shorter than the sampling period"
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


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist
    from paper_2310_14423_b200 import binding as B
    from paper_2310_14423_b200 import sharded
    from paper_2310_14423_b200 import workloads as W

    B.lib()  # fail loudly if the CUDA library is missing
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    base = W.workload(args.workload)
    K_local = base.K                          # weak scaling: every GPU holds the configuration's K workers
    K_total = K_local * world
    w = base.replace(worker_offset=rank * K_local)
    steps, warmup = args.steps, max(args.warmup, 3)
    if steps > w.T:
        raise SystemExit(f"--steps must be <= {w.T}")

    lam_h, ths_h = W.draw_inputs(w.P, w.data_seed)
    P4 = (w.P + 3) // 4 * 4
    lam = torch.zeros(P4, device=dev)
    ths = torch.zeros(P4, device=dev)
    lam[:w.P].copy_(torch.from_numpy(lam_h))
    ths[:w.P].copy_(torch.from_numpy(ths_h))
    # rows on large power-of-two boundaries (see include/qsr.h) unless asked to pack them
    stride = P4 if args.packed_rows else B.qsr_row_stride_hint(w.P)
    theta = torch.zeros(K_local, stride, device=dev)
    s1 = torch.zeros(K_local, stride, device=dev)
    s2 = torch.zeros(K_local, stride, device=dev) if w.opt == W.OPT_ADAMW else None
    stream = torch.cuda.current_stream().cuda_stream
    cfg = B.make_config(w, K=K_local, row_stride=stride)
    sharded_path = world > 1 or args.sharded_path      # rounds end with partial sums + all-reduce + finish
    sums = torch.zeros(3 * P4, device=dev) if sharded_path else None

    def all_reduce(buf):
        if world > 1:
            dist.all_reduce(buf)

    def fresh_context():
        theta.zero_()
        s1.zero_()
        if s2 is not None:
            s2.zero_()
        return B.Context(cfg, theta, s1, s2, lam, ths, stream=stream)

    def do_sync(ctx, t_next):
        if not sharded_path:
            ctx.qsr_sync(t_next)
        else:
            ctx.qsr_sync_partial(sums)
            all_reduce(sums[:ctx.qsr_sync_sum_floats()])
            ctx.qsr_sync_finish(sums, K_total, t_next)

    # ---- warm-up: a few steps and one synchronization, then start again from zero
    ctx = fresh_context()
    for t in range(warmup):
        ctx.qsr_local_step(t)
    do_sync(ctx, warmup)
    torch.cuda.synchronize()
    ctx.close()
    ctx = fresh_context()

    # ---- timed region: global steps [0, steps) with the syncs the schedule places in it
    starts, H = B.qsr_config_schedule(cfg)
    ends = set((starts + H).tolist())
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * steps + 2)]
    kinds = []
    gpu_id = "GPU-" + str(torch.cuda.get_device_properties(local_rank).uuid).replace("GPU-", "")
    sampler = ClockSampler(gpu_id) if rank == 0 else None
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    launches0 = ctx.qsr_launch_count()
    ev[0].record()
    n_ev = 1
    for t in range(steps):
        if t + 1 in ends and not sharded_path:
            ctx.qsr_local_step_sync(t, t + 1)     # last step of a round: step and averaging in one launch
            ev[n_ev].record()
            n_ev += 1
            kinds.append("sync")
            continue
        if t + 1 in ends:
            # sharded round end: last step fused with this rank's row sums, all-reduce, finish
            ctx.qsr_local_step_partial(t, sums)
            all_reduce(sums[:ctx.qsr_sync_sum_floats()])
            ctx.qsr_sync_finish(sums, K_total, t + 1)
            ev[n_ev].record()
            n_ev += 1
            kinds.append("sync")
            continue
        ctx.qsr_local_step(t)
        ev[n_ev].record()
        n_ev += 1
        kinds.append("step")
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    launches = ctx.qsr_launch_count() - launches0
    total_ms = ev[0].elapsed_time(ev[n_ev - 1])
    clocks = sampler.stop() if sampler else None
    gaps = np.array([ev[i].elapsed_time(ev[i + 1]) for i in range(n_ev - 1)])
    kinds = np.array(kinds)
    step_ms = float(gaps[kinds == "step"].mean())
    n_syncs = int((kinds == "sync").sum())
    sync_ms = float(gaps[kinds == "sync"].mean()) if n_syncs else None
    # the stand-alone averaging kernel, outside the timed window (the window's rounds end in the fused launch)
    sync_alone_ms = None
    if world == 1:
        for _ in range(3):
            ctx.qsr_sync(steps)
        sa0, sa1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sa0.record()
        for _ in range(20):
            ctx.qsr_sync(steps)
        sa1.record()
        torch.cuda.synchronize()
        sync_alone_ms = sa0.elapsed_time(sa1) / 20
    ctx.close()

    if world > 1:
        tmax = torch.tensor([total_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        total_ms = float(tmax.item())
    value = K_total * w.P * steps / (total_ms * 1e-3)

    # ---- end to end from host memory
    e2e = None
    if not args.no_e2e:
        theta0_h = torch.zeros(w.P, dtype=torch.float32).pin_memory()
        lam_p = torch.from_numpy(lam_h).pin_memory()
        ths_p = torch.from_numpy(ths_h).pin_memory()
        out_h = torch.empty(w.P, dtype=torch.float32).pin_memory()
        t_end = min(w.T, steps)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if not sharded_path:
            # the slabs above are released first: qsr_train_host works in one caller-owned workspace
            theta = s1 = s2 = None
            torch.cuda.empty_cache()
            ws = torch.empty(B.qsr_workspace_bytes(cfg), dtype=torch.uint8, device=dev)
            torch.cuda.synchronize()
            e0.record()
            r_st, r_H, _ = B.qsr_train_host(cfg, theta0_h, lam_p, ths_p, out_h, ws, t_end=t_end, stream=stream)
            e1.record()
            torch.cuda.synchronize()
            e2e_ms = e0.elapsed_time(e1)
            done = int(r_st[-1] + r_H[-1])      # whole rounds: stops at the first round end at or after t_end
        else:
            if world > 1:
                dist.barrier()
            torch.cuda.synchronize()
            e0.record()
            lam[:w.P].copy_(lam_p, non_blocking=True)
            ths[:w.P].copy_(ths_p, non_blocking=True)
            theta0_d = torch.empty(P4, device=dev)
            theta0_d[:w.P].copy_(theta0_h, non_blocking=True)
            s1.zero_()
            if s2 is not None:
                s2.zero_()
            ctx = B.Context(cfg, theta, s1, s2, lam, ths, stream=stream)
            ctx.qsr_set_params(theta0_d)
            n_sum = ctx.qsr_sync_sum_floats()
            rounds = sharded.run_rounds(ctx, sums, K_total, 0, t_end, lambda buf: all_reduce(buf[:n_sum]))
            out_h.copy_(theta[0, :w.P], non_blocking=True)
            e1.record()
            torch.cuda.synchronize()
            ctx.close()
            done = rounds[-1][0] + rounds[-1][1]
            e2e_ms = e0.elapsed_time(e1)
            if world > 1:
                dist.barrier()
                tmax = torch.tensor([e2e_ms], device=dev, dtype=torch.float64)
                dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
                e2e_ms = float(tmax.item())
        e2e = {"value": K_total * w.P * done / (e2e_ms * 1e-3), "unit": UNIT, "steps": done,
               "h2d_bytes_per_step": 3 * w.P * 4 / done, "d2h_bytes_per_step": w.P * 4 / done,
               "api": "sharded.run_rounds" if sharded_path else "qsr_train_host"}

    if rank != 0:
        dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak()
    step_bytes = step_bytes_per_update(w) * K_local * w.P
    step_gbs = step_bytes / (step_ms * 1e-3) / 1e9
    traffic = None
    n_slabs = 3 if w.opt == W.OPT_ADAMW else 2
    streams_from_hbm = n_slabs * K_local * P4 * 4 > 2 * L2_BYTES     # else the slabs stay in L2 and DRAM sees little
    if NCU_TRAFFIC["step_source_sha256"] == step_source_hash() and streams_from_hbm:
        traffic = NCU_TRAFFIC["bytes_per_update"][w.opt] * K_local * w.P
    roofline = {"bound": "hbm", "kernel": "local_step_kernel", "achieved": step_gbs, "peak": peak, "unit": "GB/s",
                "frac": step_gbs / peak, "peak_kind": f"of {peak_kind}", "traffic": traffic,
                "frac_of_nominal_8TBps": step_gbs / NOMINAL_HBM_GBS,
                "algorithmic_bytes_per_launch": step_bytes, "avg_launch_ms": step_ms}
    kernels = {"local_step": {"launches": int((kinds == "step").sum()), "avg_ms": step_ms, "GBps": step_gbs,
                              "frac_of_measured": step_gbs / peak}}
    if sync_ms is not None and not sharded_path:
        # fused: the round's last step also averages; its traffic is that of a plain step
        fused_gbs = step_bytes / (sync_ms * 1e-3) / 1e9
        kernels["local_step_with_mean"] = {"launches": n_syncs, "avg_ms": sync_ms, "GBps": fused_gbs,
                                           "frac_of_measured": fused_gbs / peak,
                                           "note": "last step of a round + replica averaging in one launch"}
    if sync_alone_ms is not None:
        sa_gbs = 8.0 * K_local * w.P / (sync_alone_ms * 1e-3) / 1e9
        kernels["sync"] = {"launches_outside_window": 20, "avg_ms": sync_alone_ms, "GBps": sa_gbs,
                           "frac_of_measured": sa_gbs / peak, "frac_of_nominal_8TBps": sa_gbs / NOMINAL_HBM_GBS,
                           "note": "stand-alone replica-mean kernel (used when the state is averaged or reset)"}
    if sync_ms is not None and sharded_path:
        # last step without the theta write-back, [P] sums out, then sums in and K rows written
        end_bytes = step_bytes - 4.0 * K_local * w.P + 8.0 * w.P + 4.0 * K_local * w.P
        end_gbs = end_bytes / (sync_ms * 1e-3) / 1e9
        kernels["sharded_round_end"] = {"launches": n_syncs, "avg_ms": sync_ms, "GBps": end_gbs,
                                        "frac_of_measured": end_gbs / peak,
                                        "note": "last step fused with row sums + NCCL all-reduce of P floats + finish kernel"}

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
    if e2e is not None:
        out["e2e"] = e2e
    if world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(base)
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
