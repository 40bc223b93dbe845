"""QSR against constant-H synchronization at the ViT-B/16 shape: sync counts and run times on one GPU.

    python -m paper_2310_14423_b200.sweep [--workload c5] [--steps T] [--eta-max 8e-4 8e-3] [--out table.md]

For every growth coefficient alpha in {0.01, 0.0175, 0.025} and minimum period H_base in {2, 4, 8}, and for constant
H in {2, 4, 8}, the whole schedule is run through qsr_run (K workers as slab rows, gradients generated in the
kernel) and timed with CUDA events.  Runs whose schedules are identical (Eq. 2 gives the same rounds when
(alpha/eta_max)^2 exceeds every H_base) are executed once and listed for each setting.  Reported per run: rounds
(= synchronizations), communication volume rounds/T as in the paper's tables, kernel launches, total time,
time per step, and replica param-updates per second.
"""
from __future__ import annotations

import argparse
import sys

import numpy as np


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c5")
    ap.add_argument("--steps", type=int, default=None, help="run only rounds starting before this step (default: all T)")
    ap.add_argument("--eta-max", type=float, nargs="*", default=None)
    ap.add_argument("--out", default=None)
    args = ap.parse_args(argv)

    import torch
    from . import binding as B
    from . import workloads as W

    B.lib()
    base = W.workload(args.workload)
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    lam_h, ths_h = W.draw_inputs(base.P, base.data_seed)
    P4 = (base.P + 3) // 4 * 4
    lam = torch.zeros(P4, device=dev)
    ths = torch.zeros(P4, device=dev)
    lam[:base.P].copy_(torch.from_numpy(lam_h))
    ths[:base.P].copy_(torch.from_numpy(ths_h))
    stride = B.qsr_row_stride_hint(base.P)
    theta = torch.zeros(base.K, stride, device=dev)
    s1 = torch.zeros_like(theta)
    s2 = torch.zeros_like(theta) if base.opt == W.OPT_ADAMW else None
    stream = torch.cuda.current_stream().cuda_stream

    settings = []
    for eta_max in (args.eta_max or [base.eta_max]):
        for alpha in (0.01, 0.0175, 0.025):
            for Hb in (2, 4, 8):
                settings.append((f"QSR alpha={alpha} H_base={Hb}", base.replace(eta_max=eta_max, alpha=alpha, H_base=Hb)))
        for Hc in (2, 4, 8):
            settings.append((f"constant H={Hc}", base.replace(eta_max=eta_max, rule=W.RULE_CONST_H, H_base=Hc)))

    done = {}
    lines = ["| eta_max | setting | rounds (syncs) | comm. % | launches | total s | ms / step | param-updates / s |",
             "|---|---|---|---|---|---|---|---|"]
    for label, w in settings:
        cfg = B.make_config(w, row_stride=stride)
        st, H = B.qsr_config_schedule(cfg)
        t_end = w.T if args.steps is None else min(w.T, args.steps)
        key = (w.eta_max, tuple(H[st < t_end].tolist()))
        if key not in done:
            theta.zero_()
            s1.zero_()
            if s2 is not None:
                s2.zero_()
            ctx = B.Context(cfg, theta, s1, s2, lam, ths, stream=stream)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            r_st, r_H = ctx.qsr_run(0, t_end)
            e1.record()
            torch.cuda.synchronize()
            steps = int(r_st[-1] + r_H[-1])
            done[key] = (len(r_st), steps, ctx.qsr_launch_count(), e0.elapsed_time(e1) * 1e-3)
            ctx.close()
        rounds, steps, launches, secs = done[key]
        lines.append(f"| {w.eta_max:g} | {label} | {rounds} | {100.0 * rounds / steps:.2f} | {launches} | {secs:.2f} | "
                     f"{1e3 * secs / steps:.3f} | {w.K * w.P * steps / secs:.4g} |")
        print(lines[-1], flush=True)
    text = (f"Workload {base.name}: K={base.K}, P={base.P}, {base.opt}, T={base.T}, warm-up {base.T_warmup}, "
            f"steps run per setting: {'all' if args.steps is None else args.steps}\n\n" + "\n".join(lines) + "\n")
    if args.out:
        with open(args.out, "w") as f:
            f.write(text)
    return 0


if __name__ == "__main__":
    sys.exit(main())
