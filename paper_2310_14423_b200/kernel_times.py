"""Device time of every kernel of the library at a run configuration's full size, one line per kernel.

    python -m paper_2310_14423_b200.kernel_times [--workload c4] [--launches 30] [--out table.md]

Back-to-back launches on one stream, timed with CUDA events after warm-up.  GB/s figures use the algorithmic bytes of
each kernel (fp32 slabs streamed once); kernels bound by the synthetic-noise arithmetic rather than by memory are
reported in noise evaluations per second instead.
"""
from __future__ import annotations

import argparse
import sys

import numpy as np


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c4")
    ap.add_argument("--launches", type=int, default=30)
    ap.add_argument("--out", default=None)
    ap.add_argument("--packed", action="store_true",
                    help="rows packed at P instead of the stride qsr_row_stride_hint recommends")
    args = ap.parse_args(argv)

    import torch
    from . import binding as B
    from . import workloads as W

    B.lib()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    w = W.workload(args.workload)
    KP = w.K * w.P
    n_slabs = 3 if w.opt == W.OPT_ADAMW else 2
    stride = (w.P + 3) // 4 * 4 if args.packed else B.qsr_row_stride_hint(w.P)
    theta = torch.zeros(w.K, stride, device=dev)
    s1 = torch.zeros_like(theta)
    s2 = torch.zeros_like(theta) if w.opt == W.OPT_ADAMW else None
    lam = torch.rand(w.P, device=dev)
    ths = torch.randn(w.P, device=dev)
    stream = torch.cuda.current_stream().cuda_stream
    t = [w.T_warmup + 100]

    def timed(fn):
        for _ in range(5):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.launches):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / args.launches

    def context(mode=W.STATE_KEEP):
        return B.Context(B.make_config(w.replace(state_sync=mode), row_stride=stride), theta, s1, s2, lam, ths, stream=stream)

    rows = []

    def add(label, ms, nbytes=None, evals=None):
        rate = f"{nbytes / ms / 1e6:.0f} GB/s" if nbytes else f"{evals / ms / 1e6:.0f} G noise evaluations/s"
        rows.append(f"| {label} | {ms:.3f} | {rate} |")
        print(rows[-1], flush=True)

    ctx = context()

    def step(grads=None):
        ctx.qsr_local_step(t[0], grads)
        t[0] += 1

    def step_mean():
        ctx.qsr_local_step_sync(t[0], t[0] + 1)
        t[0] += 1

    def parallel():
        ctx.qsr_parallel_step(t[0])
        t[0] += 1

    add("local step, generated gradient", timed(step), (n_slabs * 8 + 8 / w.K) * KP)
    add("local step + replica mean (round end, one launch)", timed(step_mean), (n_slabs * 8 + 8 / w.K) * KP)
    sums = torch.zeros(ctx.qsr_sync_sum_floats(), device=dev)

    def round_end_sharded():
        ctx.qsr_local_step_partial(t[0], sums)
        ctx.qsr_sync_finish(sums, w.K, t[0] + 1)
        t[0] += 1

    add("sharded round end: step + row sums, then finish (two launches, no all-reduce)", timed(round_end_sharded),
        (n_slabs * 8 + 8 / w.K) * KP + 8 * w.P)
    grads = torch.zeros_like(theta)
    add("local step, gradients from a slab", timed(lambda: step(grads)), (n_slabs * 8 + 4) * KP)
    del grads
    ends = torch.from_numpy(np.cumsum(w.layout.numel).astype(np.int64)).cuda()
    if int(ends[-1]) == w.P and bool((ends[:-1] % 4 == 0).all()):
        scale = torch.ones(ends.numel(), device=dev)
        scale[1::3] = 0.0
        ctx.qsr_set_tensor_table(ends, scale)
        add(f"local step with a {ends.numel()}-tensor weight-decay table", timed(step), (n_slabs * 8 + 8 / w.K) * KP)
        ctx.qsr_set_tensor_table(None, None)
    ws = torch.zeros(ctx.qsr_clip_workspace_floats(), device=dev)
    ctx.qsr_set_grad_clip(1.0, ws)
    add("clipped local step (norm pass + factors + step: three launches)", timed(step), (n_slabs * 8 + 4 + 16 / w.K) * KP)
    # inside qsr_run a step leaves its successor's norm partials behind: time a whole round and divide by its steps
    t_round = [0]

    def clipped_round():
        st_, H_ = ctx.qsr_run(0, 1)
        t_round[0] = int(H_[0])

    saved, args.launches = args.launches, max(1, args.launches // 10)
    ms_round = timed(clipped_round)
    args.launches = saved
    add(f"clipped local step inside qsr_run (round of {t_round[0]} steps; factors + step, norm pass once per round)",
        ms_round / t_round[0], (n_slabs * 8 + 8 / w.K) * KP)
    add("clipped Algorithm-1 step (row 0; three launches)", timed(parallel), evals=2 * KP)
    ctx.qsr_set_grad_clip(0.0)
    add("Algorithm-1 step (row 0, K gradients per coordinate)", timed(parallel), evals=KP)
    add("replica mean, state kept", timed(lambda: ctx.qsr_sync(t[0])), 8 * KP)
    if int(sums.numel()) <= B.QSR_STATIC_SCRATCH_FLOATS:
        add("replica mean through the static scratch (two launches)", timed(lambda: ctx.qsr_sync_static(t[0])), 8 * KP + 8 * w.P)
    ctx.close()
    for mode, per in ((W.STATE_AVERAGE, 8 + 8 * (n_slabs - 1)), (W.STATE_RESET, 8 + 4 * (n_slabs - 1))):
        c = context(mode)
        label = f"replica mean, state {mode}" + (" (mean launch + state-reset launch)" if mode == W.STATE_RESET else "")
        add(label, timed(lambda: c.qsr_sync(t[0])), per * KP)
        c.close()
    theta0 = torch.zeros(stride, device=dev)[:w.P]
    c = context()
    add("broadcast of theta_bar(0) to every worker", timed(lambda: c.qsr_set_params(theta0)), 4 * KP + 4 * w.P)
    c.close()

    text = (f"Workload {w.name}: K={w.K}, P={w.P}, {w.opt}; {args.launches} back-to-back launches per line\n\n"
            "| kernel | ms per call | rate |\n|---|---|---|\n" + "\n".join(rows) + "\n")
    if args.out:
        with open(args.out, "w") as f:
            f.write(text)
    return 0


if __name__ == "__main__":
    sys.exit(main())
