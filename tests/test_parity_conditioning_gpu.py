"""GPU parity on the runs where fp32 cannot hold 1e-5 on every coordinate, bounded instead of avoided.

Three regimes make AdamW take first steps at a non-zero learning rate (moments just zero, step eta * g / (|g| + eps)):
a short run from the full learning rate, moments reset at every synchronization, and the clipped run at P = 3e5 and
T = 30.  All coordinates are compared.  The bar is gpu_harness.assert_parity: 1e-5 everywhere, except that a coordinate
may exceed it by what the binary64 oracle itself moves there when its gradients are perturbed by one fp32 ulp
(conditioning.py).  The oracle's binary32-storage build is run beside it and its distance reported: the library must
be hit on coordinates that build is hit on too, and nowhere else.
"""
import numpy as np
import pytest
import torch

from paper_2310_14423_b200 import workloads as W

import conditioning
import gpu_harness as G

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("K,P,T,mode,clip", [
    (3, 99999, 40, W.STATE_KEEP, 0.0),
    (8, 99999, 60, W.STATE_RESET, 0.0),
    (5, 300000, 30, W.STATE_KEEP, 55.0),
])
def test_adamw_first_steps_at_full_learning_rate(K, P, T, mode, clip):
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    w = W.tiny_workload(W.OPT_ADAMW, K=K, P=P, T=T, state_sync=mode, clip_norm=clip)
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    S = G.Slabs(w)
    ctx = G.make_context(w, S, lam_d, ths_d)
    if clip > 0:
        ws = torch.zeros(ctx.qsr_clip_workspace_floats(), device="cuda")
        ctx.qsr_set_grad_clip(clip, ws)
    st, H = ctx.qsr_run()
    torch.cuda.synchronize()
    ctx.close()
    orc = G.oracle_on(w, lam, ths)
    ost, oH = orc.run()
    assert np.array_equal(st, ost) and np.array_equal(H, oH)
    theta = S.theta[0, :P].cpu().numpy()
    err = G.assert_parity(theta, w, lam, ths, orc.theta[0])
    # the same run in the oracle's binary32-storage build
    mirror = G.oracle_on(w, lam, ths, mirror=True)
    mirror.run()
    err_mirror = G.rel_err(mirror.theta[0], orc.theta[0])
    sens = conditioning.fp32_sensitivity(w, lam, ths)
    scale = np.maximum(np.abs(orc.theta[0]), np.sqrt(np.mean(orc.theta[0] ** 2)))
    marked = sens > G.REL_TOL * scale
    out_gpu = conditioning.excess_over(theta, orc.theta[0], G.REL_TOL) > 0
    assert not np.any(out_gpu & ~marked)                 # the library leaves the bar only where the run is ill-conditioned
    assert marked.sum() <= 2e-4 * P
    # away from those few coordinates the library is as close to binary64 as the best fp32 arithmetic
    rel = np.abs(theta.astype(np.float64) - orc.theta[0]) / scale
    assert rel[~marked].max() <= G.REL_TOL
    assert np.median(rel) <= 1e-7
    print(f"K={K} P={P} T={T} {mode} clip={clip}: gpu {err:.2e}, binary32-storage oracle {err_mirror:.2e}, "
          f"{int(marked.sum())} coordinates marked ill-conditioned, gpu outside the bar on {int(out_gpu.sum())}")
    assert S.guards_intact()
