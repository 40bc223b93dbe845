"""GPU parity for gradient clipping by global norm (App. C.2): Local OPT with per-worker clipping and Algorithm 1
with the averaged gradient clipped, against the oracle on ALL coordinates (clipping couples them, so there is no
coordinate subset here)."""
import numpy as np
import pytest
import torch

from oracle import qsr_oracle as O
from paper_2310_14423_b200 import binding as B
from paper_2310_14423_b200 import workloads as W

import gpu_harness as G

pytestmark = pytest.mark.gpu


def _clip_context(w, S, lam_d, ths_d):
    ctx = G.make_context(w, S, lam_d, ths_d)
    ws = torch.full((ctx.qsr_clip_workspace_floats() + 8,), 7.0, device="cuda")
    ctx.qsr_set_grad_clip(w.clip_norm, ws)
    return ctx, ws


@pytest.mark.parametrize("opt", [W.OPT_SGDM, W.OPT_ADAMW])
@pytest.mark.parametrize("K,P", [(1, 3), (3, 1001), (16, 40002), (5, 300000)])
def test_clipped_local_runs(opt, K, P):
    # the threshold sits inside the range of gradient norms of the run, so some steps clip and some do not
    clip = {3: 0.02, 1001: 3.0, 40002: 20.0, 300000: 55.0}[P]
    # the largest AdamW case starts at the full learning rate, where one coordinate in 1e5 is ill-conditioned for any
    # fp32 gradient (see conditioning.py); assert_parity bounds it by the run's own sensitivity instead of avoiding it
    w = W.tiny_workload(opt, K=K, P=P, T=30, clip_norm=clip)
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    S = G.Slabs(w)
    ctx, ws = _clip_context(w, S, lam_d, ths_d)
    st, H = ctx.qsr_run()
    torch.cuda.synchronize()
    # per step the factor pass and the step; the norm pass only at a round's first step (later steps find the partial
    # sums their predecessor left behind)
    assert ctx.qsr_launch_count() == 2 * w.T + len(st)
    orc = G.oracle_on(w, lam, ths)
    ost, oH = orc.run()
    assert np.array_equal(st, ost) and np.array_equal(H, oH)
    G.assert_parity(S.theta[0, :P].cpu().numpy(), w, lam, ths, orc.theta[0])
    assert bool((S.theta[:, :P] == S.theta[0, :P]).all())
    free = G.oracle_on(w.replace(clip_norm=0.0), lam, ths)
    free.run()
    assert G.rel_err(S.theta[0, :P].cpu().numpy(), free.theta[0]) > 1e-4   # clipping did change the run
    assert S.guards_intact() and bool((ws[-8:] == 7.0).all())
    ctx.close()


def test_clip_factors_against_numpy():
    """The factors themselves, for gradients from a slab: min(1, c / (||g_k|| + 1e-6)) per worker."""
    K, P = 6, 123457
    w = W.tiny_workload(W.OPT_SGDM, K=K, P=P, T=5, momentum=0.0, weight_decay=0.0, sched=W.SCHED_CONST, eta_max=1.0,
                        clip_norm=100.0)
    S = G.Slabs(w, n_extra=1)
    ctx = G.make_context(w, S, None, None)
    ws = torch.zeros(ctx.qsr_clip_workspace_floats(), device="cuda")
    ctx.qsr_set_grad_clip(w.clip_norm, ws)
    grads = S.extra[0]
    scale = torch.tensor([0.01, 0.1, 0.28, 0.3, 1.0, 10.0], device="cuda").view(K, 1)
    grads[:, :P] = torch.randn(K, P, device="cuda") * scale
    ctx.qsr_local_step(0, grads)
    torch.cuda.synchronize()
    g = grads[:, :P].double().cpu().numpy()
    coef = np.minimum(1.0, 100.0 / (np.sqrt((g * g).sum(axis=1)) + 1e-6))
    assert (coef < 1).any() and (coef == 1).any()
    theta = S.theta[:, :P].double().cpu().numpy()
    np.testing.assert_allclose(theta, -coef[:, None] * g, rtol=2e-6, atol=1e-9)
    ctx.close()


@pytest.mark.parametrize("opt", [W.OPT_SGDM, W.OPT_ADAMW])
def test_clipped_parallel_steps(opt):
    K, P = 8, 50003
    w = W.tiny_workload(opt, K=K, P=P, T=30, clip_norm=12.0)
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    S = G.Slabs(w)
    ctx, ws = _clip_context(w, S, lam_d, ths_d)
    orc = O.State(w, lam, ths, rows=1)
    for t in range(w.T):
        ctx.qsr_parallel_step(t)
        orc.parallel_step(t, K)
    torch.cuda.synchronize()
    assert G.rel_err(S.theta[0, :P].cpu().numpy(), orc.theta[0]) <= G.REL_TOL
    free = O.State(w.replace(clip_norm=0.0), lam, ths, rows=1)
    for t in range(w.T):
        free.parallel_step(t, K)
    assert G.rel_err(S.theta[0, :P].cpu().numpy(), free.theta[0]) > 1e-4
    ctx.close()


def test_clip_switch_and_argument_errors():
    w = W.tiny_workload(W.OPT_SGDM, K=2, P=64, T=10)
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    S = G.Slabs(w)
    ctx = G.make_context(w, S, lam_d, ths_d)
    with pytest.raises(B.QsrError) as e:
        ctx.qsr_set_grad_clip(1.0, None)
    assert e.value.status == B.QSR_EINVAL
    ws = torch.zeros(ctx.qsr_clip_workspace_floats() + 4, device="cuda")
    with pytest.raises(B.QsrError) as e:
        ctx.qsr_set_grad_clip(1.0, ws[1:])
    assert e.value.status == B.QSR_EALIGN
    ctx.qsr_set_grad_clip(1.0, ws)
    ctx.qsr_local_step(0)
    assert ctx.qsr_launch_count() == 3
    ctx.qsr_set_grad_clip(0.0)                # off again
    ctx.qsr_local_step(1)
    assert ctx.qsr_launch_count() == 4
    torch.cuda.synchronize()
    ctx.close()


@pytest.mark.parametrize("opt", [W.OPT_SGDM, W.OPT_ADAMW])
@pytest.mark.parametrize("K,P,mode", [(1, 3, W.STATE_KEEP), (3, 1001, W.STATE_KEEP), (16, 40002, W.STATE_KEEP),
                                      (5, 70003, W.STATE_RESET), (7, 4100, W.STATE_AVERAGE)])
def test_norms_left_by_the_previous_step_equal_the_norm_pass_bitwise(opt, K, P, mode):
    """Inside qsr_run a plain step also computes its successor's gradient-norm partials; driving the same steps one
    call at a time runs the stand-alone norm pass before every step.  The two must agree in every bit of every slab:
    same per-column values, same block geometry, same order of summation."""
    clip = {3: 0.02, 1001: 3.0, 40002: 20.0, 70003: 25.0, 4100: 6.0}[P]
    w = W.tiny_workload(opt, K=K, P=P, T=60, clip_norm=clip, state_sync=mode)
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    A, Bs = G.Slabs(w), G.Slabs(w)
    ca, wa = _clip_context(w, A, lam_d, ths_d)
    cb, wb = _clip_context(w, Bs, lam_d, ths_d)
    st, H = ca.qsr_run()
    t = 0
    while t < w.T:
        h = cb.qsr_round_length(t)
        for u in range(t, t + h - 1):
            cb.qsr_local_step(u)
        cb.qsr_local_step_sync(t + h - 1, t + h)
        t += h
    torch.cuda.synchronize()
    assert cb.qsr_launch_count() > ca.qsr_launch_count()
    assert torch.equal(A.theta, Bs.theta) and torch.equal(A.s1, Bs.s1)
    assert A.s2 is None or torch.equal(A.s2, Bs.s2)
    assert A.guards_intact() and Bs.guards_intact() and bool((wa[-8:] == 7.0).all())
    # and clipping was active on some steps but not on all: the factors in the workspace are not all 1
    ca.close()
    cb.close()


def test_norms_fall_back_to_the_norm_pass_when_the_block_has_no_room():
    """K x threads sums must fit next to the step's ring in shared memory; with 512-thread blocks and K = 96 (the most
    clipping takes) AdamW's 96 KiB ring (four rows in flight) leaves no room for 192 KiB more, so every step runs the
    stand-alone norm pass -- with the same result up to the order of the norms' partial sums."""
    w = W.tiny_workload(W.OPT_ADAMW, K=96, P=3001, T=24, clip_norm=6.0)
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    for threads in (256, 512):
        S = G.Slabs(w)
        ctx, ws = _clip_context(w, S, lam_d, ths_d)
        ctx.qsr_set_launch_shape(threads, 4, 0)
        st, H = ctx.qsr_run()
        torch.cuda.synchronize()
        expect = 2 * w.T + len(st) if threads == 256 else 3 * w.T
        assert ctx.qsr_launch_count() == expect
        orc = G.oracle_on(w, lam, ths)
        orc.run()
        G.assert_parity(S.theta[0, :w.P].cpu().numpy(), w, lam, ths, orc.theta[0])
        assert S.guards_intact() and bool((ws[-8:] == 7.0).all())
        ctx.close()
