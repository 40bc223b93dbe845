"""Register-resident multi-step launches (benchmark-only; qsr_set_resident_steps) against the per-step path and the
oracle.  The launches hold parameters and state in registers over up to 128 consecutive steps and average inside the
kernel at round ends; the arithmetic is the per-step kernel's, so every slab must come out bit for bit the same,
whatever the chunk length, the worker count or the state mode, and the run must meet the oracle at the usual bar."""
import numpy as np
import pytest
import torch

from paper_2310_14423_b200 import binding as B
from paper_2310_14423_b200 import workloads as W

import gpu_harness as G

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _cuda():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    B.lib()
    yield
    torch.cuda.synchronize()
    torch.cuda.empty_cache()


def _run(w, resident, t_end=None, row_stride=None):
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    S = G.Slabs(w, row_stride=row_stride)
    ctx = G.make_context(w, S, lam_d, ths_d)
    ctx.qsr_set_resident_steps(resident)
    st, H = ctx.qsr_run(0, w.T if t_end is None else t_end)
    torch.cuda.synchronize()
    launches = ctx.qsr_launch_count()
    ctx.close()
    assert S.guards_intact()
    return lam, ths, S, st, H, launches


def _same(a, b):
    return torch.equal(a.theta, b.theta) and torch.equal(a.s1, b.s1) and (a.s2 is None or torch.equal(a.s2, b.s2))


@pytest.mark.parametrize("n", [1, 5, 128])
@pytest.mark.parametrize("opt,mode", [(W.OPT_SGDM, W.STATE_KEEP), (W.OPT_ADAMW, W.STATE_KEEP),
                                      (W.OPT_ADAMW, W.STATE_RESET), (W.OPT_SGDM, W.STATE_AVERAGE),
                                      (W.OPT_ADAMW, W.STATE_AVERAGE)])
def test_resident_launches_equal_per_step_launches_bitwise(opt, mode, n):
    # rounds of 6 to about 100 steps: launches that end inside a round, on a round end, and that span several rounds
    w = W.tiny_workload(opt, K=3, P=4099, T=400, state_sync=mode)
    _, _, S0, st0, H0, n0 = _run(w, 0)
    assert H0.max() > 64 > H0.min() and n0 >= w.T
    _, _, S1, st1, H1, n1 = _run(w, n)
    assert np.array_equal(st0, st1) and np.array_equal(H0, H1)
    assert _same(S0, S1)
    if mode == W.STATE_KEEP:
        assert n1 == -(-w.T // n)                       # launches run across round ends
    else:
        per_sync = 2 if mode == W.STATE_RESET else 1           # the reset of the state is a launch of its own
        assert n1 == sum(-(-int(h) // n) for h in H0) + per_sync * len(H0)     # chunks per round, plus the syncs


@pytest.mark.parametrize("K", [1, 2, 3, 4, 8, 16, 31, 32])
@pytest.mark.parametrize("P", [1, 3, 127, 128, 129, 4100, 8191])
def test_worker_counts_and_ragged_sizes(K, P):
    opt = W.OPT_ADAMW if (K + P) % 2 else W.OPT_SGDM
    w = W.tiny_workload(opt, K=K, P=P, T=50)
    _, _, S0, st0, H0, _ = _run(w, 0, row_stride=(P + 3) // 4 * 4 + 8)
    _, _, S1, st1, H1, _ = _run(w, 7, row_stride=(P + 3) // 4 * 4 + 8)
    assert np.array_equal(st0, st1) and np.array_equal(H0, H1)
    assert _same(S0, S1)


def test_config1_resident_against_the_oracle_on_every_coordinate():
    """K=4, P=65,536, Local SGD with momentum, cosine, QSR alpha=0.2 H_base=2, T=2000: 2000 steps in 16 launches."""
    w = W.workload("c1")
    lam, ths, S, st, H, launches = _run(w, 128)
    orc = G.oracle_on(w, lam, ths)
    ost, oH = orc.run()
    assert np.array_equal(st, ost) and np.array_equal(H, oH) and len(st) == 203
    assert launches == 16
    theta = S.theta.cpu().numpy()
    assert (theta == theta[0]).all()
    assert G.rel_err(theta[0], orc.theta[0]) <= G.REL_TOL


def test_config2_resident_against_the_oracle_on_a_subset():
    """K=8, P=2^20, Local AdamW, warm-up + cosine, T=5000: device runs all of it, the oracle 8192 coordinates."""
    w = W.workload("c2")
    lam, ths, S, st, H, launches = _run(w, 128)
    idx = W.coordinate_subset(w.layout, 8192, seed=2)
    orc = G.oracle_on(w, lam, ths, idx)
    ost, oH = orc.run()
    assert np.array_equal(st, ost) and np.array_equal(H, oH) and len(st) == 8
    assert launches == -(-5000 // 128)
    theta = S.theta.cpu().numpy()
    assert (theta == theta[0]).all()
    assert G.rel_err(theta[0][idx], orc.theta[0]) <= G.REL_TOL


def test_resume_in_pieces():
    w = W.tiny_workload(W.OPT_ADAMW, K=5, P=1030, T=240)
    _, _, S0, st0, H0, _ = _run(w, 0)
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    S = G.Slabs(w)
    ctx = G.make_context(w, S, lam_d, ths_d)
    ctx.qsr_set_resident_steps(16)
    st_a, H_a = ctx.qsr_run(0, 100)
    t_mid = int(st_a[-1] + H_a[-1])
    ctx.qsr_set_resident_steps(0)                # back to per-step launches for a stretch
    st_b, H_b = ctx.qsr_run(t_mid, 170)
    t_mid2 = int(st_b[-1] + H_b[-1])
    ctx.qsr_set_resident_steps(100)
    st_c, H_c = ctx.qsr_run(t_mid2, w.T)
    torch.cuda.synchronize()
    ctx.close()
    assert np.array_equal(np.concatenate([st_a, st_b, st_c]), st0)
    assert _same(S0, S)


def test_falls_back_to_per_step_launches_with_a_tensor_table_or_clipping():
    w = W.tiny_workload(W.OPT_SGDM, K=3, P=2048, T=40, weight_decay=0.1)
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    ends = torch.tensor([1024, 2048], dtype=torch.int64, device="cuda")
    scales = torch.tensor([0.0, 1.0], device="cuda")
    runs = []
    for resident in (0, 32):
        S = G.Slabs(w)
        ctx = G.make_context(w, S, lam_d, ths_d)
        ctx.qsr_set_tensor_table(ends, scales)
        ctx.qsr_set_resident_steps(resident)
        ctx.qsr_run()
        torch.cuda.synchronize()
        assert ctx.qsr_launch_count() == w.T
        ctx.close()
        runs.append(S)
    assert _same(runs[0], runs[1])


def test_argument_errors():
    w = W.tiny_workload(W.OPT_SGDM, K=33, P=64, T=10)
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    S = G.Slabs(w)
    ctx = G.make_context(w, S, lam_d, ths_d)
    for bad in (-1, 129, 1):                      # K = 33 does not fit one block
        with pytest.raises(B.QsrError) as e:
            ctx.qsr_set_resident_steps(bad)
        assert e.value.status == B.QSR_ERANGE
    ctx.qsr_set_resident_steps(0)
    ctx.close()


def test_packed_noise_equals_scalar_noise_bitwise():
    """The resident launches evaluate the noise with packed fp32 instructions (two Box-Muller transforms per
    instruction stream), the per-step kernel one lane at a time.  With eta = 1, lambda = 0, sigma = 1, no momentum and
    no weight decay one SGD step from zero leaves theta = -z: 33.5 M normals (16.8 M words through the logarithm and
    as many through the sine / cosine: most of the 2^23-point grid of each) must agree bit for bit."""
    P, K, t = 1 << 22, 8, 12345
    w = W.tiny_workload(W.OPT_SGDM, K=K, P=P, T=20000, sched=W.SCHED_CONST, eta_max=1.0, momentum=0.0,
                        weight_decay=0.0, noise_std=1.0, rule=W.RULE_CONST_H, H_base=5)
    zero = torch.zeros(P, device="cuda")
    out = []
    for resident in (0, 1):
        theta = torch.zeros(K, P, device="cuda")
        s1 = torch.zeros(K, P, device="cuda")
        ctx = B.Context(B.make_config(w), theta, s1, None, zero, zero, stream=torch.cuda.current_stream().cuda_stream)
        if resident:
            ctx.qsr_set_resident_steps(1)
            st, H = ctx.qsr_run(10000, 10001)          # a round of 5 from t = 10000: steps 10000 .. 10004 and a mean
        else:
            for u in range(10000, 10004):
                ctx.qsr_local_step(u)
            ctx.qsr_local_step_sync(10004, 10005)
        torch.cuda.synchronize()
        ctx.close()
        out.append((theta, s1))
    assert torch.equal(out[0][0], out[1][0]) and torch.equal(out[0][1], out[1][1])
    # s1 holds the last step's gradient, i.e. that step's noise itself: not all the same, not all finite by accident
    z = out[0][1]
    assert bool(torch.isfinite(z).all()) and abs(float(z.mean())) < 1e-3 and abs(float(z.var()) - 1) < 1e-2
