"""Pins for the oracle's local steps, averaging and round loop (Eq. 1, Algorithm 2, App. C).

Expected values come from closed forms, from torch.optim on the CPU fed with the same gradients,
from invariants of the mean, and from a brute-force run of a tiny case written out in plain Python.
None of these tests touches the CUDA library.
"""
import math

import numpy as np
import pytest
import torch

from oracle import qsr_oracle as O
from paper_2310_14423_b200 import workloads as W


def _inputs(w, n=None):
    lam, ths = W.draw_inputs(w.P, w.data_seed)
    return (lam, ths) if n is None else (lam[:n], ths[:n])


# ------------------------------------------------------------------ SGD with heavy-ball momentum

def test_sgd_momentum_closed_form_constant_lr():
    """Noise-free diagonal quadratic, constant eta: x = theta - theta~ with theta~ = lam*theta_star/(lam+wd)
    obeys x_{t+1} = (1 + mu - eta*lam')*x_t - mu*x_{t-1}, x_1 = (1 - eta*lam')*x_0, lam' = lam + wd.  With r1, r2 the
    roots of r^2 - (1 + mu - eta*lam')*r + mu = 0:  x_t = x_0*(r1^(t+1)*(1-r2) - r2^(t+1)*(1-r1))/(r1 - r2)."""
    T = 57
    w = W.tiny_workload(W.OPT_SGDM, K=2, P=64, T=T, sched=W.SCHED_CONST, eta_max=0.3, momentum=0.9,
                        weight_decay=0.02, noise_std=0.0, alpha=0.5, H_base=3)
    lam = np.geomspace(1e-3, 6.0, 64)           # both real and complex root pairs occur
    ths = np.linspace(-2.0, 2.0, 64) + 0.1
    S = O.State(w, lam, ths)
    S.run()
    lp = lam + w.weight_decay
    fixed = lam * ths / lp
    b = (1 + w.momentum - w.eta_max * lp).astype(complex)
    disc = np.sqrt(b * b - 4 * w.momentum)
    r1, r2 = (b + disc) / 2, (b - disc) / 2
    assert (np.abs(disc) > 1e-6).all()
    x0 = 0.0 - fixed
    xT = x0 * (r1 ** (T + 1) * (1 - r2) - r2 ** (T + 1) * (1 - r1)) / (r1 - r2)
    expect = fixed + xT.real
    assert np.abs(xT.imag).max() < 1e-9
    for k in range(2):
        np.testing.assert_allclose(S.theta[k], expect, rtol=1e-9, atol=1e-11)


def test_sgd_momentum_time_varying_lr_matrix_product():
    """Cosine schedule, noise-free: (x, v) is mapped by [[1 - eta_t*lam', -eta_t*mu], [lam', mu]] each step."""
    w = W.tiny_workload(W.OPT_SGDM, K=3, P=16, T=80, eta_max=0.5, momentum=0.9, weight_decay=0.0,
                        noise_std=0.0, alpha=0.4, H_base=2)
    lam = np.geomspace(1e-2, 3.0, 16)
    ths = np.linspace(1.0, 2.0, 16)
    S = O.State(w, lam, ths)
    S.run()
    for c in range(16):
        M = np.eye(2)
        for t in range(w.T):
            eta = 0.5 * w.eta_max * (1 + math.cos(math.pi * t / w.T))
            M = np.array([[1 - eta * lam[c], -eta * w.momentum], [lam[c], w.momentum]]) @ M
        x = (M @ np.array([0.0 - ths[c], 0.0]))[0]
        assert S.theta[0, c] == pytest.approx(ths[c] + x, rel=1e-10, abs=1e-12)


def _grad(w, lam, ths, theta, k, t, idx=None):
    n = theta.shape[0]
    z = np.array([O.noise(w.noise_seed, k, t, int(i if idx is None else idx[i])) for i in range(n)])
    return lam * (theta - ths) + w.noise_std * z


def test_single_worker_equals_torch_sgd():
    """K = 1: averaging is the identity, so Algorithm 2 is plain SGD whatever the round lengths."""
    w = W.tiny_workload(W.OPT_SGDM, K=1, P=24, T=40, momentum=0.9, weight_decay=0.01)
    lam, ths = _inputs(w)
    lam, ths = lam.astype(np.float64), ths.astype(np.float64)
    S = O.State(w, lam, ths)
    S.run()
    p = torch.zeros(24, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.SGD([p], lr=1.0, momentum=0.9, weight_decay=0.01)
    for t in range(w.T):
        for g in opt.param_groups:
            g["lr"] = 0.5 * w.eta_max * (1 + math.cos(math.pi * t / w.T))
        p.grad = torch.from_numpy(_grad(w, lam, ths, p.detach().numpy(), 0, t))
        opt.step()
    np.testing.assert_allclose(S.theta[0], p.detach().numpy(), rtol=1e-11, atol=1e-13)


def test_single_worker_equals_torch_adamw():
    w = W.tiny_workload(W.OPT_ADAMW, K=1, P=24, T=40, T_warmup=5, eta_max=0.02, weight_decay=0.05)
    lam, ths = _inputs(w)
    lam, ths = lam.astype(np.float64), ths.astype(np.float64)
    S = O.State(w, lam, ths)
    S.run()
    p = torch.zeros(24, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.AdamW([p], lr=1.0, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.05)
    for t in range(w.T):
        eta = w.eta_max * t / 5 if t < 5 else 0.5 * w.eta_max * (1 + math.cos(math.pi * (t - 5) / (w.T - 5)))
        for g in opt.param_groups:
            g["lr"] = eta
        p.grad = torch.from_numpy(_grad(w, lam, ths, p.detach().numpy(), 0, t))
        opt.step()
    np.testing.assert_allclose(S.theta[0], p.detach().numpy(), rtol=1e-10, atol=1e-13)


def test_adamw_constant_gradient_closed_form():
    """Constant g: m_hat = g and v_hat = g^2 at every step, so theta_{t+1} = (1 - eta_t*wd)*theta_t - eta_t*g/(|g| + eps)."""
    w = W.tiny_workload(W.OPT_ADAMW, K=2, P=5, T=30, sched=W.SCHED_LINEAR, eta_max=0.05, weight_decay=0.1,
                        rule=W.RULE_CONST_H, H_base=4)
    g = np.array([0.3, -2.0, 1e-4, 5.0, -1e-9])
    S = O.State(w, np.zeros(5), np.zeros(5))
    S.theta[:] = 1.0
    theta = np.ones(5)
    for t in range(w.T):
        S.local_step(t, grads=np.tile(g, (2, 1)))
        eta = w.eta_max * (1 - t / w.T)
        theta = (1 - eta * w.weight_decay) * theta - eta * g / (np.abs(g) + w.eps)
    np.testing.assert_allclose(S.theta[0], theta, rtol=1e-9)
    np.testing.assert_allclose(S.theta[1], theta, rtol=1e-9)
    # first step from theta = 0: -eta_0 * g / (|g| + eps)
    S = O.State(w, np.zeros(5), np.zeros(5))
    S.local_step(0, grads=np.tile(g, (2, 1)))
    np.testing.assert_allclose(S.theta[0], -w.eta_max * g / (np.abs(g) + w.eps), rtol=1e-12)


def test_external_gradients_equal_internal_ones():
    for opt in (W.OPT_SGDM, W.OPT_ADAMW):
        w = W.tiny_workload(opt, K=2, P=12, T=6)
        lam, ths = _inputs(w)
        lam, ths = lam.astype(np.float64), ths.astype(np.float64)
        A, B = O.State(w, lam, ths), O.State(w, lam, ths)
        for t in range(6):
            g = np.stack([_grad(w, lam, ths, B.theta[k], k, t) for k in range(2)])
            A.local_step(t)
            B.local_step(t, grads=g)
        np.testing.assert_allclose(A.theta, B.theta, rtol=1e-13, atol=1e-15)
        assert np.abs(A.theta[0] - A.theta[1]).max() > 1e-3   # workers do see different noise


# ------------------------------------------------------------------ the mean and the round loop

def test_mean_trajectory_does_not_depend_on_the_schedule_for_sgd():
    """The SGD-momentum update is linear in (theta, v, noise) and averaging keeps the means of theta and v, so
    the final average is the same for QSR, H = 1, any constant H and a single final average."""
    base = W.tiny_workload(W.OPT_SGDM, K=4, P=40, T=48, momentum=0.9, weight_decay=0.01)
    lam, ths = _inputs(base)
    finals = []
    for kw in (dict(), dict(rule=W.RULE_CONST_H, H_base=1), dict(rule=W.RULE_CONST_H, H_base=5),
               dict(rule=W.RULE_CONST_H, H_base=48), dict(state_sync=W.STATE_AVERAGE)):
        S = O.State(base.replace(**kw), lam, ths)
        S.run()
        assert np.abs(S.theta - S.theta[0]).max() == 0.0
        finals.append(S.theta[0].copy())
    for f in finals[1:]:
        np.testing.assert_allclose(f, finals[0], rtol=1e-11, atol=1e-13)
    # and it does depend on it once the state is reset at each synchronization
    S = O.State(base.replace(state_sync=W.STATE_RESET), lam, ths)
    S.run()
    assert np.abs(S.theta[0] - finals[0]).max() > 1e-4


def test_adamw_final_point_depends_on_the_schedule():
    base = W.tiny_workload(W.OPT_ADAMW, K=4, P=40, T=48)
    lam, ths = _inputs(base)
    a = O.State(base.replace(rule=W.RULE_CONST_H, H_base=1), lam, ths)
    b = O.State(base.replace(rule=W.RULE_CONST_H, H_base=12), lam, ths)
    a.run(), b.run()
    assert np.abs(a.theta[0] - b.theta[0]).max() > 1e-5


def test_h1_local_sgd_equals_parallel_sgd():
    """Sec. 3 (remark after the theorem): with H = 1 Local SGD is parallel SGD, i.e. Algorithm 1 with the mean gradient."""
    w = W.tiny_workload(W.OPT_SGDM, K=3, P=20, T=25, momentum=0.0, weight_decay=0.0,
                        rule=W.RULE_CONST_H, H_base=1)
    lam, ths = _inputs(w)
    lam, ths = lam.astype(np.float64), ths.astype(np.float64)
    S = O.State(w, lam, ths)
    S.run()
    p = torch.zeros(20, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.SGD([p], lr=1.0)
    for t in range(w.T):
        for g in opt.param_groups:
            g["lr"] = 0.5 * w.eta_max * (1 + math.cos(math.pi * t / w.T))
        th = p.detach().numpy()
        p.grad = torch.from_numpy(np.mean([_grad(w, lam, ths, th, k, t) for k in range(3)], axis=0))
        opt.step()
    np.testing.assert_allclose(S.theta[0], p.detach().numpy(), rtol=1e-11, atol=1e-13)


def test_averaging_invariants():
    rng = np.random.default_rng(5)
    for K in (1, 2, 3, 8):
        w = W.tiny_workload(W.OPT_ADAMW, K=K, P=33)
        S = O.State(w, np.ones(33), np.zeros(33))
        S.theta[:] = rng.standard_normal((K, 33))
        S.s1[:] = rng.standard_normal((K, 33))
        before, s1_before = S.theta.copy(), S.s1.copy()
        S.sync()
        np.testing.assert_allclose(S.theta[0], before.mean(axis=0), rtol=1e-14, atol=1e-16)
        assert (S.theta == S.theta[0]).all()
        assert np.array_equal(S.s1, s1_before)          # state kept per worker
        once = S.theta.copy()
        S.sync()
        if K <= 2:
            assert np.array_equal(S.theta, once)       # x + x and (2x)/2 are exact
        else:
            np.testing.assert_allclose(S.theta, once, rtol=4e-16)   # a running sum of equal terms may round
        if K == 1:
            assert np.array_equal(once, before)


def test_state_modes_at_sync():
    rng = np.random.default_rng(6)
    for mode in (W.STATE_AVERAGE, W.STATE_RESET):
        w = W.tiny_workload(W.OPT_ADAMW, K=4, P=9, state_sync=mode)
        S = O.State(w, np.ones(9), np.zeros(9))
        S.s1[:] = rng.standard_normal((4, 9))
        S.s2[:] = rng.random((4, 9))
        m, v = S.s1.copy(), S.s2.copy()
        S.sync(t_next=17)
        if mode == W.STATE_AVERAGE:
            np.testing.assert_allclose(S.s1, np.tile(m.mean(0), (4, 1)), rtol=1e-14)
            np.testing.assert_allclose(S.s2, np.tile(v.mean(0), (4, 1)), rtol=1e-14)
            assert S.t_state_origin == 0
        else:
            assert not S.s1.any() and not S.s2.any() and S.t_state_origin == 17


def test_reset_mode_restarts_adamw_each_round():
    """K = 1, constant H, state reset: every round is a fresh torch AdamW started from the round's first iterate."""
    w = W.tiny_workload(W.OPT_ADAMW, K=1, P=10, T=12, rule=W.RULE_CONST_H, H_base=4, state_sync=W.STATE_RESET,
                        eta_max=0.02)
    lam, ths = _inputs(w)
    lam, ths = lam.astype(np.float64), ths.astype(np.float64)
    S = O.State(w, lam, ths)
    S.run()
    p = torch.zeros(10, dtype=torch.float64, requires_grad=True)
    for s in range(3):
        opt = torch.optim.AdamW([p], lr=1.0, betas=(0.9, 0.999), eps=1e-8, weight_decay=w.weight_decay)
        for t in range(4 * s, 4 * s + 4):
            for g in opt.param_groups:
                g["lr"] = 0.5 * w.eta_max * (1 + math.cos(math.pi * t / w.T))
            p.grad = torch.from_numpy(_grad(w, lam, ths, p.detach().numpy(), 0, t))
            opt.step()
    np.testing.assert_allclose(S.theta[0], p.detach().numpy(), rtol=1e-10, atol=1e-13)


def test_tiny_run_by_brute_force():
    """K=2, P=3, T=6, AdamW, QSR with alpha chosen so that the rounds are 2, 2, 2(truncated from 3): every step
    written out with Python floats -- global-step learning rates, per-worker noise, averaging at round ends,
    bias correction counted over the whole run."""
    w = W.tiny_workload(W.OPT_ADAMW, K=2, P=3, T=6, eta_max=0.1, alpha=0.12, H_base=2, weight_decay=0.1,
                        noise_std=0.2)
    lam, ths = np.array([0.5, 1.0, 0.01]), np.array([1.0, -1.0, 0.3])
    S = O.State(w, lam, ths)
    starts, H = S.run()
    eta = [0.05 * (1 + math.cos(math.pi * t / 6)) for t in range(6)]
    # Eq. 2 by hand: t=0: (0.12/0.1)^2=1.44 -> 2; t=2: eta=0.075, 2.56 -> 2; t=4: eta=0.025, 23.04 -> 23 -> 6-4=2
    assert starts.tolist() == [0, 2, 4] and H.tolist() == [2, 2, 2]
    th = [[0.0] * 3 for _ in range(2)]
    m = [[0.0] * 3 for _ in range(2)]
    v = [[0.0] * 3 for _ in range(2)]
    for t in range(6):
        for k in range(2):
            for i in range(3):
                g = lam[i] * (th[k][i] - ths[i]) + 0.2 * O.noise(w.noise_seed, k, t, i)
                th[k][i] *= 1 - eta[t] * 0.1
                m[k][i] = 0.9 * m[k][i] + 0.1 * g
                v[k][i] = 0.999 * v[k][i] + 0.001 * g * g
                th[k][i] -= eta[t] * (m[k][i] / (1 - 0.9 ** (t + 1))) / (math.sqrt(v[k][i] / (1 - 0.999 ** (t + 1))) + 1e-8)
        if t in (1, 3, 5):
            for i in range(3):
                mean = (th[0][i] + th[1][i]) / 2
                th[0][i] = th[1][i] = mean
    np.testing.assert_allclose(S.theta, np.array(th), rtol=1e-11, atol=1e-14)


def test_resume_is_exact():
    """Noise is addressed by the global step, so stopping at a round boundary and continuing changes nothing."""
    for opt in (W.OPT_SGDM, W.OPT_ADAMW):
        w = W.tiny_workload(opt, K=3, P=17, T=60)
        lam, ths = _inputs(w)
        A = O.State(w, lam, ths)
        sa, Ha = A.run()
        B = O.State(w, lam, ths)
        s1, H1 = B.run(0, 30)
        t_mid = int(s1[-1] + H1[-1])
        s2, H2 = B.run(t_mid, w.T)
        assert np.array_equal(np.concatenate([s1, s2]), sa) and np.array_equal(np.concatenate([H1, H2]), Ha)
        assert np.array_equal(A.theta, B.theta)


def test_sgd_stationary_variance():
    """Plain SGD (mu = 0) on one curvature with constant eta: Var[theta_k] -> eta*sigma^2/(lam*(2 - eta*lam)); the
    K-average under H = 1 has 1/K of it."""
    n, eta, lam_v, sigma, K = 20000, 0.2, 0.5, 0.3, 4
    w = W.tiny_workload(W.OPT_SGDM, K=K, P=n, T=200, sched=W.SCHED_CONST, eta_max=eta, momentum=0.0,
                        weight_decay=0.0, noise_std=sigma, rule=W.RULE_CONST_H, H_base=200)
    S = O.State(w, np.full(n, lam_v), np.zeros(n))
    for t in range(199):
        S.local_step(t)
    var = eta * sigma ** 2 / (lam_v * (2 - eta * lam_v))
    assert S.theta.var() == pytest.approx(var, rel=0.03)
    w1 = w.replace(H_base=1)
    S = O.State(w1, np.full(n, lam_v), np.zeros(n))
    S.run()
    assert S.theta[0].var() == pytest.approx(var / K, rel=0.05)


def test_coordinate_subset_equals_the_same_columns_of_the_full_run():
    """Coordinates never interact (diagonal loss, per-coordinate mean), so a run on a subset of columns, with the
    noise addressed by the *global* coordinate index, reproduces those columns of the full run bit for bit."""
    for opt in (W.OPT_SGDM, W.OPT_ADAMW):
        w = W.tiny_workload(opt, K=3, P=203, T=30)
        lam, ths = _inputs(w)
        full = O.State(w, lam, ths)
        full.run()
        idx = np.array([0, 1, 5, 6, 7, 100, 201, 202], np.int64)
        sub = O.State(w, lam[idx], ths[idx], idx=idx)
        sub.run()
        assert np.array_equal(sub.theta, full.theta[:, idx])


# ------------------------------------------------------------------ Algorithm 1 (Parallel OPT)

def test_parallel_opt_equals_torch_with_the_mean_gradient():
    """Algorithm 1: one model, K gradients at the same point, their mean fed to torch.optim."""
    for opt in (W.OPT_SGDM, W.OPT_ADAMW):
        K = 5
        w = W.tiny_workload(opt, K=K, P=14, T=30, weight_decay=0.02)
        lam, ths = _inputs(w)
        lam, ths = lam.astype(np.float64), ths.astype(np.float64)
        S = O.State(w, lam, ths, rows=1)
        p = torch.zeros(14, dtype=torch.float64, requires_grad=True)
        if opt == W.OPT_SGDM:
            topt = torch.optim.SGD([p], lr=1.0, momentum=w.momentum, weight_decay=w.weight_decay)
        else:
            topt = torch.optim.AdamW([p], lr=1.0, betas=(w.beta1, w.beta2), eps=w.eps, weight_decay=w.weight_decay)
        for t in range(w.T):
            S.parallel_step(t, K)
            for g in topt.param_groups:
                g["lr"] = 0.5 * w.eta_max * (1 + math.cos(math.pi * t / w.T))
            th = p.detach().numpy()
            p.grad = torch.from_numpy(np.mean([_grad(w, lam, ths, th, k, t) for k in range(K)], axis=0))
            topt.step()
        np.testing.assert_allclose(S.theta[0], p.detach().numpy(), rtol=1e-10, atol=1e-13)


def test_local_sgd_with_h1_is_parallel_sgd_also_with_momentum():
    """Sec. 3: Local SGD with H = 1 is parallel SGD.  With per-worker momentum buffers kept across rounds the mean
    buffer obeys the parallel recursion, so the statement extends to heavy-ball momentum (not to AdamW)."""
    K = 4
    w = W.tiny_workload(W.OPT_SGDM, K=K, P=22, T=40, momentum=0.9, weight_decay=0.01, rule=W.RULE_CONST_H, H_base=1)
    lam, ths = _inputs(w)
    local = O.State(w, lam, ths)
    local.run()
    par = O.State(w, lam, ths, rows=1)
    for t in range(w.T):
        par.parallel_step(t, K)
    np.testing.assert_allclose(local.theta[0], par.theta[0], rtol=1e-11, atol=1e-13)
    wa = w.replace(opt=W.OPT_ADAMW, eta_max=0.02)
    la, pa = O.State(wa, lam, ths), O.State(wa, lam, ths, rows=1)
    la.run()
    for t in range(wa.T):
        pa.parallel_step(t, K)
    assert np.abs(la.theta[0] - pa.theta[0]).max() > 1e-6


def test_parallel_opt_external_gradients():
    K = 3
    w = W.tiny_workload(W.OPT_ADAMW, K=K, P=9, T=8)
    lam, ths = _inputs(w)
    lam, ths = lam.astype(np.float64), ths.astype(np.float64)
    A, Bq = O.State(w, lam, ths, rows=1), O.State(w, lam, ths, rows=1)
    for t in range(w.T):
        g = np.stack([_grad(w, lam, ths, Bq.theta[0], k, t) for k in range(K)])
        A.parallel_step(t, K)
        Bq.parallel_step(t, K, grads=g)
    np.testing.assert_allclose(A.theta, Bq.theta, rtol=1e-13, atol=1e-15)


def test_per_tensor_weight_decay_equals_torch_param_groups():
    """Two 'tensors', one with the run's weight decay and one exempt (factor 0), against torch parameter groups."""
    for opt in (W.OPT_SGDM, W.OPT_ADAMW):
        w = W.tiny_workload(opt, K=1, P=12, T=25, weight_decay=0.1)
        lam, ths = _inputs(w)
        lam, ths = lam.astype(np.float64), ths.astype(np.float64)
        scale = np.array([1.0] * 8 + [0.0] * 4)
        S = O.State(w, lam, ths, wd_scale=scale)
        S.run()
        pa = torch.zeros(8, dtype=torch.float64, requires_grad=True)
        pb = torch.zeros(4, dtype=torch.float64, requires_grad=True)
        groups = [{"params": [pa], "weight_decay": 0.1}, {"params": [pb], "weight_decay": 0.0}]
        topt = (torch.optim.SGD(groups, lr=1.0, momentum=w.momentum) if opt == W.OPT_SGDM
                else torch.optim.AdamW(groups, lr=1.0, betas=(w.beta1, w.beta2), eps=w.eps))
        for t in range(w.T):
            for g in topt.param_groups:
                g["lr"] = 0.5 * w.eta_max * (1 + math.cos(math.pi * t / w.T))
            th = np.concatenate([pa.detach().numpy(), pb.detach().numpy()])
            g = _grad(w, lam, ths, th, 0, t)
            pa.grad, pb.grad = torch.from_numpy(g[:8].copy()), torch.from_numpy(g[8:].copy())
            topt.step()
        got = np.concatenate([pa.detach().numpy(), pb.detach().numpy()])
        np.testing.assert_allclose(S.theta[0], got, rtol=1e-10, atol=1e-13)
        plain = O.State(w, lam, ths)
        plain.run()
        assert np.abs(plain.theta[0, 8:] - S.theta[0, 8:]).max() > 1e-6


# ------------------------------------------------------------------ gradient clipping (App. C.2)

def test_clipped_single_worker_equals_torch_clip_grad_norm():
    for opt in (W.OPT_SGDM, W.OPT_ADAMW):
        w = W.tiny_workload(opt, K=1, P=18, T=30, clip_norm=0.35, noise_std=0.3)
        lam, ths = _inputs(w)
        lam, ths = lam.astype(np.float64), ths.astype(np.float64)
        S = O.State(w, lam, ths)
        S.run()
        p = torch.zeros(18, dtype=torch.float64, requires_grad=True)
        topt = (torch.optim.SGD([p], lr=1.0, momentum=w.momentum, weight_decay=w.weight_decay) if opt == W.OPT_SGDM
                else torch.optim.AdamW([p], lr=1.0, betas=(w.beta1, w.beta2), eps=w.eps, weight_decay=w.weight_decay))
        clipped = 0
        for t in range(w.T):
            for g in topt.param_groups:
                g["lr"] = 0.5 * w.eta_max * (1 + math.cos(math.pi * t / w.T))
            p.grad = torch.from_numpy(_grad(w, lam, ths, p.detach().numpy(), 0, t))
            clipped += float(torch.nn.utils.clip_grad_norm_([p], 0.35)) > 0.35
            topt.step()
        assert 0 < clipped                                  # the threshold did bite
        np.testing.assert_allclose(S.theta[0], p.detach().numpy(), rtol=1e-10, atol=1e-13)
        free = O.State(w.replace(clip_norm=0.0), lam, ths)
        free.run()
        assert np.abs(free.theta[0] - S.theta[0]).max() > 1e-4


def test_clipping_closed_form_and_inactive_threshold():
    """Plain SGD on a constant gradient g with ||g|| > c: every step moves by eta_t * c * g / (||g|| + 1e-6)."""
    w = W.tiny_workload(W.OPT_SGDM, K=2, P=4, T=10, momentum=0.0, weight_decay=0.0, sched=W.SCHED_CONST, eta_max=0.1,
                        clip_norm=0.5, rule=W.RULE_CONST_H, H_base=10)
    g = np.array([3.0, -4.0, 0.0, 12.0])                  # norm 13
    S = O.State(w, np.zeros(4), np.zeros(4))
    for t in range(w.T):
        S.local_step(t, grads=np.tile(g, (2, 1)))
    np.testing.assert_allclose(S.theta[0], -10 * 0.1 * 0.5 * g / (13.0 + 1e-6), rtol=1e-12)
    # a threshold above every gradient norm changes nothing
    a = W.tiny_workload(W.OPT_ADAMW, K=3, P=15, T=20)
    lam, ths = _inputs(a)
    x, y = O.State(a, lam, ths), O.State(a.replace(clip_norm=1e6), lam, ths)
    x.run(), y.run()
    assert np.array_equal(x.theta, y.theta)


def test_clipping_is_per_worker():
    """Each worker clips by its own gradient norm: a worker with a small gradient is left alone."""
    w = W.tiny_workload(W.OPT_SGDM, K=2, P=3, T=5, momentum=0.0, weight_decay=0.0, sched=W.SCHED_CONST, eta_max=1.0,
                        clip_norm=1.0)
    S = O.State(w, np.zeros(3), np.zeros(3))
    g = np.array([[0.3, 0.0, 0.4], [30.0, 0.0, 40.0]])   # norms 0.5 and 50
    S.local_step(0, grads=g)
    np.testing.assert_allclose(S.theta[0], -g[0], rtol=1e-13)
    np.testing.assert_allclose(S.theta[1], -g[1] / (50.0 + 1e-6), rtol=1e-13)
