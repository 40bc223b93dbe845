"""The oracle's binary32-storage build (the "mirror") and the conditioning yardstick, on the CPU alone.

The mirror stores parameters, state and gradients in binary32 and evaluates the gradient in binary32; everything else
is evaluated in binary64 and rounded once.  Its distance from the binary64 build is what fp32 costs on a run.  These
tests pin three things the GPU parity tests lean on:
  - on well-conditioned runs that distance is rounding-sized (far inside the parity bar of 1e-5);
  - on the runs where AdamW takes first steps at a non-zero learning rate a handful of coordinates leave the bar, and
    they are exactly the ones the yardstick of conditioning.py marks (binary64 oracle, gradients moved by one fp32 ulp);
  - writing AdamW's decay as theta * (1 - eta * wd) in fp32 drifts, which is why the CUDA kernel forms the decay and
    the update as one subtraction (a numpy restatement of the two orders on one coordinate).
"""
import numpy as np
import pytest

import conditioning
from oracle import qsr_oracle as O
from paper_2310_14423_b200 import workloads as W

REL_TOL = 1e-5
SENS_FACTOR = 2.0


def _rel(a, b):
    b = np.asarray(b, np.float64)
    floor = np.sqrt(np.mean(b * b))
    return np.abs(np.asarray(a, np.float64) - b) / np.maximum(np.abs(b), floor)


def _both(w):
    lam, ths = W.draw_inputs(w.P, w.data_seed)
    a = O.State(w, lam, ths)
    b = O.State(w, lam, ths, mirror=True)
    sa, sb = a.run(), b.run()
    assert np.array_equal(sa[0], sb[0]) and np.array_equal(sa[1], sb[1])       # the schedule is binary64 in both
    assert b.theta.dtype == np.float32 and a.theta.dtype == np.float64
    return lam, ths, a, b


@pytest.mark.parametrize("opt,kw", [
    (W.OPT_SGDM, dict(T=400)),
    (W.OPT_SGDM, dict(T=400, state_sync=W.STATE_RESET)),
    (W.OPT_ADAMW, dict(T=600, T_warmup=60)),                                   # warm-up from eta_0 = 0, as the run configs
    (W.OPT_ADAMW, dict(T=600, T_warmup=60, state_sync=W.STATE_AVERAGE)),
])
def test_mirror_is_rounding_close_on_well_conditioned_runs(opt, kw):
    w = W.tiny_workload(opt, K=4, P=20000, **kw)
    _, _, a, b = _both(w)
    assert _rel(b.theta[0], a.theta[0]).max() < 1.5e-6


@pytest.mark.parametrize("K,P,T,mode,clip", [
    (3, 99999, 40, W.STATE_KEEP, 0.0),        # AdamW from the full learning rate, short
    (8, 99999, 60, W.STATE_RESET, 0.0),       # moments reset at every synchronization
    (5, 300000, 30, W.STATE_KEEP, 55.0),      # with gradient clipping
])
def test_ill_conditioned_coordinates_are_the_ones_the_yardstick_marks(K, P, T, mode, clip):
    w = W.tiny_workload(W.OPT_ADAMW, K=K, P=P, T=T, state_sync=mode, clip_norm=clip)
    lam, ths, a, b = _both(w)
    rel = _rel(b.theta[0], a.theta[0])
    assert rel.max() > REL_TOL                                   # fp32 storage + fp32 gradient alone miss the bar here
    out = np.nonzero(rel > REL_TOL)[0]
    assert out.size <= 1e-4 * P                                  # ... on a handful of coordinates
    assert np.median(rel) < 1e-7                                 # ... while the bulk is at rounding level
    sens = conditioning.fp32_sensitivity(w, lam, ths)
    excess = conditioning.excess_over(b.theta[0], a.theta[0], REL_TOL)
    assert np.all(excess <= SENS_FACTOR * sens)                  # every miss is explained by the run's conditioning
    scale = np.maximum(np.abs(a.theta[0]), np.sqrt(np.mean(a.theta[0] ** 2)))
    marked = np.nonzero(sens > REL_TOL * scale)[0]
    assert set(out.tolist()) <= set(marked.tolist()) and marked.size <= 2e-4 * P


def test_yardstick_is_small_where_the_run_is_well_conditioned():
    w = W.tiny_workload(W.OPT_ADAMW, K=3, P=5000, T=200, T_warmup=40)
    lam, ths = W.draw_inputs(w.P, w.data_seed)
    a = O.State(w, lam, ths)
    a.run()
    sens = conditioning.fp32_sensitivity(w, lam, ths)
    scale = np.maximum(np.abs(a.theta[0]), np.sqrt(np.mean(a.theta[0] ** 2)))
    assert (sens / scale).max() < 2e-6


def test_fp32_decay_as_a_separate_product_drifts():
    """theta <- theta (1 - eta wd), then theta <- theta - step, in fp32, against theta <- theta - (eta wd theta + step):
    with eta wd = 4e-5 the factor 1 - eta wd keeps 2^-24 of absolute precision and the product has near-ties that
    round the same way step after step for theta just above a power of two.  5,000 steps of pure decay plus a
    constant small pull, every operation rounded to fp32 once."""
    f = np.float32
    eta_wd, step = f(8e-4 * 0.05), f(2.5e-9)
    theta0 = np.nextafter(f(1.0), f(2.0)) + f(3e-4)
    exact = float(theta0)
    a = b = theta0
    one_minus = f(1.0) - eta_wd
    for _ in range(5000):
        exact = exact - (float(eta_wd) * exact + float(step))
        a = f(a * one_minus) - step                                     # product rounded, then the subtraction
        fused = f(np.float64(eta_wd) * np.float64(b) + np.float64(step))    # one rounding, as a fused multiply-add
        b = b - fused
    err_a, err_b = abs(float(a) - exact) / exact, abs(float(b) - exact) / exact
    assert err_a > 1e-5 and err_b < 2e-6, (err_a, err_b)
    print(f"separate product: {err_a:.2e}; one subtraction: {err_b:.2e}")
