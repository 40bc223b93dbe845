"""How far fp32 rounding of the gradient can move a run: a per-coordinate yardstick taken from the binary64 oracle.

Almost every run of the path is well conditioned and the parity bar (REL_TOL of gpu_harness) holds on every
coordinate.  The exception is AdamW's first step after its moments were zero -- the start of a run, and every round
start in state mode RESET: it moves a coordinate by eta * g / (|g| + eps) with eps = 1e-8, and where the two terms of
g = lambda (theta - theta*) + sigma z happen to cancel to within a few eps, the ~1e-8 absolute rounding error of that
fp32 sum decides the size of the step.  About one coordinate-worker in 1e6 is hit per such step, the damage is at most
eta, and later steps contract it away.  Which coordinates are hit, and how hard, is a property of the run, not of the
kernel, and the oracle can measure it: run it in binary64 with every gradient moved by one binary32 ulp of its two
terms and see how far each coordinate goes.
"""
from __future__ import annotations

import numpy as np

from oracle import qsr_oracle as O

ULP32 = 2.0 ** -23


def fp32_sensitivity(w, lam: np.ndarray, ths: np.ndarray) -> np.ndarray:
    """|theta_perturbed - theta| of worker 0 at the end of the run, per coordinate [P], the larger of the two signs,
    where every gradient of the perturbed run is g +- ULP32 * (|lambda (theta - theta*)| + sigma |z|).
    All coordinates, all workers, the whole schedule (clipping included: it acts on the gradient handed over)."""
    starts, H = O.schedule(w)
    ends = set((starts + H).tolist())
    lam64, ths64 = lam.astype(np.float64), ths.astype(np.float64)
    base = O.State(w, lam, ths)
    base.run()
    worst = np.zeros(w.P)
    for sign in (1.0, -1.0):
        S = O.State(w, lam, ths)
        for t in range(w.T):
            z = np.stack([O.noise_fill(w.noise_seed, k, t, 0, w.P) for k in range(w.K)])
            pull = lam64 * (S.theta - ths64)
            g = pull + w.noise_std * z
            S.local_step(t, grads=g + sign * ULP32 * (np.abs(pull) + w.noise_std * np.abs(z)))
            if t + 1 in ends:
                S.sync(t + 1)
        worst = np.maximum(worst, np.abs(S.theta[0] - base.theta[0]))
    return worst


def excess_over(theta: np.ndarray, ref: np.ndarray, rel_tol: float) -> np.ndarray:
    """Per coordinate, what |theta - ref| exceeds rel_tol * max(|ref|, rms(ref)) by (zero where it does not)."""
    ref = np.asarray(ref, np.float64)
    floor = float(np.sqrt(np.mean(ref * ref)))
    return np.maximum(0.0, np.abs(np.asarray(theta, np.float64) - ref) - rel_tol * np.maximum(np.abs(ref), max(floor, 1e-30)))
