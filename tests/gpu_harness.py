"""Helpers shared by the GPU parity tests: device slabs with guard regions, the error metric, oracle runs."""
from __future__ import annotations

import numpy as np
import torch

import conditioning
from oracle import qsr_oracle as O
from paper_2310_14423_b200 import binding as B
from paper_2310_14423_b200 import workloads as W

GUARD = 64          # floats of canary before and after every slab
CANARY = 1234.5

# Parity bound for final parameters (fp32 path against the binary64 oracle):
#   max_i |theta_gpu[i] - theta_oracle[i]| / max(|theta_oracle[i]|, rms(theta_oracle))  <=  1e-5
REL_TOL = 1e-5
SENS_FACTOR = 2.0    # see assert_parity


def rel_err(gpu: np.ndarray, orc: np.ndarray) -> float:
    orc = np.asarray(orc, np.float64)
    gpu = np.asarray(gpu, np.float64)
    floor = float(np.sqrt(np.mean(orc * orc)))
    denom = np.maximum(np.abs(orc), max(floor, 1e-30))
    return float(np.max(np.abs(gpu - orc) / denom))


def assert_parity(theta_gpu, w, lam, ths, orc_theta, context=None) -> float:
    """The parity bar for one finished all-coordinate run: rel_err <= REL_TOL on every coordinate.  Where a coordinate
    misses it, the miss must be explained by the run's own conditioning (see conditioning.py): the excess over REL_TOL
    may be at most SENS_FACTOR times what the binary64 oracle itself moves on that coordinate when its gradients are
    perturbed by one fp32 ulp.  Returns the relative error."""
    err = rel_err(theta_gpu, orc_theta)
    if err > REL_TOL:
        sens = conditioning.fp32_sensitivity(w, lam, ths)
        excess = conditioning.excess_over(theta_gpu, orc_theta, REL_TOL)
        bad = np.nonzero(excess > SENS_FACTOR * sens)[0]
        assert bad.size == 0, (err, bad[:8], excess[bad[:8]], sens[bad[:8]], context)
    return err


class Slabs:
    """[K, row_stride] fp32 slabs on the device, each inside a guarded allocation."""

    def __init__(self, w, K=None, row_stride=None, n_extra=0, device="cuda:0"):
        self.w = w
        self.K = int(w.K if K is None else K)
        self.P = int(w.P)
        self.stride = int((self.P + 3) // 4 * 4 if row_stride is None else row_stride)
        self.device = device
        self._raw = []
        self.theta = self._slab()
        self.s1 = self._slab()
        self.s2 = self._slab() if w.opt == W.OPT_ADAMW else None
        self.extra = [self._slab() for _ in range(n_extra)]

    def _slab(self):
        raw = torch.full((GUARD + self.K * self.stride + GUARD,), CANARY, dtype=torch.float32, device=self.device)
        self._raw.append(raw)
        body = raw[GUARD:GUARD + self.K * self.stride].view(self.K, self.stride)
        body[:, :self.P] = 0.0
        return body

    def guards_intact(self) -> bool:
        ok = True
        for raw in self._raw:
            ok &= bool((raw[:GUARD] == CANARY).all()) and bool((raw[-GUARD:] == CANARY).all())
            body = raw[GUARD:GUARD + self.K * self.stride].view(self.K, self.stride)
            if self.stride > self.P:
                ok &= bool((body[:, self.P:] == CANARY).all())
        return ok


def device_inputs(w, device="cuda:0"):
    lam, ths = W.draw_inputs(w.P, w.data_seed)
    pad = (-w.P) % 4
    lam_d = torch.from_numpy(np.concatenate([lam, np.zeros(pad, np.float32)])).to(device)[:w.P]
    ths_d = torch.from_numpy(np.concatenate([ths, np.zeros(pad, np.float32)])).to(device)[:w.P]
    return lam, ths, lam_d, ths_d


def make_context(w, slabs: Slabs, lam_d, ths_d, **cfg_kw):
    cfg = B.make_config(w, K=slabs.K, row_stride=slabs.stride, **cfg_kw)
    return B.Context(cfg, slabs.theta, slabs.s1, slabs.s2, lam_d, ths_d,
                     stream=torch.cuda.current_stream().cuda_stream)


def oracle_on(w, lam, ths, idx=None, mirror=False):
    if idx is None:
        return O.State(w, lam, ths, mirror=mirror)
    return O.State(w, lam[idx], ths[idx], idx=idx, mirror=mirror)
