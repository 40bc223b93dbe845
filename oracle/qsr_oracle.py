"""ctypes front end of the CPU oracle (qsr_oracle.c)  --  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this module.
It compiles the C file with gcc on first use (binary64 build, and a "mirror" build with binary32
storage used only to size rounding error) and marshals numpy arrays; it contains no arithmetic of its own
and imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "qsr_oracle.c")
_LOCK = threading.Lock()
_LIBS = {}

OPT = {"sgdm": 0, "adamw": 1}
SCHED = {"cosine": 0, "step_pow2": 1, "linear": 2, "const": 3, "halving": 4, "cosine_held": 5}
RULE = {"qsr": 0, "const_h": 1, "power": 2, "post_local": 3, "swap": 4}
STATE = {"keep": 0, "average": 1, "reset": 2}


class OrcConfig(C.Structure):
    _fields_ = [("opt", C.c_int32), ("sched", C.c_int32), ("rule", C.c_int32), ("state_sync", C.c_int32),
                ("momentum", C.c_double), ("beta1", C.c_double), ("beta2", C.c_double), ("eps", C.c_double),
                ("weight_decay", C.c_double), ("eta_max", C.c_double), ("eta_min", C.c_double),
                ("alpha", C.c_double), ("noise_std", C.c_double),
                ("T", C.c_int64), ("T_warmup", C.c_int64), ("H_base", C.c_int64), ("seed", C.c_uint64),
                ("gamma", C.c_double), ("t_switch", C.c_int64), ("t_hold", C.c_int64), ("t_period", C.c_int64),
                ("wd_scale", C.c_void_p), ("clip_norm", C.c_double)]


def build(force: bool = False) -> None:
    """Compile both builds of the oracle next to its source (no-op when they are up to date)."""
    for mirror in (False, True):
        out = _so_path(mirror)
        if not force and os.path.exists(out) and os.path.getmtime(out) >= os.path.getmtime(_SRC):
            continue
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off", _SRC, "-o", out + ".tmp", "-lm"]
        if mirror:
            cmd.insert(1, "-DORC_REAL=float")
        subprocess.run(cmd, check=True)
        os.replace(out + ".tmp", out)


def _so_path(mirror: bool) -> str:
    return os.path.join(_HERE, "liborc_f32.so" if mirror else "liborc_f64.so")


def _lib(mirror: bool = False):
    with _LOCK:
        if mirror not in _LIBS:
            build()
            lib = C.CDLL(_so_path(mirror))
            p = C.c_void_p
            cfg = C.POINTER(OrcConfig)
            lib.orc_sizeof_real.restype = C.c_int
            lib.orc_lr.restype = C.c_double
            lib.orc_lr.argtypes = [cfg, C.c_int64]
            lib.orc_round_length.restype = C.c_int64
            lib.orc_round_length.argtypes = [cfg, C.c_int64]
            lib.orc_philox4x32_10.restype = None
            lib.orc_philox4x32_10.argtypes = [p, p, p]
            lib.orc_noise.restype = C.c_double
            lib.orc_noise.argtypes = [C.c_uint64, C.c_int64, C.c_int64, C.c_int64]
            lib.orc_noise_fill.restype = None
            lib.orc_noise_fill.argtypes = [C.c_uint64, C.c_int64, C.c_int64, C.c_int64, C.c_int64, p]
            lib.orc_box_muller_parts_fill.restype = None
            lib.orc_box_muller_parts_fill.argtypes = [p, p, C.c_int64, p, p, p]
            lib.orc_local_step.restype = C.c_int
            lib.orc_local_step.argtypes = [cfg, C.c_int64, C.c_int64, C.c_int64, p, p, p, p, p, p, p, C.c_int64, C.c_int64]
            lib.orc_parallel_step.restype = C.c_int
            lib.orc_parallel_step.argtypes = [cfg, C.c_int64, C.c_int64, p, p, p, p, p, p, p, C.c_int64, C.c_int64]
            lib.orc_sync.restype = None
            lib.orc_sync.argtypes = [cfg, C.c_int64, C.c_int64, p, p, p]
            lib.orc_run.restype = C.c_int64
            lib.orc_run.argtypes = [cfg, C.c_int64, C.c_int64, p, p, p, p, p, p, C.c_int64, C.c_int64, p, p, p, C.c_int64]
            lib.orc_schedule.restype = C.c_int64
            lib.orc_schedule.argtypes = [cfg, p, p, C.c_int64]
            assert lib.orc_sizeof_real() == (4 if mirror else 8)
            _LIBS[mirror] = lib
        return _LIBS[mirror]


def config_from(w) -> OrcConfig:
    """Translate a workload description (any object with the Workload fields) into the oracle's struct."""
    return OrcConfig(opt=OPT[w.opt], sched=SCHED[w.sched], rule=RULE[w.rule], state_sync=STATE[w.state_sync],
                     momentum=w.momentum, beta1=w.beta1, beta2=w.beta2, eps=w.eps, weight_decay=w.weight_decay,
                     eta_max=w.eta_max, eta_min=w.eta_min, alpha=w.alpha, noise_std=w.noise_std,
                     T=w.T, T_warmup=w.T_warmup, H_base=w.H_base, seed=w.noise_seed,
                     gamma=getattr(w, "gamma", 2.0), t_switch=getattr(w, "t_switch", 0),
                     t_hold=getattr(w, "t_hold", 0), t_period=max(1, getattr(w, "t_period", 1)),
                     clip_norm=float(getattr(w, "clip_norm", 0.0)))


def set_threads(n: int) -> None:
    os.environ["OMP_NUM_THREADS"] = str(n)


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def lr(w, t: int) -> float:
    return float(_lib().orc_lr(C.byref(config_from(w)), int(t)))


def round_length(w, t: int) -> int:
    return int(_lib().orc_round_length(C.byref(config_from(w)), int(t)))


def schedule(w) -> Tuple[np.ndarray, np.ndarray]:
    """(round starts, round lengths) of the whole run, as int64 arrays."""
    cap = int(w.T)
    st = np.empty(cap, np.int64)
    H = np.empty(cap, np.int64)
    n = _lib().orc_schedule(C.byref(config_from(w)), _ptr(st), _ptr(H), cap)
    if n < 0:
        raise ValueError("bad schedule arguments")
    return st[:n].copy(), H[:n].copy()


def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, np.uint32).copy()
    k = np.asarray(key, np.uint32).copy()
    out = np.empty(4, np.uint32)
    _lib().orc_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def noise(seed: int, k: int, u: int, i: int) -> float:
    return float(_lib().orc_noise(C.c_uint64(seed), int(k), int(u), int(i)))


def noise_fill(seed: int, k: int, u: int, i0: int, n: int) -> np.ndarray:
    out = np.empty(int(n), np.float64)
    _lib().orc_noise_fill(C.c_uint64(seed), int(k), int(u), int(i0), int(n), _ptr(out))
    return out


def box_muller_parts(a, b) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """(radius, sine, cosine) of the Box-Muller transform for arrays of 23-bit fields a (radius) and b (angle)."""
    a = np.ascontiguousarray(a, np.uint32)
    b = np.ascontiguousarray(b, np.uint32)
    assert a.shape == b.shape and a.ndim == 1
    radius, sine, cosine = (np.empty(a.size, np.float64) for _ in range(3))
    _lib().orc_box_muller_parts_fill(_ptr(a), _ptr(b), a.size, _ptr(radius), _ptr(sine), _ptr(cosine))
    return radius, sine, cosine


class State:
    """Parameters and optimizer state of K workers on a set of coordinates, in the oracle's precision."""

    def __init__(self, w, lam: np.ndarray, theta_star: np.ndarray, idx: Optional[np.ndarray] = None,
                 mirror: bool = False, rows: Optional[int] = None, k0: int = 0,
                 wd_scale: Optional[np.ndarray] = None):
        self.w = w
        self.mirror = mirror
        self.dtype = np.float32 if mirror else np.float64
        self.rows = int(w.K if rows is None else rows)
        self.k0 = int(k0)
        self.n = int(lam.shape[0])
        self.idx = None if idx is None else np.ascontiguousarray(idx, np.int64)
        assert self.idx is None or self.idx.shape[0] == self.n
        self.lam = np.ascontiguousarray(lam, self.dtype)
        self.theta_star = np.ascontiguousarray(theta_star, self.dtype)
        self.theta = np.zeros((self.rows, self.n), self.dtype)
        self.s1 = np.zeros((self.rows, self.n), self.dtype)
        self.s2 = np.zeros((self.rows, self.n), self.dtype)
        self.t_state_origin = 0
        self.cfg = config_from(w)
        self.wd_scale = None
        if wd_scale is not None:                       # one weight-decay factor per column, always binary64
            self.wd_scale = np.ascontiguousarray(wd_scale, np.float64)
            assert self.wd_scale.shape == (self.n,)
            self.cfg.wd_scale = self.wd_scale.ctypes.data

    def local_step(self, t: int, grads: Optional[np.ndarray] = None) -> None:
        g = None if grads is None else np.ascontiguousarray(grads, self.dtype)
        _lib(self.mirror).orc_local_step(C.byref(self.cfg), self.rows, self.k0, self.n, _ptr(self.idx),
                                         _ptr(self.lam), _ptr(self.theta_star), _ptr(self.theta), _ptr(self.s1),
                                         _ptr(self.s2), _ptr(g), int(t), int(t - self.t_state_origin))

    def parallel_step(self, t: int, K: int, grads: Optional[np.ndarray] = None) -> None:
        """Algorithm 1 on row 0 (the single model): K workers' gradients at the same point, averaged, one OPT step."""
        g = None if grads is None else np.ascontiguousarray(grads, self.dtype)
        assert g is None or g.shape == (K, self.n)
        rc = _lib(self.mirror).orc_parallel_step(C.byref(self.cfg), int(K), self.n, _ptr(self.idx), _ptr(self.lam),
                                                 _ptr(self.theta_star), _ptr(self.theta[0]), _ptr(self.s1[0]),
                                                 _ptr(self.s2[0]), _ptr(g), int(t), int(t - self.t_state_origin))
        assert rc == 0

    def sync(self, t_next: Optional[int] = None) -> None:
        _lib(self.mirror).orc_sync(C.byref(self.cfg), self.rows, self.n, _ptr(self.theta), _ptr(self.s1), _ptr(self.s2))
        if self.w.state_sync == "reset":
            assert t_next is not None
            self.t_state_origin = int(t_next)

    def run(self, t_begin: int = 0, t_end: Optional[int] = None) -> Tuple[np.ndarray, np.ndarray]:
        """Algorithm 2 from t_begin (a round start) until the first round end at or after t_end."""
        t_end = int(self.w.T if t_end is None else t_end)
        cap = int(self.w.T)
        st = np.empty(cap, np.int64)
        H = np.empty(cap, np.int64)
        origin = C.c_int64(self.t_state_origin)
        assert self.rows == self.w.K and self.k0 == 0
        n = _lib(self.mirror).orc_run(C.byref(self.cfg), self.rows, self.n, _ptr(self.idx), _ptr(self.lam),
                                      _ptr(self.theta_star), _ptr(self.theta), _ptr(self.s1), _ptr(self.s2),
                                      int(t_begin), t_end, C.byref(origin), _ptr(st), _ptr(H), cap)
        if n < 0:
            raise ValueError("bad run arguments")
        self.t_state_origin = int(origin.value)
        return st[:n].copy(), H[:n].copy()
