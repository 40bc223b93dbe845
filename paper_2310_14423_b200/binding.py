"""Thin ctypes binding over libqsr.so: the same names as include/qsr.h, argument marshalling only.

Every step of the path runs in the library's CUDA kernels.  There is no CPU fallback: loading fails loudly if
the library has not been built (`python -m paper_2310_14423_b200.build`), and calls that need a device return
the library's error codes, raised here as QsrError.

torch is used by callers for device memory and streams; this module only needs `tensor.data_ptr()`.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libqsr.so")

OPT = {"sgdm": 0, "adamw": 1}
SCHED = {"cosine": 0, "step_pow2": 1, "linear": 2, "const": 3, "halving": 4, "cosine_held": 5}
RULE = {"qsr": 0, "const_h": 1, "power": 2, "post_local": 3, "swap": 4}
STATE = {"keep": 0, "average": 1, "reset": 2}

QSR_OK, QSR_EINVAL, QSR_EALIGN, QSR_ECUDA, QSR_ERANGE, QSR_ESTATE = 0, -1, -2, -3, -4, -5
QSR_STATIC_SCRATCH_FLOATS = 1 << 20

EXPORTS = ("qsr_config_check", "qsr_row_stride_hint", "qsr_config_learning_rate", "qsr_config_round_length", "qsr_config_schedule",
           "qsr_workspace_bytes", "qsr_init", "qsr_destroy", "qsr_round_length", "qsr_set_tensor_table", "qsr_clip_workspace_floats", "qsr_set_grad_clip", "qsr_set_params", "qsr_local_step",
           "qsr_local_step_sync", "qsr_parallel_step", "qsr_sync", "qsr_sync_sum_floats", "qsr_sync_partial", "qsr_local_step_partial", "qsr_sync_finish", "qsr_sync_static", "qsr_run", "qsr_launch_count",
           "qsr_set_launch_shape", "qsr_set_graph_replay", "qsr_set_resident_steps", "qsr_train_host", "qsr_debug_box_muller", "qsr_debug_fast_math", "qsr_strerror")


class QsrConfig(C.Structure):
    """Mirror of `qsr_config` in include/qsr.h (field order and types must match)."""
    _fields_ = [("K", C.c_int32), ("worker_offset", C.c_int32), ("P", C.c_int64), ("row_stride", C.c_int64),
                ("opt", C.c_int32), ("sched", C.c_int32), ("rule", C.c_int32), ("state_sync", C.c_int32),
                ("momentum", C.c_double), ("beta1", C.c_double), ("beta2", C.c_double), ("eps", C.c_double),
                ("weight_decay", C.c_double), ("eta_max", C.c_double), ("eta_min", C.c_double),
                ("alpha", C.c_double), ("noise_std", C.c_double),
                ("T", C.c_int64), ("T_warmup", C.c_int64), ("H_base", C.c_int64), ("t_state_origin", C.c_int64),
                ("seed", C.c_uint64), ("gamma", C.c_double), ("t_switch", C.c_int64), ("t_hold", C.c_int64),
                ("t_period", C.c_int64)]


class QsrError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__(f"{where}: {strerror(status)} (status {status})")


_lib = None


def lib():
    """The loaded library.  Raises if it is missing: the product has no other implementation to fall back to."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not found; build it with `python -m paper_2310_14423_b200.build` "
                              "(needs nvcc; there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        cfg, vp, i64, i32 = C.POINTER(QsrConfig), C.c_void_p, C.c_int64, C.c_int32
        sig = {
            "qsr_config_check": (C.c_int, [cfg]),
            "qsr_row_stride_hint": (i64, [i64]),
            "qsr_config_learning_rate": (C.c_double, [cfg, i64]),
            "qsr_config_round_length": (i64, [cfg, i64]),
            "qsr_config_schedule": (i64, [cfg, vp, vp, i64]),
            "qsr_workspace_bytes": (i64, [cfg]),
            "qsr_init": (C.c_int, [C.POINTER(vp), cfg, vp, vp, vp, vp, vp, vp]),
            "qsr_destroy": (C.c_int, [vp]),
            "qsr_round_length": (i64, [vp, i64]),
            "qsr_set_tensor_table": (C.c_int, [vp, i32, vp, vp]),
            "qsr_clip_workspace_floats": (i64, [vp]),
            "qsr_set_grad_clip": (C.c_int, [vp, C.c_double, vp]),
            "qsr_set_params": (C.c_int, [vp, vp]),
            "qsr_local_step": (C.c_int, [vp, i64, vp]),
            "qsr_local_step_sync": (C.c_int, [vp, i64, vp, i64]),
            "qsr_parallel_step": (C.c_int, [vp, i64, vp]),
            "qsr_sync": (C.c_int, [vp, i64]),
            "qsr_sync_sum_floats": (i64, [vp]),
            "qsr_sync_partial": (C.c_int, [vp, vp]),
            "qsr_local_step_partial": (C.c_int, [vp, i64, vp, vp]),
            "qsr_sync_finish": (C.c_int, [vp, vp, i32, i64]),
            "qsr_sync_static": (C.c_int, [vp, i64]),
            "qsr_run": (C.c_int, [vp, i64, i64, vp, vp, i64, C.POINTER(i64)]),
            "qsr_launch_count": (i64, [vp]),
            "qsr_set_launch_shape": (C.c_int, [vp, i32, i32, i32]),
            "qsr_set_graph_replay": (C.c_int, [vp, i32]),
            "qsr_set_resident_steps": (C.c_int, [vp, i32]),
            "qsr_train_host": (C.c_int, [cfg, vp, vp, vp, vp, vp, i64, i64, vp, vp, vp, i64, C.POINTER(i64), C.POINTER(i64)]),
            "qsr_debug_box_muller": (C.c_int, [vp, i64, vp, vp, vp, vp]),
            "qsr_debug_fast_math": (C.c_int, [vp, i64, vp, vp, vp]),
            "qsr_strerror": (C.c_char_p, [C.c_int]),
        }
        for name in EXPORTS:
            fn = getattr(L, name)
            fn.restype, fn.argtypes = sig[name]
        _lib = L
    return _lib


def strerror(status: int) -> str:
    return lib().qsr_strerror(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != QSR_OK:
        raise QsrError(status, where)


def make_config(w, K: Optional[int] = None, row_stride: Optional[int] = None, worker_offset: Optional[int] = None,
                t_state_origin: int = 0) -> QsrConfig:
    """qsr_config from a workload description (an object with the fields of workloads.Workload)."""
    P = int(w.P)
    return QsrConfig(K=int(w.K if K is None else K),
                     worker_offset=int(w.worker_offset if worker_offset is None else worker_offset),
                     P=P, row_stride=int((P + 3) // 4 * 4 if row_stride is None else row_stride),
                     opt=OPT[w.opt], sched=SCHED[w.sched], rule=RULE[w.rule], state_sync=STATE[w.state_sync],
                     momentum=w.momentum, beta1=w.beta1, beta2=w.beta2, eps=w.eps, weight_decay=w.weight_decay,
                     eta_max=w.eta_max, eta_min=w.eta_min, alpha=w.alpha, noise_std=w.noise_std,
                     T=int(w.T), T_warmup=int(w.T_warmup), H_base=int(w.H_base), t_state_origin=int(t_state_origin),
                     seed=int(w.noise_seed), gamma=float(getattr(w, "gamma", 2.0)),
                     t_switch=int(getattr(w, "t_switch", 0)), t_hold=int(getattr(w, "t_hold", 0)),
                     t_period=max(1, int(getattr(w, "t_period", 1))))


# ---- host-only schedule ---------------------------------------------------------------------------------

def qsr_config_check(cfg: QsrConfig) -> int:
    return int(lib().qsr_config_check(C.byref(cfg)))


def qsr_config_learning_rate(cfg: QsrConfig, t: int) -> float:
    return float(lib().qsr_config_learning_rate(C.byref(cfg), int(t)))


def qsr_config_round_length(cfg: QsrConfig, t: int) -> int:
    H = int(lib().qsr_config_round_length(C.byref(cfg), int(t)))
    if H < 0:
        raise QsrError(H, "qsr_config_round_length")
    return H


def qsr_config_schedule(cfg: QsrConfig) -> Tuple[np.ndarray, np.ndarray]:
    cap = int(cfg.T)
    st, H = np.empty(cap, np.int64), np.empty(cap, np.int64)
    n = int(lib().qsr_config_schedule(C.byref(cfg), st.ctypes.data, H.ctypes.data, cap))
    if n < 0:
        raise QsrError(n, "qsr_config_schedule")
    return st[:n].copy(), H[:n].copy()


def qsr_row_stride_hint(P: int) -> int:
    n = int(lib().qsr_row_stride_hint(int(P)))
    if n < 0:
        raise QsrError(n, "qsr_row_stride_hint")
    return n


def qsr_workspace_bytes(cfg: QsrConfig) -> int:
    n = int(lib().qsr_workspace_bytes(C.byref(cfg)))
    if n < 0:
        raise QsrError(n, "qsr_workspace_bytes")
    return n


# ---- context --------------------------------------------------------------------------------------------

def _dptr(t) -> Optional[int]:
    """Device address of a torch tensor (or None)."""
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return int(t.data_ptr())


class Context:
    """Owner of one `qsr_ctx`.  Keeps references to the tensors whose memory the library borrows."""

    def __init__(self, cfg: QsrConfig, params, state1, state2=None, lam=None, theta_star=None, stream: int = 0):
        self.cfg = cfg
        self._keep = (params, state1, state2, lam, theta_star)
        self._h = C.c_void_p()
        _check(lib().qsr_init(C.byref(self._h), C.byref(cfg), _dptr(params), _dptr(state1), _dptr(state2),
                              _dptr(lam), _dptr(theta_star), C.c_void_p(stream)), "qsr_init")

    def close(self) -> None:
        if self._h:
            lib().qsr_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def qsr_round_length(self, t: int) -> int:
        H = int(lib().qsr_round_length(self._h, int(t)))
        if H < 0:
            raise QsrError(H, "qsr_round_length")
        return H

    def qsr_set_tensor_table(self, tensor_end=None, wd_scale=None) -> None:
        """tensor_end: CUDA int64 tensor [n]; wd_scale: CUDA float32 tensor [n]; None clears the table."""
        n = 0 if tensor_end is None else int(tensor_end.numel())
        self._table = (tensor_end, wd_scale)
        _check(lib().qsr_set_tensor_table(self._h, n, _dptr(tensor_end), _dptr(wd_scale)), "qsr_set_tensor_table")

    def qsr_clip_workspace_floats(self) -> int:
        return int(lib().qsr_clip_workspace_floats(self._h))

    def qsr_set_grad_clip(self, max_norm: float, workspace=None) -> None:
        self._clip_ws = workspace
        _check(lib().qsr_set_grad_clip(self._h, float(max_norm), _dptr(workspace)), "qsr_set_grad_clip")

    def qsr_set_params(self, theta0) -> None:
        _check(lib().qsr_set_params(self._h, _dptr(theta0)), "qsr_set_params")

    def qsr_local_step(self, t: int, grads=None) -> None:
        _check(lib().qsr_local_step(self._h, int(t), _dptr(grads)), "qsr_local_step")

    def qsr_local_step_sync(self, t: int, t_next: int, grads=None) -> None:
        _check(lib().qsr_local_step_sync(self._h, int(t), _dptr(grads), int(t_next)), "qsr_local_step_sync")

    def qsr_parallel_step(self, t: int, grads=None) -> None:
        _check(lib().qsr_parallel_step(self._h, int(t), _dptr(grads)), "qsr_parallel_step")

    def qsr_sync(self, t_next: int) -> None:
        _check(lib().qsr_sync(self._h, int(t_next)), "qsr_sync")

    def qsr_sync_sum_floats(self) -> int:
        return int(lib().qsr_sync_sum_floats(self._h))

    def qsr_sync_partial(self, sums) -> None:
        _check(lib().qsr_sync_partial(self._h, _dptr(sums)), "qsr_sync_partial")

    def qsr_local_step_partial(self, t: int, sums, grads=None) -> None:
        _check(lib().qsr_local_step_partial(self._h, int(t), _dptr(grads), _dptr(sums)), "qsr_local_step_partial")

    def qsr_sync_finish(self, sums, K_total: int, t_next: int) -> None:
        _check(lib().qsr_sync_finish(self._h, _dptr(sums), int(K_total), int(t_next)), "qsr_sync_finish")

    def qsr_sync_static(self, t_next: int) -> None:
        """qsr_sync through the library's built-in scratch array: for callers that cannot allocate the `sum` buffer.
        Raises QsrError(QSR_ERANGE) when the problem exceeds QSR_STATIC_SCRATCH_FLOATS."""
        _check(lib().qsr_sync_static(self._h, int(t_next)), "qsr_sync_static")

    def qsr_run(self, t_begin: int = 0, t_end: Optional[int] = None) -> Tuple[np.ndarray, np.ndarray]:
        t_end = int(self.cfg.T if t_end is None else t_end)
        cap = max(1, t_end - int(t_begin))
        st, H = np.empty(cap, np.int64), np.empty(cap, np.int64)
        n = C.c_int64(0)
        _check(lib().qsr_run(self._h, int(t_begin), t_end, st.ctypes.data, H.ctypes.data, cap, C.byref(n)), "qsr_run")
        return st[:n.value].copy(), H[:n.value].copy()

    def qsr_launch_count(self) -> int:
        return int(lib().qsr_launch_count(self._h))

    def qsr_set_graph_replay(self, max_steps_per_graph: int) -> None:
        _check(lib().qsr_set_graph_replay(self._h, max_steps_per_graph), "qsr_set_graph_replay")

    def qsr_set_resident_steps(self, max_steps_per_launch: int) -> None:
        """Benchmark-only: up to this many consecutive steps per launch, state held in registers (0 = off)."""
        _check(lib().qsr_set_resident_steps(self._h, max_steps_per_launch), "qsr_set_resident_steps")

    def qsr_set_launch_shape(self, step_threads: int = 0, step_rows_in_flight: int = 0, sync_threads: int = 0) -> None:
        _check(lib().qsr_set_launch_shape(self._h, step_threads, step_rows_in_flight, sync_threads), "qsr_set_launch_shape")


def qsr_train_host(cfg: QsrConfig, theta0: np.ndarray, lam: np.ndarray, theta_star: np.ndarray, theta_out: np.ndarray,
                   workspace, t_end: Optional[int] = None, stream: int = 0):
    """Whole run from host arrays (numpy float32 [P], or pinned torch CPU tensors exposing data_ptr()).
    `workspace` is a CUDA tensor of at least qsr_workspace_bytes(cfg) bytes.
    Returns (round starts, round lengths, kernel launches)."""
    def hptr(a):
        return int(a.ctypes.data) if isinstance(a, np.ndarray) else int(a.data_ptr())
    t_end = int(cfg.T if t_end is None else t_end)
    cap = max(1, t_end)
    st, H = np.empty(cap, np.int64), np.empty(cap, np.int64)
    n, launches = C.c_int64(0), C.c_int64(0)
    nbytes = int(workspace.numel() * workspace.element_size())
    _check(lib().qsr_train_host(C.byref(cfg), hptr(theta0), hptr(lam), hptr(theta_star), hptr(theta_out),
                                _dptr(workspace), nbytes, t_end, C.c_void_p(stream),
                                st.ctypes.data, H.ctypes.data, cap, C.byref(n), C.byref(launches)), "qsr_train_host")
    return st[:n.value].copy(), H[:n.value].copy(), int(launches.value)


def qsr_debug_box_muller(words, radius, sine, cosine, stream: int = 0) -> None:
    """Test hook: Box-Muller radius / sine / cosine of each uint32 generator word (CUDA tensors; words as int32 bits)."""
    n = int(words.numel())
    _check(lib().qsr_debug_box_muller(_dptr(words), n, _dptr(radius), _dptr(sine), _dptr(cosine), C.c_void_p(stream)),
           "qsr_debug_box_muller")


def qsr_debug_fast_math(x, root, reciprocal, stream: int = 0) -> None:
    """Test hook: the library's single-instruction square root and reciprocal of each float of x (CUDA tensors)."""
    _check(lib().qsr_debug_fast_math(_dptr(x), int(x.numel()), _dptr(root), _dptr(reciprocal), C.c_void_p(stream)),
           "qsr_debug_fast_math")
