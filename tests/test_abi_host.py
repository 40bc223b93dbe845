"""CPU-side checks of the C-ABI library: it loads, exports every symbol the header declares, validates its
arguments, and its host schedule (learning rate, round lengths) equals the oracle's bit for bit.
No device work is issued here."""
import ctypes as C
import math
import os
import re

import numpy as np
import pytest

from oracle import qsr_oracle as O
from paper_2310_14423_b200 import binding as B
from paper_2310_14423_b200 import build as qsr_build
from paper_2310_14423_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
IMAGENET_TRAIN = 1_281_167


@pytest.fixture(scope="module", autouse=True)
def _built():
    qsr_build.build()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "qsr.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(qsr_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    declared = _declared_functions()
    assert len(declared) >= 15
    raw = C.CDLL(B.LIB_PATH)
    for name in declared:
        assert hasattr(raw, name), name
    assert sorted(B.EXPORTS) == declared


def test_config_struct_matches_header_size():
    # 2 int32, 2 int64, 4 int32, 9 doubles, 4 int64, 1 uint64, 1 double, 3 int64: 8 + 16 + 16 + 72 + 32 + 8 + 8 + 24
    assert C.sizeof(B.QsrConfig) == 184


def test_strerror_and_status_codes():
    assert B.strerror(0) == "ok"
    for code in (-1, -2, -3, -4, -5, -99):
        assert B.strerror(code)


def test_config_validation():
    w = W.workload("c1")
    ok = B.make_config(w)
    assert B.qsr_config_check(ok) == B.QSR_OK

    def bad(**kw):
        c = B.make_config(w)
        for k, v in kw.items():
            setattr(c, k, v)
        return B.qsr_config_check(c)

    assert bad(K=0) == B.QSR_EINVAL
    assert bad(P=0) == B.QSR_EINVAL
    assert bad(opt=7) == B.QSR_EINVAL
    assert bad(sched=-1) == B.QSR_EINVAL
    assert bad(sched=6) == B.QSR_EINVAL
    assert bad(rule=5) == B.QSR_EINVAL
    assert bad(rule=2, gamma=0.0) == B.QSR_EINVAL
    assert bad(rule=3, t_switch=-1) == B.QSR_ERANGE
    assert bad(sched=4, t_period=0) == B.QSR_ERANGE
    assert bad(state_sync=3) == B.QSR_EINVAL
    assert bad(eta_max=float("nan")) == B.QSR_EINVAL
    assert bad(alpha=float("inf")) == B.QSR_EINVAL
    assert bad(eta_max=-0.1) == B.QSR_EINVAL
    assert bad(row_stride=65538) == B.QSR_EALIGN
    assert bad(row_stride=65532) == B.QSR_EALIGN
    assert bad(T=0) == B.QSR_ERANGE
    assert bad(T_warmup=2000) == B.QSR_ERANGE
    assert bad(H_base=0) == B.QSR_ERANGE
    assert bad(T=(1 << 32) + 1) == B.QSR_ERANGE
    assert math.isnan(B.qsr_config_learning_rate(ok, -1))
    assert math.isnan(B.qsr_config_learning_rate(ok, 2000))
    with pytest.raises(B.QsrError) as e:
        B.qsr_config_round_length(ok, 2000)
    assert e.value.status == B.QSR_ERANGE
    assert B.lib().qsr_config_round_length(None, 0) == B.QSR_EINVAL
    assert B.lib().qsr_round_length(None, 0) == B.QSR_EINVAL
    assert B.lib().qsr_local_step(None, 0, None) == B.QSR_EINVAL
    assert B.lib().qsr_sync(None, 0) == B.QSR_EINVAL
    assert B.lib().qsr_destroy(None) == B.QSR_OK


def test_init_rejects_bad_pointers_without_touching_a_device():
    cfg = B.make_config(W.workload("c2"))
    h = C.c_void_p()
    L = B.lib()
    assert L.qsr_init(None, C.byref(cfg), 256, 256, 256, 256, 256, None) == B.QSR_EINVAL
    assert L.qsr_init(C.byref(h), None, 256, 256, 256, 256, 256, None) == B.QSR_EINVAL
    assert L.qsr_init(C.byref(h), C.byref(cfg), None, 256, 256, 256, 256, None) == B.QSR_EINVAL
    assert L.qsr_init(C.byref(h), C.byref(cfg), 256, 256, None, 256, 256, None) == B.QSR_EINVAL   # AdamW needs state2
    assert L.qsr_init(C.byref(h), C.byref(cfg), 256, 256, 256, 256, None, None) == B.QSR_EINVAL   # lambda without theta*
    assert L.qsr_init(C.byref(h), C.byref(cfg), 260, 256, 256, 256, 256, None) == B.QSR_EALIGN
    assert L.qsr_init(C.byref(h), C.byref(cfg), 256, 256, 256, 264, 256, None) == B.QSR_EALIGN
    assert not h.value


def test_workspace_bytes():
    w = W.workload("c2")
    cfg = B.make_config(w)
    assert B.qsr_workspace_bytes(cfg) == (3 * w.K * w.P + 3 * w.P) * 4
    w = W.tiny_workload(W.OPT_SGDM, K=3, P=1001)
    stride = B.qsr_row_stride_hint(1001)
    assert stride == 1024
    assert B.qsr_workspace_bytes(B.make_config(w)) == (2 * 3 * stride + 3 * stride) * 4


def test_row_stride_hint():
    """A legal stride (multiple of 4, >= P) on a power-of-two boundary of at most 2^20 floats, padding below P/16."""
    for P in (1, 2, 3, 4, 5, 63, 64, 65, 1000, 65535, 65536, 65537, 1 << 20, (1 << 20) + 1, 60_192_808, 86_415_592,
              (1 << 31) + 12345):
        s = B.qsr_row_stride_hint(P)
        assert s >= P and s % 4 == 0
        unit = s & -s                        # largest power of two dividing the stride
        assert s - P < max(4, P / 16)
        assert unit >= min(1 << 20, max(4, 1 << max(0, P.bit_length() - 5)))
        cfg = B.make_config(W.tiny_workload(W.OPT_SGDM, K=2, P=P), row_stride=s)
        assert B.qsr_config_check(cfg) == B.QSR_OK
    assert B.qsr_row_stride_hint(86_415_592) == 83 * (1 << 20)
    for bad in (0, -7):
        with pytest.raises(B.QsrError) as e:
            B.qsr_row_stride_hint(bad)
        assert e.value.status == B.QSR_EINVAL


def _same_schedule(w):
    cfg = B.make_config(w)
    st, H = B.qsr_config_schedule(cfg)
    ost, oH = O.schedule(w)
    assert np.array_equal(st, ost) and np.array_equal(H, oH)
    return st, H


def test_schedule_equals_oracle_on_the_run_configurations():
    for name in ("c1", "c2", "c3", "c4", "c4p", "c5"):
        w = W.workload(name)
        st, H = _same_schedule(w)
        for sched in (W.SCHED_STEP_POW2, W.SCHED_LINEAR, W.SCHED_CONST):
            _same_schedule(w.replace(sched=sched))
        _same_schedule(w.replace(eta_min=1e-6))
    # the sweep: growth coefficients x minimum periods, and constant periods, at both peak learning rates
    for eta_max in (8e-4, 8e-3):
        for alpha in (0.01, 0.0175, 0.025):
            for Hb in (2, 4, 8):
                _same_schedule(W.workload("c5").replace(eta_max=eta_max, alpha=alpha, H_base=Hb))
    for Hb in (2, 4, 8):
        _same_schedule(W.workload("c5").replace(rule=W.RULE_CONST_H, H_base=Hb))


def test_schedule_equals_oracle_on_the_papers_runs(golden_dir):
    """The 13 runs of Tables 1-3 / the linear-decay figure: same rounds as the oracle, hence the printed volumes."""
    n = 0
    with open(os.path.join(golden_dir, "paper_comm_volumes.txt")) as f:
        for line in f:
            if not line.strip() or line.startswith("#"):
                continue
            label, model, sched, batch, epochs, warm, eta_max, alpha, Hb, comm, src = line.split()
            per_epoch = IMAGENET_TRAIN // int(batch)
            T = int(epochs) * per_epoch
            T_w = int(warm[:-2]) * per_epoch if warm.endswith("ep") else int(warm[:-2])
            w = W.Workload(label, 1, W.flat_layout(4), W.OPT_SGDM, T=T, T_warmup=T_w, eta_max=float(eta_max),
                           sched=sched, alpha=float(alpha), H_base=int(Hb))
            st, H = _same_schedule(w)
            assert abs(100.0 * len(st) / T - float(comm)) <= 0.055
            n += 1
    assert n == 13


def test_learning_rate_equals_oracle_bitwise():
    for name in ("c1", "c2", "c4"):
        for sched in (W.SCHED_COSINE, W.SCHED_STEP_POW2, W.SCHED_LINEAR, W.SCHED_CONST):
            w = W.workload(name).replace(sched=sched)
            cfg = B.make_config(w)
            for t in list(range(0, w.T, 97)) + [w.T - 1, w.T_warmup, max(0, w.T_warmup - 1)]:
                assert B.qsr_config_learning_rate(cfg, t) == O.lr(w, t), (name, sched, t)


def test_round_length_pointwise_and_truncation():
    w = W.workload("c1")
    cfg = B.make_config(w)
    for t in range(0, w.T, 13):
        assert B.qsr_config_round_length(cfg, t) == O.round_length(w, t)
    assert B.qsr_config_round_length(cfg, 1999) == 1
    assert B.qsr_config_round_length(cfg, 0) == 4          # (0.2/0.1)^2 is exactly 4 in binary64


def test_other_rules_and_schedules_equal_oracle():
    """Power rule (gamma = 1, 3, 1.5), post-local, modified SWAP; halving and held-cosine schedules (App. G, App. H)."""
    per_epoch = IMAGENET_TRAIN // 4096
    vit = W.Workload("vit", 1, W.flat_layout(4), W.OPT_ADAMW, T=300 * per_epoch, T_warmup=10000, eta_max=0.008,
                     alpha=0.0175, H_base=4)
    halving = dict(sched=W.SCHED_HALVING, t_hold=150 * per_epoch, t_period=30 * per_epoch)
    cases = [
        vit.replace(**halving),
        vit.replace(rule=W.RULE_POWER, gamma=3.0, alpha=0.0075, **halving),
        vit.replace(rule=W.RULE_POWER, gamma=3.0, alpha=0.0075, eta_min=1e-6),
        vit.replace(rule=W.RULE_POWER, gamma=1.0, alpha=0.03),
        vit.replace(rule=W.RULE_POWER, gamma=1.5, alpha=0.02, H_base=2),
        vit.replace(sched=W.SCHED_COSINE_HELD, t_hold=250 * per_epoch),
        vit.replace(sched=W.SCHED_COSINE_HELD, t_hold=250 * per_epoch, rule=W.RULE_POWER, gamma=3.0, alpha=0.0075),
        vit.replace(rule=W.RULE_POST_LOCAL, t_switch=100 * per_epoch, H_base=8),
        vit.replace(rule=W.RULE_SWAP, t_switch=280 * per_epoch + 1, H_base=4),
        W.workload("c1").replace(rule=W.RULE_POWER, gamma=3.0, alpha=0.13),
    ]
    for w in cases:
        st, H = _same_schedule(w)
        assert H.sum() == w.T
        cfg = B.make_config(w)
        for t in range(0, w.T, 4999):
            assert B.qsr_config_learning_rate(cfg, t) == O.lr(w, t)
    st, H = _same_schedule(cases[0])
    assert abs(100.0 * len(st) / cases[0].T - 13.2) <= 0.055      # step-decay table of App. G
    st, H = _same_schedule(cases[1])
    assert abs(100.0 * len(st) / cases[1].T - 14.4) <= 0.055


def test_train_host_fails_before_touching_a_device_and_zeroes_its_outputs():
    """Every check of qsr_train_host that can fail on the host comes before its first copy is enqueued, and the output
    counters are zeroed at entry: bad arguments return their status with *launches = *n_rounds = 0 (no device needed;
    on a machine without a GPU the valid call stops at the context's device query, QSR_ECUDA, also before any copy)."""
    L = B.lib()
    w = W.tiny_workload(W.OPT_ADAMW, K=2, P=64, T=10)
    cfg = B.make_config(w)
    host = np.zeros(64, np.float32)
    ws_bytes = B.qsr_workspace_bytes(cfg)

    def call(cfg_, workspace=4096, nbytes=ws_bytes, t_end=10, theta0=host):
        n, launches = C.c_int64(77), C.c_int64(77)
        st = np.empty(16, np.int64)
        rc = L.qsr_train_host(C.byref(cfg_) if cfg_ is not None else None,
                              theta0.ctypes.data if theta0 is not None else None, host.ctypes.data, host.ctypes.data,
                              host.ctypes.data, workspace, nbytes, t_end, None, st.ctypes.data, st.ctypes.data, 16,
                              C.byref(n), C.byref(launches))
        return rc, n.value, launches.value

    assert call(None) == (B.QSR_EINVAL, 0, 0)
    assert call(cfg, theta0=None) == (B.QSR_EINVAL, 0, 0)
    assert call(cfg, workspace=4096 + 16) == (B.QSR_EALIGN, 0, 0)          # workspace must be 256-byte aligned
    assert call(cfg, nbytes=ws_bytes - 1) == (B.QSR_ERANGE, 0, 0)
    assert call(cfg, t_end=11) == (B.QSR_ERANGE, 0, 0)
    bad = B.make_config(w)
    bad.K = 0
    assert call(bad)[1:] == (0, 0) and call(bad)[0] < 0
    import torch
    if not torch.cuda.is_available():
        # a valid call on a machine without a device: the context cannot be created, nothing was enqueued
        assert call(cfg) == (B.QSR_ECUDA, 0, 0)


def test_header_is_plain_c(tmp_path):
    """include/qsr.h is a C header: plain pointers and sizes, no C++ in the signatures.  gcc -std=c99 -pedantic must take it."""
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler here")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    src = tmp_path / "use_header.c"
    src.write_text('#include "include/qsr.h"\nint main(void) { qsr_config c; (void)c; return QSR_OK; }\n')
    r = subprocess.run([gcc, "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only", "-I", root, str(src)],
                       capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
