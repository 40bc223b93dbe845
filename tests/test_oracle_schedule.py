"""Pins for the oracle's learning-rate schedule and round-length rule (Sec. 2, Eq. 2; Tables 1-3).

None of these tests touches the CUDA library.  The expected values come from the paper's printed
communication volumes, from inverting the cosine in high precision (a different route from the
oracle's forward evaluation), and from small hand calculations written out below.
"""
import math
import os

import mpmath as mp
import numpy as np
import pytest

from oracle import qsr_oracle as O
from paper_2310_14423_b200 import workloads as W

IMAGENET_TRAIN = 1_281_167  # outside fact: the paper names ImageNet-1k but not its size


def _paper_case(cols):
    label, model, sched, batch, epochs, warm, eta_max, alpha, H_base, comm, source = cols
    per_epoch = IMAGENET_TRAIN // int(batch)
    T = int(epochs) * per_epoch
    T_w = int(warm[:-2]) * per_epoch if warm.endswith("ep") else int(warm[:-2])
    w = W.Workload(label, 1, W.flat_layout(4), W.OPT_SGDM, T=T, T_warmup=T_w, eta_max=float(eta_max),
                   sched=sched, alpha=float(alpha), H_base=int(H_base))
    return w, float(comm)


def _paper_cases(golden_dir):
    out = []
    with open(os.path.join(golden_dir, "paper_comm_volumes.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                out.append(_paper_case(line.split()))
    return out


def test_paper_communication_volumes(golden_dir):
    """Tables 1-3 and the linear-decay figure: 100 * (#rounds) / T, to the printed digit."""
    cases = _paper_cases(golden_dir)
    assert len(cases) == 13
    for w, printed in cases:
        starts, H = O.schedule(w)
        assert H.sum() == w.T
        ours = 100.0 * len(starts) / w.T
        assert abs(ours - printed) <= 0.055, (w.name, ours, printed)


def _py_schedule(T, T_w, eta_max, alpha, H_base, variant):
    """Alternative readings of Eq. 2, in plain Python, to show that the printed values tell them apart."""
    t = n = 0
    while t < T:
        te = max(t, T_w)
        if variant == "cosine_over_all_T":
            eta = 0.5 * eta_max * (1 + math.cos(math.pi * te / T))
        else:
            eta = 0.5 * eta_max * (1 + math.cos(math.pi * (te - T_w) / (T - T_w)))
        q = (alpha / eta) ** 2 if eta > 0 else 1e18
        H = {"ceil": math.ceil(q), "nearest": math.floor(q + 0.5)}.get(variant, math.floor(q))
        H = min(max(H_base, H), T - t)
        t += H
        n += 1
    return 100.0 * n / T


def test_printed_volumes_reject_other_readings():
    # ViT-B, B=4096, H_base=4 (Table 1b): 10.4 printed.
    T, T_w = 300 * (IMAGENET_TRAIN // 4096), 10000
    assert abs(_py_schedule(T, T_w, 0.008, 0.0175, 4, "floor") - 10.4) <= 0.055
    for variant in ("ceil", "nearest", "cosine_over_all_T"):
        assert abs(_py_schedule(T, T_w, 0.008, 0.0175, 4, variant) - 10.4) > 0.5, variant


def _schedule_from_thresholds(T, eta_max, alpha, H_base):
    """Config with no warm-up and cosine to zero: H(t) = max(H_base, n(t)) where n(t) is the largest n
    with (alpha/eta_t)^2 >= n, i.e. t >= (T/pi) * arccos(2*alpha/(eta_max*sqrt(n)) - 1).  The crossing
    points are computed with 50 digits, so this never evaluates eta_t in binary64."""
    mp.mp.dps = 50
    # the exact values of the binary64 inputs, so that a knife edge (t = 0 here) falls on the oracle's side
    a, e = mp.mpf(alpha), mp.mpf(eta_max)

    def first_t(n):
        c = 2 * a / (e * mp.sqrt(n)) - 1
        if c >= 1:
            return 0
        if c <= -1:
            return None
        return int(mp.ceil(mp.mpf(T) / mp.pi * mp.acos(c)))

    starts, Hs = [], []
    t = 0
    n = 1
    while t < T:
        while True:
            ft = first_t(n + 1)
            if ft is not None and ft <= t:
                n += 1
            else:
                break
        H = min(max(H_base, n), T - t)
        starts.append(t)
        Hs.append(H)
        t += H
    return np.asarray(starts), np.asarray(Hs)


def test_config1_sequence_from_inverse_cosine():
    w = W.workload("c1")
    starts, H = O.schedule(w)
    ref_starts, ref_H = _schedule_from_thresholds(w.T, w.eta_max, w.alpha, w.H_base)
    assert np.array_equal(starts, ref_starts)
    assert np.array_equal(H, ref_H)


def test_config1_hand_worked_anchors():
    """T=2000, eta_max=0.1, alpha=0.2, H_base=2, cosine to 0, no warm-up.
    t=0: (0.2/0.1)^2 = 4 exactly -> H=4.  H stays 4 while eta > 0.2/sqrt(5) = 0.0894427, i.e. while
    (1+cos(pi t/2000))/2 > 0.894427, i.e. t < 2000/pi * arccos(0.788854) = 421.3; rounds of 4 start at
    multiples of 4, so the first round with H=5 starts at t=424.  H=6 needs t >= 2000/pi*arccos(0.632993)
    = 561.1; from 424 in strides of 5 the first start past it is 564.  The last round starts at 1593,
    where eta = 0.05*(1+cos(pi*1593/2000)) = 0.0098737 and (0.2/eta)^2 = 410.3 -> 410 > 2000-1593 = 407."""
    w = W.workload("c1")
    starts, H = O.schedule(w)
    d = dict(zip(starts.tolist(), H.tolist()))
    assert d[0] == 4 and d[420] == 4 and d[424] == 5 and 421 not in d
    assert d[559] == 5 and d[564] == 6
    assert starts[-1] == 1593 and H[-1] == 407
    assert len(starts) == 203
    assert (H[:106] == 4).all() and H[106] == 5


def test_sum_and_chain_invariants():
    for name in ("c1", "c2", "c3", "c4", "c4p"):
        w = W.workload(name)
        starts, H = O.schedule(w)
        assert starts[0] == 0 and H.sum() == w.T
        assert np.array_equal(starts[1:], np.cumsum(H)[:-1])
        assert (H[:-1] >= w.H_base).all() and H[-1] >= 1
        # decaying schedule after warm-up => H never shrinks, except for the truncated last round
        assert (np.diff(H[:-1]) >= 0).all()


def test_truncation_forces_last_sync_at_T():
    w = W.workload("c1").replace(T=1999)
    starts, H = O.schedule(w)
    assert starts[-1] + H[-1] == 1999
    w = W.workload("c1").replace(rule=W.RULE_CONST_H, H_base=7)
    starts, H = O.schedule(w)
    assert (H[:-1] == 7).all() and H[-1] == 2000 - 7 * (2000 // 7) and len(H) == 2000 // 7 + 1


def test_constant_h_rule_ignores_learning_rate():
    for Hc in (2, 4, 8):
        w = W.workload("c4").replace(rule=W.RULE_CONST_H, H_base=Hc)
        starts, H = O.schedule(w)
        assert (H == Hc).all() and len(H) == w.T // Hc


def test_warmup_rounds_use_the_post_warmup_value():
    """Sec. 2: during warm-up H is the value of the round right after warm-up, i.e. Eq. 2 at eta_max."""
    w = W.workload("c2")  # (0.0175/1e-3)^2 = 306.25
    assert O.round_length(w, 0) == 306
    assert O.round_length(w, 50) == 306
    assert O.round_length(w, 99) == 306
    assert O.round_length(w, 100) == 306
    w = W.workload("c4p")  # (0.0175/0.008)^2 = 4.785 -> 4 = H_base
    assert O.round_length(w, 0) == 4
    # paper's own runs: (alpha/eta_max)^2 < H_base + 1, so warm-up rounds have H_base steps
    assert O.round_length(W.workload("c4p").replace(H_base=8), 3) == 8


def test_learning_rate_values():
    w = W.workload("c2")  # warm-up 100, peak 1e-3, T=5000, cosine to 0
    assert O.lr(w, 0) == 0.0
    assert O.lr(w, 50) == pytest.approx(0.5e-3, rel=1e-15)
    assert O.lr(w, 100) == 1e-3
    assert O.lr(w, 100 + 2450) == pytest.approx(0.5e-3, rel=1e-12)   # midpoint of the cosine
    assert O.lr(w, 100 + 1225) == pytest.approx(1e-3 * (1 + math.sqrt(0.5)) / 2, rel=1e-12)  # quarter point
    assert 0 < O.lr(w, 4999) < 1e-9
    wmin = w.replace(eta_min=1e-6)
    assert O.lr(wmin, 4999) == pytest.approx(1e-6, rel=1e-3)
    wl = w.replace(sched=W.SCHED_LINEAR)
    assert O.lr(wl, 100) == 1e-3 and O.lr(wl, 2550) == pytest.approx(0.5e-3, rel=1e-12)
    wc = w.replace(sched=W.SCHED_CONST)
    assert O.lr(wc, 4000) == 1e-3
    ws = w.replace(sched=W.SCHED_STEP_POW2)
    for t in range(100, 5000, 37):
        e_cos, e_step = O.lr(w, t), O.lr(ws, t)
        m, ex = math.frexp(e_step)
        assert m == 0.5  # a power of two
        assert 2 ** -0.5 <= e_step / e_cos <= 2 ** 0.5 * (1 + 1e-12)


def test_lr_is_monotone_after_warmup():
    for name in ("c1", "c3", "c4"):
        w = W.workload(name)
        eta = np.array([O.lr(w, t) for t in range(w.T_warmup, w.T)])
        assert (np.diff(eta) <= 0).all() and eta[0] == w.eta_max


def test_round_counts_of_the_configs():
    """Round counts by the thresholds route (c1) and by direct reasoning on the first round (others)."""
    assert len(O.schedule(W.workload("c1"))[0]) == 203
    st, H = O.schedule(W.workload("c2"))
    assert H[0] == 306 and st[1] == 306 and H.sum() == 5000
    st, H = O.schedule(W.workload("c4"))
    assert H[0] == 478 and H.sum() == 10000  # (0.0175/8e-4)^2 = 478.5
    st, H = O.schedule(W.workload("c3"))
    assert H[0] == 2  # (0.2/0.8)^2 < 1 -> H_base
