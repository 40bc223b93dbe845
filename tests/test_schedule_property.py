"""Randomised agreement of the library's host schedule with the oracle's: for seeded random hyper-parameters over every
rule and schedule, the round starts and lengths must be identical, sum to T, and respect the rule's invariants.  CPU only."""
import numpy as np
import pytest

from oracle import qsr_oracle as O
from paper_2310_14423_b200 import binding as B
from paper_2310_14423_b200 import build as qsr_build
from paper_2310_14423_b200 import workloads as W

SCHEDS = [W.SCHED_COSINE, W.SCHED_STEP_POW2, W.SCHED_LINEAR, W.SCHED_CONST, W.SCHED_HALVING, W.SCHED_COSINE_HELD]
RULES = [W.RULE_QSR, W.RULE_CONST_H, W.RULE_POWER, W.RULE_POST_LOCAL, W.RULE_SWAP]


@pytest.fixture(scope="module", autouse=True)
def _built():
    qsr_build.build()


def _random_workload(rng):
    T = int(rng.integers(1, 30000))
    T_w = int(rng.integers(0, max(1, T // 3))) if T > 1 else 0
    eta_max = float(10 ** rng.uniform(-4, 0.5))
    sched = SCHEDS[int(rng.integers(len(SCHEDS)))]
    rule = RULES[int(rng.integers(len(RULES)))]
    t_hold = int(rng.integers(T_w, T + 1))
    return W.Workload("rnd", 1, W.flat_layout(4), W.OPT_SGDM, T=T, T_warmup=T_w, eta_max=eta_max,
                      eta_min=float(eta_max * rng.choice([0.0, 0.0, 1e-3, 0.1])), sched=sched, rule=rule,
                      alpha=float(eta_max * 10 ** rng.uniform(-1, 1.5)), H_base=int(rng.integers(1, 17)),
                      gamma=float(rng.choice([0.5, 1.0, 1.5, 2.0, 3.0])), t_switch=int(rng.integers(0, T + 1)),
                      t_hold=t_hold, t_period=int(rng.integers(1, max(2, T // 4))))


def test_random_schedules_equal_oracle():
    rng = np.random.default_rng(20231014)
    seen = set()
    for _ in range(400):
        w = _random_workload(rng)
        cfg = B.make_config(w)
        assert B.qsr_config_check(cfg) == B.QSR_OK, w
        st, H = B.qsr_config_schedule(cfg)
        ost, oH = O.schedule(w)
        assert np.array_equal(st, ost) and np.array_equal(H, oH), w
        assert st[0] == 0 and H.sum() == w.T and (H >= 1).all()
        assert np.array_equal(st[1:], np.cumsum(H)[:-1])
        if w.rule in (W.RULE_QSR, W.RULE_POWER, W.RULE_CONST_H):
            assert (H[:-1] >= w.H_base).all()
        if w.rule == W.RULE_CONST_H:
            assert (H[:-1] == w.H_base).all()
        if w.rule == W.RULE_POST_LOCAL:
            assert (H[st < w.t_switch] == 1).all()
        if w.rule == W.RULE_SWAP and w.t_switch < w.T:
            assert st[-1] == w.t_switch and H[-1] == w.T - w.t_switch      # one final round after the switch
            assert (H[:-1] <= w.H_base).all()
        for t in rng.integers(0, w.T, size=5):
            assert B.qsr_config_learning_rate(cfg, int(t)) == O.lr(w, int(t)), (w, t)
        seen.add((w.rule, w.sched))
    assert len(seen) >= 25      # the draw covered most rule x schedule pairs
