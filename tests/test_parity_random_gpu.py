"""Seeded random configurations through the C ABI against the CPU oracle: worker counts, ragged sizes, padded row
strides, launch shapes, every round-length rule, learning-rate schedule and state mode in combinations that the
hand-picked cases of test_parity_gpu.py do not enumerate -- AdamW started at full learning rate and AdamW whose
moments are reset at every synchronization included.  Bars: the round log bit-exact; parameters within REL_TOL on every
coordinate; a coordinate may miss it only by what the run's own conditioning explains (gpu_harness.assert_parity:
the binary64 oracle, its gradients perturbed by one fp32 ulp, must move that coordinate as far)."""
import numpy as np
import pytest
import torch

from paper_2310_14423_b200 import binding as B
from paper_2310_14423_b200 import workloads as W

import gpu_harness as G

pytestmark = pytest.mark.gpu

N_CASES = 36


def _draw(case):
    rng = np.random.default_rng([20231014, case])
    opt = (W.OPT_SGDM, W.OPT_ADAMW)[int(rng.integers(2))]
    K = int(rng.choice([1, 2, 3, 4, 7, 8, 9, 16, 19, 33]))
    P = int(rng.choice([1, 6, 7, 255, 1000, 1025, 2047, 4100, 9999]))
    T = int(rng.integers(30, 90)) if rng.integers(2) else int(rng.integers(300, 420))
    T_warmup = int(rng.integers(0, T // 3))
    sched = str(rng.choice([W.SCHED_COSINE, W.SCHED_STEP_POW2, W.SCHED_LINEAR, W.SCHED_CONST, W.SCHED_HALVING,
                            W.SCHED_COSINE_HELD]))
    rule = str(rng.choice([W.RULE_QSR, W.RULE_QSR, W.RULE_CONST_H, W.RULE_POWER, W.RULE_POST_LOCAL, W.RULE_SWAP]))
    eta_max = float(rng.choice([0.05, 0.1, 0.3])) if opt == W.OPT_SGDM else float(rng.choice([2e-3, 5e-3, 1e-2]))
    kw = dict(sched=sched, rule=rule, eta_max=eta_max, T_warmup=T_warmup,
              alpha=eta_max * float(rng.uniform(1.2, 3.0)), H_base=int(rng.integers(1, 6)),
              gamma=float(rng.choice([1.0, 1.5, 2.0, 3.0])), t_switch=int(rng.integers(0, T + 1)),
              t_hold=int(rng.integers(T_warmup, T)), t_period=int(rng.integers(1, 12)),
              momentum=float(rng.choice([0.0, 0.5, 0.9])), weight_decay=float(rng.choice([0.0, 1e-4, 0.05])),
              noise_std=float(rng.choice([0.0, 0.05, 0.2])),
              state_sync=str(rng.choice([W.STATE_KEEP, W.STATE_KEEP, W.STATE_AVERAGE, W.STATE_RESET])),
              noise_seed=int(rng.integers(1, 2 ** 62)))
    w = W.tiny_workload(opt, K=K, P=P, T=T, **kw)
    P4 = (P + 3) // 4 * 4
    stride = int(rng.choice([P4, P4 + 4, P4 + 36, B.qsr_row_stride_hint(P)]))
    shape = (int(rng.choice([64, 128, 256, 512])), int(rng.choice([1, 2, 4, 8])), int(rng.choice([64, 128, 512])))
    graph_steps = int(rng.choice([0, 0, 5, 64]))
    return w, stride, shape, graph_steps


@pytest.mark.parametrize("case", range(N_CASES))
def test_random_configuration(case):
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    w, stride, shape, graph_steps = _draw(case)
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    S = G.Slabs(w, row_stride=stride)
    ctx = G.make_context(w, S, lam_d, ths_d)
    ctx.qsr_set_launch_shape(*shape)
    ctx.qsr_set_graph_replay(graph_steps)
    st, H = ctx.qsr_run()
    torch.cuda.synchronize()
    ctx.close()
    orc = G.oracle_on(w, lam, ths)
    ost, oH = orc.run()
    assert np.array_equal(st, ost) and np.array_equal(H, oH), (w, st, ost)
    assert int(st[-1] + H[-1]) == w.T
    theta = S.theta[:, :w.P].cpu().numpy()
    assert (theta == theta[0]).all()                    # the run ends with a synchronization
    G.assert_parity(theta[0], w, lam, ths, orc.theta[0], context=(w, stride, shape))
    assert S.guards_intact()
