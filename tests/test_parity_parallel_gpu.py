"""GPU parity for Algorithm 1 (Parallel OPT): qsr_parallel_step against the oracle's mean-gradient step, and the
paper's remark that Local SGD with H = 1 is parallel SGD (Sec. 3), checked between the two CUDA paths."""
import numpy as np
import pytest
import torch

from oracle import qsr_oracle as O
from paper_2310_14423_b200 import binding as B
from paper_2310_14423_b200 import workloads as W

import gpu_harness as G

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("opt", [W.OPT_SGDM, W.OPT_ADAMW])
@pytest.mark.parametrize("K,P", [(1, 5), (4, 1003), (16, 4096), (7, 2050)])
def test_parallel_step_matches_oracle(opt, K, P):
    w = W.tiny_workload(opt, K=K, P=P, T=50)
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    S = G.Slabs(w)
    S.theta[1:, :P] = 7.0                       # rows beyond the model must stay untouched
    ctx = G.make_context(w, S, lam_d, ths_d)
    orc = O.State(w, lam, ths, rows=1)
    for t in range(w.T):
        ctx.qsr_parallel_step(t)
        orc.parallel_step(t, K)
    torch.cuda.synchronize()
    assert ctx.qsr_launch_count() == w.T
    assert G.rel_err(S.theta[0, :P].cpu().numpy(), orc.theta[0]) <= G.REL_TOL
    assert bool((S.theta[1:, :P] == 7.0).all()) and not S.s1[1:, :P].any()
    assert S.guards_intact()
    ctx.close()


def test_parallel_step_external_gradients():
    K, P = 5, 3001
    w = W.tiny_workload(W.OPT_ADAMW, K=K, P=P, T=10)
    S = G.Slabs(w, n_extra=1)
    ctx = G.make_context(w, S, None, None)
    orc = O.State(w, np.zeros(P), np.zeros(P), rows=1)
    gen = torch.Generator(device="cuda").manual_seed(9)
    grads = S.extra[0]
    for t in range(w.T):
        grads[:, :P] = torch.randn(K, P, device="cuda", generator=gen)
        ctx.qsr_parallel_step(t, grads)
        orc.parallel_step(t, K, grads=grads[:, :P].cpu().numpy().astype(np.float64))
    torch.cuda.synchronize()
    assert G.rel_err(S.theta[0, :P].cpu().numpy(), orc.theta[0]) <= G.REL_TOL
    assert S.guards_intact()
    ctx.close()


def test_local_sgd_h1_is_parallel_sgd_on_the_device():
    """Local SGD (momentum 0.9, state kept) with a synchronization after every step, against Algorithm 1."""
    K, P = 8, 20011
    w = W.tiny_workload(W.OPT_SGDM, K=K, P=P, T=60, momentum=0.9, weight_decay=0.01, rule=W.RULE_CONST_H, H_base=1)
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    A, Bs = G.Slabs(w), G.Slabs(w)
    ca, cb = G.make_context(w, A, lam_d, ths_d), G.make_context(w, Bs, lam_d, ths_d)
    st, H = ca.qsr_run()
    assert (H == 1).all()
    for t in range(w.T):
        cb.qsr_parallel_step(t)
    torch.cuda.synchronize()
    local = A.theta[0, :P].double().cpu().numpy()
    par = Bs.theta[0, :P].double().cpu().numpy()
    assert G.rel_err(par, local) <= G.REL_TOL
    ca.close()
    cb.close()
