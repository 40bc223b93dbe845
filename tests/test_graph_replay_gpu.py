"""qsr_run with its rounds replayed from CUDA graphs against the same run with direct launches.

The graphs hold the same kernels in the same order with the same arguments, so everything must agree bit for bit:
parameters, optimizer state, the round log and the number of kernels that ran.  The direct path itself is checked
against the CPU oracle (once more here, and throughout test_parity_gpu.py)."""
import numpy as np
import pytest
import torch

from paper_2310_14423_b200 import binding as B
from paper_2310_14423_b200 import workloads as W

import gpu_harness as G

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _cuda():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    B.lib()
    yield
    torch.cuda.synchronize()
    torch.cuda.empty_cache()


def _run(w, graph_steps, t_end=None, shape=None):
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    S = G.Slabs(w)
    ctx = G.make_context(w, S, lam_d, ths_d)
    if shape:
        ctx.qsr_set_launch_shape(*shape)
    ctx.qsr_set_graph_replay(graph_steps)
    st, H = ctx.qsr_run(0, w.T if t_end is None else t_end)
    torch.cuda.synchronize()
    launches = ctx.qsr_launch_count()
    ctx.close()
    assert S.guards_intact()
    return lam, ths, S, st, H, launches


def _same(a, b):
    return torch.equal(a.theta, b.theta) and torch.equal(a.s1, b.s1) and (a.s2 is None or torch.equal(a.s2, b.s2))


@pytest.mark.parametrize("graph_steps", [1, 3, 7, 64])
@pytest.mark.parametrize("opt,mode", [(W.OPT_SGDM, W.STATE_KEEP), (W.OPT_ADAMW, W.STATE_KEEP),
                                      (W.OPT_ADAMW, W.STATE_RESET), (W.OPT_SGDM, W.STATE_AVERAGE)])
def test_replayed_rounds_equal_direct_launches(opt, mode, graph_steps):
    # rounds of 6 to about 100 steps: chains shorter than, equal to and longer than the limit
    w = W.tiny_workload(opt, K=3, P=4099, T=400, state_sync=mode)
    _, _, S0, st0, H0, n0 = _run(w, 0)
    assert len(set(H0.tolist())) >= 6 and H0.max() > 64 > H0.min()
    _, _, S1, st1, H1, n1 = _run(w, graph_steps)
    assert np.array_equal(st0, st1) and np.array_equal(H0, H1)
    assert n0 == n1
    assert _same(S0, S1)


def test_replay_matches_the_oracle():
    w = W.tiny_workload(W.OPT_ADAMW, K=4, P=3001, T=300)
    lam, ths, S, st, H, _ = _run(w, 16)
    orc = G.oracle_on(w, lam, ths)
    o_st, o_H = orc.run()
    assert np.array_equal(st, o_st) and np.array_equal(H, o_H)
    assert G.rel_err(S.theta[:, :w.P].cpu().numpy(), orc.theta) <= G.REL_TOL


def test_more_chain_lengths_than_the_cache_holds():
    """With a limit above every round length each distinct H needs its own chain; this run has more distinct
    lengths than a context keeps, so the later ones fall back to direct launches -- with the same result."""
    w = W.tiny_workload(W.OPT_SGDM, K=2, P=515, T=6000, alpha=0.3)
    _, _, S0, st0, H0, n0 = _run(w, 0)
    assert len(set(H0.tolist())) > 48
    _, _, S1, st1, H1, n1 = _run(w, 1024)
    assert np.array_equal(st0, st1) and np.array_equal(H0, H1) and n0 == n1
    assert _same(S0, S1)


def test_replay_in_pieces_and_after_a_shape_change():
    w = W.tiny_workload(W.OPT_ADAMW, K=5, P=1030, T=240)
    _, _, S0, st0, H0, _ = _run(w, 0)
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    S = G.Slabs(w)
    ctx = G.make_context(w, S, lam_d, ths_d)
    ctx.qsr_set_graph_replay(8)
    st_a, H_a = ctx.qsr_run(0, 100)
    t_mid = int(st_a[-1] + H_a[-1])
    ctx.qsr_set_launch_shape(128, 4, 0)          # discards the cached chains; the next ones use the new geometry
    st_b, H_b = ctx.qsr_run(t_mid, w.T)
    torch.cuda.synchronize()
    ctx.close()
    assert np.array_equal(np.concatenate([st_a, st_b]), st0) and np.array_equal(np.concatenate([H_a, H_b]), H0)
    assert _same(S0, S)


def test_argument_errors():
    w = W.tiny_workload(W.OPT_SGDM, K=2, P=64, T=10)
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    S = G.Slabs(w)
    ctx = G.make_context(w, S, lam_d, ths_d)
    for bad in (-1, 1025):
        with pytest.raises(B.QsrError) as e:
            ctx.qsr_set_graph_replay(bad)
        assert e.value.status == B.QSR_ERANGE
    ctx.qsr_set_graph_replay(0)
    ctx.close()


def test_tensor_table_set_between_replayed_runs():
    """A per-tensor weight-decay table set (or cleared) between two replayed runs switches the step to another kernel
    instance; the cached chains must not go on replaying the old one.  Replay on, a stretch of rounds, a table that
    switches weight decay off for one tensor, the rest of the run, the table cleared, and again -- against a context
    that launches everything directly."""
    w = W.tiny_workload(W.OPT_ADAMW, K=3, P=4096, T=300, weight_decay=0.1)
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    ends = torch.tensor([1024, 2048, 4096], dtype=torch.int64, device="cuda")
    scales = torch.tensor([1.0, 0.0, 2.0], device="cuda")
    runs = []
    for graph_steps in (0, 16):
        S = G.Slabs(w)
        ctx = G.make_context(w, S, lam_d, ths_d)
        ctx.qsr_set_graph_replay(graph_steps)
        st_a, H_a = ctx.qsr_run(0, 100)
        t1 = int(st_a[-1] + H_a[-1])
        ctx.qsr_set_tensor_table(ends, scales)
        st_b, H_b = ctx.qsr_run(t1, 200)
        t2 = int(st_b[-1] + H_b[-1])
        ctx.qsr_set_tensor_table(None, None)
        ctx.qsr_run(t2, w.T)
        torch.cuda.synchronize()
        ctx.close()
        runs.append(S)
    assert _same(runs[0], runs[1])
    # and the table did act in the middle stretch: a run without it ends elsewhere
    _, _, plain, _, _, _ = _run(w, 0)
    assert not torch.equal(plain.theta, runs[0].theta)
