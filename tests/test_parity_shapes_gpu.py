"""GPU parity at the full sizes of the shaped configurations (ResNet-152 and ViT-B/16 parameter sets).

The device runs every coordinate of every worker for the whole schedule, in the launch configuration the
benchmark uses (library defaults).  The oracle follows a subset of coordinates -- the first and last element of
each tensor and their neighbours, the row ends, and random fill -- through all K workers and all steps; since
coordinates never interact, those columns are the exact algorithm.  Bars as in test_parity_gpu.py.
"""
import numpy as np
import pytest
import torch

from paper_2310_14423_b200 import binding as B
from paper_2310_14423_b200 import workloads as W

import gpu_harness as G

pytestmark = pytest.mark.gpu

N_SUBSET = 4096


def _run_device(w, t_end=None):
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    stride = B.qsr_row_stride_hint(w.P)              # the layout bench.py uses
    theta = torch.zeros(w.K, stride, device="cuda")
    s1 = torch.zeros(w.K, stride, device="cuda")
    s2 = torch.zeros(w.K, stride, device="cuda") if w.opt == W.OPT_ADAMW else None
    cfg = B.make_config(w, row_stride=stride)
    ctx = B.Context(cfg, theta, s1, s2, lam_d, ths_d, stream=torch.cuda.current_stream().cuda_stream)
    st, H = ctx.qsr_run(0, t_end)
    torch.cuda.synchronize()
    ctx.close()
    return lam, ths, theta, st, H


def _compare(w, lam, ths, theta, st, H, t_end=None):
    idx = W.coordinate_subset(w.layout, N_SUBSET, seed=7)
    orc = G.oracle_on(w, lam, ths, idx)
    ost, oH = orc.run(0, t_end)
    assert np.array_equal(st, ost) and np.array_equal(H, oH)
    idx_d = torch.from_numpy(idx).cuda()
    cols = theta[:, idx_d].cpu().numpy()
    assert (cols == cols[0]).all()                       # every worker holds the average
    err = G.rel_err(cols[0], orc.theta[0])
    assert err <= G.REL_TOL, err
    return err


@pytest.fixture(autouse=True)
def _free():
    assert torch.cuda.is_available()
    yield
    torch.cuda.synchronize()
    torch.cuda.empty_cache()


def test_resnet152_shape_full_schedule():
    """K=16, P=60,192,808 in 467 tensors, Local SGD momentum 0.9 wd 1e-4, cosine from 0.8, T=10,000."""
    w = W.workload("c3")
    assert len(w.layout.names) == 467 and w.P == 60_192_808
    lam, ths, theta, st, H = _run_device(w)
    assert len(st) == 3950 and st[-1] + H[-1] == w.T
    _compare(w, lam, ths, theta, st, H)


def test_vit_b16_shape_full_schedule():
    """K=16, P=86,415,592, Local AdamW wd 0.05, warm-up 100 + cosine from 8e-4, T=10,000: the benchmark's workload."""
    w = W.workload("c4")
    assert w.P == 86_415_592
    lam, ths, theta, st, H = _run_device(w)
    assert len(st) == 10 and H[0] == 478
    _compare(w, lam, ths, theta, st, H)


def test_vit_b16_paper_learning_rate_first_rounds():
    """Peak learning rate 0.008 as in the paper's ViT-B runs: H_base = 4 rules the first rounds; 600 steps, 150 syncs."""
    w = W.workload("c4p")
    lam, ths, theta, st, H = _run_device(w, t_end=600)
    assert (H == 4).all() and len(st) == 150
    _compare(w, lam, ths, theta, st, H, t_end=600)


def test_k32_slab_beyond_32bit_indexing():
    """K=32 workers of the ViT-B/16 set: K*P = 2.77e9 elements per slab, so element offsets need 64 bits.
    The first two rounds (478 + 481 steps) are enough to visit every element."""
    w = W.workload("c5")
    assert w.K * w.P > 2 ** 31
    lam, ths, theta, st, H = _run_device(w, t_end=500)
    assert st.tolist() == [0, 478] and H.tolist() == [478, 481]
    _compare(w, lam, ths, theta, st, H, t_end=500)
    assert bool((theta[31, :w.P] == theta[0, :w.P]).all())


def test_k32_reset_and_replica_copy_at_full_size():
    """K=32 at the paper's peak learning rate with the optimizer state reset at every synchronization, from a non-zero
    theta_bar(0): the replica copy and the state-reset launches write rows whose element offsets need 64 bits; three
    rounds of four steps, compared on the coordinate subset, and the state slabs must be zero everywhere afterwards."""
    w = W.workload("c5").replace(eta_max=8e-3, state_sync=W.STATE_RESET)
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    stride = B.qsr_row_stride_hint(w.P)
    theta = torch.full((w.K, stride), 7.0, device="cuda")          # 7.0 marks what must be overwritten or left alone
    s1 = torch.full((w.K, stride), 7.0, device="cuda")
    s2 = torch.full((w.K, stride), 7.0, device="cuda")
    s1[:, :w.P] = 0.0
    s2[:, :w.P] = 0.0
    gen = torch.Generator(device="cuda").manual_seed(3)
    theta0 = torch.randn(w.P, device="cuda", generator=gen) * 0.1
    ctx = B.Context(B.make_config(w, row_stride=stride), theta, s1, s2, lam_d, ths_d,
                    stream=torch.cuda.current_stream().cuda_stream)
    ctx.qsr_set_params(theta0)
    torch.cuda.synchronize()
    assert bool((theta[31, :w.P] == theta0).all()) and bool((theta[0, :w.P] == theta0).all())
    st, H = ctx.qsr_run(0, 12)
    torch.cuda.synchronize()
    ctx.close()
    assert st.tolist() == [0, 4, 8] and H.tolist() == [4, 4, 4]
    idx = W.coordinate_subset(w.layout, N_SUBSET, seed=7)
    orc = G.oracle_on(w, lam, ths, idx)
    orc.theta[:] = theta0[torch.from_numpy(idx).cuda()].double().cpu().numpy()
    orc.run(0, 12)
    cols = theta[:, torch.from_numpy(idx).cuda()].cpu().numpy()
    assert (cols == cols[0]).all()
    assert G.rel_err(cols[0], orc.theta[0]) <= G.REL_TOL
    assert not bool(s1[:, :w.P].any()) and not bool(s2[:, :w.P].any())          # reset: zero on every row
    if stride > w.P:                                                            # padding is never written
        assert bool((theta[:, w.P:] == 7.0).all()) and bool((s1[:, w.P:] == 7.0).all()) and bool((s2[:, w.P:] == 7.0).all())


def test_k32_resident_launches_at_full_size():
    """The register-resident launches (benchmark-only) on the K=32 slabs: 64-bit offsets, 1024-thread blocks (32 columns
    x 32 rows); the first round of 478 steps in four launches, against the oracle on the coordinate subset."""
    w = W.workload("c5")
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    stride = B.qsr_row_stride_hint(w.P)
    theta = torch.zeros(w.K, stride, device="cuda")
    s1 = torch.zeros(w.K, stride, device="cuda")
    s2 = torch.zeros(w.K, stride, device="cuda")
    ctx = B.Context(B.make_config(w, row_stride=stride), theta, s1, s2, lam_d, ths_d,
                    stream=torch.cuda.current_stream().cuda_stream)
    ctx.qsr_set_resident_steps(128)
    st, H = ctx.qsr_run(0, 400)
    torch.cuda.synchronize()
    assert ctx.qsr_launch_count() == 4 and st.tolist() == [0] and H.tolist() == [478]
    ctx.close()
    _compare(w, lam, ths, theta, st, H, t_end=400)
    assert bool((theta[31, :w.P] == theta[0, :w.P]).all())
