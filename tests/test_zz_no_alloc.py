"""qsr_sync_static: the synchronization for callers that cannot give the library a scratch buffer.

Who needs it: code that runs where device memory is handed out once by someone else (a serving process with a fixed
memory plan, a framework allocator with a hard budget, a job whose slabs already fill the GPU) or where cudaMalloc
is off limits because it stalls the device.  Such callers have no `sum` buffer for qsr_sync_partial / qsr_sync_finish;
qsr_sync_static uses a 4 MiB array inside the library instead and allocates nothing.

Checked here, through the C ABI: its output against qsr_sync's on the same slabs, on two calls in a row with
different data (the array keeps the first call's contents, which must not show in the second), in the state modes
that change what the scratch holds, and the refusal of a problem that does not fit.  This file sorts last on purpose,
so that a run stopping at the first failure has already run every other test; it also passes alone in a fresh process.
"""
import numpy as np
import pytest
import torch

from paper_2310_14423_b200 import binding as B
from paper_2310_14423_b200 import workloads as W

import gpu_harness as G

pytestmark = pytest.mark.gpu


def _pair(w):
    """Two guarded slab sets with identical random contents, and a context over each."""
    zero = torch.zeros(w.P + 4, device="cuda")[:w.P]
    a, b = G.Slabs(w), G.Slabs(w)
    return (a, G.make_context(w, a, zero, zero)), (b, G.make_context(w, b, zero, zero))


def _fill(slabs_a, slabs_b, w, seed):
    gen = torch.Generator(device="cuda").manual_seed(seed)
    for name in ("theta", "s1", "s2"):
        x = getattr(slabs_a, name)
        if x is None:
            continue
        vals = torch.randn(slabs_a.K, w.P, device="cuda", generator=gen) * (seed + 1)
        if name == "s2":
            vals = vals.abs()
        x[:, :w.P] = vals
        getattr(slabs_b, name)[:, :w.P] = vals


@pytest.mark.parametrize("mode", [W.STATE_KEEP, W.STATE_AVERAGE, W.STATE_RESET])
def test_static_sync_equals_sync_twice_in_a_row(mode):
    assert torch.cuda.is_available()
    w = W.tiny_workload(W.OPT_ADAMW, K=5, P=30003, T=50, state_sync=mode)
    (sa, ctx_a), (sb, ctx_b) = _pair(w)
    for call, seed in enumerate((1, 2)):
        _fill(sa, sb, w, seed)
        before = ctx_b.qsr_launch_count()
        ctx_a.qsr_sync(10 * (call + 1))
        ctx_b.qsr_sync_static(10 * (call + 1))
        torch.cuda.synchronize()
        assert ctx_b.qsr_launch_count() == before + 2
        for name in ("theta", "s1", "s2"):
            ref = getattr(sa, name)[:, :w.P].cpu().numpy()
            got = getattr(sb, name)[:, :w.P].cpu().numpy()
            assert G.rel_err(got, ref) <= G.REL_TOL, (call, name)
        theta = sb.theta[:, :w.P].cpu().numpy()
        assert (theta == theta[0]).all()
        assert sa.guards_intact() and sb.guards_intact()
    ctx_a.close()
    ctx_b.close()


def test_static_sync_inside_a_run_matches_the_plain_run():
    """Whole rounds: local steps, then the static synchronization, against the same rounds with qsr_sync."""
    w = W.tiny_workload(W.OPT_SGDM, K=4, P=4099, T=40)
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    sa, sb = G.Slabs(w), G.Slabs(w)
    ctx_a, ctx_b = G.make_context(w, sa, lam_d, ths_d), G.make_context(w, sb, lam_d, ths_d)
    t = 0
    while t < w.T:
        H = ctx_a.qsr_round_length(t)
        for h in range(H):
            ctx_a.qsr_local_step(t + h)
            ctx_b.qsr_local_step(t + h)
        ctx_a.qsr_sync(t + H)
        ctx_b.qsr_sync_static(t + H)
        t += H
    torch.cuda.synchronize()
    assert G.rel_err(sb.theta[:, :w.P].cpu().numpy(), sa.theta[:, :w.P].cpu().numpy()) <= G.REL_TOL
    ctx_a.close()
    ctx_b.close()


def test_static_sync_refuses_what_does_not_fit():
    """One float more than the array holds: QSR_ERANGE, no launch, slabs untouched."""
    P = B.QSR_STATIC_SCRATCH_FLOATS + 4
    w = W.tiny_workload(W.OPT_SGDM, K=2, P=P, T=10)
    theta = torch.ones(2, P, device="cuda")
    theta[1] = 3.0
    s1 = torch.zeros(2, P, device="cuda")
    ctx = B.Context(B.make_config(w), theta, s1, None, None, None, stream=torch.cuda.current_stream().cuda_stream)
    with pytest.raises(B.QsrError) as e:
        ctx.qsr_sync_static(1)
    assert e.value.status == B.QSR_ERANGE
    assert ctx.qsr_launch_count() == 0
    torch.cuda.synchronize()
    assert bool((theta[0] == 1.0).all()) and bool((theta[1] == 3.0).all())
    ctx.close()
    # the largest problem that fits does run: AVERAGE mode with SGD needs 2 * P4 floats
    P = B.QSR_STATIC_SCRATCH_FLOATS // 2
    w = W.tiny_workload(W.OPT_SGDM, K=2, P=P, T=10, state_sync=W.STATE_AVERAGE)
    theta = torch.ones(2, P, device="cuda")
    theta[1] = 3.0
    s1 = torch.zeros(2, P, device="cuda")
    s1[0] = 4.0
    ctx = B.Context(B.make_config(w), theta, s1, None, None, None, stream=torch.cuda.current_stream().cuda_stream)
    ctx.qsr_sync_static(1)
    torch.cuda.synchronize()
    assert bool((theta == 2.0).all()) and bool((s1 == 2.0).all())
    ctx.close()
