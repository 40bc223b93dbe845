"""qsr_sync_static: the synchronization for callers that cannot give the library a scratch buffer.

Who needs it: code that runs where device memory is handed out once by someone else (a serving process with a fixed
memory plan, a framework allocator with a hard budget, a job whose slabs already fill the GPU) or where cudaMalloc
is off limits because it stalls the device.  Such callers have no `sum` buffer for qsr_sync_partial / qsr_sync_finish;
qsr_sync_static uses a 4 MiB array inside the library instead and allocates nothing.

Checked here, through the C ABI:
  - its output against qsr_sync's on the same slabs, BIT FOR BIT (the header promises the same fp32 sum over
    k = 0..K-1 and the same single division), on two calls in a row with different data, for both optimizers and the
    three state modes (they change what the scratch holds);
  - its output against the CPU oracle's synchronization (orc_sync, binary64) at the parity tolerance, same modes;
  - that a call changes neither the free device memory nor torch's allocation count;
  - that what a large call leaves in the array does not show in a smaller call whose regions sit elsewhere in it;
  - the refusal of a problem that does not fit.
This file sorts last on purpose, so that a run stopping at the first failure has already run every other test; it
also passes alone in a fresh process.
"""
import numpy as np
import pytest
import torch

from oracle import qsr_oracle as O
from paper_2310_14423_b200 import binding as B
from paper_2310_14423_b200 import workloads as W

import gpu_harness as G

pytestmark = pytest.mark.gpu

SLABS = ("theta", "s1", "s2")


def _pair(w):
    """Two guarded slab sets and a context over each."""
    zero = torch.zeros(w.P + 4, device="cuda")[:w.P]
    a, b = G.Slabs(w), G.Slabs(w)
    return (a, G.make_context(w, a, zero, zero)), (b, G.make_context(w, b, zero, zero))


def _fill(slabs_a, slabs_b, w, seed):
    """The same seeded random contents in both slab sets; returns them as binary64 host arrays."""
    gen = torch.Generator(device="cuda").manual_seed(seed)
    host = {}
    for name in SLABS:
        x = getattr(slabs_a, name)
        if x is None:
            continue
        vals = torch.randn(slabs_a.K, w.P, device="cuda", generator=gen) * (seed + 1)
        if name == "s2":
            vals = vals.abs()
        x[:, :w.P] = vals
        getattr(slabs_b, name)[:, :w.P] = vals
        host[name] = vals.double().cpu().numpy()
    return host


def _same_bits(sa, sb):
    return all(getattr(sa, n) is None or torch.equal(getattr(sa, n), getattr(sb, n)) for n in SLABS)


@pytest.mark.parametrize("opt", [W.OPT_SGDM, W.OPT_ADAMW])
@pytest.mark.parametrize("mode", [W.STATE_KEEP, W.STATE_AVERAGE, W.STATE_RESET])
def test_static_sync_equals_sync_bitwise_and_the_oracle_twice_in_a_row(mode, opt):
    assert torch.cuda.is_available()
    w = W.tiny_workload(opt, K=5, P=30003, T=50, state_sync=mode)
    (sa, ctx_a), (sb, ctx_b) = _pair(w)
    for call, seed in enumerate((1, 2)):
        host = _fill(sa, sb, w, seed)
        before = ctx_b.qsr_launch_count()
        ctx_a.qsr_sync(10 * (call + 1))
        ctx_b.qsr_sync_static(10 * (call + 1))
        torch.cuda.synchronize()
        assert ctx_b.qsr_launch_count() == before + (3 if mode == W.STATE_RESET else 2)    # sums, rows, [state reset]
        assert _same_bits(sa, sb), (call, mode, opt)
        # the oracle's synchronization on the same numbers
        orc = O.State(w, np.zeros(w.P), np.zeros(w.P))
        orc.theta[:] = host["theta"]
        orc.s1[:] = host["s1"]
        if "s2" in host:
            orc.s2[:] = host["s2"]
        orc.sync(10 * (call + 1))
        for name in host:
            got = getattr(sb, name)[:, :w.P].cpu().numpy()
            ref = getattr(orc, name)
            if mode == W.STATE_RESET and name != "theta":
                assert not got.any() and not ref.any()
            else:
                assert G.rel_err(got, ref) <= G.REL_TOL, (call, name)
        theta = sb.theta[:, :w.P].cpu().numpy()
        assert (theta == theta[0]).all()
        assert sa.guards_intact() and sb.guards_intact()
    ctx_a.close()
    ctx_b.close()


def test_static_sync_allocates_no_device_memory():
    """After the first call (which looks the array's address up) a call leaves the device's free memory and torch's
    books exactly as they were."""
    w = W.tiny_workload(W.OPT_ADAMW, K=4, P=100003, T=20, state_sync=W.STATE_AVERAGE)
    (sa, ctx_a), (sb, ctx_b) = _pair(w)
    _fill(sa, sb, w, 3)
    ctx_b.qsr_sync_static(1)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for t in (2, 3, 4):
        ctx_b.qsr_sync_static(t)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
    ctx_a.close()
    ctx_b.close()


def test_leftovers_of_a_large_call_do_not_show_in_a_smaller_one():
    """AVERAGE mode with AdamW keeps three regions in the array, at multiples of P rounded up to 4.  A call with a
    large P fills the array far beyond where a later call with a small P puts its second and third regions, so that
    call finds the large one's sums everywhere it has not yet written.  Results must still equal qsr_sync's bits."""
    big = W.tiny_workload(W.OPT_ADAMW, K=3, P=B.QSR_STATIC_SCRATCH_FLOATS // 3 - 5, T=20, state_sync=W.STATE_AVERAGE)
    (sa, ctx_a), (sb, ctx_b) = _pair(big)
    _fill(sa, sb, big, 5)
    ctx_a.qsr_sync(1)
    ctx_b.qsr_sync_static(1)
    torch.cuda.synchronize()
    assert _same_bits(sa, sb)
    ctx_a.close()
    ctx_b.close()
    for P in (1001, 70001):
        small = W.tiny_workload(W.OPT_ADAMW, K=7, P=P, T=20, state_sync=W.STATE_AVERAGE)
        (sa, ctx_a), (sb, ctx_b) = _pair(small)
        _fill(sa, sb, small, 6)
        ctx_a.qsr_sync(1)
        ctx_b.qsr_sync_static(1)
        torch.cuda.synchronize()
        assert _same_bits(sa, sb), P
        assert sa.guards_intact() and sb.guards_intact()
        ctx_a.close()
        ctx_b.close()


def test_static_sync_inside_a_run_matches_the_plain_run():
    """Whole rounds: local steps, then the static synchronization, against the same rounds with qsr_sync (same bits)
    and against the oracle's run (parity tolerance)."""
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
    assert _same_bits(sa, sb)
    orc = G.oracle_on(w, lam, ths)
    orc.run()
    assert G.rel_err(sb.theta[:, :w.P].cpu().numpy(), orc.theta) <= G.REL_TOL
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
