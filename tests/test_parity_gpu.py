"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same seeded inputs.

Bars: round starts / lengths (hence sync step indices) bit-exact; final parameters within REL_TOL = 1e-5 under
    max_i |gpu - oracle| / max(|oracle_i|, rms(oracle)),
the oracle in binary64, the library in fp32.  Small cases are compared on every coordinate; the shaped
configurations run at full size on the device and are compared on a coordinate subset (first / last element of
every tensor, row ends, random fill) that the oracle follows through all K workers and all T steps.
"""
import numpy as np
import pytest
import torch

from oracle import qsr_oracle as O
from paper_2310_14423_b200 import binding as B
from paper_2310_14423_b200 import workloads as W

import gpu_harness as G

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _cuda():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    B.lib()  # must be the built CUDA library; there is nothing else to fall back to
    yield
    torch.cuda.synchronize()
    torch.cuda.empty_cache()


def _run_full(w, row_stride=None, shape=None):
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    S = G.Slabs(w, row_stride=row_stride)
    ctx = G.make_context(w, S, lam_d, ths_d)
    if shape:
        ctx.qsr_set_launch_shape(*shape)
    st, H = ctx.qsr_run()
    torch.cuda.synchronize()
    launches = ctx.qsr_launch_count()
    ctx.close()
    return lam, ths, S, st, H, launches


# ------------------------------------------------------------------ noise generator

def test_noise_matches_oracle_elementwise():
    """SGD with mu = 0, wd = 0, lambda = 0, eta = 1, sigma = 1 turns theta into -z after one step from zero."""
    P, K, t = 40000 + 3, 3, 77
    w = W.tiny_workload(W.OPT_SGDM, K=K, P=P, T=100, sched=W.SCHED_CONST, eta_max=1.0, momentum=0.0,
                        weight_decay=0.0, noise_std=1.0, noise_seed=0xDEADBEEF12345678 % (1 << 63))
    S = G.Slabs(w)
    zero = torch.zeros(P + 1, device="cuda")[:P]
    ctx = G.make_context(w, S, zero, zero)
    ctx.qsr_local_step(t)
    torch.cuda.synchronize()
    z_gpu = -S.theta[:, :P].cpu().numpy().astype(np.float64)
    for k in range(K):
        z = O.noise_fill(w.noise_seed, k, t, 0, P)
        assert np.abs(z_gpu[k] - z).max() < 2e-6
    ctx.close()


def test_noise_has_no_bias_against_oracle():
    """4 M normals: the fp32 generator's error against the binary64 oracle is rounding-sized and averages out.
    A bias b in the noise would shift a coordinate of curvature lambda by sigma*b/lambda, so it is bounded tightly."""
    P, K, t = 1 << 20, 4, 4242
    w = W.tiny_workload(W.OPT_SGDM, K=K, P=P, T=5000, sched=W.SCHED_CONST, eta_max=1.0, momentum=0.0,
                        weight_decay=0.0, noise_std=1.0)
    S = G.Slabs(w)
    zero = torch.zeros(P, device="cuda")
    ctx = G.make_context(w, S, zero, zero)
    ctx.qsr_local_step(t)
    torch.cuda.synchronize()
    z_gpu = -S.theta[:, :P].cpu().numpy().astype(np.float64)
    err = np.concatenate([z_gpu[k] - O.noise_fill(w.noise_seed, k, t, 0, P) for k in range(K)])
    assert np.abs(err).max() < 2e-6
    assert np.sqrt(np.mean(err * err)) < 1.5e-7
    assert abs(err.mean()) < 2e-9
    assert abs(z_gpu.mean()) < 4 / np.sqrt(K * P) and abs(z_gpu.var() - 1) < 6 / np.sqrt(K * P)
    ctx.close()


def test_noise_high_counter_words():
    """Worker offset, a step beyond 2^16 and the last coordinates of a long row reach the counter unchanged."""
    P = 1 << 16
    w = W.tiny_workload(W.OPT_SGDM, K=2, P=P, T=1 << 20, sched=W.SCHED_CONST, eta_max=1.0, momentum=0.0,
                        weight_decay=0.0, noise_std=1.0, worker_offset=1000)
    S = G.Slabs(w)
    zero = torch.zeros(P, device="cuda")
    ctx = G.make_context(w, S, zero, zero)
    t = 777777
    ctx.qsr_local_step(t)
    torch.cuda.synchronize()
    z_gpu = -S.theta.cpu().numpy().astype(np.float64)
    for k in range(2):
        assert np.abs(z_gpu[k] - O.noise_fill(w.noise_seed, 1000 + k, t, 0, P)).max() < 2e-6
    ctx.close()


# ------------------------------------------------------------------ small cases, every coordinate

@pytest.mark.parametrize("opt", [W.OPT_SGDM, W.OPT_ADAMW])
@pytest.mark.parametrize("P", [1, 2, 3, 4, 5, 1001, 1002, 1003, 4096])
def test_tiny_ragged_runs(opt, P):
    w = W.tiny_workload(opt, K=3, P=P, T=60)
    lam, ths, S, st, H, launches = _run_full(w, row_stride=(P + 3) // 4 * 4 + 8)
    orc = G.oracle_on(w, lam, ths)
    ost, oH = orc.run()
    assert np.array_equal(st, ost) and np.array_equal(H, oH)
    assert launches == w.T          # the last step of each round carries the averaging
    theta = S.theta[:, :P].cpu().numpy()
    assert (theta == theta[0]).all()
    assert G.rel_err(theta[0], orc.theta[0]) <= G.REL_TOL
    assert S.guards_intact()


@pytest.mark.parametrize("rows", [1, 2, 4, 8])
@pytest.mark.parametrize("K", [1, 2, 5, 8, 17])
def test_rows_in_flight_and_worker_counts(rows, K):
    w = W.tiny_workload(W.OPT_ADAMW, K=K, P=2051, T=24)
    lam, ths, S, st, H, _ = _run_full(w, shape=(128, rows, 128))
    orc = G.oracle_on(w, lam, ths)
    ost, oH = orc.run()
    assert np.array_equal(st, ost) and np.array_equal(H, oH)
    assert G.rel_err(S.theta[0, :w.P].cpu().numpy(), orc.theta[0]) <= G.REL_TOL
    assert S.guards_intact()


def test_config1_full():
    """K=4, P=65,536, Local SGD with momentum, cosine, QSR alpha=0.2 H_base=2, T=2000: every coordinate."""
    w = W.workload("c1")
    lam, ths, S, st, H, launches = _run_full(w)
    orc = G.oracle_on(w, lam, ths)
    ost, oH = orc.run()
    assert np.array_equal(st, ost) and np.array_equal(H, oH)
    assert np.array_equal(st + H, ost + oH)            # sync step indices
    assert len(st) == 203 and launches == 2000
    theta = S.theta.cpu().numpy()
    assert (theta == theta[0]).all()
    assert G.rel_err(theta[0], orc.theta[0]) <= G.REL_TOL


def test_config2_subset():
    """K=8, P=2^20, Local AdamW, warm-up + cosine, T=5000: device runs all of it, the oracle 8192 coordinates."""
    w = W.workload("c2")
    lam, ths, S, st, H, _ = _run_full(w)
    idx = W.coordinate_subset(w.layout, 8192, seed=2)
    orc = G.oracle_on(w, lam, ths, idx)
    ost, oH = orc.run()
    assert np.array_equal(st, ost) and np.array_equal(H, oH) and len(st) == 8
    theta = S.theta[0].cpu().numpy()
    assert G.rel_err(theta[idx], orc.theta[0]) <= G.REL_TOL


# ------------------------------------------------------------------ the pieces of the ABI

def test_external_gradients():
    for opt in (W.OPT_SGDM, W.OPT_ADAMW):
        w = W.tiny_workload(opt, K=3, P=3001, T=12)
        S = G.Slabs(w, n_extra=1)
        ctx = G.make_context(w, S, None, None)
        orc = O.State(w, np.zeros(w.P), np.zeros(w.P))
        gen = torch.Generator(device="cuda").manual_seed(5)
        grads = S.extra[0]
        for t in range(w.T):
            grads[:, :w.P] = torch.randn(3, w.P, device="cuda", generator=gen)
            ctx.qsr_local_step(t, grads)
            orc.local_step(t, grads=grads[:, :w.P].cpu().numpy().astype(np.float64))
            if t % 4 == 3:
                ctx.qsr_sync(t + 1)
                orc.sync(t + 1)
        torch.cuda.synchronize()
        assert G.rel_err(S.theta[:, :w.P].cpu().numpy(), orc.theta) <= G.REL_TOL
        assert S.guards_intact()
        with pytest.raises(B.QsrError):
            ctx.qsr_run()            # no lambda / theta_star: generated gradients are unavailable
        ctx.close()


@pytest.mark.parametrize("mode", [W.STATE_KEEP, W.STATE_AVERAGE, W.STATE_RESET])
@pytest.mark.parametrize("opt", [W.OPT_SGDM, W.OPT_ADAMW])
def test_state_modes(mode, opt):
    w = W.tiny_workload(opt, K=4, P=1003, T=48, state_sync=mode)
    lam, ths, S, st, H, _ = _run_full(w)
    orc = G.oracle_on(w, lam, ths)
    ost, oH = orc.run()
    assert np.array_equal(st, ost) and np.array_equal(H, oH)
    assert G.rel_err(S.theta[:, :w.P].cpu().numpy(), orc.theta) <= G.REL_TOL
    s1 = S.s1[:, :w.P].cpu().numpy()
    if mode == W.STATE_RESET:
        assert not s1.any()
    elif mode == W.STATE_AVERAGE:
        assert (s1 == s1[0]).all()
        assert G.rel_err(s1, orc.s1) <= 1e-4
    else:
        assert np.abs(s1 - s1[0]).max() > 0


def test_sync_invariants():
    w = W.tiny_workload(W.OPT_SGDM, K=8, P=5003, T=10)
    S = G.Slabs(w)
    zero = torch.zeros(w.P + 1, device="cuda")[:w.P]
    ctx = G.make_context(w, S, zero, zero)
    S.theta[:, :w.P] = torch.randn(8, w.P, device="cuda")
    S.s1[:, :w.P] = 3.0
    before = S.theta[:, :w.P].double().cpu().numpy()
    ctx.qsr_sync(1)
    torch.cuda.synchronize()
    after = S.theta[:, :w.P].cpu().numpy()
    assert (after == after[0]).all()
    # fp32 running sum over k ascending, then one division by K
    acc = np.zeros(w.P, np.float32)
    for k in range(8):
        acc = acc + before[k].astype(np.float32)
    assert np.array_equal(after[0], acc / np.float32(8))
    assert np.abs(after[0] - before.mean(0)).max() < 1e-6
    assert bool((S.s1[:, :w.P] == 3.0).all())
    ctx.close()
    # K = 1: the mean of one row is the row
    w1 = W.tiny_workload(W.OPT_SGDM, K=1, P=77)
    S1 = G.Slabs(w1)
    ctx = G.make_context(w1, S1, zero[:77], zero[:77])
    S1.theta[:, :77] = torch.randn(1, 77, device="cuda")
    ref = S1.theta.clone()
    ctx.qsr_sync(1)
    torch.cuda.synchronize()
    assert torch.equal(S1.theta, ref)
    ctx.close()


def test_sharded_sync_equals_single_process():
    """Workers split over two contexts (as over two GPUs): partial sums, SUM all-reduce (here an add), finish."""
    for mode in (W.STATE_KEEP, W.STATE_AVERAGE, W.STATE_RESET):
        w = W.tiny_workload(W.OPT_ADAMW, K=6, P=2003, T=40, state_sync=mode)
        lam, ths, lam_d, ths_d = G.device_inputs(w)
        parts = []
        for r in range(2):
            S = G.Slabs(w, K=3)
            parts.append((S, G.make_context(w, S, lam_d, ths_d, worker_offset=3 * r)))
        n_sum = parts[0][1].qsr_sync_sum_floats()
        sums = [torch.zeros(n_sum, device="cuda") for _ in range(2)]
        t = 0
        rounds = []
        while t < w.T:
            H = parts[0][1].qsr_round_length(t)
            assert H == parts[1][1].qsr_round_length(t)
            for h in range(H - 1):
                for S, ctx in parts:
                    ctx.qsr_local_step(t + h)
            for r, ((S, ctx), buf) in enumerate(zip(parts, sums)):
                if r == 0:                       # one rank takes the two-launch route, the other the fused one
                    ctx.qsr_local_step(t + H - 1)
                    ctx.qsr_sync_partial(buf)
                else:
                    ctx.qsr_local_step_partial(t + H - 1, buf)
            total = sums[0] + sums[1]
            for S, ctx in parts:
                ctx.qsr_sync_finish(total, 6, t + H)
            rounds.append((t, H))
            t += H
        torch.cuda.synchronize()
        orc = G.oracle_on(w, lam, ths)
        ost, oH = orc.run()
        assert [r[0] for r in rounds] == ost.tolist() and [r[1] for r in rounds] == oH.tolist()
        for r, (S, ctx) in enumerate(parts):
            assert G.rel_err(S.theta[:, :w.P].cpu().numpy(), orc.theta[3 * r:3 * r + 3]) <= G.REL_TOL
            assert S.guards_intact()
            with pytest.raises(B.QsrError) as e:
                ctx.qsr_sync_finish(total, 6, w.T)     # no partial pending
            assert e.value.status == B.QSR_ESTATE
            ctx.close()


class _TwoShards:
    """Two contexts on one GPU behind the interface of one engine: every call goes to both, each shard writes its
    partial sums to its own half of the buffer, and the 'all-reduce' adds the halves, as the exchange would."""

    def __init__(self, parts, n_sum):
        self.parts, self.n = parts, n_sum

    def qsr_round_length(self, t):
        H = {ctx.qsr_round_length(t) for _, ctx in self.parts}
        assert len(H) == 1
        return H.pop()

    def qsr_local_step(self, t):
        for _, ctx in self.parts:
            ctx.qsr_local_step(t)

    def qsr_local_step_partial(self, t, sums):
        for r, (_, ctx) in enumerate(self.parts):
            ctx.qsr_local_step_partial(t, sums[r * self.n:(r + 1) * self.n])

    def all_reduce(self, sums):
        total = sums[:self.n] + sums[self.n:]
        sums[:self.n] = total
        sums[self.n:] = total

    def qsr_sync_finish(self, sums, K_total, t_next):
        for r, (_, ctx) in enumerate(self.parts):
            ctx.qsr_sync_finish(sums[r * self.n:(r + 1) * self.n], K_total, t_next)


@pytest.mark.parametrize("mode", [W.STATE_KEEP, W.STATE_AVERAGE, W.STATE_RESET])
@pytest.mark.parametrize("opt", [W.OPT_SGDM, W.OPT_ADAMW])
def test_sharded_loop_over_two_contexts(opt, mode):
    """The product's round loop (sharded.run_steps, the one the benchmark times and the gloo tests drive) over the
    library's own partial-sum and finish launches: 7 workers split 4 + 3 over two contexts, all state modes -- in
    AVERAGE mode the exchanged buffer carries the sums of the state slabs after those of the parameters."""
    from paper_2310_14423_b200 import sharded
    w = W.tiny_workload(opt, K=7, P=2003, T=40, state_sync=mode)
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    parts = []
    for r in range(2):
        rows, k0 = sharded.shard(7, 2, r)
        S = G.Slabs(w, K=rows)
        parts.append((S, G.make_context(w, S, lam_d, ths_d, worker_offset=k0)))
    n_sum = parts[0][1].qsr_sync_sum_floats()
    assert n_sum == (1 if mode != W.STATE_AVERAGE else (3 if opt == W.OPT_ADAMW else 2)) * 2004
    pair = _TwoShards(parts, n_sum)
    sums = torch.zeros(2 * n_sum, device="cuda")
    rounds = sharded.run_steps(pair, 0, w.T, sharded.Exchange(sums, 7, pair.all_reduce), whole_rounds=True)
    torch.cuda.synchronize()
    orc = G.oracle_on(w, lam, ths)
    ost, oH = orc.run()
    assert [r[0] for r in rounds] == ost.tolist() and [r[1] for r in rounds] == oH.tolist()
    for r, (S, ctx) in enumerate(parts):
        rows, k0 = sharded.shard(7, 2, r)
        assert G.rel_err(S.theta[:, :w.P].cpu().numpy(), orc.theta[k0:k0 + rows]) <= G.REL_TOL
        if mode == W.STATE_AVERAGE:
            assert G.rel_err(S.s1[:, :w.P].cpu().numpy(), orc.s1[k0:k0 + rows]) <= 1e-4
        if mode == W.STATE_RESET:
            assert not S.s1[:, :w.P].any()
        assert S.guards_intact()
        ctx.close()


def test_train_host_equals_context_path():
    for opt in (W.OPT_SGDM, W.OPT_ADAMW):
        w = W.tiny_workload(opt, K=4, P=10007, T=50)
        lam, ths, S, st, H, launches = _run_full(w)
        cfg = B.make_config(w)
        ws = torch.empty(B.qsr_workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
        out = np.empty(w.P, np.float32)
        st2, H2, launches2 = B.qsr_train_host(cfg, np.zeros(w.P, np.float32), lam, ths, out, ws,
                                              stream=torch.cuda.current_stream().cuda_stream)
        assert np.array_equal(st, st2) and np.array_equal(H, H2)
        assert launches2 == launches + 1               # plus the copy of theta_bar(0) to every worker
        assert np.array_equal(out, S.theta[0, :w.P].cpu().numpy())
        small = torch.empty(1024, dtype=torch.uint8, device="cuda")
        with pytest.raises(B.QsrError) as e:
            B.qsr_train_host(cfg, np.zeros(w.P, np.float32), lam, ths, out, small)
        assert e.value.status == B.QSR_ERANGE


@pytest.mark.parametrize("opt", [W.OPT_SGDM, W.OPT_ADAMW])
@pytest.mark.parametrize("K,P", [(3, 1001), (5, 4098), (16, 2051), (1, 7)])
def test_fused_last_step_equals_step_then_sync_bitwise(opt, K, P):
    """qsr_local_step_sync (one launch) against qsr_local_step + qsr_sync (two): same bits in every slab."""
    w = W.tiny_workload(opt, K=K, P=P, T=36)
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    A, Bs = G.Slabs(w), G.Slabs(w)
    ca, cb = G.make_context(w, A, lam_d, ths_d), G.make_context(w, Bs, lam_d, ths_d)
    t = 0
    while t < w.T:
        H = ca.qsr_round_length(t)
        for h in range(H - 1):
            ca.qsr_local_step(t + h)
            cb.qsr_local_step(t + h)
        ca.qsr_local_step(t + H - 1)
        ca.qsr_sync(t + H)
        cb.qsr_local_step_sync(t + H - 1, t + H)
        t += H
    torch.cuda.synchronize()
    assert cb.qsr_launch_count() == w.T and ca.qsr_launch_count() > w.T
    assert torch.equal(A.theta, Bs.theta) and torch.equal(A.s1, Bs.s1)
    if opt == W.OPT_ADAMW:
        assert torch.equal(A.s2, Bs.s2)
    assert Bs.guards_intact()
    ca.close()
    cb.close()


@pytest.mark.parametrize("opt", [W.OPT_SGDM, W.OPT_ADAMW])
def test_row_stride_does_not_change_the_bits(opt):
    """Rows packed at P, at the stride the library recommends and at an odd padded stride: the layout is a matter of
    speed only, every parameter and state value is bit-identical (padding stays untouched: the guards check it)."""
    w = W.tiny_workload(opt, K=5, P=70003, T=60)
    hinted = B.qsr_row_stride_hint(w.P)
    assert hinted % 4096 == 0 and hinted >= w.P
    runs = []
    for stride in ((w.P + 3) // 4 * 4, hinted, (w.P + 3) // 4 * 4 + 36):
        lam, ths, S, st, H, _ = _run_full(w, row_stride=stride)
        assert S.guards_intact()
        runs.append(S)
    for S in runs[1:]:
        assert torch.equal(S.theta[:, :w.P], runs[0].theta[:, :w.P])
        assert torch.equal(S.s1[:, :w.P], runs[0].s1[:, :w.P])
        assert S.s2 is None or torch.equal(S.s2[:, :w.P], runs[0].s2[:, :w.P])


def test_nonzero_start_and_set_params():
    w = W.tiny_workload(W.OPT_SGDM, K=3, P=999, T=30)
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    S = G.Slabs(w)
    ctx = G.make_context(w, S, lam_d, ths_d)
    theta0 = torch.randn(w.P + 1, device="cuda")[:w.P]
    ctx.qsr_set_params(theta0)
    st, H = ctx.qsr_run()
    torch.cuda.synchronize()
    orc = G.oracle_on(w, lam, ths)
    orc.theta[:] = theta0.cpu().numpy().astype(np.float64)
    orc.run()
    assert G.rel_err(S.theta[:, :w.P].cpu().numpy(), orc.theta) <= G.REL_TOL
    assert S.guards_intact()
    ctx.close()


def test_resume_is_bit_identical():
    for opt, mode in ((W.OPT_SGDM, W.STATE_KEEP), (W.OPT_ADAMW, W.STATE_KEEP), (W.OPT_ADAMW, W.STATE_RESET)):
        w = W.tiny_workload(opt, K=3, P=2001, T=80, state_sync=mode)
        lam, ths, S, st, H, _ = _run_full(w)
        lam, ths, lam_d, ths_d = G.device_inputs(w)
        S2 = G.Slabs(w)
        ctx = G.make_context(w, S2, lam_d, ths_d)
        st_a, H_a = ctx.qsr_run(0, 40)
        t_mid = int(st_a[-1] + H_a[-1])
        ctx.close()
        torch.cuda.synchronize()
        # a new context over the same memory, told where the optimizer state was last zero
        origin = t_mid if mode == W.STATE_RESET else 0
        ctx = G.make_context(w, S2, lam_d, ths_d, t_state_origin=origin)
        st_b, H_b = ctx.qsr_run(t_mid, w.T)
        torch.cuda.synchronize()
        assert np.array_equal(np.concatenate([st_a, st_b]), st) and np.array_equal(np.concatenate([H_a, H_b]), H)
        assert torch.equal(S.theta, S2.theta) and torch.equal(S.s1, S2.s1)
        ctx.close()


def test_step_argument_errors():
    w = W.tiny_workload(W.OPT_SGDM, K=2, P=64, T=10)
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    S = G.Slabs(w)
    ctx = G.make_context(w, S, lam_d, ths_d)
    for t in (-1, 10):
        with pytest.raises(B.QsrError) as e:
            ctx.qsr_local_step(t)
        assert e.value.status == B.QSR_ERANGE
    with pytest.raises(B.QsrError) as e:
        ctx.qsr_local_step(0, S.theta.view(-1)[1:5])       # misaligned gradient pointer
    assert e.value.status == B.QSR_EALIGN
    with pytest.raises(B.QsrError):
        ctx.qsr_set_launch_shape(100, 0, 0)
    with pytest.raises(B.QsrError):
        ctx.qsr_set_launch_shape(0, 3, 0)
    assert not S.theta[:, :w.P].any()                      # failed calls wrote nothing
    ctx.close()


@pytest.mark.parametrize("opt", [W.OPT_SGDM, W.OPT_ADAMW])
def test_per_tensor_weight_decay_table(opt):
    """A tensor table with factors 1, 0, 0.5, 2 on the weight decay (tensor ends multiples of 4, the last one ragged)."""
    ends = np.array([400, 404, 2000, 3003], np.int64)
    scales = np.array([1.0, 0.0, 0.5, 2.0], np.float32)
    w = W.tiny_workload(opt, K=3, P=3003, T=40, weight_decay=0.1)
    lam, ths, lam_d, ths_d = G.device_inputs(w)
    S = G.Slabs(w)
    ctx = G.make_context(w, S, lam_d, ths_d)
    ctx.qsr_set_tensor_table(torch.from_numpy(ends).cuda(), torch.from_numpy(scales).cuda())
    st, H = ctx.qsr_run()
    torch.cuda.synchronize()
    per_coord = np.repeat(scales.astype(np.float64), np.diff(np.concatenate([[0], ends])))
    orc = O.State(w, lam, ths, wd_scale=per_coord)
    ost, oH = orc.run()
    assert np.array_equal(st, ost) and np.array_equal(H, oH)
    got = S.theta[0, :w.P].cpu().numpy()
    assert G.rel_err(got, orc.theta[0]) <= G.REL_TOL
    plain = G.oracle_on(w, lam, ths)
    plain.run()
    assert G.rel_err(got, plain.theta[0]) > 1e-4          # the table does change the result
    # clearing the table restores the uniform weight decay
    S2 = G.Slabs(w)
    ctx2 = G.make_context(w, S2, lam_d, ths_d)
    ctx2.qsr_set_tensor_table(torch.from_numpy(ends).cuda(), torch.from_numpy(scales).cuda())
    ctx2.qsr_set_tensor_table(None, None)
    ctx2.qsr_run()
    torch.cuda.synchronize()
    assert G.rel_err(S2.theta[0, :w.P].cpu().numpy(), plain.theta[0]) <= G.REL_TOL
    ctx.close()
    ctx2.close()
