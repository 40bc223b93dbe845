"""The device code of the Box-Muller transform on EVERY input it can meet, against the binary64 oracle.

The synthetic gradient's noise is radius(u1) * cos / sin(angle(u2)) with u1, u2 on a grid of 2^23 points each, and the
library evaluates -2 ln u1, the square root and the sine / cosine with code written for exactly that grid (polynomials
and single special-function instructions, no math library).  Their accuracy claims are therefore checked exhaustively:
all 2^23 fields through `qsr_debug_box_muller` (the same device functions the step kernels inline) against
`orc_box_muller_parts`.  What matters for parity is stated with each bound: a relative error of the radius scales the
noise and averages out over the angle; a BIAS in sine or cosine would shift the fixed point of a coordinate of
curvature lambda by sigma * bias / lambda, so the mean error over the grid is held to 1e-9.
"""
import numpy as np
import pytest
import torch

from oracle import qsr_oracle as O
from paper_2310_14423_b200 import binding as B

pytestmark = pytest.mark.gpu

N_GRID = 1 << 23


def _device_parts(words_u32: np.ndarray):
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    words = torch.from_numpy(words_u32.view(np.int32)).cuda()
    out = [torch.full((words.numel() + 8,), -7.0, device="cuda") for _ in range(3)]
    B.qsr_debug_box_muller(words, *[o[:words.numel()] for o in out], stream=torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    for o in out:
        assert bool((o[words.numel():] == -7.0).all())           # nothing written past n
    return [o[:words.numel()].cpu().numpy() for o in out]


@pytest.fixture(scope="module")
def grid():
    fields = np.arange(N_GRID, dtype=np.uint32)
    radius, sine, cosine = _device_parts(fields << np.uint32(9))
    o_radius, o_sine, o_cosine = O.box_muller_parts(fields, fields)
    return fields, (radius, sine, cosine), (o_radius, o_sine, o_cosine)


def test_radius_over_all_fields(grid):
    _, (radius, _, _), (o_radius, _, _) = grid
    rel = (radius.astype(np.float64) - o_radius) / o_radius
    # -2 ln u is within 1e-7 (relative) of exact, the root halves that, the root instruction itself adds up to 1e-7
    assert np.abs(rel).max() <= 1.5e-7, np.abs(rel).max()
    assert np.sqrt(np.mean(rel * rel)) <= 5e-8
    assert abs(rel.mean()) <= 2e-8                                # a common scale error of the noise, not a shift
    print("radius: max rel err %.3e, rms %.2e, mean %.2e" % (np.abs(rel).max(), np.sqrt(np.mean(rel * rel)), rel.mean()))
    assert np.all(np.diff(radius.astype(np.float64)) <= 0)        # monotone like the exact function
    assert radius[0] < 5.77 and radius[-1] > 3.4e-4               # sqrt(2*24*ln 2) = 5.768..., sqrt(2^-23) = 3.45e-4


def test_sine_and_cosine_over_all_fields(grid):
    _, (_, sine, cosine), (_, o_sine, o_cosine) = grid
    for name, got, ref in (("sine", sine, o_sine), ("cosine", cosine, o_cosine)):
        err = got.astype(np.float64) - ref
        assert np.abs(err).max() <= 9e-8, (name, np.abs(err).max())
        assert abs(err.mean()) <= 1e-9, (name, err.mean())        # no bias: see the module docstring
        assert abs(got.astype(np.float64).mean()) <= 1e-9, name   # the grid is symmetric: the exact mean is zero
        # per quadrant the mean need not vanish (an odd polynomial's error has a sign on each half of its range, and
        # the halves land in different quadrants); it is held to rounding size so that the zero mean over the circle
        # is not the difference of two large numbers
        quadrant_means = [err[q * (N_GRID // 4):(q + 1) * (N_GRID // 4)].mean() for q in range(4)]
        print(name, "max |err| %.2e, mean %.2e, per quadrant" % (np.abs(err).max(), err.mean()),
              ["%.1e" % m for m in quadrant_means])
        assert max(abs(m) for m in quadrant_means) <= 1e-8, (name, quadrant_means)
    norm = sine.astype(np.float64) ** 2 + cosine.astype(np.float64) ** 2
    assert np.abs(norm - 1).max() <= 2.5e-7


def test_bits_below_the_field_are_ignored(grid):
    """A word's low 9 bits do not belong to the field: any value there gives the same three results."""
    fields, (radius, sine, cosine), _ = grid
    rng = np.random.default_rng(9)
    sel = np.concatenate([np.arange(4096), rng.integers(0, N_GRID, 1 << 18), np.arange(N_GRID - 4096, N_GRID)])
    low = rng.integers(0, 512, sel.size).astype(np.uint32)
    low[:3] = (0x1FF, 0x100, 1)
    r2, s2, c2 = _device_parts((fields[sel] << np.uint32(9)) | low)
    assert np.array_equal(r2, radius[sel]) and np.array_equal(s2, sine[sel]) and np.array_equal(c2, cosine[sel])


def test_noise_is_the_product_of_the_parts():
    """The step kernel's normal for a coordinate equals radius * cosine (even lane) or radius * sine (odd lane) of the
    hook's outputs for the generator words of that coordinate, bit for bit: the hook runs the kernel's own code."""
    import gpu_harness as G
    from paper_2310_14423_b200 import workloads as W
    P, K, t = 4096, 2, 31
    w = W.tiny_workload(W.OPT_SGDM, K=K, P=P, T=100, sched=W.SCHED_CONST, eta_max=1.0, momentum=0.0,
                        weight_decay=0.0, noise_std=1.0)
    S = G.Slabs(w)
    zero = torch.zeros(P, device="cuda")
    ctx = G.make_context(w, S, zero, zero)
    ctx.qsr_local_step(t)
    torch.cuda.synchronize()
    z_gpu = -S.theta[:, :P].cpu().numpy()
    ctx.close()
    seed = w.noise_seed
    for k in range(K):
        words = np.array([O.philox4x32_10([j, 0, t, k], [seed & 0xFFFFFFFF, seed >> 32]) for j in range(P // 4)],
                         np.uint32).reshape(-1)                   # [P/4 blocks x 4 words], published generator
        radius, sine, cosine = _device_parts(words)
        z = np.empty(P, np.float32)
        z[0::4] = radius[0::4] * cosine[1::4]
        z[1::4] = radius[0::4] * sine[1::4]
        z[2::4] = radius[2::4] * cosine[3::4]
        z[3::4] = radius[2::4] * sine[3::4]
        assert np.array_equal(z, z_gpu[k])


def test_argument_errors():
    buf = torch.zeros(16, device="cuda")
    words = torch.zeros(16, dtype=torch.int32, device="cuda")
    L = B.lib()
    st = torch.cuda.current_stream().cuda_stream
    assert L.qsr_debug_box_muller(words.data_ptr(), -1, buf.data_ptr(), buf.data_ptr(), buf.data_ptr(), st) == B.QSR_EINVAL
    assert L.qsr_debug_box_muller(None, 4, buf.data_ptr(), buf.data_ptr(), buf.data_ptr(), st) == B.QSR_EINVAL
    assert L.qsr_debug_box_muller(words.data_ptr(), 4, buf.data_ptr() + 2, buf.data_ptr(), buf.data_ptr(), st) == B.QSR_EALIGN
    assert L.qsr_debug_box_muller(None, 0, None, None, None, st) == B.QSR_OK
    torch.cuda.synchronize()
    assert not buf.any()


def test_fast_square_root_and_reciprocal():
    """The optimizer update's two special-function instructions against binary64: every fp32 mantissa (2^23 values) in
    two binades each for the root (its error pattern repeats every two binades) and one for the reciprocal, plus the
    ranges the path feeds them -- second moments down to 1e-30, denominators from eps = 1e-8 up."""
    mant = np.arange(N_GRID, dtype=np.uint32)
    parts = [(mant | np.uint32(0x3f800000)).view(np.float32),          # [1, 2)
             (mant | np.uint32(0x40000000)).view(np.float32)]          # [2, 4)
    rng = np.random.default_rng(4)
    parts.append(np.exp(rng.uniform(np.log(1e-30), np.log(1e4), 1 << 22)).astype(np.float32))
    x = np.concatenate(parts)
    xd = torch.from_numpy(x).cuda()
    root, rcp = torch.empty_like(xd), torch.empty_like(xd)
    B.qsr_debug_fast_math(xd, root, rcp, stream=torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    x64 = x.astype(np.float64)
    rel_root = root.cpu().numpy().astype(np.float64) / np.sqrt(x64) - 1
    rel_rcp = rcp.cpu().numpy().astype(np.float64) * x64 - 1
    print("sqrt.approx.ftz: max rel err %.3e, mean %.2e; rcp.approx.ftz: max %.3e, mean %.2e"
          % (np.abs(rel_root).max(), rel_root.mean(), np.abs(rel_rcp).max(), rel_rcp.mean()))
    assert np.abs(rel_root).max() <= 1.2e-7 and abs(rel_root.mean()) <= 2e-8
    assert np.abs(rel_rcp).max() <= 1.6e-7 and abs(rel_rcp.mean()) <= 1e-8
