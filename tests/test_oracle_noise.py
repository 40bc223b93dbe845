"""Pins for the oracle's counter-based Gaussian noise: Philox-4x32-10 against its published known-answer
vectors, the uniforms' grid, and the moments / independence of the Box-Muller normals.  CPU only."""
import math
import os

import numpy as np
from scipy import stats

from oracle import qsr_oracle as O

SEED = 0x231014423000


def test_philox_known_answers(golden_dir):
    n = 0
    with open(os.path.join(golden_dir, "philox4x32_10_kat.txt")) as f:
        for line in f:
            if not line.strip() or line.startswith("#"):
                continue
            words = [int(x, 16) for x in line.split()]
            out = O.philox4x32_10(words[0:4], words[4:6])
            assert out.tolist() == words[6:10]
            n += 1
    assert n == 3


def test_counter_layout_and_branches():
    """Coordinates 4j..4j+3 share one block with counter (low j, high j, step, worker) and key = seed words;
    words (0,1) give the cosine/sine pair of 4j, 4j+1 and words (2,3) that of 4j+2, 4j+3."""
    for (k, u, i) in [(0, 0, 0), (3, 17, 5), (15, 9999, 86415591), (2, 123, (1 << 34) + 6)]:
        j = i >> 2
        r = O.philox4x32_10([j & 0xFFFFFFFF, j >> 32, u, k], [SEED & 0xFFFFFFFF, SEED >> 32])
        lane = i & 3
        a, b = int(r[2 * (lane >> 1)]) >> 9, int(r[2 * (lane >> 1) + 1]) >> 9
        u1, u2 = (a + 0.5) / 2 ** 23, (b + 0.5) / 2 ** 23
        rad = math.sqrt(-2 * math.log(u1))
        z = rad * (math.sin(2 * math.pi * u2) if lane & 1 else math.cos(2 * math.pi * u2))
        assert abs(O.noise(SEED, k, u, i) - z) <= 1e-14 * max(1.0, abs(z))


def test_pair_lies_on_one_circle():
    """The two normals of a pair are radius*(cos, sin) of one angle: z0^2 + z1^2 = -2 ln(u1) <= 2*24*ln 2."""
    z = O.noise_fill(SEED, 1, 2, 0, 4000)
    r2 = z[0::2] ** 2 + z[1::2] ** 2
    assert r2.max() <= 2 * 24 * math.log(2) and r2.min() > 0
    # -2 ln(u1) with u1 uniform is exponential with mean 2
    assert abs(r2.mean() - 2.0) < 4 * 2.0 / math.sqrt(r2.size)


N_DRAWS = 1 << 24          # 1.7e7 normals per statistical test


def test_moments_and_uniformity():
    n = N_DRAWS
    z = O.noise_fill(SEED, 0, 0, 0, n)
    se = 1 / math.sqrt(n)
    assert abs(z.mean()) < 4 * se
    assert abs(z.var() - 1) < 4 * math.sqrt(2) * se          # far inside the 1 % band
    assert abs((z ** 3).mean()) < 4 * math.sqrt(15) * se
    assert abs((z ** 4).mean() - 3) < 4 * math.sqrt(96) * se
    assert np.abs(z).max() < math.sqrt(2 * 24 * math.log(2)) + 1e-9
    for lane in range(4):
        p = stats.kstest(z[lane::4], "norm").pvalue
        assert p > 1e-4, (lane, p)
    # the two uniforms behind every pair, recovered from the normals: u1 = exp(-(z0^2 + z1^2)/2), u2 = angle / 2 pi
    z0, z1 = z[0::2], z[1::2]
    u1 = np.exp(-0.5 * (z0 * z0 + z1 * z1))
    u2 = np.mod(np.arctan2(z1, z0) / (2 * math.pi), 1.0)
    for name, u in (("u1", u1), ("u2", u2)):
        p = stats.kstest(u, "uniform").pvalue
        assert p > 1e-4, (name, p)
        # they sit on the grid (a + 1/2) / 2^23
        a = u[:100000] * 2 ** 23 - 0.5
        assert np.abs(a - np.round(a)).max() < 1e-3, name
    assert abs(np.corrcoef(u1, u2)[0, 1]) < 4.5 / math.sqrt(u1.size)


def test_independence_across_workers_steps_and_neighbours():
    n = N_DRAWS
    bound = 4 / math.sqrt(n)
    base = O.noise_fill(SEED, 0, 0, 0, n)
    others = {
        "worker": O.noise_fill(SEED, 1, 0, 0, n),
        "step": O.noise_fill(SEED, 0, 1, 0, n),
        "seed": O.noise_fill(SEED + 1, 0, 0, 0, n),
        "shifted by one block": O.noise_fill(SEED, 0, 0, 4, n),
    }
    for name, o in others.items():
        assert abs(np.corrcoef(base, o)[0, 1]) < bound, name
    for lag in (1, 2, 3):
        assert abs(np.corrcoef(base[:-lag], base[lag:])[0, 1]) < bound, lag
    # within a pair the two branches are uncorrelated, also in their squares
    assert abs(np.corrcoef(base[0::2] ** 2, base[1::2] ** 2)[0, 1]) < 2 * bound


def test_box_muller_parts_against_40_digit_arithmetic():
    """radius = sqrt(-2 ln u1), sin / cos(2 pi u2) on the 23-bit grid: the ends of the grid, the quadrant borders and
    seeded random fields, against mpmath at 40 digits."""
    import mpmath
    mpmath.mp.dps = 40
    rng = np.random.default_rng(7)
    n_grid = 1 << 23
    edge = [0, 1, 2, n_grid - 1, n_grid - 2, n_grid // 2, n_grid // 2 - 1, n_grid // 4, n_grid // 4 - 1,
            3 * n_grid // 4, 3 * n_grid // 4 - 1, n_grid // 8, 12345]
    a = np.array(edge + rng.integers(0, n_grid, 1500).tolist(), np.uint32)
    b = np.array(edge[::-1] + rng.integers(0, n_grid, 1500).tolist(), np.uint32)
    radius, sine, cosine = O.box_muller_parts(a, b)
    for i in range(a.size):
        u1 = (mpmath.mpf(int(a[i])) + mpmath.mpf(1) / 2) / n_grid
        u2 = (mpmath.mpf(int(b[i])) + mpmath.mpf(1) / 2) / n_grid
        r = mpmath.sqrt(-2 * mpmath.log(u1))
        assert abs(mpmath.mpf(float(radius[i])) - r) <= 4e-16 * r
        # the product 2 pi u2 is rounded to binary64 before the sine: an argument error of up to 4e-16 near 2 pi
        assert abs(mpmath.mpf(float(sine[i])) - mpmath.sin(2 * mpmath.pi * u2)) <= 1e-15
        assert abs(mpmath.mpf(float(cosine[i])) - mpmath.cos(2 * mpmath.pi * u2)) <= 1e-15


def test_box_muller_parts_over_the_whole_grid():
    """All 2^23 fields: the angle grid is symmetric, so sine and cosine average to zero; sin^2 + cos^2 = 1; the mean of
    radius^2 = -2 ln u1 over the midpoint grid is 2 (the integral) up to the midpoint rule's error at the singularity."""
    n_grid = 1 << 23
    f = np.arange(n_grid, dtype=np.uint32)
    radius, sine, cosine = O.box_muller_parts(f, f)
    assert abs(sine.mean()) < 1e-13 and abs(cosine.mean()) < 1e-13
    assert np.abs(sine * sine + cosine * cosine - 1).max() < 1e-15
    assert np.array_equal(np.sign(sine[:n_grid // 2]), np.ones(n_grid // 2))          # first half turn: sine > 0
    assert np.abs(sine + sine[::-1]).max() < 1e-15 and np.abs(cosine - cosine[::-1]).max() < 1e-15
    assert np.all(np.diff(radius) < 0)                                                # radius falls as u1 grows
    # midpoint rule for the integral of -2 ln u over (0,1): error ~ ln(2)/N from the first cell
    assert abs((radius * radius).mean() - 2.0) < 2.0 / n_grid
    assert radius[0] == math.sqrt(2 * 24 * math.log(2))


def test_noise_is_radius_times_branch():
    """orc_noise for coordinate i equals the parts' radius times cosine (even lane) or sine (odd lane), bit for bit."""
    for (k, u, i0) in [(0, 0, 0), (7, 4242, 4 * 10 ** 6)]:
        z = O.noise_fill(SEED, k, u, i0, 64)
        for c in range(64):
            i = i0 + c
            j = i >> 2
            r = O.philox4x32_10([j & 0xFFFFFFFF, j >> 32, u, k], [SEED & 0xFFFFFFFF, SEED >> 32])
            lane = i & 3
            a, b = int(r[2 * (lane >> 1)]) >> 9, int(r[2 * (lane >> 1) + 1]) >> 9
            radius, sine, cosine = O.box_muller_parts([a], [b])
            assert z[c] == radius[0] * (sine[0] if lane & 1 else cosine[0])


def test_noise_is_a_pure_function_of_its_four_integers():
    a = O.noise_fill(SEED, 5, 77, 1000, 64)
    b = np.array([O.noise(SEED, 5, 77, 1000 + c) for c in range(64)])
    assert np.array_equal(a, b)
    assert O.noise(SEED, 5, 77, 1000) != O.noise(SEED, 5, 78, 1000)
    assert O.noise(SEED, 5, 77, 1000) != O.noise(SEED, 6, 77, 1000)
