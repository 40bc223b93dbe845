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


def test_moments_and_uniformity():
    n = 1 << 21
    z = O.noise_fill(SEED, 0, 0, 0, n)
    se = 1 / math.sqrt(n)
    assert abs(z.mean()) < 4 * se
    assert abs(z.var() - 1) < 4 * math.sqrt(2) * se
    assert abs((z ** 3).mean()) < 4 * math.sqrt(15) * se
    assert abs((z ** 4).mean() - 3) < 4 * math.sqrt(96) * se
    assert np.abs(z).max() < math.sqrt(2 * 24 * math.log(2)) + 1e-9
    for lane in range(4):
        p = stats.kstest(z[lane::4][:200000], "norm").pvalue
        assert p > 1e-4, (lane, p)


def test_independence_across_workers_steps_and_neighbours():
    n = 1 << 19
    bound = 4.5 / math.sqrt(n)
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


def test_noise_is_a_pure_function_of_its_four_integers():
    a = O.noise_fill(SEED, 5, 77, 1000, 64)
    b = np.array([O.noise(SEED, 5, 77, 1000 + c) for c in range(64)])
    assert np.array_equal(a, b)
    assert O.noise(SEED, 5, 77, 1000) != O.noise(SEED, 5, 78, 1000)
    assert O.noise(SEED, 5, 77, 1000) != O.noise(SEED, 6, 77, 1000)
