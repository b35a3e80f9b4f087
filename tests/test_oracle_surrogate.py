"""Pins of the oracle's Gaussian surrogate (Sec. 3.2): the noise scale against the paper's printed table,
the normal variates against the moments and the distribution function of N(0, 1), and the algebra of the output."""
import math
import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def test_alpha_of_L_matches_the_printed_table(oracle):
    table = np.loadtxt(os.path.join(GOLDEN, "surrogate_alpha_table.txt"))
    for L, alpha in table:
        # the paper prints three significant digits: the rule must land within half a unit of the last digit
        assert abs(oracle.SURROGATE_COEFF / L - alpha) <= 0.5e-4 + 1e-12, (L, alpha)
    # and the product alpha * L is constant to the printed precision
    prod = table[:, 0] * table[:, 1]
    assert prod.max() - prod.min() < 0.01 and abs(prod.mean() - oracle.SURROGATE_COEFF) < 0.01


def test_standard_normal_moments_and_distribution(oracle):
    n = 200000
    z = np.array([oracle.standard_normal(12345, 0, k) for k in range(n)])
    assert abs(z.mean()) < 4 / math.sqrt(n)
    assert abs(z.var() - 1.0) < 4 * math.sqrt(2.0 / n)
    assert abs((z ** 3).mean()) < 4 * math.sqrt(15.0 / n)
    assert abs((z ** 4).mean() - 3.0) < 4 * math.sqrt(96.0 / n)
    # Kolmogorov distance to the normal distribution function
    zs = np.sort(z)
    cdf = 0.5 * (1.0 + np.vectorize(math.erf)(zs / math.sqrt(2.0)))
    d = np.max(np.abs(cdf - (np.arange(1, n + 1) - 0.5) / n))
    assert d < 1.63 / math.sqrt(n) + 0.5 / n          # 1 % critical value
    # neighbouring cells and other streams / seeds are uncorrelated and different
    z2 = np.array([oracle.standard_normal(12345, 1, k) for k in range(20000)])
    z3 = np.array([oracle.standard_normal(12346, 0, k) for k in range(20000)])
    for other in (z2, z3, np.roll(z[:20000], 1)):
        assert abs(np.corrcoef(z[:20000], other)[0, 1]) < 0.03


def test_surrogate_output_algebra(oracle):
    rng = np.random.default_rng(9)
    Y = rng.standard_normal((6, 50)).astype(np.float32)
    L = np.array([0, 8, 32, 128, 256, 1024], dtype=np.int32)
    out = oracle.surrogate_noise(Y, L, oracle.SURROGATE_COEFF, seed=77, stream_id=3)
    assert (out[0] == 0).all()                                   # no stream, no output
    for i in range(1, 6):
        for j in (0, 17, 49):
            z = oracle.standard_normal(77, 3, i * 50 + j)
            want = float(Y[i, j]) * (1.0 + oracle.SURROGATE_COEFF / L[i] * z)
            assert abs(out[i, j] - want) <= 1e-6 * abs(want) + 1e-12
    # zero noise scale returns the input; doubling the scale doubles the deviation
    assert np.array_equal(oracle.surrogate_noise(Y, L[1:2].repeat(6), 0.0, 77), Y)
    d1 = oracle.surrogate_noise(Y, np.full(6, 64, np.int32), 1.0, 5).astype(np.float64) - Y
    d2 = oracle.surrogate_noise(Y, np.full(6, 64, np.int32), 2.0, 5).astype(np.float64) - Y
    assert np.allclose(d2, 2 * d1, rtol=1e-4, atol=1e-7)
    # relative deviation has standard deviation alpha(L)
    Yb = np.ones((1, 100000), dtype=np.float32)
    dev = oracle.surrogate_noise(Yb, np.array([64], np.int32), oracle.SURROGATE_COEFF, 3)[0] - 1.0
    assert abs(dev.std() - oracle.SURROGATE_COEFF / 64) < 0.02 * oracle.SURROGATE_COEFF / 64
