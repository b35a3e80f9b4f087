"""Pins of the oracle's Sobol-8 / conditional-generation streams (Sec. 4.2, Appendix A.1).

The cycle-by-cycle multiplier is checked against: the structure of the Sobol sequences (permutations, stratified
prefixes, the joint net of dimensions 1 and 2), a closed form of the XNOR count written here from cumulative counts,
exactness at full length for boundaries on coarse grids (an 8-bit operand is recovered exactly at L = 256, Sec. 3.2),
zero cross-correlation there (Appendix A.1), and an error that falls like 1/L rather than 1/sqrt(L) (Sec. 3.2's table).
The match with the authors' own kernel cannot be checked: parity unpinned."""
import numpy as np

PER_ROW, PER_TENSOR, NONE = 1, 2, 0


def test_sobol_sequences_are_stratified_permutations(oracle):
    for dim in (1, 2):
        seq = [oracle.sobol8(dim, n) for n in range(256)]
        assert sorted(seq) == list(range(256))
        for k in range(1, 9):                       # every aligned block of 2^k points hits each of 2^k equal bins once
            size = 1 << k
            for start in range(0, 256, size):
                bins = sorted(v >> (8 - k) for v in seq[start:start + size])
                assert bins == list(range(size)), (dim, k, start)
    # dimension 1 is the base-2 radical inverse
    assert [oracle.sobol8(1, n) for n in range(256)] == [int(format(n, "08b")[::-1], 2) for n in range(256)]
    # dimensions (1, 2) form a (0, 8, 2)-net: every 2^a x 2^(8-a) box of the 256 x 256 square holds exactly one point
    pts = [(oracle.sobol8(1, n), oracle.sobol8(2, n)) for n in range(256)]
    for a in range(9):
        cells = {(x >> (8 - a), y >> a) for x, y in pts}
        assert len(cells) == 256, a


def _closed_form(oracle, Ta, Tw, L, scr):
    """XNOR count from cumulative counts: n1 ones of the activation stream consume the first n1 draws of one weight
    generator, the n0 zeros the first n0 draws of the other."""
    sA = [oracle.sobol8(1, n) ^ int(scr[0]) for n in range(256)]
    s1 = [oracle.sobol8(2, n) ^ int(scr[1]) for n in range(256)]
    s0 = [oracle.sobol8(2, n) ^ int(scr[2]) for n in range(256)]
    n1 = sum(1 for l in range(L) if sA[l] < Ta)
    n0 = L - n1
    return sum(1 for k in range(n1) if s1[k] < Tw) + sum(1 for k in range(n0) if s0[k] >= Tw)


def test_multiplier_equals_closed_form(oracle):
    rng = np.random.default_rng(0)
    for seed in (0, 1, 99):
        scr = oracle.cbsg_scramble(seed, 3)
        for _ in range(150):
            Ta, Tw, L = int(rng.integers(0, 257)), int(rng.integers(0, 257)), int(rng.integers(0, 257))
            p, counts = oracle.cbsg_pair(Ta, Tw, L, scr)
            assert p == _closed_form(oracle, Ta, Tw, L, scr)
            assert counts.sum() == L and p == counts[0] + counts[3]
    # different seeds / stream ids scramble differently
    assert len({tuple(oracle.cbsg_scramble(s, i)) for s in range(4) for i in range(4)}) > 8


def test_special_boundaries(oracle):
    scr = oracle.cbsg_scramble(7)
    for L in (1, 17, 100, 256):
        for T in (0, 1, 100, 255, 256):
            ones = oracle.cbsg_pair(T, 256, L, scr)[0]          # weight +1: output = activation stream
            assert ones == oracle.cbsg_pair(T, 0, L, scr)[1][1] + oracle.cbsg_pair(T, 0, L, scr)[1][0]
            assert oracle.cbsg_pair(T, 0, L, scr)[0] == L - ones   # weight -1: output = inverted activation stream
        assert oracle.cbsg_pair(256, 256, L, scr)[0] == L and oracle.cbsg_pair(0, 0, L, scr)[0] == L
        assert oracle.cbsg_pair(256, 0, L, scr)[0] == 0
    # full length: an 8-bit boundary is recovered exactly (count of ones = T)
    for T in range(0, 257, 7):
        assert oracle.cbsg_pair(T, 256, 256, scr)[0] == T
        assert oracle.cbsg_pair(256, T, 256, scr)[0] == T


def test_exact_products_and_zero_correlation_on_coarse_grids(oracle):
    """Boundaries that are multiples of 16 (activation) and 16 (weight): at L = 256 the XNOR count is exactly
    L (1 + a w) / 2 and ad - bc = 0, so the stochastic cross-correlation vanishes."""
    for seed in (0, 5):
        scr = oracle.cbsg_scramble(seed)
        for Ta in range(0, 257, 16):
            for Tw in range(0, 257, 16):
                p, (a, b, c, d) = oracle.cbsg_pair(Ta, Tw, 256, scr)
                va, vw = Ta / 128.0 - 1.0, Tw / 128.0 - 1.0
                assert p == round(128 * (1 + va * vw)), (Ta, Tw)
                assert int(a) * int(d) == int(b) * int(c)
                assert oracle.scc(int(a), int(b), int(c), int(d)) == 0.0
    # the correlation measure itself: identical streams +1, complementary streams -1
    assert oracle.scc(100, 0, 0, 156) == 1.0 and oracle.scc(0, 100, 156, 0) == -1.0


def test_scc_piecewise_definition_hand_worked(oracle):
    """Appendix A.1's two-case normalisation, worked by hand (a, b, c, d = cycles with the bit pair 11, 10, 01, 00).
    Negative branch with a > d, where the max(a - d, 0) term matters:
      (50, 30, 20, 0): ad - bc = -600, D = 80 * 70 - 100 * 50 = 600            -> -1 (as anti-correlated as the marginals allow)
      (40, 30, 20, 10): ad - bc = -200, D = 70 * 60 - 100 * 30 = 1200          -> -1/6 (without the max term: -200/4200)
    Negative branch with a <= d (the term vanishes): (5, 30, 20, 45): (225 - 600) / (35 * 25) = -3/7.
    Positive branch: (40, 10, 20, 30): ad - bc = 1000, D = 100 * min(50, 60) - 50 * 60 = 2000 -> 1/2;
    with the roles of the marginals swapped, (40, 20, 10, 30): D = 100 * 50 - 60 * 50 = 2000 -> 1/2.
    Independent pair counts (ad = bc) give 0 in either branch."""
    assert oracle.scc(50, 30, 20, 0) == -1.0
    assert abs(oracle.scc(40, 30, 20, 10) - (-1.0 / 6.0)) < 1e-15
    assert abs(oracle.scc(5, 30, 20, 45) - (-3.0 / 7.0)) < 1e-15
    assert oracle.scc(40, 10, 20, 30) == 0.5 and oracle.scc(40, 20, 10, 30) == 0.5
    assert oracle.scc(20, 20, 30, 30) == 0.0 and oracle.scc(0, 0, 0, 0) == 0.0
    # bounded by 1 in magnitude over every table with L = 12
    for a in range(13):
        for b in range(13 - a):
            for c in range(13 - a - b):
                assert -1.0 - 1e-12 <= oracle.scc(a, b, c, 12 - a - b - c) <= 1.0 + 1e-12


def test_error_falls_like_one_over_L(oracle):
    """Root-mean-square error of the decoded pair product over random boundaries: error x L stays within a band
    (decay like 1/L, the law of Sec. 3.2's table, whose alpha x L is 2.32), far below the sqrt((1 - (a w)^2) / L) of
    independent streams at the same length."""
    rng = np.random.default_rng(3)
    pairs = [(int(rng.integers(0, 257)), int(rng.integers(0, 257))) for _ in range(400)]
    for seed in (11, 12):
        scr = oracle.cbsg_scramble(seed)
        for L in (32, 64, 128, 192, 256):
            sq, iid = [], []
            for Ta, Tw in pairs:
                p, _ = oracle.cbsg_pair(Ta, Tw, L, scr)
                t = (Ta / 128.0 - 1) * (Tw / 128.0 - 1)
                sq.append(((2 * p - L) / L - t) ** 2)
                iid.append((1 - t * t) / L)
            rms = float(np.sqrt(np.mean(sq)))
            assert 1.0 < rms * L < 3.0, (seed, L, rms * L)
            assert rms < 0.4 * float(np.sqrt(np.mean(iid))), (seed, L)


def test_matmul_composition(oracle):
    rng = np.random.default_rng(4)
    A = rng.standard_normal((5, 12)).astype(np.float32)
    W = (0.02 * rng.standard_normal((12, 7))).astype(np.float32)
    L = np.array([0, 1, 64, 200, 256], dtype=np.int32)
    out = oracle.matmul_cbsg(A, W, L, PER_ROW, PER_TENSOR, seed=2, stream_id=1)
    scr = oracle.cbsg_scramble(2, 1)
    for i in range(5):
        for j in range(7):
            want = 0
            for d in range(12):
                Ta = oracle.boundary_bipolar(oracle.normalise(float(A[i, d]), float(out["sigma_a"][i])))
                Tw = oracle.boundary_bipolar(oracle.normalise(float(W[d, j]), float(out["sigma_w"][j])))
                want += oracle.cbsg_pair(Ta, Tw, int(L[i]), scr)[0]
            assert out["P"][i, j] == want
    assert (out["C"][0] == 0).all()
    # at full length the decoded product is the product of the quantised operands up to the generator's discrepancy
    Aq = np.round((np.clip(A[4] / out["sigma_a"][4], -1, 1) + 1) * 128) / 128 - 1
    Wq = np.round((np.clip(W / out["sigma_w"][0], -1, 1) + 1) * 128) / 128 - 1
    exact = out["sigma_a"][4] * out["sigma_w"][0] * (Aq @ Wq)
    assert np.abs(out["C"][4] - exact).max() < 0.05 * out["sigma_a"][4] * out["sigma_w"][0] * np.sqrt(12)
    sub = oracle.matmul_cbsg(A, W, L, PER_ROW, PER_TENSOR, seed=2, stream_id=1, row_sel=[3, 4], col_sel=[0, 6])
    assert np.array_equal(sub["P"], out["P"][np.ix_([3, 4], [0, 6])])
