"""Pins for the oracle's generator, boundary map and SNG (Sec. 3.1 Encoding / Bitstream generation).

None of these tests re-types the oracle's formulas: they compare it with an independent
library generator, with closed forms, and with statistics the definitions fix.
"""
import ctypes
import ctypes.util
import glob
import math

import numpy as np
import pytest


def _curand_host():
    names = sorted(glob.glob("/usr/local/cuda/lib64/libcurand.so*")) + [ctypes.util.find_library("curand") or ""]
    for n in names:
        if n:
            try:
                return ctypes.CDLL(n)
            except OSError:
                continue
    return None


def _curand_host_philox(lib, seed, n_groups):
    """First 4*n_groups outputs of cuRAND's HOST Philox4_32_10 generator (runs on the CPU)."""
    lib.curandSetPseudoRandomGeneratorSeed.argtypes = [ctypes.c_void_p, ctypes.c_ulonglong]
    lib.curandGenerate.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t]
    gen = ctypes.c_void_p()
    assert lib.curandCreateGeneratorHost(ctypes.byref(gen), 161) == 0      # CURAND_RNG_PSEUDO_PHILOX4_32_10
    assert lib.curandSetPseudoRandomGeneratorSeed(gen, seed) == 0
    out = np.zeros(4 * n_groups, dtype=np.uint32)
    assert lib.curandGenerate(gen, out.ctypes.data, out.size) == 0
    lib.curandDestroyGenerator(gen)
    return out.reshape(n_groups, 4)


def test_philox_matches_library_generator(oracle):
    """Independent implementation: cuRAND's host generator emits, as its g-th group of four words,
    Philox4x32-10 of counter (0, 0, g, 0) under key = (seed_lo, seed_hi)."""
    lib = _curand_host()
    if lib is None:
        pytest.skip("libcurand not present")
    for seed in (0, 1, 0x0123456789ABCDEF, 0xFFFFFFFFFFFFFFFF, 4):
        ref = _curand_host_philox(lib, seed, 257)
        key = [seed & 0xFFFFFFFF, seed >> 32]
        for g in (0, 1, 2, 3, 31, 32, 255, 256):
            got = oracle.philox4x32_10([0, 0, g, 0], key)
            assert [int(x) for x in got] == [int(x) for x in ref[g]], (seed, g)


def test_philox_counter_words_all_matter(oracle):
    """Each counter word and each key word changes the output (no word is dropped), and about
    half of the 128 output bits flip (avalanche) for a one-bit input change."""
    base_c, base_k = [5, 6, 7, 8], [9, 10]
    base = oracle.philox4x32_10(base_c, base_k)
    for word in range(6):
        for bit in (0, 13, 31):
            c, k = list(base_c), list(base_k)
            if word < 4:
                c[word] ^= 1 << bit
            else:
                k[word - 4] ^= 1 << bit
            out = oracle.philox4x32_10(c, k)
            flipped = sum(bin(int(a) ^ int(b)).count("1") for a, b in zip(out, base))
            assert 32 <= flipped <= 96, (word, bit, flipped)


def test_boundary_closed_forms(oracle):
    assert oracle.boundary_bipolar(-1.0) == 0
    assert oracle.boundary_bipolar(0.0) == 128
    assert oracle.boundary_bipolar(1.0) == 256
    assert oracle.boundary_unipolar(0.0) == (0, 0)
    assert oracle.boundary_unipolar(1.0) == (256, 0)
    assert oracle.boundary_unipolar(-1.0) == (256, 1)
    assert oracle.boundary_unipolar(-0.25) == (64, 1)
    # on-grid values map to themselves, ties go to even
    for T in range(257):
        assert oracle.boundary_bipolar(T / 128.0 - 1.0) == T
        assert oracle.boundary_unipolar(T / 256.0)[0] == T
    assert oracle.boundary_bipolar((0.5) / 128.0 - 1.0) == 0        # 0.5 -> 0 (even)
    assert oracle.boundary_bipolar((1.5) / 128.0 - 1.0) == 2        # 1.5 -> 2 (even)
    assert oracle.boundary_unipolar(2.5 / 256.0)[0] == 2


def test_boundary_monotone_and_within_half_step(oracle):
    vs = np.linspace(-1.0, 1.0, 4001, dtype=np.float32)
    Ts = [oracle.boundary_bipolar(float(v)) for v in vs]
    assert all(b >= a for a, b in zip(Ts, Ts[1:]))
    # Pr[z=1] = T/256 approximates (v+1)/2 to half a grid step: |T/128 - 1 - v| <= 1/256
    assert max(abs(T / 128.0 - 1.0 - float(v)) for T, v in zip(Ts, vs)) <= 1.0 / 256 + 1e-7
    Tu = [oracle.boundary_unipolar(float(v))[0] for v in vs]
    assert max(abs(T / 256.0 - abs(float(v))) for T, v in zip(Tu, vs)) <= 1.0 / 512 + 1e-7


def test_normalise_is_ieee_division_clamped(oracle):
    rng = np.random.default_rng(0)
    x = rng.standard_normal(2000).astype(np.float32)
    s = np.abs(rng.standard_normal(2000)).astype(np.float32) + np.float32(0.1)
    for xi, si in zip(x, s):
        expect = np.clip(np.float32(xi) / np.float32(si), np.float32(-1), np.float32(1))
        assert oracle.normalise(float(xi), float(si)) == float(expect)


def test_draws_are_uniform_bytes(oracle):
    """r_l is uniform on 0..255: chi-square over 2^16 draws taken across elements and positions."""
    counts = np.zeros(256, dtype=np.int64)
    n = 0
    for elem in range(64):
        for l in range(1024):
            counts[oracle.random_byte(7, 0, 0, elem * 977 + 3, l)] += 1
            n += 1
    expected = n / 256.0
    chi2 = float(((counts - expected) ** 2 / expected).sum())
    # 255 degrees of freedom: mean 255, sd ~22.6; 6 sd window
    assert 255 - 6 * 22.6 < chi2 < 255 + 6 * 22.6, chi2


def test_comparator_is_strictly_below(oracle):
    """z_l = [r_l < T] for every boundary, including the exact 0 and exact 1 at T = 0 and T = 256."""
    for T in range(257):
        for l in (0, 1, 31, 32, 33, 500):
            r = oracle.random_byte(3, 2, 1, 12345, l)
            assert oracle.stream_bit(3, 2, 1, 12345, l, T) == (1 if r < T else 0)
    assert all(oracle.stream_bit(9, 0, 0, e, l, 0) == 0 for e in range(5) for l in range(100))
    assert all(oracle.stream_bit(9, 0, 0, e, l, 256) == 1 for e in range(5) for l in range(100))


def test_stream_popcount_statistics(oracle):
    """The count of ones over L positions is Binomial(L, T/256): mean and variance over streams."""
    L, T = 256, 96
    counts = []
    for elem in range(600):
        counts.append(sum(oracle.stream_bit(11, 0, 0, elem, l, T) for l in range(L)))
    counts = np.array(counts, dtype=np.float64)
    p = T / 256.0
    se_mean = math.sqrt(L * p * (1 - p) / counts.size)
    assert abs(counts.mean() - L * p) < 5 * se_mean
    assert 0.8 * L * p * (1 - p) < counts.var() < 1.2 * L * p * (1 - p)


def test_streams_of_distinct_elements_tensors_ids_seeds_differ(oracle):
    L = 128

    def stream(seed, sid, tid, elem):
        return tuple(oracle.random_byte(seed, sid, tid, elem, l) for l in range(L))

    base = stream(1, 0, 0, 10)
    for other in (stream(2, 0, 0, 10), stream(1, 1, 0, 10), stream(1, 0, 1, 10), stream(1, 0, 0, 11),
                  stream(1, 0, 0, 10 + (1 << 32))):
        agree = sum(a == b for a, b in zip(base, other))
        assert agree <= 8           # independent bytes agree with probability 1/256
    assert base == stream(1, 0, 0, 10)     # deterministic for a fixed configuration


def test_encode_is_the_per_bit_definition_and_has_the_prefix_property(oracle):
    """Tensor encode == scale, normalise, boundary, comparator applied element by element; a shorter
    stream is the prefix of a longer one (early termination); sub-selections keep element indices."""
    rng = np.random.default_rng(5)
    X = rng.standard_normal((6, 10)).astype(np.float32)
    sig = oracle.scales(X, oracle.SCALE_PER_ROW, "row")
    assert np.array_equal(sig, np.abs(X).max(axis=1))
    bits, T, sign = oracle.encode(X, 0, oracle.BIPOLAR_XNOR, 70, seed=21, stream_id=3, sigma_row=sig)
    for r in range(6):
        for c in range(10):
            v = oracle.normalise(float(X[r, c]), float(sig[r]))
            t = oracle.boundary_bipolar(v)
            assert T[r, c] == t
            for l in (0, 1, 31, 32, 63, 64, 69):
                assert bits[r, c, l] == oracle.stream_bit(21, 3, 0, r * 10 + c, l, t)
    short, _, _ = oracle.encode(X, 0, oracle.BIPOLAR_XNOR, 33, seed=21, stream_id=3, sigma_row=sig)
    assert np.array_equal(short, bits[:, :, :33])
    sub, _, _ = oracle.encode(X, 0, oracle.BIPOLAR_XNOR, 70, seed=21, stream_id=3, sigma_row=sig,
                              row_sel=[4, 1], col_sel=[9, 0, 3])
    assert np.array_equal(sub, bits[[4, 1]][:, [9, 0, 3]])
    # the row maximum maps to the top boundary: an all-ones (or all-zeros) stream
    r, c = 2, int(np.argmax(np.abs(X[2])))
    assert bits[r, c].all() or not bits[r, c].any()


def test_scales(oracle):
    X = np.array([[1.0, -3.0, 2.0], [0.0, 0.0, 0.0]], dtype=np.float32)
    assert oracle.scales(X, oracle.SCALE_PER_ROW, "row").tolist() == [3.0, 1.0]      # zero row -> 1
    assert oracle.scales(X, oracle.SCALE_PER_ROW, "col").tolist() == [1.0, 3.0, 2.0]
    assert oracle.scales(X, oracle.SCALE_PER_TENSOR, "col").tolist() == [3.0, 3.0, 3.0]
    assert oracle.scales(X, oracle.SCALE_NONE, "row").tolist() == [1.0, 1.0]
    assert oracle.row_absmax(X).tolist() == [3.0, 0.0]
    bad = X.copy()
    bad[0, 1] = np.nan
    with pytest.raises(oracle.OracleError) as e:
        oracle.scales(bad, oracle.SCALE_PER_ROW, "row")
    assert e.value.code == oracle.ERR_NONFINITE


def test_int8_two_step_boundaries(oracle):
    """Sec. 4.2's fused quantisation: the int8 grid (q_max = 127, Sec. 3.1) first, then one of the 257 boundaries.
    Fixed by the text: the grid has 255 points, -1 / 0 / +1 are grid points, and the bipolar stream probability of a
    grid point is (x_hat + q_max) / (2 q_max) (Sec. 3.1), so the boundary is the one nearest to 256 times that."""
    from fractions import Fraction
    assert oracle.boundary_bipolar_int8(-1.0) == 0
    assert oracle.boundary_bipolar_int8(0.0) == 128
    assert oracle.boundary_bipolar_int8(1.0) == 256
    levels = []
    for q in range(-127, 128):
        T = oracle.boundary_bipolar_int8(q / 127.0)
        target = Fraction(q + 127, 254) * 256                      # exact position of the grid point on the 0..256 scale
        assert abs(T - target) < Fraction(1, 2)                    # nearest boundary; never a tie (127 is odd)
        levels.append(T)
    assert levels == sorted(levels) and len(set(levels)) == 255    # monotone, the 255 grid points stay distinct
    assert set(range(257)) - set(levels) == {64, 192}              # two of the 257 boundaries are never used
    # values between grid points snap to the grid first (round half to even in binary32), e.g. 0.004 -> x_hat = 1
    assert oracle.boundary_bipolar_int8(0.004) == oracle.boundary_bipolar_int8(1 / 127.0) == 129
    assert oracle.boundary_bipolar_int8(0.0039) == 128             # 127 * 0.0039 = 0.4953 -> 0
    xs = np.linspace(-1, 1, 4001)
    Ts = [oracle.boundary_bipolar_int8(float(x)) for x in xs]
    assert Ts == sorted(Ts)
    assert max(abs(T / 128.0 - 1.0 - x) for T, x in zip(Ts, xs)) <= 1 / 254 + 1 / 256 + 1e-6   # half a grid step + half a boundary step
    # unipolar: sign and magnitude, magnitude grid 0..127 -> boundary nearest to 256 |x_hat| / 127
    assert oracle.boundary_unipolar_int8(0.0) == (0, 0)
    assert oracle.boundary_unipolar_int8(1.0) == (256, 0) and oracle.boundary_unipolar_int8(-1.0) == (256, 1)
    mags = []
    for q in range(128):
        T, s = oracle.boundary_unipolar_int8(-q / 127.0)
        assert s == (1 if q else 0) and abs(T - Fraction(q, 127) * 256) < Fraction(1, 2)
        mags.append(T)
    assert mags == sorted(mags) and len(set(mags)) == 128


def test_int8_variant_changes_only_the_boundary(oracle):
    """Streams of the two-step variant are the comparator outputs of its own boundaries on the same draws."""
    rng = np.random.default_rng(2)
    X = rng.uniform(-1, 1, size=(5, 9)).astype(np.float32)
    for mode in (0, 1):
        b0, T0, s0 = oracle.encode(X, 0, mode, 40, seed=9, stream_id=2)
        b1, T1, s1 = oracle.encode(X, 0, mode, 40, seed=9, stream_id=2, quant=oracle.QUANT_INT8_THEN_257)
        assert np.array_equal(s0, s1) and not np.array_equal(T0, T1) and np.abs(T0 - T1).max() <= 2
        for i in range(5):
            for d in range(9):
                want = oracle.boundary_bipolar_int8(float(X[i, d])) if mode == 0 else oracle.boundary_unipolar_int8(float(X[i, d]))[0]
                assert T1[i, d] == want
                for l in range(40):
                    assert b1[i, d, l] == (1 if oracle.random_byte(9, 2, 0, i * 9 + d, l) < want else 0)
