"""Pins of the oracle's extensions: gradient clipping, base-s packing, quantization error and the
refinement sweeps over the greedy ORQ levels.

As in test_oracle_pins.py no expected value comes from the function under test: library routines
on the special case they cover (numpy variance and clip, Python's positional-notation parser),
size arithmetic from the paper's compression ratios, brute force on tiny inputs and invariants
that a dropped term, a wrong sign or a shifted index would break.
"""
import math

import numpy as np
import pytest

import oracle
import ogq_workloads as wl


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


# ------------------------------------------------------------------ clipping


def test_clip_threshold_is_c_times_population_std():
    """sigma^2 is the variance about the mean over all n elements; numpy's var computes exactly that
    (ddof = 0) in fp64 on the widened values."""
    for seed, n, shift in [(1, 10007, 0.0), (2, 257, 3e-3), (3, 5, -1e-2)]:
        v = (wl.laplace(rng(seed), n, 1e-3) + np.float32(shift)).astype(np.float32)
        for c in (2.5, 1.7):
            tau, st = oracle.clip_threshold(v, c)
            assert st == 0
            want = c * math.sqrt(np.var(v.astype(np.float64)))
            assert float(tau) == pytest.approx(want, rel=2e-7)
            # a non-zero mean must not leak into sigma (variance about the mean, not about zero)
            about_zero = c * math.sqrt(np.mean(v.astype(np.float64) ** 2))
            if shift != 0.0:
                assert abs(float(tau) - about_zero) > 1e-3 * about_zero
    assert oracle.clip_threshold(np.zeros(0, np.float32), 2.5)[1] & 1
    assert oracle.clip_threshold(np.array([1.0, np.nan], np.float32), 2.5)[1] & 2
    assert float(oracle.clip_threshold(np.full(9, 0.25, np.float32), 2.5)[0]) == 0.0


def test_clip_is_the_symmetric_clamp():
    v = wl.student_t(rng(4), 4001, 3.0, 1e-3)
    tau = np.float32(2.0e-3)
    got = oracle.clip(v, tau)
    assert np.array_equal(got, np.clip(v, -tau, tau))
    # sign(v) min(|v|, tau): untouched inside, exactly +-tau outside, sign kept
    inside = np.abs(v) <= tau
    assert np.array_equal(got[inside], v[inside])
    assert np.all(got[~inside] == np.sign(v[~inside]) * tau)
    assert np.any(~inside) and np.any(inside)


def test_clipping_then_orq_uses_the_clipped_extremes():
    """Corollary 1 on the clipped gradient: the end levels are the clipped minimum and maximum."""
    v = wl.student_t(rng(6), 20000, 3.0, 1e-3)
    tau, _ = oracle.clip_threshold(v, 2.5)
    cv = oracle.clip(v, tau)
    assert v.max() > tau and v.min() < -tau
    lv, st = oracle.levels_orq(cv, 5)
    assert st == 0 and lv[0] == -tau and lv[-1] == tau


# ------------------------------------------------------------------ base-s packing


def test_dense_digits_and_the_papers_compression_ratios():
    """m codes per 32-bit word, the largest m with s^m <= 2^32; the resulting ratio 32 / (32/m) = m
    approaches the paper's 32 / log2(s) (x20.2, x13.8, x10.1) from below."""
    want = {2: 32, 3: 20, 5: 13, 9: 10, 17: 7}
    for s, m in want.items():
        assert oracle.dense_digits(s) == m
        assert s ** m <= 2 ** 32 < s ** (m + 1)
        ideal = 32.0 / math.log2(s)
        assert m <= ideal < m + 1
    assert oracle.dense_digits(3) == math.floor(20.2) and oracle.dense_digits(9) == math.floor(10.1)
    assert oracle.dense_digits(5) == math.floor(13.8)
    for s, m in want.items():
        for n in (0, 1, m - 1, m, m + 1, 4 * m, 4 * m + 1, 1000):
            w = oracle.dense_words(n, s)
            assert w % 4 == 0 and w >= -(-n // m) and w - 4 < -(-n // m) + (1 if n == 0 else 0) + 3


def test_pack_dense_against_positional_notation():
    """Each word is the number whose base-s digits, least significant first, are its m codes:
    Python's int(text, base) parses exactly that (most significant digit first)."""
    digits = "0123456789abcdefg"
    for s in (2, 3, 5, 9, 17):
        m = oracle.dense_digits(s)
        for n in (1, m - 1, m, m + 1, 5 * m + 3, 997):
            codes = rng(100 * s + n).integers(0, s, n).astype(np.uint8)
            words = oracle.pack_dense(codes, s)
            assert words.size == oracle.dense_words(n, s)
            for j in range(words.size):
                chunk = codes[j * m : (j + 1) * m]
                text = "".join(digits[c] for c in chunk[::-1]) or "0"
                assert int(words[j]) == int(text, s)
            assert np.array_equal(oracle.unpack_dense(words, n, s), codes)
    # the largest code in every position still fits a word
    for s in (3, 5, 9, 17):
        m = oracle.dense_digits(s)
        codes = np.full(2 * m, s - 1, np.uint8)
        words = oracle.pack_dense(codes, s)
        assert int(words[0]) == s ** m - 1 and np.array_equal(oracle.unpack_dense(words, 2 * m, s), codes)


def test_dense_with_two_levels_is_the_bit_stream():
    codes = rng(8).integers(0, 2, 1000).astype(np.uint8)
    assert np.array_equal(oracle.pack_dense(codes, 2), oracle.pack(codes, 1))


def test_unpack_sum_dense_matches_numpy_gather():
    r = rng(9)
    for s in (3, 5, 9, 17):
        n, K = 1234, 3
        codes = [r.integers(0, s, n).astype(np.uint8) for _ in range(K)]
        levels = [np.sort(r.standard_normal(s)).astype(np.float32) for _ in range(K)]
        got = oracle.unpack_sum_dense([oracle.pack_dense(c, s) for c in codes], levels, n, s, 1.0 / K)
        want = sum(l.astype(np.float64)[c] for l, c in zip(levels, codes)) / K
        assert np.allclose(got, want, rtol=1e-6, atol=1e-9)


# ------------------------------------------------------------------ quantization error


def numpy_expected_error(v, lv):
    """sum (v - lo)(hi - v) inside the levels, squared distance to the end level outside."""
    v = v.astype(np.float64)
    lv = lv.astype(np.float64)
    k = np.clip(np.searchsorted(lv, v, side="right"), 1, lv.size - 1)
    lo, hi = lv[k - 1], lv[k]
    inside = (v >= lv[0]) & (v <= lv[-1])
    e = np.where(inside, (v - lo) * (hi - v), np.minimum((v - lv[0]) ** 2, (v - lv[-1]) ** 2))
    return math.fsum(e)


def test_quant_error_is_the_squared_distance():
    v = wl.gaussian(rng(10), 5000, 1e-3)
    lv = np.array([-2e-3, -5e-4, 0.0, 6e-4, 2.5e-3], np.float32)
    codes = rng(11).integers(0, 5, v.size).astype(np.uint8)
    want = math.fsum((lv.astype(np.float64)[codes] - v.astype(np.float64)) ** 2)
    assert oracle.quant_error(v, lv, codes) == pytest.approx(want, rel=1e-13)


def test_expected_error_formula_and_monte_carlo():
    v = wl.laplace(rng(12), 3000, 1e-3)
    lv, _ = oracle.levels_orq(v, 5)
    e = oracle.expected_error(v, lv)
    assert e == pytest.approx(numpy_expected_error(v, lv), rel=1e-12)
    # the mean realised error over many independent draws converges to it
    M = 400
    tot = 0.0
    for m in range(M):
        codes = oracle.quantize(v, oracle.ORQ, 5, lv, 0.0, 3, 0, m)
        tot += oracle.quant_error(v, lv, codes)
    assert tot / M == pytest.approx(e, rel=0.01)
    # levels that do not span the data: the clipped part counts with its squared distance
    narrow = np.array([-1e-3, 1e-3], np.float32)
    assert oracle.expected_error(v, narrow) == pytest.approx(numpy_expected_error(v, narrow), rel=1e-12)
    assert np.any(np.abs(v) > 1e-3)


def test_bingrad_b_error_is_below_pb_error():
    """BinGrad-b minimises the error of a deterministic two-level quantizer, so its realised error is
    not above the expected error of the unbiased-inside BinGrad-pb (Section 'Binary Quantization')."""
    v = wl.laplace(rng(13), 20000, 1e-3)
    lb, th, _ = oracle.levels_bingrad_b(v, 0)
    cb = oracle.quantize(v, oracle.B, 2, lb, th, 0, 0, 0)
    lpb, _ = oracle.levels_bingrad_pb(v)
    assert oracle.quant_error(v, lb, cb) < oracle.expected_error(v, lpb)


# ------------------------------------------------------------------ refinement sweeps


def discrete_condition_holds(v, L, b, R):
    seg = v[(v >= L) & (v <= R)].astype(np.float64)
    T = (seg.sum() - float(L) * seg.size) / (float(R) - float(L))
    ge, gt = np.count_nonzero(seg >= b), np.count_nonzero(seg > b)
    return ge > gt and ge >= T - 1e-9 * seg.size and gt <= T + 1e-9 * seg.size


@pytest.mark.parametrize("s", [3, 5, 9])
def test_refinement_never_increases_the_error_and_reaches_a_fixed_point(s):
    for seed, gen in [(20, lambda r: wl.laplace(r, 3000, 1e-3)), (21, lambda r: wl.student_t(r, 2000, 3.0, 1e-3)),
                      (22, lambda r: wl.mixture(r, 2500, 0.9, 1e-4, 1e-2))]:
        v = gen(rng(seed))
        lv0, _ = oracle.levels_orq(v, s)
        errs = [numpy_expected_error(v, lv0)]
        lv = lv0
        for _ in range(64):
            nxt, changed = oracle.refine_orq(v, lv, 1)
            errs.append(numpy_expected_error(v, nxt))
            assert errs[-1] <= errs[-2] * (1 + 1e-12)
            assert nxt[0] == lv0[0] and nxt[-1] == lv0[-1] and np.all(np.diff(nxt) >= 0)
            if changed == 0:
                assert np.array_equal(nxt, lv)
                break
            lv = nxt
        else:
            pytest.fail("no fixed point within 64 sweeps")
        # one call with a large cap lands on the same levels
        full, _ = oracle.refine_orq(v, lv0, 1000)
        assert np.array_equal(full, lv)
        # fixed point: every interior level meets the discrete condition against its FINAL neighbours
        for k in range(1, s - 1):
            if lv[k + 1] > lv[k - 1]:
                assert discrete_condition_holds(v, lv[k - 1], lv[k], lv[k + 1]), k
        if s == 3:
            assert np.array_equal(lv, lv0)  # one interior level: the greedy solve is already optimal
        else:
            assert errs[-1] < errs[0]  # deeper recursions leave room


def test_refinement_fixed_point_is_coordinatewise_optimal_by_brute_force():
    v = wl.laplace(rng(23), 300, 1e-3)
    lv0, _ = oracle.levels_orq(v, 5)
    lv, _ = oracle.refine_orq(v, lv0, 1000)
    base = numpy_expected_error(v, lv)
    cand = np.unique(v)
    for k in range(1, 4):
        for b in cand[(cand >= lv[k - 1]) & (cand <= lv[k + 1])]:
            trial = lv.copy()
            trial[k] = b
            assert numpy_expected_error(v, trial) >= base * (1 - 1e-12)


def test_refinement_order_is_ascending_gauss_seidel():
    """One sweep updates level 1 first and level 2 sees the new level 1: redo it by hand with Q*."""
    v = wl.student_t(rng(24), 1500, 3.0, 1e-3)
    lv0, _ = oracle.levels_orq(v, 5)
    got, _ = oracle.refine_orq(v, lv0, 1)
    hand = lv0.copy()
    for k in (1, 2, 3):
        hand[k] = np.float32(oracle.qstar(v, float(hand[k - 1]), float(hand[k + 1])))
    assert np.array_equal(got, hand)
