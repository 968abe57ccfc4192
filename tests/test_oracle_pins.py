"""Pins for the CPU oracle: what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Each one is chosen so that a
plausible mistake in the oracle (a dropped term, a wrong sign or index, a
transposed operand, an off-by-one level) fails it.
"""
import math
import os
import re
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import literal
from paper_2112_10769_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_values.txt")


def golden():
    rec = {}
    with open(GOLDEN) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, vals, _cite = [p.strip() for p in line.split("|", 2)]
            rec[name] = [float(v) for v in vals.split()]
    return rec


def decode_luq(codes, n, alpha):
    nib = oracle.unpack(codes, n).astype(np.int64)
    c = nib & 7
    mag = np.where(c > 0, np.exp2((c - 1).astype(np.float64)), 0.0) * float(alpha)
    return np.where(nib & 8, -mag, mag), c


# ---------------------------------------------------------------- Philox ----

def test_philox_weyl_constants_closed_form():
    """The two key increments are floor(2^32 (phi - 1)) and floor(2^32 (sqrt 3 - 1))."""
    c = oracle.philox_constants()
    phi = (1 + Fraction(math.isqrt(5 * 10 ** 40), 10 ** 20)) / 2
    assert int(c[2]) == int((phi - 1) * 2 ** 32)
    sqrt3 = Fraction(math.isqrt(3 * 10 ** 40), 10 ** 20)
    assert int(c[3]) == int((sqrt3 - 1) * 2 ** 32)


def test_philox_constants_match_curand_header():
    path = "/usr/local/cuda/include/curand_philox4x32_x.h"
    if not os.path.exists(path):
        pytest.skip("cuRAND header not on this machine")
    text = open(path).read()
    want = {}
    for name in ("PHILOX_M4x32_0", "PHILOX_M4x32_1", "PHILOX_W32_0", "PHILOX_W32_1"):
        m = re.search(r"#define\s+%s\s+\(?(0x[0-9A-Fa-f]+)" % name, text)
        assert m, name
        want[name] = int(m.group(1), 16)
    c = [int(v) for v in oracle.philox_constants()]
    assert c == [want["PHILOX_M4x32_0"], want["PHILOX_M4x32_1"], want["PHILOX_W32_0"], want["PHILOX_W32_1"]]


def _inverse_round(c, k):
    """Inverse of one Philox round, built from modular inverses of the multipliers
    (a round is a bijection of the 128-bit counter for a fixed key)."""
    ma, mb = int(oracle.philox_constants()[0]), int(oracle.philox_constants()[1])
    inv_a, inv_b = pow(ma, -1, 2 ** 32), pow(mb, -1, 2 ** 32)
    n0, n1, n2, n3 = c
    c0 = (n3 * inv_a) % 2 ** 32          # n3 = lo(ma*c0)
    c2 = (n1 * inv_b) % 2 ** 32          # n1 = lo(mb*c2)
    c1 = n0 ^ ((mb * c2) >> 32) ^ k[0]   # n0 = hi(mb*c2)^c1^k0
    c3 = n2 ^ ((ma * c0) >> 32) ^ k[1]   # n2 = hi(ma*c0)^c3^k1
    return [c0, c1, c2, c3]


def test_philox_ten_rounds_invert():
    """Undoing ten rounds with the key schedule run backwards recovers the counter:
    checks the round structure, the word routing and the number of rounds."""
    w0, w1 = int(oracle.philox_constants()[2]), int(oracle.philox_constants()[3])
    rng = np.random.default_rng(7)
    for _ in range(50):
        ctr = [int(v) for v in rng.integers(0, 2 ** 32, 4)]
        key = [int(v) for v in rng.integers(0, 2 ** 32, 2)]
        out = [int(v) for v in oracle.philox4x32_10(ctr, key)]
        c = out
        for r in range(9, -1, -1):
            k = [(key[0] + r * w0) % 2 ** 32, (key[1] + r * w1) % 2 ** 32]
            c = _inverse_round(c, k)
        assert c == ctr


def test_philox_words_uniform_and_keyed():
    n = 1 << 16
    w = np.array([oracle.random_word(0, 0, i) for i in range(n)], dtype=np.uint64)
    # chi-square on the top byte: 255 dof, mean 255, sd ~22.6
    counts = np.bincount((w >> 24).astype(np.int64), minlength=256)
    chi2 = float(((counts - n / 256) ** 2 / (n / 256)).sum())
    assert 150 < chi2 < 380
    # bit balance of every bit position
    for b in range(32):
        ones = int(((w >> b) & 1).sum())
        assert abs(ones - n / 2) < 5 * math.sqrt(n) / 2
    # sample s of seed equals sample 0 of seed+s; different seeds differ
    assert all(oracle.random_word(5, 2, i) == oracle.random_word(7, 0, i) for i in range(64))
    assert sum(oracle.random_word(5, 0, i) == oracle.random_word(6, 0, i) for i in range(64)) == 0
    # element i uses word i%4 of block i//4
    blk = oracle.philox4x32_10([3, 0, 0, 0], [9, 0])
    assert [oracle.random_word(9, 0, 12 + j) for j in range(4)] == [int(v) for v in blk]
    # 64-bit index and seed reach the high counter/key words
    blk = oracle.philox4x32_10([1, 2, 0, 0], [4, 3])
    assert oracle.random_word((3 << 32) + 4, 0, ((2 << 32) + 1) * 4 + 1) == int(blk[1])


# ------------------------------------------------------------------ amax ----

def test_amax_basic_and_nonfinite():
    x = np.array([0.5, -3.25, 2.0, -0.0], dtype=np.float32)
    v, fl = oracle.amax(x)
    assert v == np.float32(3.25) and fl == 0
    x = inputs.log_uniform_magnitudes(10001, -40, 10, 3)
    v, fl = oracle.amax(x)
    assert v == np.abs(x).max() and fl == 0
    for bad in (np.inf, -np.inf, np.nan):
        y = x.copy()
        y[17] = bad
        _, fl = oracle.amax(y)
        assert fl == oracle.FLAG_NONFINITE
    v, fl = oracle.amax(np.zeros(5, dtype=np.float32))
    assert v == 0 and fl == 0
    b = inputs.to_bf16_bits(np.array([1.0, -2.5, 0.3], dtype=np.float32))
    v, _ = oracle.amax(b)
    assert v == np.float32(2.5)


# ------------------------------------------------------------------ INT4 ----

def test_int4_error_bound_grid_and_extremes():
    x = inputs.normal((4096,), 1.0, 11)
    clip, _ = oracle.amax(x)
    codes, s, fl = oracle.quant_int4(x, clip)
    assert fl == 0 and s == np.float32(clip) / np.float32(7)
    q = oracle.unpack(codes, x.size).astype(np.int64)
    q = np.where(q >= 8, q - 16, q)
    assert q.min() >= -7 and q.max() <= 7 and (oracle.unpack(codes, x.size) != 8).all()
    err = np.abs(x.astype(np.float64) - q * float(s))
    assert err.max() <= float(s) / 2 * (1 + 1e-5)
    # the element of largest magnitude maps to +-7
    i = int(np.abs(x).argmax())
    assert abs(q[i]) == 7 and np.sign(q[i]) == np.sign(x[i])
    # dequantised values agree with the C dequantiser
    np.testing.assert_array_equal(oracle.dequant(codes, x.size, s, "int4"), q * float(s))


def test_int4_idempotent_on_grid_and_ties_to_even():
    clip = np.float32(7.0)  # step exactly 1
    grid = np.arange(-7, 8, dtype=np.float32)
    codes, s, _ = oracle.quant_int4(grid, clip)
    assert s == 1.0
    q = oracle.unpack(codes, grid.size).astype(np.int64)
    q = np.where(q >= 8, q - 16, q)
    np.testing.assert_array_equal(q, np.arange(-7, 8))
    halves = np.array([0.5, 1.5, 2.5, 3.5, 4.5, 5.5, 6.5, -0.5, -1.5, -2.5, -6.5], dtype=np.float32)
    codes, _, _ = oracle.quant_int4(halves, clip)
    q = oracle.unpack(codes, halves.size).astype(np.int64)
    q = np.where(q >= 8, q - 16, q)
    np.testing.assert_array_equal(q, [0, 2, 2, 4, 4, 6, 6, 0, -2, -2, -6])
    # a caller-supplied clip below the maximum saturates at +-7
    big = np.array([100.0, -100.0, 7.49, 7.51], dtype=np.float32)
    codes, _, _ = oracle.quant_int4(big, clip)
    q = oracle.unpack(codes, 4).astype(np.int64)
    np.testing.assert_array_equal(np.where(q >= 8, q - 16, q), [7, -7, 7, 7])


def test_int4_brute_force_window():
    """Every float in a small window around a decision boundary rounds to the
    nearest grid point (checked against exact rational arithmetic)."""
    clip = np.float32(3.0)
    s = np.float32(clip) / np.float32(7)
    inv = np.float32(7) / np.float32(clip)
    start = np.float32(2.5 * float(s))
    bits = np.arange(-300, 300, dtype=np.int64) + int(np.array([start]).view(np.uint32)[0])
    x = bits.astype(np.uint32).view(np.float32)
    codes, _, _ = oracle.quant_int4(x, clip)
    q = oracle.unpack(codes, x.size).astype(np.int64)
    # the oracle's rule: nearest integer to fl(x * fl(7/clip)); near the boundary the
    # result must be 2 or 3 and must switch exactly once, where fl(x*inv) crosses 2.5
    y = (x * inv).astype(np.float32)
    want = np.where(y > 2.5, 3, 2)  # 2.5 ties to even -> 2
    np.testing.assert_array_equal(q, want)
    assert set(q.tolist()) == {2, 3}
    # and the exact quotient agrees away from the last-ulp neighbourhood
    exact = np.array([Fraction(float(v)) / Fraction(float(s)) for v in x])
    far = np.array([abs(e - Fraction(5, 2)) > Fraction(1, 10 ** 6) for e in exact])
    np.testing.assert_array_equal(q[far], np.array([round(e) for e in exact])[far])


def test_int4_zero_and_unusable_clip():
    x = np.ones(6, dtype=np.float32)
    for clip, flag in ((0.0, 0), (np.inf, oracle.FLAG_NONFINITE), (np.nan, oracle.FLAG_NONFINITE),
                       (2.0 ** -120, oracle.FLAG_RANGE), (2.0 ** 110, oracle.FLAG_RANGE)):
        codes, s, fl = oracle.quant_int4(x, clip)
        assert s == 0 and fl == flag and not codes.any()


# ------------------------------------------------------------------- LUQ ----

def luq_test_tensor(seed=21, n=4096):
    x = inputs.log_uniform_magnitudes(n, -30, 3, seed)
    x[:8] = [0.0, -0.0, 8.0, -8.0, 1e-30, -1e-30, 3.0, -5.0]
    return x


@pytest.mark.parametrize("kmax", [4, 6, 2])
def test_luq_grid_and_top_level(kmax):
    x = luq_test_tensor()
    mx, _ = oracle.amax(x)
    codes, alpha, fl = oracle.quant_luq(x, mx, seed=3, n_samples=2, kmax=kmax)
    assert fl == 0 and float(alpha) * 2 ** kmax == float(mx)
    for s in range(2):
        val, c = decode_luq(codes[s], x.size, alpha)
        assert c.max() <= kmax + 1
        levels = {0.0} | {float(alpha) * 2 ** k for k in range(kmax + 1)}
        assert set(np.abs(val).tolist()) <= levels
        # sign kept, zero is always the 0x0 nibble
        nz = val != 0
        assert (np.sign(val[nz]) == np.sign(x[nz])).all()
        assert (oracle.unpack(codes[s], x.size)[~nz] == 0).all()
        # the maximum is represented exactly by the top level
        i = int(np.abs(x).argmax())
        assert abs(val[i]) == float(mx)
        # a value never moves further than to the two levels around it
        lo, hi, _ = oracle.luq_bins(x, mx, kmax)
        a = np.abs(val) / float(alpha)
        assert ((a == lo) | (a == hi)).all()
        assert (lo * float(alpha) <= np.abs(x).astype(np.float64) * (1 + 1e-6)).all()
        assert (np.abs(x).astype(np.float64) <= hi * float(alpha) * (1 + 1e-6)).all()


def test_luq_fixed_points_every_seed():
    kmax = 4
    mx = np.float32(0.37)
    alpha = oracle.luq_alpha(mx, kmax)
    grid = [0.0, -0.0] + [s * float(alpha) * 2 ** k for k in range(kmax + 1) for s in (1, -1)]
    x = np.array(grid, dtype=np.float32)
    for seed in range(40):
        codes, a, _ = oracle.quant_luq(x, mx, seed)
        val, _ = decode_luq(codes[0], x.size, a)
        np.testing.assert_array_equal(val, x.astype(np.float64))
        assert (oracle.unpack(codes[0], x.size)[:2] == 0).all()
    # on-grid inputs stay fixed for many different scales (true IEEE division)
    rng = np.random.default_rng(5)
    for mxv in np.exp2(rng.uniform(-20, 20, 300)).astype(np.float32):
        al = oracle.luq_alpha(mxv, kmax)
        xs = np.array([float(al) * 2 ** k for k in range(kmax + 1)], dtype=np.float32)
        lo, hi, thr = oracle.luq_bins(xs, mxv, kmax)
        np.testing.assert_array_equal(lo, [1, 2, 4, 8, 16])
        assert not thr.any()


def test_luq_exact_expectation_closed_form():
    """E[Q(x)] = alpha (lo + (hi - lo) thr / 2^32) equals x up to one fp32 rounding
    of the quotient and the 2^-32 truncation of the threshold."""
    for kmax in (4, 6):
        x = luq_test_tensor(seed=33, n=20000)
        mx, _ = oracle.amax(x)
        alpha = float(oracle.luq_alpha(mx, kmax))
        lo, hi, thr = oracle.luq_bins(x, mx, kmax)
        e = alpha * (lo + (hi - lo) * thr.astype(np.float64) / 2.0 ** 32)
        a = np.abs(x).astype(np.float64)
        bound = 2.0 ** -23 * a + 2.0 ** -32 * alpha
        assert (np.abs(e - a) <= bound).all()


def test_luq_matches_literal_two_stage_distribution():
    """The single-draw rule has the same outcome probabilities as applying the
    paper's T_alpha and then Q_alpha with independent draws (exact fractions)."""
    kmax = 4
    mx = np.float32(16.0)  # alpha = 1: thresholds are exact
    picks = [0.25, 0.5, 0.75, 1.0, 1.5, 3.0, 5.0, 6.0, 12.0, 15.0, 16.0, -0.25, -3.0, -12.0,
             2.0 ** -20, 1.0 - 2.0 ** -24, 1.0 + 2.0 ** -23]
    x = np.array(picks, dtype=np.float32)
    lo, hi, thr = oracle.luq_bins(x, mx, kmax)
    for xi, l, h, t in zip(x, lo, hi, thr):
        dist = literal.luq_distribution(Fraction(float(xi)), Fraction(1), kmax)
        sign = -1 if xi < 0 else 1
        p_hi = Fraction(int(t), 2 ** 32)
        got = {}
        if p_hi < 1:
            got[Fraction(sign * l)] = 1 - p_hi
        if p_hi > 0:
            got[Fraction(sign * h)] = got.get(Fraction(sign * h), 0) + p_hi
        assert got == dist, (xi, got, dist)
        assert literal.expectation(dist) == Fraction(float(xi))
    # mid-bin values have probability exactly one half, a quarter of alpha one quarter
    assert int(thr[picks.index(1.5)]) == 2 ** 31 and int(thr[picks.index(0.25)]) == 2 ** 30
    # a general scale: probabilities agree with the exact ones to fp32 rounding
    mx = np.float32(0.123456)
    alpha = Fraction(float(oracle.luq_alpha(mx, kmax)))
    x = inputs.log_uniform_magnitudes(400, -12, -3.1, 44)
    x = x[np.abs(x) <= mx]
    lo, hi, thr = oracle.luq_bins(x, mx, kmax)
    for xi, l, h, t in zip(x, lo, hi, thr):
        dist = literal.luq_distribution(Fraction(float(xi)), alpha, kmax)
        sign = -1 if xi < 0 else 1
        p_exact = dist.get(sign * Fraction(h) * alpha, Fraction(0)) if h != l else Fraction(0)
        assert abs(Fraction(int(t), 2 ** 32) - p_exact) <= Fraction(1, 2 ** 21)


def test_luq_codes_follow_the_random_word():
    """code = lo + (word < thr): ties the codes to the documented stream."""
    x = luq_test_tensor(seed=8, n=3000)
    mx, _ = oracle.amax(x)
    lo, hi, thr = oracle.luq_bins(x, mx, 4)
    codes, alpha, _ = oracle.quant_luq(x, mx, seed=77, n_samples=3)
    for s in range(3):
        words = np.array([oracle.random_word(77, s, i) for i in range(x.size)], dtype=np.uint64)
        up = words < thr.astype(np.uint64)
        val, _ = decode_luq(codes[s], x.size, alpha)
        want = np.where(up, hi, lo) * float(alpha)
        np.testing.assert_array_equal(np.abs(val), want)
    # planes are independent draws: sample s of seed 77 is sample 0 of seed 77+s
    again, _, _ = oracle.quant_luq(x, mx, seed=79, n_samples=1)
    np.testing.assert_array_equal(again[0], codes[2])


def test_luq_statistically_unbiased_and_variance():
    """Mean over seeds approaches x; per-element variance follows Table 1:
    Var[SR(x)] = (x - l)(u - x)."""
    kmax = 4
    x = inputs.log_uniform_magnitudes(512, -8, 0, 55)
    mx, _ = oracle.amax(x)
    alpha = float(oracle.luq_alpha(mx, kmax))
    S = 2048
    acc = np.zeros(x.size)
    acc2 = np.zeros(x.size)
    for seed in range(S):
        codes, a, _ = oracle.quant_luq(x, mx, seed)
        v, _ = decode_luq(codes[0], x.size, a)
        acc += v
        acc2 += v * v
    mean = acc / S
    lo, hi, _ = oracle.luq_bins(x, mx, kmax)
    ax = np.abs(x).astype(np.float64)
    var_closed = (ax - lo * alpha) * (hi * alpha - ax)
    var_closed = np.maximum(var_closed, 0)
    z = np.abs(mean - x) / np.sqrt(var_closed / S + 1e-300)
    assert (z[var_closed > 0] < 5.5).all()
    assert (mean[var_closed == 0] == x[var_closed == 0]).all()
    var_emp = acc2 / S - mean ** 2
    big = var_closed > 0
    # aggregate check: total empirical variance within a few percent of the closed form
    assert abs(var_emp[big].sum() / var_closed[big].sum() - 1) < 0.05
    # tensor-level sum is unbiased as well
    total_sd = math.sqrt(var_closed.sum() / S)
    assert abs(mean.sum() - x.astype(np.float64).sum()) < 5 * total_sd


def test_smp_two_samples_halve_the_variance():
    """Sec. 5.1: averaging N independent samples divides the variance by N."""
    x = inputs.log_uniform_magnitudes(256, -6, 0, 66)
    mx, _ = oracle.amax(x)
    S = 1500
    one, two = [], []
    for t in range(S):
        codes, a, _ = oracle.quant_luq(x, mx, seed=2 * t, n_samples=2)
        v0, _ = decode_luq(codes[0], x.size, a)
        v1, _ = decode_luq(codes[1], x.size, a)
        one.append(v0)
        two.append((v0 + v1) / 2)
    v1 = np.var(np.array(one), axis=0).sum()
    v2 = np.var(np.array(two), axis=0).sum()
    assert abs(v2 / v1 - 0.5) < 0.04
    assert abs(np.mean(two, axis=0).sum() - x.astype(np.float64).sum()) < 5 * math.sqrt(v2 / S)


def test_luq_zero_and_unusable_max():
    x = np.ones(6, dtype=np.float32)
    for mx, flag in ((0.0, 0), (np.inf, oracle.FLAG_NONFINITE), (np.nan, oracle.FLAG_NONFINITE),
                     (2.0 ** -120, oracle.FLAG_RANGE)):
        codes, a, fl = oracle.quant_luq(x, mx, 1, n_samples=2)
        assert a == 0 and fl == flag and not codes.any()
    # a caller-supplied max below the true one clips to the top level
    x = np.array([100.0, -100.0, 1.0], dtype=np.float32)
    codes, a, _ = oracle.quant_luq(x, np.float32(16.0), 0)
    np.testing.assert_array_equal(oracle.unpack(codes[0], 3), [5, 13, 1])


# ---------------------------------------------------- the paper's numbers ----

def test_worked_values_from_the_paper():
    g = golden()
    bins = g["radix2_bins"]
    # 4.5 lies in the bin [4, 8]: nearest is 4, stochastic rounding goes up w.p. 1/8
    lo = max(b for b in bins if b <= 4.5)
    hi = min(b for b in bins if b > 4.5)
    assert literal.round_nearest_in_bin(4.5, lo, hi) == g["radix2_nearest_of_4p5"][0]
    dist = literal.log_stochastic_round(Fraction(9, 2), Fraction(1), 3)
    assert dist == {Fraction(4): Fraction(7, 8), Fraction(8): Fraction(1, 8)}
    x = np.array([4.5, 8.0], dtype=np.float32)
    lo_, hi_, thr = oracle.luq_bins(x, np.float32(8.0), 3)
    assert (lo_[0], hi_[0], int(thr[0])) == (4.0, 8.0, 2 ** 29)
    # FP4 [1,3,0]: magnitude code 011 represents 4; INT4 3 times FP4 4 is 12
    packed = np.array([0b0011 | (0b0011 << 4)], dtype=np.uint8)
    assert oracle.dequant(packed, 1, 1.0, "luq")[0] == g["fp4_code_011_value"][0]
    prod = oracle.gemm_int64("bwd", packed, 1, np.array([0x03, 0x00], dtype=np.uint8), 1, 2, 2)
    # G = [4, 4] (codes 3,3), W = [[3, 0], [0, 0]] -> dA[0,0] = 4*3
    assert prod[0, 0] == g["int4_3_times_fp4_4"][0]
    # FP2 [1,1,0]: three levels from 2^0 to 2^2 when the maximum is 4
    x = np.array([4.0, 0.3, 1.7, 2.9], dtype=np.float32)
    codes, a, _ = oracle.quant_luq(x, np.float32(4.0), 0, kmax=2)
    val, _ = decode_luq(codes[0], 4, a)
    assert float(a) == g["fp2_min_max"][0] and abs(val[0]) == g["fp2_min_max"][1]
    # Eq. alpha with b = 3
    assert 2 ** (2 ** (3 - 1)) == g["fp4_alpha_divisor"][0]
    assert float(oracle.luq_alpha(np.float32(1.0), oracle.KMAX_DEFAULT)) == 1 / g["fp4_alpha_divisor"][0]
    assert abs((math.log2(4 / 3) - 0.5) - g["rdnp_shift"][0]) < 1e-4


def test_table1_closed_forms_and_mse_ordering():
    """Table 1 against the exact distribution of stochastic rounding."""
    for xf in [Fraction(9, 2), Fraction(5), Fraction(7, 1), Fraction(33, 8), Fraction(4), Fraction(6)]:
        lo, hi = Fraction(4), Fraction(8)
        dist = literal.log_stochastic_round(xf, Fraction(1), 3)
        b_rdn, v_rdn, mse_rdn, b_sr, v_sr, mse_sr = literal.table1(xf, lo, hi)
        assert literal.expectation(dist) - xf == b_sr == 0
        assert literal.variance(dist) == v_sr == (xf - lo) * (hi - xf)
        r = literal.round_nearest_in_bin(xf, lo, hi)
        assert abs(r - xf) == b_rdn and (r - xf) ** 2 == mse_rdn and v_rdn == 0
        assert mse_sr >= mse_rdn


# ------------------------------------------------------------------ GEMMs ----

def small_codes(M, K, N, seed, n_samples=1):
    A, W, G = inputs.small_layer(M, K, N, seed)
    ca, sa, _ = oracle.quant_int4(A, oracle.amax(A)[0])
    cw, sw, _ = oracle.quant_int4(W, oracle.amax(W)[0])
    cg, al, _ = oracle.quant_luq(G, oracle.amax(G)[0], seed=seed, n_samples=n_samples)
    return (A, W, G), (ca, sa), (cw, sw), (cg, al)


@pytest.mark.parametrize("M,K,N,ns", [(6, 8, 4, 1), (5, 6, 8, 2), (16, 10, 12, 3)])
def test_gemms_against_numpy_and_int64(M, K, N, ns):
    _, (ca, sa), (cw, sw), (cg, al) = small_codes(M, K, N, 100 + M, ns)
    Ad = oracle.dequant(ca, M * K, sa, "int4").reshape(M, K)
    Wd = oracle.dequant(cw, N * K, sw, "int4").reshape(N, K)
    Gd = np.mean([oracle.dequant(cg[s], M * N, al, "luq").reshape(M, N) for s in range(ns)], axis=0)
    Z = oracle.gemm_fwd(ca, sa, cw, sw, M, N, K)
    dA = oracle.gemm_bwd(cg, al, ns, cw, sw, M, N, K)
    dW = oracle.gemm_wgrad(cg, al, ns, ca, sa, M, N, K)
    np.testing.assert_allclose(Z, Ad @ Wd.T, rtol=1e-13, atol=1e-300)
    np.testing.assert_allclose(dA, Gd @ Wd, rtol=1e-13, atol=1e-300)
    np.testing.assert_allclose(dW, Gd.T @ Ad, rtol=1e-13, atol=1e-300)
    # scale factoring (Appendix A.1): integer sums times one scale product
    zi = oracle.gemm_int64("fwd", ca, 1, cw, M, N, K)
    np.testing.assert_allclose(Z, zi * (float(sa) * float(sw)), rtol=1e-13)
    di = oracle.gemm_int64("bwd", cg, ns, cw, M, N, K)
    np.testing.assert_allclose(dA, di * (float(al) * float(sw) / ns), rtol=1e-13)
    wi = oracle.gemm_int64("wgrad", cg, ns, ca, M, N, K)
    np.testing.assert_allclose(dW, wi * (float(al) * float(sa) / ns), rtol=1e-13)
    # entries computed one by one
    rows = np.array([0, M - 1, 1]); cols = np.array([N - 1, 0, 2])
    np.testing.assert_allclose(oracle.gemm_entries("fwd", ca, sa, 1, cw, sw, M, N, K, rows, cols),
                               Z[rows, cols], rtol=1e-13)
    cols = np.array([K - 1, 0, 2])
    np.testing.assert_allclose(oracle.gemm_entries("bwd", cg, al, ns, cw, sw, M, N, K, rows, cols),
                               dA[rows, cols], rtol=1e-13)
    rows = np.array([0, N - 1, 1])
    np.testing.assert_allclose(oracle.gemm_entries("wgrad", cg, al, ns, ca, sa, M, N, K, rows, cols),
                               dW[rows, cols], rtol=1e-13)


def test_general_kind_products_against_numpy_and_the_named_products():
    """oracle.gemm_general (operands of any code kind) against numpy on the dequantized values, and equal
    to gemm_fwd / gemm_bwd / gemm_wgrad for the kinds those take."""
    M, K, N, ns = 10, 12, 8, 3
    (A, W, G), (ca, sa), (cw, sw), (cg, al) = small_codes(M, K, N, 321, ns)
    np.testing.assert_array_equal(oracle.gemm_general("fwd", ca, "int4", sa, 1, cw, "int4", sw, M, N, K),
                                  oracle.gemm_fwd(ca, sa, cw, sw, M, N, K))
    np.testing.assert_array_equal(oracle.gemm_general("bwd", cg, "luq", al, ns, cw, "int4", sw, M, N, K),
                                  oracle.gemm_bwd(cg, al, ns, cw, sw, M, N, K))
    np.testing.assert_array_equal(oracle.gemm_general("wgrad", cg, "luq", al, ns, ca, "int4", sa, M, N, K),
                                  oracle.gemm_wgrad(cg, al, ns, ca, sa, M, N, K))
    cu, su, _ = oracle.quant_uint4(np.maximum(A, 0), oracle.amax(A)[0])
    gi, sg, _ = oracle.quant_int4_sr(G, oracle.amax(G)[0], 5, n_samples=ns)
    Au = oracle.dequant(cu, M * K, su, "uint4").reshape(M, K)
    Wd = oracle.dequant(cw, N * K, sw, "int4").reshape(N, K)
    Gi = np.mean([oracle.dequant(gi[s], M * N, sg, "int4").reshape(M, N) for s in range(ns)], axis=0)
    np.testing.assert_allclose(oracle.gemm_general("fwd", cu, "uint4", su, 1, cw, "int4", sw, M, N, K), Au @ Wd.T,
                               rtol=1e-13, atol=1e-300)
    np.testing.assert_allclose(oracle.gemm_general("bwd", gi, "int4", sg, ns, cw, "int4", sw, M, N, K), Gi @ Wd,
                               rtol=1e-13, atol=1e-18)
    np.testing.assert_allclose(oracle.gemm_general("wgrad", gi, "int4", sg, ns, cu, "uint4", su, M, N, K), Gi.T @ Au,
                               rtol=1e-13, atol=1e-18)


def test_gemm_orientation_with_unit_vectors():
    """One non-zero per operand: the product lands where the definition puts it
    (catches transposed operands and swapped index roles)."""
    M, K, N = 4, 6, 8
    def int4_plane(rows, cols, r, c, q):
        p = np.zeros((rows, cols // 2), dtype=np.uint8)
        p[r, c // 2] = (q & 0xF) << (4 * (c % 2))
        return p
    def luq_plane(rows, cols, r, c, nib):
        p = np.zeros((rows, cols // 2), dtype=np.uint8)
        p[r, c // 2] = nib << (4 * (c % 2))
        return p
    a = int4_plane(M, K, 2, 5, 3)          # A[2,5] = 3
    w = int4_plane(N, K, 7, 5, -2)         # W[7,5] = -2
    Z = oracle.gemm_fwd(a, 1.0, w, 1.0, M, N, K)
    assert Z[2, 7] == -6 and np.count_nonzero(Z) == 1
    g = luq_plane(M, N, 1, 7, 0b1011)      # G[1,7] = -4
    dA = oracle.gemm_bwd(g, 1.0, 1, w, 1.0, M, N, K)
    assert dA[1, 5] == 8 and np.count_nonzero(dA) == 1
    g = luq_plane(M, N, 2, 3, 0b0100)      # G[2,3] = 8
    dW = oracle.gemm_wgrad(g, 0.5, 1, a, 2.0, M, N, K)
    assert dW[3, 5] == 24 and np.count_nonzero(dW) == 1


def test_wgrad_is_unbiased_over_seeds():
    """E[Q(G)^T A_q] = G^T A_q (Sec. 3.2, Eq. 'update' expectation)."""
    M, K, N = 24, 8, 6
    A, W, G = inputs.small_layer(M, K, N, 9, g_mu=-2.0, g_sigma=1.5, zero_frac=0.1)
    ca, sa, _ = oracle.quant_int4(A, oracle.amax(A)[0])
    Ad = oracle.dequant(ca, M * K, sa, "int4").reshape(M, K)
    target = G.astype(np.float64).T @ Ad
    mx = oracle.amax(G)[0]
    S = 3000
    acc = np.zeros((N, K)); acc2 = np.zeros((N, K))
    for seed in range(S):
        cg, al, _ = oracle.quant_luq(G, mx, seed)
        dW = oracle.gemm_wgrad(cg, al, 1, ca, sa, M, N, K)
        acc += dW; acc2 += dW * dW
    mean = acc / S
    sd = np.sqrt(np.maximum(acc2 / S - mean ** 2, 0) / S)
    assert (np.abs(mean - target) <= 5.5 * sd + 1e-12).all()
    # closed-form variance: sum_m A_q[m,k]^2 (|G|-lo)(hi-|G|)
    lo, hi, _ = oracle.luq_bins(G, mx, 4)
    al = float(oracle.luq_alpha(mx, 4))
    g = np.abs(G.astype(np.float64)).reshape(-1)
    v = np.maximum((g - lo * al) * (hi * al - g), 0).reshape(M, N)
    var_closed = v.T @ (Ad ** 2)
    var_emp = acc2 / S - mean ** 2
    assert abs(var_emp.sum() / var_closed.sum() - 1) < 0.1


def test_integer_partial_sums_fit_fp32():
    """All products are small integers; the largest possible sum over the
    benchmark shapes stays below 2^24, so fp32 accumulation is exact."""
    kmax = oracle.KMAX_DEFAULT
    worst_fwd = 49 * 2304
    worst_bwd = 7 * 2 ** kmax * 4096 * 1
    worst_wgrad = 7 * 2 ** kmax * 50176 * 2
    assert max(worst_fwd, worst_bwd, worst_wgrad) < 2 ** 24


def test_philox_stream_matches_curand_host_function(tmp_path):
    """The generator equals NVIDIA's own Philox4x32-10 block function, compiled
    for the host from the cuRAND header (an implementation independent of the oracle)."""
    import ctypes
    import shutil
    import subprocess
    if shutil.which("nvcc") is None:
        pytest.skip("nvcc not on this machine")
    src = os.path.join(os.path.dirname(__file__), "curand_philox_host.cu")
    so = str(tmp_path / "libcurand_philox_host.so")
    subprocess.run(["nvcc", "-Wno-deprecated-gpu-targets", "-shared", "-Xcompiler", "-fPIC", "-o", so, src], check=True)
    L = ctypes.CDLL(so)
    u32p = ctypes.POINTER(ctypes.c_uint32)
    rng = np.random.default_rng(1)
    cases = [(np.zeros(4, np.uint32), np.zeros(2, np.uint32)),
             (np.full(4, 0xFFFFFFFF, np.uint32), np.full(2, 0xFFFFFFFF, np.uint32))]
    cases += [(rng.integers(0, 2 ** 32, 4, dtype=np.uint32), rng.integers(0, 2 ** 32, 2, dtype=np.uint32))
              for _ in range(200)]
    for c, k in cases:
        out = np.zeros(4, dtype=np.uint32)
        L.curand_philox_block(c.ctypes.data_as(u32p), k.ctypes.data_as(u32p), out.ctypes.data_as(u32p))
        np.testing.assert_array_equal(out, oracle.philox4x32_10(c, k))


def test_luq_window_equals_slice_of_full_tensor():
    x = luq_test_tensor(seed=91, n=5000)
    mx, _ = oracle.amax(x)
    full, _, _ = oracle.quant_luq(x, mx, seed=5, n_samples=2)
    win, _, _ = oracle.quant_luq(x[1000:3000], mx, seed=5, n_samples=2, first_index=1000)
    np.testing.assert_array_equal(win, full[:, 500:1500])


# ------------------------------------------- power-of-two scale and hindsight ----

def test_pw2_ceiling_of_the_maximum():
    """alpha_PW2 = 2^ceil(log2 max) / 2^kmax (Appendix A.7): checked against exact rationals."""
    rng = np.random.default_rng(12)
    vals = list(np.exp2(rng.uniform(-90, 90, 500)).astype(np.float32)) + \
        [np.float32(2.0 ** k) for k in range(-20, 21)] + [np.float32(1.0000001), np.float32(0.99999994)]
    for v in vals:
        p = float(oracle.pw2_ceil(v))
        m, e = math.frexp(p)
        assert m == 0.5                                   # a power of two
        assert Fraction(p) >= Fraction(float(v)) and Fraction(p) < 2 * Fraction(float(v))
        assert float(oracle.pw2_ceil(np.float32(p))) == p  # idempotent
    assert oracle.pw2_ceil(0.0) == 0.0


def test_pw2_luq_levels_are_powers_of_two_and_still_unbiased():
    x = luq_test_tensor(seed=71, n=6000)
    mx, _ = oracle.amax(x)
    codes, alpha, fl = oracle.quant_luq_pw2(x, mx, seed=4)
    assert fl == 0 and math.frexp(float(alpha))[0] == 0.5
    assert float(alpha) * 16 >= float(mx) > float(alpha) * 8          # ceiling: no clipping, less than one binade of slack
    val, c = decode_luq(codes[0], x.size, alpha)
    assert all(math.frexp(abs(v))[0] == 0.5 for v in val[val != 0][:200])
    p2 = oracle.pw2_ceil(mx)
    lo, hi, thr = oracle.luq_bins(x, p2)
    e = float(alpha) * (lo + (hi - lo) * thr.astype(np.float64) / 2.0 ** 32)
    a = np.abs(x).astype(np.float64)
    assert (np.abs(e - a) <= 2.0 ** -32 * float(alpha) + 1e-300).all()  # division by a power of two is exact
    np.testing.assert_array_equal(codes, oracle.quant_luq(x, p2, seed=4)[0])


def test_hindsight_recursion_closed_form_and_limits():
    """m_hat^t - max = eta^t (m_hat^0 - max) for a constant maximum; eta = 0 copies the
    previous maximum, eta = 1 never moves."""
    mx, m0, eta = 3.0, 11.0, 0.1
    m = np.float32(m0)
    for t in range(1, 12):
        m = oracle.hindsight_next(mx, m, eta)
        want = mx + (eta ** t) * (m0 - mx)
        assert abs(float(m) - want) <= 4e-7 * want
    assert oracle.hindsight_next(2.5, 100.0, 0.0) == np.float32(2.5)
    assert oracle.hindsight_next(2.5, 100.0, 1.0) == np.float32(100.0)
    # one rounding per operation, in binary32
    a = np.float32(np.float32(1.0) - np.float32(0.1)) * np.float32(0.7)
    b = np.float32(0.1) * np.float32(0.3)
    assert oracle.hindsight_next(0.7, 0.3, 0.1) == np.float32(np.float32(a) + np.float32(b))


def test_hindsight_recursion_ignores_non_finite_measurements_and_replaces_unusable_estimates():
    """Reading where the paper is silent: an Inf/NaN measurement leaves the estimate unchanged (so the
    sequence [m, Inf, m, m] never leaves the finite numbers), and an estimate without usable history
    (0, negative, Inf, NaN) is replaced by the measurement instead of being blended with it."""
    inf, nan = np.float32(np.inf), np.float32(np.nan)
    assert oracle.hindsight_next(inf, 3.0, 0.1) == np.float32(3.0)
    assert oracle.hindsight_next(nan, 3.0, 0.1) == np.float32(3.0)
    for bad in (0.0, -0.0, -2.0, inf, nan):
        assert oracle.hindsight_next(2.5, bad, 0.1) == np.float32(2.5)
    assert np.isnan(oracle.hindsight_next(nan, nan, 0.1)) and oracle.hindsight_next(inf, 0.0, 0.1) == 0
    m = np.float32(4.0)
    for measured in (np.float32(2.0), inf, np.float32(2.0), np.float32(2.0)):
        m = oracle.hindsight_next(measured, m, 0.1)
        assert np.isfinite(m)
    # three finite steps from 4 towards 2: 2 + 2 * 0.1^3 up to the binary32 roundings
    assert abs(float(m) - (2.0 + 2.0 * 0.1 ** 3)) < 1e-6
    # the ordinary case is untouched: one rounding per operation
    keep = np.float32(1.0) - np.float32(0.1)
    assert oracle.hindsight_next(0.7, 0.3, 0.1) == np.float32(keep * np.float32(0.7)) + np.float32(np.float32(0.1) * np.float32(0.3))


def test_hindsight_step_uses_the_estimate_and_clips_above_it():
    x = luq_test_tensor(seed=81, n=4000)
    true_max, _ = oracle.amax(x)
    m_hat = np.float32(float(true_max) / 8)                 # stale, too small estimate
    codes, alpha, fl, measured, nxt = oracle.quant_luq_hindsight(x, m_hat, 0.1, seed=9, n_samples=2)
    assert fl == 0 and measured == true_max and float(alpha) * 16 == float(m_hat)
    assert nxt == oracle.hindsight_next(true_max, m_hat, 0.1)
    val, c = decode_luq(codes[0], x.size, alpha)
    above = np.abs(x) >= m_hat
    assert above.sum() > 0 and (np.abs(val[above]) == float(m_hat)).all() and (c[above] == 5).all()
    np.testing.assert_array_equal(codes, oracle.quant_luq(x, m_hat, 9, 2)[0])
    # an estimate at or above the maximum changes nothing but the scale: still unbiased
    big = np.float32(float(true_max) * 1.7)
    lo, hi, thr = oracle.luq_bins(x, big)
    al = float(oracle.luq_alpha(big))
    e = al * (lo + (hi - lo) * thr.astype(np.float64) / 2.0 ** 32)
    a = np.abs(x).astype(np.float64)
    assert (np.abs(e - a) <= 2.0 ** -23 * a + 2.0 ** -32 * al).all()
    # with the power-of-two option the estimate is rounded up first
    codes2, alpha2, _, _, nxt2 = oracle.quant_luq_hindsight(x, m_hat, 0.1, seed=9, pw2=True)
    assert float(alpha2) * 16 == float(oracle.pw2_ceil(m_hat)) and nxt2 == nxt


# ------------------------------------- biased FP4 baseline: round-to-nearest-power (Eq. RC) ----

def _levels(kmax):
    return np.array([0.0] + [2.0 ** k for k in range(kmax + 1)])


@pytest.mark.parametrize("kmax", [2, 4, 6])
def test_nearest_power_is_the_linear_nearest_level(kmax):
    """RDNP exists because rounding the EXPONENT to nearest is biased; Eq. (RC) shifts it so that the
    chosen level is the nearest one in linear distance.  Brute force over the levels, away from ties."""
    rng = np.random.default_rng(70 + kmax)
    mx = np.float32(3.7)
    alpha = float(oracle.luq_alpha(mx, kmax))
    t = np.exp2(rng.uniform(-6, kmax, 20000))
    lv = _levels(kmax)
    mids = (lv[:-1] + lv[1:]) / 2
    t = t[np.min(np.abs(t[:, None] - mids[None, :]), axis=1) > 1e-4]
    x = (t * alpha * np.where(rng.random(t.size) < 0.5, -1, 1)).astype(np.float32)
    if x.size % 2:
        x = x[:-1]
    codes, a, fl = oracle.quant_fp_nearest(x, mx, kmax)
    assert fl == 0 and float(a) == alpha
    got = oracle.dequant(codes[0], x.size, 1.0, "luq")
    tt = np.abs(x.astype(np.float64)) / alpha
    want = lv[np.argmin(np.abs(tt[:, None] - lv[None, :]), axis=1)] * np.sign(x)
    np.testing.assert_array_equal(got, want)


def test_nearest_power_matches_the_printed_formulas():
    """2^floor(log2(4/3 * 2^x)) and the printed 2^RDN(x - 0.085), evaluated in float64 away from ties."""
    shift = golden()["rdnp_shift"][0]                      # -0.085, printed in Eq. (RC)
    rng = np.random.default_rng(5)
    xs = rng.uniform(0.0, 4.0, 20000)                       # exponents inside the range of kmax = 4
    frac = (xs + math.log2(4 / 3)) % 1.0
    xs = xs[np.minimum(frac, 1 - frac) > 1e-3]
    mx = np.float32(16.0)                                   # alpha = 1
    x = np.exp2(xs).astype(np.float32)
    if x.size % 2:
        x, xs = x[:-1], xs[:-1]
    xs = np.log2(x.astype(np.float64))
    codes, a, _ = oracle.quant_fp_nearest(x, mx, 4)
    assert float(a) == 1.0
    got = oracle.dequant(codes[0], x.size, 1.0, "luq")
    np.testing.assert_array_equal(got, np.exp2(np.floor(xs + math.log2(4 / 3))))
    np.testing.assert_array_equal(got, np.exp2(np.rint(xs + shift)))


def test_nearest_power_ties_underflow_clipping_and_bias():
    mx = np.float32(16.0)
    x = np.array([1.5, 3.0, 6.0, 12.0, 0.5, 0.49999997, 0.0, -0.75, 1.0, 2.0, 16.0, 40.0, -1.4999999, 11.999999],
                 dtype=np.float32)
    codes, _, _ = oracle.quant_fp_nearest(x, mx, 4)
    got = oracle.dequant(codes[0], x.size, 1.0, "luq")
    # midpoints go up (the floor of an exact power of two), alpha/2 goes up, values above max clip
    np.testing.assert_array_equal(got, [2, 4, 8, 16, 1, 0, 0, -1, 1, 2, 16, 16, -1, 8])
    # on-grid values are fixed points
    grid = np.array([0, 1, 2, 4, 8, 16, -1, -2, -4, -8, -16, 0], dtype=np.float32)
    c2, _, _ = oracle.quant_fp_nearest(grid, mx, 4)
    np.testing.assert_array_equal(oracle.dequant(c2[0], grid.size, 1.0, "luq"), grid)
    # it is biased, unlike LUQ: for a log-uniform density on one bin the mean error is
    # (2 ln 2 - ln 1.5 - 1) / ln 2 of the bin's lower edge (closed form of the two integrals)
    n = 1 << 20
    u = (np.arange(n) + 0.5) / n
    t = np.exp2(u).astype(np.float32)                       # log-uniform on [1, 2), alpha = 1
    c3, _, _ = oracle.quant_fp_nearest(t, mx, 4)
    err = (oracle.dequant(c3[0], n, 1.0, "luq") - t.astype(np.float64)).mean()
    closed = (2 * math.log(2) - math.log(1.5) - 1) / math.log(2)
    assert abs(err - closed) < 1e-5 and closed < -0.02
    # and it is the LUQ decision taken at probability one half: up exactly when the up-threshold >= 2^31
    xr = inputs.log_uniform_magnitudes(20000, -6, 4.5, 9)
    m2 = np.float32(np.abs(xr).max())
    lo, hi, thr = oracle.luq_bins(xr, m2)
    c4, al, _ = oracle.quant_fp_nearest(xr, m2, 4)
    got = np.abs(oracle.dequant(c4[0], xr.size, 1.0, "luq"))
    np.testing.assert_array_equal(got, np.where(thr >= 2 ** 31, hi, lo))


# ------------------------------------------------- unsigned INT4 for non-negative tensors ----

def test_uint4_grid_error_bound_and_edges():
    rng = np.random.default_rng(11)
    x = np.maximum(rng.standard_normal(100_000), 0).astype(np.float32)      # post-ReLU: half zeros
    clip, _ = oracle.amax(x)
    codes, s, fl = oracle.quant_uint4(x, clip)
    assert fl == 0 and s == np.float32(clip) / np.float32(15)
    q = oracle.unpack(codes, x.size)
    assert q.max() == 15 and q.min() == 0                                   # the maximum takes the top code
    deq = oracle.dequant(codes, x.size, float(s), "uint4")
    np.testing.assert_array_equal(deq, q.astype(np.float64) * float(s))
    assert np.abs(deq - x).max() <= float(s) / 2 * (1 + 1e-6)               # round to nearest
    assert (q[x == 0] == 0).all()
    # half the step of the signed grid on the same range: Delta/(2^b - 1) with all levels on one side
    _, s_signed, _ = oracle.quant_int4(x, clip)
    assert abs(float(s) / float(s_signed) - 7 / 15) < 1e-6
    # negative inputs clamp to zero, values above the clip to 15, ties go to even, NaN to 0
    c = np.float32(15.0)
    y = np.array([-3.0, 0.5, 1.5, 2.5, 14.5, 15.5, 99.0, np.nan, 7.49, 7.51], dtype=np.float32)
    cy, sy, _ = oracle.quant_uint4(y, c)
    assert sy == 1.0
    np.testing.assert_array_equal(oracle.unpack(cy, y.size), [0, 0, 2, 2, 14, 15, 15, 0, 7, 8])
    # idempotent on its own grid, and brute force against the nearest of the sixteen levels
    g = (np.arange(16, dtype=np.float32) * np.float32(0.25))
    cg, sg, _ = oracle.quant_uint4(g, np.float32(3.75))
    np.testing.assert_array_equal(oracle.unpack(cg, 16), np.arange(16))
    z = rng.uniform(0, 3.75, 4000).astype(np.float32)
    z = z[np.abs((z / 0.25) % 1.0 - 0.5) > 1e-3]
    z = z[: z.size // 2 * 2]
    cz, _, _ = oracle.quant_uint4(z, np.float32(3.75))
    want = np.argmin(np.abs(z.astype(np.float64)[:, None] - g.astype(np.float64)[None, :]), axis=1)
    np.testing.assert_array_equal(oracle.unpack(cz, z.size), want)
    # unusable clips behave like the signed quantizer's
    for bad, flag in ((0.0, 0), (np.inf, oracle.FLAG_NONFINITE), (1e-35, oracle.FLAG_RANGE)):
        cb, sb, fb = oracle.quant_uint4(x[:10], np.float32(bad))
        assert sb == 0 and not cb.any() and fb == flag


# ------------------------------------------ ablation arms (Sec. 4, ablation figure) ----


def test_ablation_arms_reduce_to_luq_and_to_the_biased_baseline_region_by_region():
    """SR+SU is LUQ, neither is the deterministic baseline; a mixed arm has LUQ's codes in its
    stochastic region and the baseline's in the other."""
    for kmax in (2, 4):
        x = luq_test_tensor(seed=91, n=6000)
        mx, _ = oracle.amax(x)
        alpha = oracle.luq_alpha(mx, kmax)
        luq, a0, _ = oracle.quant_luq(x, mx, seed=5, n_samples=2, kmax=kmax)
        near, _, _ = oracle.quant_fp_nearest(x, mx, kmax=kmax)
        both, a1, _ = oracle.quant_fp_ablation(x, mx, 5, True, True, n_samples=2, kmax=kmax)
        none, _, _ = oracle.quant_fp_ablation(x, mx, 5, False, False, n_samples=2, kmax=kmax)
        assert a0 == a1 == alpha
        np.testing.assert_array_equal(both, luq)
        np.testing.assert_array_equal(none[0], near[0])
        np.testing.assert_array_equal(none[1], near[0])           # no randomness: every sample equal
        below = np.abs(x) < alpha
        assert below.sum() > 100 and (~below).sum() > 100
        for sr, su in ((True, False), (False, True)):
            got, _, _ = oracle.quant_fp_ablation(x, mx, 5, sr, su, n_samples=2, kmax=kmax)
            for s in range(2):
                g = oracle.unpack(got[s], x.size)
                l = oracle.unpack(luq[s], x.size)
                d = oracle.unpack(near[0], x.size)
                np.testing.assert_array_equal(g[below], (l if su else d)[below])
                np.testing.assert_array_equal(g[~below], (l if sr else d)[~below])


def test_ablation_arms_are_unbiased_exactly_where_the_caption_says():
    """"FP4+SR" is unbiased inside the range and biased below it; stochastic underflow alone the
    other way round.  The deterministic region's error is the nearest-level error, the same for
    every seed."""
    kmax = 4
    x = inputs.log_uniform_magnitudes(384, -9, 0, 71)
    mx, _ = oracle.amax(x)
    alpha = float(oracle.luq_alpha(mx, kmax))
    below = np.abs(x) < alpha
    assert below.sum() > 60 and (~below).sum() > 60
    S = 1500
    lo, hi, _ = oracle.luq_bins(x, mx, kmax)
    ax = np.abs(x).astype(np.float64)
    var_closed = np.maximum((ax - lo * alpha) * (hi * alpha - ax), 0)     # Table 1: Var[SR]
    for sr, su in ((True, False), (False, True)):
        acc = np.zeros(x.size)
        first = None
        for seed in range(S):
            codes, a, _ = oracle.quant_fp_ablation(x, mx, seed, sr, su, kmax=kmax)
            v, _ = decode_luq(codes[0], x.size, a)
            acc += v
            if first is None:
                first = v
            det = ~below if su else below
            assert (v[det] == first[det]).all()                            # the deterministic region never moves
        mean = acc / S
        sto = below if su else ~below
        z = np.abs(mean - x)[sto] / np.sqrt(var_closed[sto] / S + 1e-300)
        assert (z[var_closed[sto] > 0] < 5.5).all()
        # deterministic region: nearest level, so the error is min(x - l, u - x) (Table 1: Bias[RDN])
        det = ~sto
        bias = np.abs(mean - x)[det]
        want = np.minimum(ax - lo * alpha, hi * alpha - ax)[det]
        assert np.allclose(bias, want, rtol=1e-5, atol=1e-12)
        assert bias.max() > 0.1 * alpha


def decode_int4(codes, n, s):
    q = oracle.unpack(codes, n).astype(np.int64)
    q = np.where(q >= 8, q - 16, q)
    return q * float(s), q


def test_int4_sr_brackets_fixed_points_and_symmetry():
    rng = np.random.default_rng(17)
    x = rng.standard_normal(20000).astype(np.float32)
    mx, _ = oracle.amax(x)
    codes, s, fl = oracle.quant_int4_sr(x, mx, seed=3, n_samples=2)
    assert fl == 0 and s == np.float32(mx) / np.float32(7)
    for p in range(2):
        v, q = decode_int4(codes[p], x.size, s)
        assert np.abs(q).max() == 7 and (np.abs(v - x) < float(s) * (1 + 1e-6)).all()   # floor or ceiling of x/s
        assert (np.sign(v) * np.sign(x) >= 0).all()                                    # never crosses zero
    assert (codes[0] != codes[1]).any()
    # the maximum itself takes +-7 with every seed, on-grid values are fixed points, zero stays zero
    g = (np.arange(-7, 8, dtype=np.float32) * np.float32(0.5))
    g = np.concatenate([g, np.float32([0.0])])
    for seed in range(30):
        cg, sg, _ = oracle.quant_int4_sr(g, np.float32(3.5), seed)
        vg, _ = decode_int4(cg[0], g.size, sg)
        np.testing.assert_array_equal(vg, g.astype(np.float64))
    # Q(-x) = -Q(x) with the same random words
    cn, _, _ = oracle.quant_int4_sr(-x, mx, seed=3)
    vn, _ = decode_int4(cn[0], x.size, s)
    vp, _ = decode_int4(codes[0], x.size, s)
    np.testing.assert_array_equal(vn, -vp)
    # values beyond a smaller caller-supplied maximum clamp to the top level; NaN goes to zero
    y = np.array([9.0, -9.0, np.nan, 7.0, -7.0, 0.25], dtype=np.float32)
    cy, sy, _ = oracle.quant_int4_sr(y, np.float32(7.0), seed=1)
    _, qy = decode_int4(cy[0], y.size, sy)
    assert sy == 1.0 and list(qy[:5]) == [7, -7, 0, 7, -7] and qy[5] in (0, 1)
    for bad, flag in ((0.0, 0), (np.inf, oracle.FLAG_NONFINITE), (1e-35, oracle.FLAG_RANGE)):
        cb, sb, fb = oracle.quant_int4_sr(x[:10], np.float32(bad), seed=1)
        assert sb == 0 and not cb.any() and fb == flag


def test_int4_sr_follows_the_random_word_and_is_exactly_half_at_midpoints():
    x = np.array([0.5, 1.5, -2.5, 0.25, 6.75, -0.125, 3.0], dtype=np.float32)
    mx = np.float32(7.0)                                                    # s = 1: fractions are exact
    frac = np.abs(x) - np.floor(np.abs(x))
    for seed in (0, 9, 123456789):
        codes, s, _ = oracle.quant_int4_sr(x, mx, seed, n_samples=2)
        for p in range(2):
            words = np.array([oracle.random_word(seed, p, i) for i in range(x.size)], dtype=np.float64)
            up = words < frac * 2.0 ** 32
            _, q = decode_int4(codes[p], x.size, s)
            np.testing.assert_array_equal(np.abs(q), np.floor(np.abs(x)) + up)
    # over many seeds a midpoint goes up half of the time, a quarter point a quarter of the time
    ups = np.zeros(x.size)
    S = 4000
    for seed in range(S):
        codes, s, _ = oracle.quant_int4_sr(x, mx, seed)
        _, q = decode_int4(codes[0], x.size, s)
        ups += np.abs(q) > np.floor(np.abs(x))
    p_hat = ups / S
    assert (np.abs(p_hat - frac) < 5 * np.sqrt(frac * (1 - frac) / S) + 1e-12).all()


def test_int4_sr_unbiased_with_table1_variance_and_twice_the_rdn_error():
    """Eq. SR: E[SR(x)] = x and Var = (x - l)(u - x); Table 1: MSE[SR] >= MSE[RDN] - on fractions
    spread evenly over the bins E[f(1-f)] = 1/6 against E[min(f,1-f)^2] = 1/12, a factor of two."""
    rng = np.random.default_rng(23)
    x = rng.uniform(-1, 1, 600).astype(np.float32)
    x[0] = 1.0
    mx, _ = oracle.amax(x)
    S = 1500
    acc = np.zeros(x.size)
    acc2 = np.zeros(x.size)
    s = None
    for seed in range(S):
        codes, s, _ = oracle.quant_int4_sr(x, mx, seed)
        v, _ = decode_int4(codes[0], x.size, s)
        acc += v
        acc2 += (v - x) ** 2
    mean = acc / S
    y = np.abs(x).astype(np.float64) / float(s)
    f = y - np.floor(y)
    var_closed = f * (1 - f) * float(s) ** 2
    z = np.abs(mean - x) / np.sqrt(var_closed / S + 1e-300)
    assert (z[var_closed > 1e-12] < 5.5).all()
    assert abs((acc2 / S).sum() / var_closed.sum() - 1) < 0.05
    crn, srn, _ = oracle.quant_int4(x, mx)
    vr, _ = decode_int4(crn, x.size, srn)
    mse_rdn = ((vr - x) ** 2).mean()
    mse_sr = (acc2 / S).mean()
    assert abs(mse_sr / mse_rdn - 2.0) < 0.2


# ------------------------------------------ in-hindsight range for the INT4 tensors (Sec. 7) ----


def test_int4_hindsight_step_saturates_beyond_the_estimate_and_follows_the_recursion():
    rng = np.random.default_rng(31)
    x = rng.standard_normal(6000).astype(np.float32)
    true_max, _ = oracle.amax(x)
    c_hat = np.float32(float(true_max) / 3)                  # stale, too small estimate
    codes, s, fl, measured, nxt = oracle.quant_int4_hindsight(x, c_hat, 0.1)
    assert fl == 0 and measured == true_max and s == c_hat / np.float32(7)
    assert nxt == oracle.hindsight_next(true_max, c_hat, 0.1)
    val, q = decode_int4(codes, x.size, s)
    beyond = np.abs(x) >= c_hat
    assert beyond.sum() > 50 and (np.abs(q[beyond]) == 7).all()          # saturation, sign kept
    assert (np.sign(val[beyond]) == np.sign(x[beyond])).all()
    inside = ~beyond
    assert (np.abs(val[inside] - x[inside]) <= float(s) / 2 * (1 + 1e-6)).all()   # nearest inside the range
    # with an estimate equal to the maximum the step is the plain quantizer
    plain, s_plain, _ = oracle.quant_int4(x, true_max)
    same, s_same, _, _, _ = oracle.quant_int4_hindsight(x, true_max, 0.1)
    np.testing.assert_array_equal(same, plain)
    assert s_same == s_plain
    # a constant maximum is approached geometrically: error eta^t after t steps
    est = np.float32(1.0)
    for t in range(1, 8):
        _, _, _, m, est = oracle.quant_int4_hindsight(x, est, 0.25)
        assert abs(float(est) - float(true_max)) <= abs(1.0 - float(true_max)) * 0.25 ** t * (1 + 1e-5) + 1e-6
    # a non-finite element is reported, the codes stay defined
    y = x.copy(); y[5] = np.inf
    cy, _, fy, my, ny = oracle.quant_int4_hindsight(y, c_hat, 0.1)
    assert fy & oracle.FLAG_NONFINITE
    _, qy = decode_int4(cy, y.size, s)
    assert qy[5] == 7
