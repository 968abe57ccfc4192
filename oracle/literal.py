"""Literal, exact-rational transcription of the paper's gradient quantizer.
TEST INFRASTRUCTURE ONLY (used to pin ``luq_oracle.c``).

The two stages are applied one after the other exactly as the paper states
them, each with its own randomness, and the outcome distribution is returned
as exact fractions:

* stochastic underflow T_alpha (Eq. StochasticPruning): |x| >= alpha passes;
  otherwise sign(x)*alpha with probability |x|/alpha, else 0;
* logarithmic stochastic rounding Q_alpha (Eq. unbiasedFpQ) on the bins
  [2^(n-1) alpha, 2^n alpha]: up with probability (x - 2^(n-1) alpha)/(2^(n-1) alpha).

Also the deterministic rules used as pins: round-to-nearest in a bin and the
closed forms of Table 1.
"""
from __future__ import annotations

from fractions import Fraction


def stochastic_underflow(x: Fraction, alpha: Fraction) -> dict:
    """Distribution {value: probability} of T_alpha(x)."""
    if abs(x) >= alpha:
        return {x: Fraction(1)}
    p = abs(x) / alpha
    sign = 1 if x > 0 else -1
    out = {}
    if p > 0:
        out[sign * alpha] = p
    if p < 1:
        out[Fraction(0)] = out.get(Fraction(0), Fraction(0)) + (1 - p)
    return out


def log_stochastic_round(y: Fraction, alpha: Fraction, kmax: int) -> dict:
    """Distribution of Q_alpha(y) for y = 0 or alpha <= |y| <= 2^kmax alpha."""
    if y == 0:
        return {Fraction(0): Fraction(1)}
    a = abs(y)
    sign = 1 if y > 0 else -1
    top = alpha * 2 ** kmax
    if a >= top:  # the largest level is the tensor maximum: nothing lies above it
        return {sign * top: Fraction(1)}
    n = 1
    while not (alpha * 2 ** (n - 1) <= a < alpha * 2 ** n):
        n += 1
    lo, hi = alpha * 2 ** (n - 1), alpha * 2 ** n
    p_up = (a - lo) / lo
    out = {}
    if p_up < 1:
        out[sign * lo] = 1 - p_up
    if p_up > 0:
        out[sign * hi] = p_up
    return out


def luq_distribution(x: Fraction, alpha: Fraction, kmax: int) -> dict:
    """Distribution of X_q = Q_alpha(T_alpha(x)) (law of total probability)."""
    out = {}
    for y, py in stochastic_underflow(x, alpha).items():
        for z, pz in log_stochastic_round(y, alpha, kmax).items():
            out[z] = out.get(z, Fraction(0)) + py * pz
    return out


def expectation(dist: dict) -> Fraction:
    return sum((v * p for v, p in dist.items()), Fraction(0))


def variance(dist: dict) -> Fraction:
    m = expectation(dist)
    return sum(((v - m) ** 2 * p for v, p in dist.items()), Fraction(0))


def round_nearest_in_bin(x, lo, hi):
    """RDN inside a bin [lo, hi] (Sec. 3.1)."""
    return lo if (x - lo) <= (hi - x) else hi


def table1(x, lo, hi):
    """Closed forms of Table 1: (bias_rdn, var_rdn, mse_rdn, bias_sr, var_sr, mse_sr)."""
    b = min(x - lo, hi - x)
    v = (x - lo) * (hi - x)
    return b, 0, b * b, 0, v, v
