"""Pins for the noise law R (Eq. 9 / Eq. 10, Section 3.4) and the packed format."""
import os
from fractions import Fraction

import numpy as np
import pytest
from scipy import stats

from oracle import gws_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")

# Eq. 10, as exact rationals
P2 = Fraction(3, 4) * Fraction(1, 2 ** 9)                      # each of +-2
P1 = Fraction(3, 4) ** 2 * Fraction(1, 4) * (1 - 2 * P2)       # each of +-1
P0 = 1 - 2 * P1 - 2 * P2
PMF = {-2: P2, -1: P1, 0: P0, 1: P1, 2: P2}


def test_eq10_printed_values():
    rows = {}
    with open(os.path.join(GOLDEN, "eq10_pmf.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, num, den, printed = line.split()
            rows[name] = (Fraction(int(num), int(den)), printed)
    assert rows["p2"][0] == P2 and rows["p1"][0] == P1 and rows["p0"][0] == P0
    assert round(float(1 / P2), 1) == 682.7
    assert round(float(1 / P1), 1) == 7.1
    assert round(float(P0), 3) == 0.717


def test_decode_exhaustive_counts_match_eq10():
    counts = {k: 0 for k in PMF}
    for field in range(1 << 16):
        counts[orc.decode_field(field)] += 1
    # 16 independent fair bits: every probability is a multiple of 2^-16
    for k, p in PMF.items():
        assert Fraction(counts[k], 1 << 16) == p, (k, counts[k])
    assert counts == {-2: 96, -1: 9189, 0: 46966, 1: 9189, 2: 96}


def test_decode_is_and_or_of_the_stated_bits():
    # Eq. 9: the events are ANDs / ORs of independent bits.  Check the bit roles one at a time.
    def bits(**kw):
        v = 0
        for k, on in kw.items():
            if on:
                v |= 1 << int(k[1:])
        return v

    low8 = 0xFF
    assert orc.decode_field(low8 | 1 << 8) == 2 and orc.decode_field(low8 | 1 << 9) == 2
    assert orc.decode_field(low8) == 0                      # needs x8 | x9
    for k in range(8):                                      # every low bit is required
        assert orc.decode_field((low8 & ~(1 << k)) | 3 << 8) == 0
    for a in (10, 11):
        for b in (12, 13):
            assert orc.decode_field(1 << a | 1 << b | 1 << 14) == 1
            assert orc.decode_field(1 << a | 1 << b) == 0            # needs x14
            assert orc.decode_field(1 << a | 1 << b | 1 << 14 | 1 << 15) == -1
    assert orc.decode_field(1 << 10 | 1 << 11 | 1 << 14) == 0         # needs x12 | x13
    assert orc.decode_field(1 << 12 | 1 << 13 | 1 << 14) == 0         # needs x10 | x11
    assert orc.decode_field(low8 | 3 << 8 | 0x7C00) == 2              # |R| = 2 wins over 1
    assert orc.decode_field(low8 | 3 << 8 | 1 << 15) == -2
    assert orc.decode_field(1 << 15) == 0                             # sign alone is zero


def test_closed_form_moments_of_eq10():
    mean = sum(k * p for k, p in PMF.items())
    var = sum(k * k * p for k, p in PMF.items())
    assert mean == 0
    assert var == Fraction(9573, 32768)
    assert sum(abs(k) * p for k, p in PMF.items()) == Fraction(9381, 32768)
    assert sum(k ** 4 * p for k, p in PMF.items()) == Fraction(10725, 32768)
    # Section 3.3: precision of w is annealed with probability <~ 0.317 = Pr(|N(0,1)| > 1)
    assert float(1 - P0) <= 2 * stats.norm.sf(1.0)
    # the law approximates round(N(0,1)/2): P(0) within 0.04 of P(|N| < 1)
    assert abs(float(P0) - (1 - 2 * stats.norm.sf(1.0))) < 0.04


@pytest.fixture(scope="module")
def draws():
    return orc.noise_r(seed=20250511, step=0, first_elem=0, n=10 ** 7).astype(np.int64)


def test_support_symmetry_and_moments_on_1e7_draws(draws):
    n = draws.size
    assert draws.min() >= -2 and draws.max() <= 2
    var = float(Fraction(9573, 32768))
    m4 = float(Fraction(10725, 32768))
    assert abs(draws.mean()) < 5 * np.sqrt(var / n)
    assert abs((draws ** 2).mean() - var) < 5 * np.sqrt((m4 - var ** 2) / n)
    assert abs((draws ** 3).mean()) < 5 * np.sqrt(float(sum(k ** 6 * p for k, p in PMF.items())) / n)
    assert abs(np.abs(draws).mean() - 9381 / 32768) < 5 * np.sqrt((var - (9381 / 32768) ** 2) / n)
    # symmetry: +k and -k counts agree within 5 s.e. of their difference
    for k, p in ((1, P1), (2, P2)):
        d = (draws == k).sum() - (draws == -k).sum()
        assert abs(d) < 5 * np.sqrt(2 * float(p) * n)


def test_ks_and_chi_square_against_eq10_on_1e7_draws(draws):
    n = draws.size
    counts = np.array([(draws == k).sum() for k in (-2, -1, 0, 1, 2)], dtype=np.float64)
    probs = np.array([float(PMF[k]) for k in (-2, -1, 0, 1, 2)])
    # Kolmogorov-Smirnov statistic of a discrete law: sup over the atoms of |F_n - F|,
    # accepted below the Dvoretzky-Kiefer-Wolfowitz bound at alpha = 1e-3
    ks = np.abs(np.cumsum(counts) / n - np.cumsum(probs)).max()
    assert ks < np.sqrt(np.log(2 / 1e-3) / (2 * n))
    chi2 = ((counts - n * probs) ** 2 / (n * probs)).sum()
    assert chi2 < stats.chi2.ppf(1 - 1e-4, df=4)
    # the target is Eq. 10, not the exact rounded normal: that one is rejected by the same data
    z = stats.norm
    exact = np.array([z.cdf(-3), z.cdf(-1) - z.cdf(-3), z.cdf(1) - z.cdf(-1), z.cdf(3) - z.cdf(1), z.sf(3)])
    assert ((counts - n * exact) ** 2 / (n * exact)).sum() > 1e4


def test_independence_between_neighbours_steps_and_seeds(draws):
    n = 1 << 20
    a = draws[:n].astype(np.float64)
    bound = 5 / np.sqrt(n)
    for lag in (1, 2, 7, 8, 9):
        assert abs(np.corrcoef(a[:-lag], a[lag:])[0, 1]) < bound
    other_step = orc.noise_r(20250511, 1, 0, n).astype(np.float64)
    other_seed = orc.noise_r(20250512, 0, 0, n).astype(np.float64)
    assert abs(np.corrcoef(a, other_step)[0, 1]) < bound
    assert abs(np.corrcoef(a, other_seed)[0, 1]) < bound
    # magnitudes are uncorrelated too (no shared bits between |R| of neighbours)
    assert abs(np.corrcoef(np.abs(a[:-1]), np.abs(a[1:]))[0, 1]) < bound


def test_packed_format_sign_magnitude_nibbles():
    seed, step, first, n = 5, 9, 8 * 1000, 8 * 513
    r = orc.noise_r(seed, step, first, n).astype(np.int64)
    p = orc.noise_packed(seed, step, first, n)
    assert p.dtype == np.uint32 and p.size == n // 8           # 0.5 byte per element
    for t in range(8):
        nib = (p >> np.uint32(4 * t)) & np.uint32(0xF)
        mag = (nib & 7).astype(np.int64)
        neg = (nib >> 3).astype(np.int64)
        assert (mag <= 2).all()
        assert ((mag == 0) <= (neg == 0)).all()                # zero is never negative
        assert (np.where(neg == 1, -mag, mag) == r[t::8]).all()
    # ragged tail: unused nibbles of the last word are zero
    q = orc.noise_packed(seed, step, first, 13)
    assert q.size == 2 and (q[1] >> np.uint32(4 * 5)) == 0
    assert q[0] == p[0] and (q[1] & np.uint32(0xFFFFF)) == (p[1] & np.uint32(0xFFFFF))
