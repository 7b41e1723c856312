"""Pins for the comparison noises of the oracle: the "DiffQ" BF16 U(-0.5, 0.5) noise (Section 4, first paragraph) and the
Box-Muller rounded normal ("bm" in the forward benchmark; Section 3.4 names the transform).  Nothing here uses the GPU."""
import math
from fractions import Fraction

import numpy as np

from oracle import gws_oracle as orc

N = 2_000_000


def _bf16_value(bits: int) -> Fraction:
    sign, exp, man = bits >> 15, (bits >> 7) & 0xFF, bits & 0x7F
    mag = Fraction(man, 128) * Fraction(2) ** (-126) if exp == 0 else (1 + Fraction(man, 128)) * Fraction(2) ** (exp - 127)
    return -mag if sign else mag


def test_uniform_noise_is_the_nearest_bf16_number_to_the_midpoint_rule():
    # element e of a vector uses the 16-bit field at bits [16 (e & 1), +16) of word (e >> 1) & 3; the exact value is
    # (x + 1/2) / 2^16 - 1/2, and the stored pattern must be its nearest BF16 neighbour (ties to the even mantissa),
    # found here by exact rational comparison with the two patterns around it
    seed, step = 0xABCDEF, 11
    words = orc.philox_words(seed, step, 0, 512).reshape(-1, 4)
    got = orc.noise_uniform(seed, step, 0, 512 * 8)
    for e in list(range(0, 64)) + list(range(4000, 4096)):
        x = (int(words[e >> 3][(e & 7) >> 1]) >> (16 * (e & 1))) & 0xFFFF
        exact = Fraction(2 * x + 1 - 65536, 131072)
        bits = int(got[e])
        v = _bf16_value(bits)
        assert abs(v - exact) <= Fraction(1, 2) ** 8 * abs(exact) + Fraction(1, 2) ** 140      # half an ulp is at most 2^-8 of the value
        for other in (bits - 1, bits + 1):
            if (other & 0x7FFF) < 0x7F80 and (other >> 15) == (bits >> 15) and other >= 0:
                d_here, d_other = abs(v - exact), abs(_bf16_value(other) - exact)
                assert d_here < d_other or (d_here == d_other and bits % 2 == 0), (e, hex(bits))


def test_uniform_noise_is_symmetric_bounded_and_has_the_uniform_moments():
    u = orc.noise_uniform(3, 4, 0, N)
    f = (u.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    assert f.min() >= -0.5 and f.max() <= 0.5
    se = math.sqrt(1.0 / 12.0 / N)
    assert abs(f.mean()) < 5 * se
    assert abs(f.var() - 1.0 / 12.0) < 5 * math.sqrt((1.0 / 80.0 - 1.0 / 144.0) / N) + 1e-5     # Var(U^2) = 1/80 - 1/144; 1e-5: BF16 rounding
    # as many values on one side of zero as on the other, and a KS test against the uniform law
    assert abs((f > 0).mean() - 0.5) < 5 * 0.5 / math.sqrt(N)
    xs = np.sort(f)
    ks = np.abs(np.arange(1, N + 1) / N - (xs + 0.5)).max()
    assert ks < math.sqrt(math.log(2 / 1e-3) / (2 * N)) + 2.0 ** -9                                # + the BF16 grid's coarsest step (2^-9 near 0.5)
    # neighbouring elements, steps and seeds are uncorrelated
    g = (orc.noise_uniform(3, 5, 0, N).astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    for a, b in ((f[:-1], f[1:]), (f, g)):
        assert abs(np.corrcoef(a, b)[0, 1]) < 5 / math.sqrt(N)


def _phi(x):
    return 0.5 * (1.0 + math.erf(x / math.sqrt(2.0)))


def test_box_muller_normals_pass_ks_and_moment_tests():
    z = orc.noise_bm_z(9, 1, 0, N)
    assert np.abs(z).max() <= math.sqrt(2 * 24 * math.log(2)) + 1e-9           # u1 >= 2^-24 bounds the radius
    xs = np.sort(z)
    cdf = np.array([_phi(v) for v in xs[::200]])
    emp = (np.arange(N)[::200] + 0.5) / N
    assert np.abs(cdf - emp).max() < math.sqrt(math.log(2 / 1e-3) / (2 * N)) + 1e-4
    assert abs(z.mean()) < 5 / math.sqrt(N)
    assert abs(z.var() - 1.0) < 5 * math.sqrt(2.0 / N)
    assert abs((z ** 4).mean() - 3.0) < 5 * math.sqrt(96.0 / N)
    # the two normals of a pair, neighbouring pairs and consecutive steps are uncorrelated
    z2 = orc.noise_bm_z(9, 2, 0, N)
    for a, b in ((z[0::2], z[1::2]), (z[:-2], z[2:]), (z, z2)):
        assert abs(np.corrcoef(a, b)[0, 1]) < 5 / math.sqrt(a.size)


def test_box_muller_r_is_the_rounded_half_normal_with_its_exact_law():
    z = orc.noise_bm_z(5, 0, 0, N)
    r = orc.noise_bm_r(5, 0, 0, N)
    assert np.array_equal(r, np.rint(0.5 * z).astype(np.int8))               # numpy's rint also rounds ties to even
    assert set(np.unique(r)) <= {-3, -2, -1, 0, 1, 2, 3}
    # P(R = k) = Phi(2k + 1) - Phi(2k - 1): 0.6827 / 0.1573 / 0.00135 / 2.9e-7, the law Eq. 10 approximates
    for k in (0, 1, 2):
        p = _phi(2 * k + 1) - _phi(2 * k - 1)
        for sign in ((1,) if k == 0 else (1, -1)):
            freq = (r == sign * k).mean()
            assert abs(freq - p) < 5 * math.sqrt(p * (1 - p) / N), (k, sign, freq, p)
    assert (np.abs(r) == 3).mean() < 1e-5
    # first elements of a run reproduce when asked for one by one, at any offset (the counter is the element index)
    assert np.array_equal(orc.noise_bm_r(5, 0, 1000, 64), r[1000:1064])
    assert np.array_equal(orc.noise_bm_z(5, 0, 7, 9), z[7:16])


def test_forward_with_a_bf16_noise_reduces_to_the_pinned_forward_when_the_noise_is_r():
    # with u = float(R) (exactly representable) the comparison forward must give the bits of the method's own forward
    rng = np.random.default_rng(2)
    rows, cols, gc = 12, 256, 128
    w = (rng.integers(0, 2 ** 16, size=rows * cols, dtype=np.uint16) & 0xBFFF).astype(np.uint16)
    w[5] = 0x8000                                                           # -0
    bt = rng.integers(4, 10, size=rows * cols // gc).astype(np.float32)
    r = orc.noise_r(77, 3, 0, rows * cols)
    as_bf16 = {0: 0x0000, 1: 0x3F80, -1: 0xBF80, 2: 0x4000, -2: 0xC000}
    u = np.array([as_bf16[int(v)] for v in r], dtype=np.uint16)
    got_hat, got_scale = orc.sample_fwd_bf16_noise(w, bt, u, rows, cols, 1, gc)
    want_hat, want_scale = orc.sample_fwd(w, bt, rows, cols, 1, gc, seed=77, step=3)
    assert np.array_equal(got_hat, want_hat) and np.array_equal(got_scale.view(np.uint32), want_scale.view(np.uint32))
    # zero noise leaves every weight as it is (-0 becomes +0, as in the method's forward)
    zero_hat, _ = orc.sample_fwd_bf16_noise(w, bt, np.zeros_like(u), rows, cols, 1, gc)
    keep = w != 0x8000
    assert np.array_equal(zero_hat[keep], w[keep]) and (zero_hat[~keep] == 0).all()
    # a hand case: absmax 1, b = 4 -> s = 0.125; w = 0.5, u = 0.25 -> 0.53125 (0x3F08)
    w1 = np.array([0x3F80, 0x3F00] + [0] * 6, dtype=np.uint16)
    u1 = np.array([0, 0x3E80] + [0] * 6, dtype=np.uint16)
    hat1, sc1 = orc.sample_fwd_bf16_noise(w1, np.array([4.0], np.float32), u1, 1, 8, 1, 8)
    assert sc1[0] == 0.125 and hat1[1] == 0x3F08 and hat1[0] == 0x3F80
