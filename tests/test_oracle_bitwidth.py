"""Pins of the oracle's bit-width parametrisation (Eq. 11), bit-width loss (Eq. 12) and layer seeds (Section 3.6)."""
import numpy as np

from oracle import gws_oracle as orc


def test_eq11_end_points_and_linearity():
    bi = np.array([1.0, 0.0, 0.5, 0.25, 2.0, -1.0], np.float32)
    bt = orc.bitwidth(bi, 6.0, 4.0)
    # b_i = 1 is the initial bit-width, b_i = 0 the target (what weight decay pulls towards); linear in between
    assert bt.tolist() == [6.0, 4.0, 5.0, 4.5, 8.0, 2.0]
    assert orc.bitwidth(bi, 8.0, 6.0).tolist() == [8.0, 6.0, 7.0, 6.5, 10.0, 4.0]
    assert orc.bitwidth(bi, 4.0, 4.0).tolist() == [4.0] * 6            # b_init = b_target: b_i has no effect


def test_eq11_rounds_once_per_operation_in_fp32():
    rng = np.random.default_rng(0)
    bi = rng.uniform(-0.5, 1.5, 20000).astype(np.float32)
    b_init, b_target = np.float32(6.3), np.float32(3.9)
    delta = np.float32(b_init - b_target)
    want = (b_target + (bi * delta).astype(np.float32)).astype(np.float32)     # numpy float32 ops round once each
    got = orc.bitwidth(bi, float(b_init), float(b_target))
    assert (got.view(np.uint32) == want.view(np.uint32)).all()
    # and it is not the double-precision result rounded at the end (that differs in some last bits)
    dbl = (float(b_target) + bi.astype(np.float64) * (float(b_init) - float(b_target))).astype(np.float32)
    assert (got != dbl).any() and np.abs(got - dbl).max() <= 1e-6


def test_eq12_loss_is_the_mean_absolute_distance():
    assert orc.bitwidth_loss(np.array([6.0, 4.0, 5.0, 3.0], np.float32), 4.0) == (2 + 0 + 1 + 1) / 4
    assert orc.bitwidth_loss(np.full(1000, 4.0, np.float32), 4.0) == 0.0
    bt = np.random.default_rng(1).uniform(2, 9, 4096).astype(np.float32)
    assert abs(orc.bitwidth_loss(bt, 4.0) - np.abs(bt.astype(np.float64) - 4.0).mean()) < 1e-12


def test_gradient_matches_finite_differences_of_the_total_loss():
    # L'(b_i) = sum_k c_k * b_t,k + lam * mean_k |b_t,k - b_target|  with  b_t = Eq. 11 (evaluated in float64 here, so
    # the difference quotient is clean); dL/db_t = c.
    rng = np.random.default_rng(2)
    m, b_init, b_target, lam = 64, 6.0, 4.0, 0.37
    bi = rng.uniform(-0.8, 1.2, m)
    c = rng.normal(0, 1, m)

    def total(b):
        bt = b_target + b * (b_init - b_target)
        return float((c * bt).sum() + lam * np.abs(bt - b_target).mean())

    bt32 = orc.bitwidth(bi.astype(np.float32), b_init, b_target)
    got = orc.bitwidth_grad(c.astype(np.float32), bt32, b_init, b_target, lam)
    h = 1e-6
    for k in range(m):
        e = np.zeros(m)
        e[k] = h
        fd = (total(bi + e) - total(bi - e)) / (2 * h)
        assert abs(got[k] - fd) < 1e-5 * max(1.0, abs(fd)), (k, got[k], fd)
    # the pieces: without lambda only the chain-rule factor of Eq. 11 remains; at b_t == b_target the |.| term adds 0
    plain = orc.bitwidth_grad(c.astype(np.float32), bt32, b_init, b_target, 0.0)
    assert np.allclose(plain, (b_init - b_target) * c.astype(np.float32).astype(np.float64), rtol=0, atol=1e-12)
    at_target = orc.bitwidth_grad(np.zeros(4, np.float32), np.full(4, 4.0, np.float32), 6.0, 4.0, 1.0)
    assert (at_target == 0).all()
    above = orc.bitwidth_grad(np.zeros(4, np.float32), np.array([5, 3, 4.5, 3.5], np.float32), 6.0, 4.0, 2.0)
    assert above.tolist() == [1.0, -1.0, 1.0, -1.0]                     # (6 - 4) * 2 / 4 * sign


def test_layer_seeds_are_philox_outputs_distinct_and_balanced():
    user = 0x0123456789ABCDEF
    for layer in (0, 1, 77, 1 << 33):
        o = orc.philox4x32_10([layer & 0xFFFFFFFF, layer >> 32, 0, 0], [user & 0xFFFFFFFF, user >> 32])
        assert orc.layer_seed(user, layer) == int(o[0]) | (int(o[1]) << 32)
    seeds = [orc.layer_seed(user, k) for k in range(4096)]
    assert len(set(seeds)) == 4096 and len({orc.layer_seed(user + 1, k) for k in range(64)} & set(seeds)) == 0
    bits = np.unpackbits(np.array(seeds, np.uint64).view(np.uint8))
    assert abs(bits.mean() - 0.5) < 5 * 0.5 / np.sqrt(bits.size)
    # independent layers: the noise of two layers at the same step and element index is uncorrelated
    a = orc.noise_r(seeds[0], 3, 0, 200000).astype(np.float64)
    b = orc.noise_r(seeds[1], 3, 0, 200000).astype(np.float64)
    assert abs(np.corrcoef(a, b)[0, 1]) < 5 / np.sqrt(a.size)
