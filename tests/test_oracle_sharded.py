"""Pins for the oracle's given-scale forward pass and for the facts a sharded sampling pass rests on.

A tensor cut into shards (Section 3.5 leaves the 2 bytes per parameter of w_hat to training parallelism)
must give the bits of the uncut tensor.  That holds because (a) the noise of an element depends on its
logical index alone, (b) the group maximum is a maximum of partial maxima, and (c) Eq. 4's group sum is a
sum of partial sums.  The tests below check each on the oracle, and pin gwso_sample_fwd_scaled against the
pinned gwso_sample_fwd and against the definition written with numpy and torch's BF16 cast.
"""
import numpy as np
import pytest
import torch

from oracle import gws_oracle as orc
from util import bits_of, f32_of_bits


def _weights(n, seed, sigma=0.02):
    g = torch.Generator().manual_seed(seed)
    return bits_of((torch.randn(n, generator=g) * sigma).to(torch.bfloat16))


@pytest.mark.parametrize("rows,cols,gr,gc", [(6, 64, 1, 16), (5, 40, 1, 0), (64, 64, 32, 32), (7, 24, 2, 9)])
def test_given_scale_forward_equals_the_fused_forward_when_given_its_scale(rows, cols, gr, gc):
    w = _weights(rows * cols, 1)
    ng = orc.n_groups(rows, cols, gr, gc)
    bt = np.random.default_rng(2).integers(4, 10, ng).astype(np.float32)
    want, sc = orc.sample_fwd(w, bt, rows, cols, gr, gc, seed=11, step=3, elem_offset=64)
    got = orc.sample_fwd_scaled(w, sc, rows, cols, gr, gc, seed=11, step=3, elem_offset=64)
    assert np.array_equal(got, want)


def test_given_scale_forward_against_numpy_and_torch_cast():
    rows, cols, gc = 9, 48, 16
    w = _weights(rows * cols, 3, sigma=0.5)
    ng = orc.n_groups(rows, cols, 1, gc)
    # arbitrary positive factors, not derived from w: the function must use exactly what it is given
    sc = np.exp(np.random.default_rng(4).normal(-4.0, 1.0, ng)).astype(np.float32)
    got = orc.sample_fwd_scaled(w, sc, rows, cols, 1, gc, seed=5, step=9, elem_offset=8)
    r = orc.noise_r(5, 9, 8, rows * cols).astype(np.float32)
    per_elem = np.repeat(sc.reshape(rows, cols // gc), gc, axis=1).ravel()
    y = (f32_of_bits(w) + r * per_elem).astype(np.float32)          # product exact, one float32 add
    want = bits_of(torch.from_numpy(y).to(torch.bfloat16))          # library round-to-nearest-even
    assert np.array_equal(got, want)


def test_given_scale_forward_with_zero_scale_returns_w_up_to_the_sign_of_zero():
    w = _weights(64, 6)
    w[:16] = 0x8000            # sixteen negative zeros: R * 0 is -0 for R < 0 and +0 otherwise
    r = orc.noise_r(1, 1, 0, 64)
    assert (r[:16] < 0).any() and (r[:16] >= 0).any()
    got = orc.sample_fwd_scaled(w, np.zeros(4, np.float32), 4, 16, 1, 16, seed=1, step=1)
    want = w.copy()
    want[:16] = np.where(r[:16] < 0, 0x8000, 0x0000)     # IEEE: -0 + -0 = -0, -0 + +0 = +0
    assert np.array_equal(got, want)


def test_given_scale_forward_respects_ld_padding():
    rows, cols, ld = 3, 16, 24
    w = _weights(rows * ld, 7)
    sc = np.array([0.01, 0.02, 0.03], np.float32)
    got = orc.sample_fwd_scaled(w, sc, rows, cols, 1, 0, seed=2, step=0, ld=ld)
    dense = np.concatenate([w[i * ld:i * ld + cols] for i in range(rows)])
    want = orc.sample_fwd_scaled(dense, sc, rows, cols, 1, 0, seed=2, step=0)
    for i in range(rows):
        assert np.array_equal(got[i * ld:i * ld + cols], want[i * cols:(i + 1) * cols])
        assert np.array_equal(got[i * ld + cols:(i + 1) * ld], w[i * ld + cols:(i + 1) * ld])


# ---- the three facts behind sharding, on a flat tensor cut at arbitrary multiples of 8 ------------------

def _cut_points(n, rng, k):
    cuts = np.sort(rng.choice(np.arange(8, n, 8), size=k, replace=False))
    return [0, *cuts.tolist(), n]


@pytest.mark.parametrize("group", [32, 128, 1024])
def test_shards_with_reduced_maxima_give_the_bits_of_the_uncut_tensor(group):
    rng = np.random.default_rng(group)
    n = group * 11
    w = _weights(n, 8)
    n_groups = n // group
    bt = rng.integers(4, 10, n_groups).astype(np.float32)
    want, want_scale = orc.sample_fwd(w, bt, n_groups, group, 1, 0, seed=21, step=4, elem_offset=1 << 20)
    bounds = _cut_points(n, rng, 4)
    # (b) partial maxima per shard and touched group, reduced by max
    absmax = np.zeros(n_groups, np.float32)
    for lo, hi in zip(bounds[:-1], bounds[1:]):
        for g in range(lo // group, (hi - 1) // group + 1):
            a, b = max(lo, g * group), min(hi, (g + 1) * group)
            part = orc.group_absmax(w[a:b], 1, b - a)[0]
            absmax[g] = max(absmax[g], part)
    assert np.array_equal(absmax, orc.group_absmax(w, n_groups, group))
    sc = orc.scale(absmax, bt)
    assert np.array_equal(sc, want_scale)
    # (a) every shard samples its own run of logical indices
    got = np.empty_like(w)
    for lo, hi in zip(bounds[:-1], bounds[1:]):
        for g in range(lo // group, (hi - 1) // group + 1):
            a, b = max(lo, g * group), min(hi, (g + 1) * group)
            got[a:b] = orc.sample_fwd_scaled(w[a:b], sc[g:g + 1], 1, b - a, seed=21, step=4, elem_offset=(1 << 20) + a)
    assert np.array_equal(got, want)


def test_partial_group_gradients_add_up_to_the_uncut_gradient():
    group, n_groups = 256, 6
    n = group * n_groups
    rng = np.random.default_rng(5)
    g = _weights(n, 9, sigma=1e-4)
    sc = np.exp(rng.normal(-6.0, 0.5, n_groups)).astype(np.float32)
    _, want = orc.sample_bwd(g, sc, n_groups, group, 1, 0, seed=3, step=7, elem_offset=4096)
    bounds = _cut_points(n, rng, 5)
    total = np.zeros(n_groups, np.float64)
    bound = np.zeros(n_groups, np.float64)
    for lo, hi in zip(bounds[:-1], bounds[1:]):
        for k in range(lo // group, (hi - 1) // group + 1):
            a, b = max(lo, k * group), min(hi, (k + 1) * group)
            _, part = orc.sample_bwd(g[a:b], sc[k:k + 1], 1, b - a, seed=3, step=7, elem_offset=4096 + a)
            total[k] += float(part[0])
            r = orc.noise_r(3, 7, 4096 + a, b - a).astype(np.float64)
            bound[k] += np.abs(f32_of_bits(g[a:b]).astype(np.float64) * r).sum()
    # each part is rounded to float32 once: the sum differs from the uncut value by a few float32 roundings
    tol = 4 * 2.0 ** -24 * np.log(2.0) * sc * bound + 1e-45
    assert np.all(np.abs(total - want.astype(np.float64)) <= tol)
    assert np.any(want != 0)


def test_factor_of_a_whole_group_is_the_largest_of_its_parts_factors():
    # fl32(a * p) is non-decreasing in a for p > 0, so reducing the parts' FACTORS by max gives the factor of the
    # reduced maximum exactly, for integer and fractional bit-widths alike (each part uses the same b)
    rng = np.random.default_rng(17)
    n_groups, n_parts = 4000, 5
    parts = np.abs(rng.normal(0.0, 0.05, (n_parts, n_groups))).astype(np.float32)
    parts[:, :50] = np.float32(2.0 ** -127) * rng.integers(0, 4, (n_parts, 50)).astype(np.float32)   # subnormal maxima
    bt = np.where(rng.random(n_groups) < 0.5, rng.integers(2, 12, n_groups), rng.uniform(2.0, 12.0, n_groups)).astype(np.float32)
    of_parts = np.stack([orc.scale(parts[k], bt) for k in range(n_parts)]).max(axis=0)
    of_whole = orc.scale(parts.max(axis=0), bt)
    assert np.array_equal(of_parts.view(np.uint32), of_whole.view(np.uint32))
