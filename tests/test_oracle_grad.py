"""Pins for the oracle's backward pass (Eq. 4)."""
import numpy as np
import pytest
import torch

from oracle import gws_oracle as orc
from util import bits_of, f32_of_bits

LN2 = float(np.log(2.0))


def _uncast_forward(w, b, r, gr, gc):
    """Eq. 3 in float64 without the cast: the differentiable map the paper takes gradients of."""
    rows, cols = w.shape
    out = np.empty_like(w)
    gcc = cols if gc == 0 else gc
    k = 0
    for bi in range(0, rows, gr):
        for bj in range(0, cols, gcc):
            blk = (slice(bi, bi + gr), slice(bj, bj + gcc))
            out[blk] = w[blk] + r[blk] * np.abs(w[blk]).max() * 2.0 ** (1.0 - b[k])
            k += 1
    return out


@pytest.mark.parametrize("gr,gc", [(1, 0), (1, 4), (2, 2)])
def test_finite_differences_on_4x8(gr, gc):
    rows, cols = 4, 8
    rng = np.random.default_rng(7)
    w_t = (torch.from_numpy(rng.standard_normal((rows, cols))).float() * 0.02).to(torch.bfloat16)
    c_t = (torch.from_numpy(rng.standard_normal((rows, cols))).float() * 1e-2).to(torch.bfloat16)   # dL/dw_hat
    w = w_t.double().numpy()
    c = c_t.double().numpy()
    ng = orc.n_groups(rows, cols, gr, gc)
    b = rng.integers(4, 10, ng).astype(np.float64) + 0.25          # non-integer on purpose
    r = rng.integers(-2, 3, (rows, cols)).astype(np.float64)
    loss = lambda w_, b_: float((c * _uncast_forward(w_, b_, r, gr, gc)).sum())

    absmax = orc.group_absmax(bits_of(w_t), rows, cols, gr, gc)
    scale = orc.scale(absmax, b.astype(np.float32))
    gw, gbt = orc.sample_bwd(bits_of(c_t), scale, rows, cols, gr, gc, r=r.astype(np.int8).ravel())

    # dL/db_t: central differences match Eq. 4
    h = 1e-5
    for k in range(ng):
        bp, bm = b.copy(), b.copy()
        bp[k] += h
        bm[k] -= h
        fd = (loss(w, bp) - loss(w, bm)) / (2 * h)
        assert abs(fd - float(gbt[k])) <= 1e-6 * max(1.0, abs(fd)) + 1e-7 * abs(fd) + 1e-9, (k, fd, gbt[k])

    # dL/dw: identity, except at the arg-max element of each group where the true derivative has the
    # extra term sign(w_max) * 2^(1-b) * sum(c R) that the paper drops (the max's gradient is taken as 0)
    assert (gw == bits_of(c_t).ravel()).all()
    gcc = cols if gc == 0 else gc
    hw = 1e-7
    for i in range(rows):
        for j in range(cols):
            wp, wm = w.copy(), w.copy()
            wp[i, j] += hw
            wm[i, j] -= hw
            fd = (loss(wp, b) - loss(wm, b)) / (2 * hw)
            k = (i // gr) * (-(-cols // gcc)) + j // gcc
            blk = (slice((i // gr) * gr, (i // gr) * gr + gr), slice((j // gcc) * gcc, (j // gcc) * gcc + gcc))
            is_argmax = abs(w[i, j]) == np.abs(w[blk]).max()
            if is_argmax:
                dropped = np.sign(w[i, j]) * 2.0 ** (1.0 - b[k]) * float((c[blk] * r[blk]).sum())
                assert abs(fd - (c[i, j] + dropped)) < 1e-6
            else:
                assert abs(fd - c[i, j]) < 1e-6


def test_constant_upstream_gradient_closed_form():
    # g == c on a group  =>  grad_b = -ln2 * s * c * sum(R), an integer sum
    rows, cols, c = 8, 256, 0.015625
    g = torch.full((rows, cols), c, dtype=torch.bfloat16)
    scale = np.linspace(0.001, 0.004, rows * 2).astype(np.float32)
    seed, step = 42, 3
    _, gbt = orc.sample_bwd(bits_of(g), scale, rows, cols, 1, 128, seed=seed, step=step)
    r = orc.noise_r(seed, step, 0, rows * cols).astype(np.int64).reshape(rows * 2, 128)
    want = (-LN2 * scale.astype(np.float64) * c * r.sum(axis=1)).astype(np.float32)
    assert (gbt == want).all()
    assert (r.sum(axis=1) != 0).any()


@pytest.mark.parametrize("rows,cols,gr,gc", [(16, 256, 1, 128), (8, 96, 1, 32), (6, 768, 1, 0), (64, 64, 32, 32),
                                             (5, 72, 1, 32)])
def test_backward_against_numpy_float64(rows, cols, gr, gc):
    gen = torch.Generator().manual_seed(9)
    g = (torch.randn(rows, cols, generator=gen) * 1e-4).to(torch.bfloat16)
    ng = orc.n_groups(rows, cols, gr, gc)
    scale = (torch.rand(ng, generator=gen) * 1e-2).numpy().astype(np.float32)
    seed, step = 1234567, 8
    gw, gbt = orc.sample_bwd(bits_of(g), scale, rows, cols, gr, gc, seed=seed, step=step)
    assert (gw == bits_of(g).ravel()).all()
    r = orc.noise_r(seed, step, 0, rows * cols).astype(np.float64).reshape(rows, cols)
    prod = g.double().numpy() * r
    gcc = cols if gc == 0 else gc
    want = []
    for bi in range(0, rows, gr):
        for bj in range(0, cols, gcc):
            want.append(prod[bi:bi + gr, bj:bj + gcc].sum())
    want = -LN2 * scale.astype(np.float64) * np.array(want)
    assert np.allclose(gbt, want, rtol=1e-6, atol=0)
    assert (np.sign(gbt[want != 0]) == np.sign(want[want != 0])).all()


def test_forward_and_backward_use_the_same_noise():
    # R implied by the forward pass equals R used by the backward pass (Section 3.6)
    rows, cols = 16, 256
    gen = torch.Generator().manual_seed(3)
    w = (torch.randn(rows, cols, generator=gen) * 0.02).to(torch.bfloat16)
    bt = np.full(rows * 2, 4, np.float32)
    seed, step = 77, 5
    w_hat, sc = orc.sample_fwd(bits_of(w), bt, rows, cols, 1, 128, seed=seed, step=step)
    # with b_t = 4 the noise step is large against BF16 rounding: recover R = round((w_hat - w) / s)
    d = f32_of_bits(w_hat).astype(np.float64) - f32_of_bits(bits_of(w).ravel()).astype(np.float64)
    r_implied = np.rint(d.reshape(rows * 2, 128) / sc.reshape(-1, 1).astype(np.float64)).astype(np.int64)
    # backward with g = one-hot picks out single R values: use g == 1 on one element per group
    for col in (0, 17, 127):
        g = torch.zeros(rows, cols, dtype=torch.bfloat16)
        g.view(rows * 2, 128)[:, col] = 1.0
        ones = np.ones(rows * 2, np.float32)
        _, gbt = orc.sample_bwd(bits_of(g), ones, rows, cols, 1, 128, seed=seed, step=step)
        r_bwd = np.rint(gbt.astype(np.float64) / -LN2).astype(np.int64)
        assert (r_bwd == r_implied[:, col]).all()
    assert (orc.noise_r(seed, step, 0, rows * cols).reshape(rows * 2, 128) == r_implied).all()
