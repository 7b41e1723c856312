"""Pins for the oracle's forward pass: group absmax, scale, Eq. 3 and the BF16 cast (Section 3.3)."""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import gws_oracle as orc
from util import bf16_from_bits, bits_of, f32_of_bits

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---- an independent, definition-level BF16 rounding: exact rationals, nearest of all candidates ----

def _bf16_value(bits: int) -> Fraction:
    sign = -1 if bits & 0x8000 else 1
    e = (bits >> 7) & 0xFF
    m = bits & 0x7F
    assert e != 0xFF
    if e == 0:
        return sign * Fraction(m, 1 << 7) * Fraction(2) ** (-126)
    return sign * (1 + Fraction(m, 1 << 7)) * Fraction(2) ** (e - 127)


_FINITE_POS = [(b, _bf16_value(b)) for b in range(0x0000, 0x7F80)]


def nearest_bf16_even(x: Fraction) -> int:
    """Nearest BF16 to the exact rational x, ties to the even significand (brute force)."""
    neg = x < 0
    a = -x if neg else x
    lo, hi = 0, len(_FINITE_POS) - 1
    while hi - lo > 1:                       # bisect the sorted positive values
        mid = (lo + hi) // 2
        if _FINITE_POS[mid][1] <= a:
            lo = mid
        else:
            hi = mid
    (b0, v0), (b1, v1) = _FINITE_POS[lo], _FINITE_POS[hi]
    if a - v0 < v1 - a:
        b = b0
    elif a - v0 > v1 - a:
        b = b1
    else:
        b = b0 if b0 % 2 == 0 else b1
    return (b | 0x8000) if neg else b


def test_bf16_widening_is_exact():
    for bits in list(range(0, 0x7F80, 37)) + [0x0001, 0x007F, 0x0080, 0x7F7F]:
        assert Fraction(orc.bf16_to_f32(bits)) == _bf16_value(bits)
        assert Fraction(orc.bf16_to_f32(bits | 0x8000)) == -_bf16_value(bits)


def test_cast_matches_bruteforce_nearest_even():
    rng = np.random.default_rng(1)
    xs = np.concatenate([
        rng.standard_normal(300).astype(np.float32) * np.float32(0.02),
        (rng.standard_normal(100) * 1e-3).astype(np.float32),
        np.array([1.00390625, 1.01171875, 1.0039062, 1.0039063, 0.0, 3.3895314e38, 1e-40, 6e-39], np.float32),
    ])
    for x in xs:
        got = orc.f32_to_bf16_rne(float(x))
        want = nearest_bf16_even(Fraction(float(x)))
        assert (got & 0x7FFF) == (want & 0x7FFF) and (got >> 15) == (1 if x < 0 else 0), (float(x), hex(got), hex(want))


def test_cast_matches_library_cast_on_many_values():
    # torch's float32 -> bfloat16 conversion is IEEE round-to-nearest-even: a library routine
    rng = np.random.default_rng(2)
    raw = rng.integers(0, 1 << 32, size=200000, dtype=np.uint64).astype(np.uint32)
    x = raw.view(np.float32)
    x = x[np.isfinite(x)]
    # plus every tie pattern in one binade and values around the overflow threshold
    ties = ((np.arange(0x3F80, 0x4000, dtype=np.uint32) << 16) | 0x8000).view(np.float32)
    edge = np.array([3.3895314e38, 3.3961775e38, 3.4e38, -3.4e38, 1e-45, -1e-45], np.float32)
    x = np.concatenate([x[:50000], ties, edge])
    want = bits_of(torch.from_numpy(x.copy()).to(torch.bfloat16))
    got = orc.f32_array_to_bf16(x)
    assert (got == want).all()
    assert orc.f32_to_bf16_rne(float("inf")) == 0x7F80 and orc.f32_to_bf16_rne(float("-inf")) == 0xFF80
    nan = orc.f32_to_bf16_rne(float("nan"))
    assert (nan & 0x7F80) == 0x7F80 and (nan & 0x7F) != 0


def _hand_cases():
    rows = []
    with open(os.path.join(GOLDEN, "add_then_cast_cases.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            a, b, w, r, e = line.split()
            rows.append((int(a, 16), int(b), int(w, 16), int(r), int(e, 16)))
    return rows


def test_hand_computed_add_then_cast_cases():
    cases = _hand_cases()
    assert len(cases) == 12
    for a_bits, b, w_bits, r, want in cases:
        # a 1x8 group whose absmax element is a_bits; the element under test sits at column 1
        w = np.zeros(8, np.uint16)
        w[0] = a_bits
        w[1] = w_bits
        rr = np.zeros(8, np.int8)
        rr[1] = r
        w_hat, sc = orc.sample_fwd(w, [float(b)], 1, 8, 1, 0, r=rr)
        assert int(w_hat[1]) == want, (hex(a_bits), b, hex(w_bits), r, hex(int(w_hat[1])), hex(want))
        assert int(w_hat[0]) == a_bits
        # and against exact rational arithmetic rounded by brute force (single rounding = double rounding here
        # because every sum in the file is exact in FP32)
        if w_bits != 0x8000:
            exact = _bf16_value(w_bits) + r * _bf16_value(a_bits) * Fraction(2) ** (1 - b)
            assert nearest_bf16_even(exact) == want


def test_4x8_matrix_of_hand_cases():
    # four of the absmax-1.0 hand cases as one 4x8 weight matrix with one group per row:
    # row = [1.0, 0, 0, case element, 0, 0, 0, 0], a different b_t per row
    cases = [c for c in _hand_cases() if c[0] == 0x3F80]
    rows = [(b, w_bits, r, want) for (a_bits, b, w_bits, r, want) in (cases[0], cases[1], cases[3], cases[6])]
    w = np.zeros((4, 8), np.uint16)
    rr = np.zeros((4, 8), np.int8)
    bt = np.zeros(4, np.float32)
    for i, (b, w_bits, r, want) in enumerate(rows):
        w[i, 0] = 0x3F80
        w[i, 3] = w_bits
        rr[i, 3] = r
        bt[i] = b
    w_hat, sc = orc.sample_fwd(w, bt, 4, 8, 1, 0, r=rr.ravel())
    w_hat = w_hat.reshape(4, 8)
    for i, (b, w_bits, r, want) in enumerate(rows):
        assert int(w_hat[i, 3]) == want
        assert sc[i] == np.float32(2.0 ** (1 - b))
    mask = np.ones((4, 8), bool)
    mask[:, 3] = False
    assert (w_hat[mask] == w[mask]).all()


def _random_case(rows, cols, seed, sigma=0.02):
    g = torch.Generator().manual_seed(seed)
    w = (torch.randn(rows, cols, generator=g) * sigma).to(torch.bfloat16)
    return w


@pytest.mark.parametrize("rows,cols,gr,gc", [(4, 8, 1, 0), (6, 64, 1, 32), (5, 72, 1, 32), (64, 96, 32, 32),
                                             (33, 40, 32, 32), (3, 256, 1, 128), (7, 13, 2, 5)])
def test_group_absmax_and_order_against_numpy(rows, cols, gr, gc):
    w = _random_case(rows, cols, 10 + rows)
    a = orc.group_absmax(bits_of(w), rows, cols, gr, gc)
    wf = np.abs(w.float().numpy())
    gcc = cols if gc == 0 else gc
    nbr, nbc = -(-rows // gr), -(-cols // gcc)
    want = np.zeros((nbr, nbc), np.float32)
    for bi in range(nbr):
        for bj in range(nbc):
            want[bi, bj] = wf[bi * gr:(bi + 1) * gr, bj * gcc:(bj + 1) * gcc].max()
    assert a.shape == (nbr * nbc,)
    assert (a == want.ravel()).all()            # row-major group numbering, exact values


def test_transposed_matrix_gives_transposed_square_block_maxima():
    # Section 3.1: square blocks make the grouping commute with transposition
    w = _random_case(64, 96, 3)
    a = orc.group_absmax(bits_of(w), 64, 96, 32, 32).reshape(2, 3)
    at = orc.group_absmax(bits_of(w.t().contiguous()), 96, 64, 32, 32).reshape(3, 2)
    assert (a.T == at).all()


def test_scale_is_exact_for_integer_bits():
    a = np.array([1.0, 0.0625, 0.02001953125, 3.0, 0.0], np.float32)
    for b in range(0, 13):
        s = orc.scale(a, np.full(a.size, b, np.float32))
        assert (s == np.ldexp(a, 1 - b)).all()
    # fractional bit-widths: 2^(1-b) in double, rounded once to float, one float multiply
    b = np.array([4.5, 6.25, 7.75, 0.5, 8.125], np.float32)
    s = orc.scale(a, b)
    p = np.exp2(1.0 - b.astype(np.float64)).astype(np.float32)
    assert (s == a * p).all()


@pytest.mark.parametrize("rows,cols,gr,gc", [(16, 256, 1, 128), (8, 96, 1, 32), (12, 768, 1, 0), (64, 64, 32, 32),
                                             (5, 72, 1, 32)])
def test_forward_against_library_ops_with_generated_noise(rows, cols, gr, gc):
    # Eq. 3 + cast written with torch CPU tensor ops (float32 multiply, add, library RNE cast)
    w = _random_case(rows, cols, 77)
    ng = orc.n_groups(rows, cols, gr, gc)
    bt = torch.randint(4, 10, (ng,), generator=torch.Generator().manual_seed(5)).float().numpy()
    seed, step = 0xABCDEF0123, 17
    w_hat, sc = orc.sample_fwd(bits_of(w), bt, rows, cols, gr, gc, seed=seed, step=step)
    r = torch.from_numpy(orc.noise_r(seed, step, 0, rows * cols).astype(np.float32)).view(rows, cols)
    gcc = cols if gc == 0 else gc
    gi = (torch.arange(rows) // gr)[:, None] * (-(-cols // gcc)) + (torch.arange(cols) // gcc)[None, :]
    absmax = torch.zeros(ng).scatter_reduce(0, gi.reshape(-1), w.float().abs().reshape(-1), "amax")
    scale = absmax * torch.exp2(1.0 - torch.from_numpy(bt))
    want = (w.float() + r * scale[gi]).to(torch.bfloat16)
    assert (sc == scale.numpy()).all()
    assert (w_hat.reshape(rows, cols) == bits_of(want).reshape(rows, cols)).all()
    # a wrong sign, a dropped scale factor or a transposed group map would each change many elements
    changed = (w_hat.reshape(rows, cols) != bits_of(w).reshape(rows, cols)).mean()
    assert 0.15 < changed < 0.40            # about Pr(R != 0) = 0.283


def test_leading_dimension_does_not_change_noise_or_groups():
    rows, cols, ld = 6, 64, 80
    w = _random_case(rows, cols, 4)
    buf = np.full(rows * ld, 0x7FC1, np.uint16)       # padding holds a marker pattern
    buf.reshape(rows, ld)[:, :cols] = bits_of(w).reshape(rows, cols)
    bt = np.full(orc.n_groups(rows, cols, 1, 32), 6, np.float32)
    dense, sc0 = orc.sample_fwd(bits_of(w), bt, rows, cols, 1, 32, seed=3, step=1)
    padded, sc1 = orc.sample_fwd(buf, bt, rows, cols, 1, 32, seed=3, step=1, ld=ld)
    assert (padded.reshape(rows, ld)[:, :cols] == dense.reshape(rows, cols)).all()
    assert (padded.reshape(rows, ld)[:, cols:] == 0x7FC1).all()
    assert (sc0 == sc1).all()


def test_elem_offset_reproduces_the_unsharded_stream():
    # rows 4..7 of an 8-row tensor, sampled alone with elem_offset = 4*cols, equal the same rows sampled in place
    rows, cols = 8, 128
    w = _random_case(rows, cols, 8)
    bt = np.full(rows * 4, 5, np.float32)
    full, _ = orc.sample_fwd(bits_of(w), bt, rows, cols, 1, 32, seed=11, step=2)
    part, _ = orc.sample_fwd(bits_of(w[4:]), bt[16:], 4, cols, 1, 32, seed=11, step=2, elem_offset=4 * cols)
    assert (part == full[4 * cols:]).all()


@pytest.mark.parametrize("b", [4, 6, 8])
def test_lemma1_no_underflow_of_noise_below_9_bits(b):
    # Lemma 1 with BF16 (m = 7) and tau = 0: b_t < 9 => R != 0 changes the stored value (Eq. 5)
    rows, cols = 64, 512
    for sigma in (0.002, 0.02, 3.0):
        w = _random_case(rows, cols, 100 + b, sigma)
        wb = bits_of(w).ravel()
        w_hat, _ = orc.sample_fwd(wb, np.full(rows * 4, b, np.float32), rows, cols, 1, 128, seed=b, step=0)
        r = orc.noise_r(b, 0, 0, rows * cols)
        nz = r != 0
        assert nz.sum() > 5000
        assert (w_hat[nz] != wb[nz]).all()


def test_lemma1_bound_is_sharp_at_9_bits():
    # b_t = 9 violates the strict inequality: a weight of magnitude absmax with R = +-1 can keep its value
    w = np.array([0x3F80] * 8, np.uint16)
    r = np.array([1, -1, 1, 1, 0, 0, 0, 0], np.int8)
    w_hat, _ = orc.sample_fwd(w, [9.0], 1, 8, 1, 0, r=r)
    assert int(w_hat[0]) == 0x3F80          # +2^-8 is a tie, lost to ties-to-even
    assert int(w_hat[1]) != 0x3F80          # -2^-8 lands in the finer binade below


def test_prop2_zero_noise_preserves_weights_and_zero_groups_stay_zero():
    rows, cols = 32, 256
    w = _random_case(rows, cols, 55)
    wb = bits_of(w).ravel()
    wb[5] = 0x8000                           # a negative zero in the data
    bt = np.full(rows * 2, 6, np.float32)
    w_hat, sc = orc.sample_fwd(wb, bt, rows, cols, 1, 128, seed=1, step=1)
    r = orc.noise_r(1, 1, 0, rows * cols)
    z = r == 0
    keep = z.copy()
    keep[5] = False
    assert (w_hat[keep] == wb[keep]).all()
    if z[5]:
        assert w_hat[5] == 0x0000
    # |w_hat - w| <= 2 s + half a BF16 step of the result
    diff = np.abs(f32_of_bits(w_hat).astype(np.float64) - f32_of_bits(wb).astype(np.float64)).reshape(rows, 2, 128)
    s64 = sc.reshape(rows, 2, 1).astype(np.float64)
    absw = np.abs(f32_of_bits(wb).astype(np.float64)).reshape(rows, 2, 128)
    bound = 2 * s64 + 2.0 ** -8 * (absw + 2 * s64)     # half a BF16 step of the largest possible result
    assert (diff <= bound).all()
    zero = np.zeros(256, np.uint16)
    zh, zs = orc.sample_fwd(zero, [4.0, 4.0], 1, 256, 1, 128, seed=1, step=1)
    assert (zh == 0).all() and (zs == 0).all()


def test_table_c1_formulas():
    with open(os.path.join(GOLDEN, "table_c1.txt")) as f:
        rows = [tuple(int(x) for x in l.split()) for l in f if l.strip() and not l.startswith("#")]
    assert len(rows) == 11
    for b, e_w, e_hat, m_hat in rows:
        assert e_w == int(np.ceil(np.log2(b + 1)))
        assert e_hat == int(np.ceil(np.log2(b + 3)))
        assert m_hat == b - 2
