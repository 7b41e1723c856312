"""Pins for the oracle's MX emission of w_hat (Section 3.1 MXFP target, Table C.1 datatypes, the square-block sharing
rule of Section 3.2): element grids against their definition and a library cast, rounding against brute force, the
shared exponent against its formula, and the properties the emission must have."""
import math

import numpy as np
import pytest
import torch

from oracle import gws_oracle as orc
from util import bits_of, f32_of_bits

E4M3, E3M2, E3M4 = orc.MX_E4M3, orc.MX_E3M2, orc.MX_E3M4
FORMATS = {E4M3: dict(width=8, mbits=3, bias=7, emax=8, max=448.0, finite=[c for c in range(256) if c & 0x7F != 0x7F]),
           E3M2: dict(width=6, mbits=2, bias=3, emax=4, max=28.0, finite=list(range(64))),
           E3M4: dict(width=8, mbits=4, bias=3, emax=4, max=31.0, finite=list(range(256)))}


def test_element_grids_match_their_definition():
    assert orc.mx_decode(E4M3, 0x7E) == 448.0 and orc.mx_decode(E4M3, 0x38) == 1.0
    assert orc.mx_decode(E4M3, 0x08) == 2.0 ** -6 and orc.mx_decode(E4M3, 0x01) == 2.0 ** -9
    assert orc.mx_decode(E4M3, 0xFE) == -448.0 and math.isnan(orc.mx_decode(E4M3, 0x7F))
    assert orc.mx_decode(E3M2, 0x1F) == 28.0 and orc.mx_decode(E3M2, 0x0C) == 1.0
    assert orc.mx_decode(E3M2, 0x04) == 0.25 and orc.mx_decode(E3M2, 0x01) == 0.0625 and orc.mx_decode(E3M2, 0x3F) == -28.0
    assert orc.mx_decode(E3M4, 0x7F) == 31.0 and orc.mx_decode(E3M4, 0x30) == 1.0 and orc.mx_decode(E3M4, 0x10) == 0.25
    assert orc.mx_decode(E3M4, 0x01) == 2.0 ** -6 and orc.mx_decode(E3M4, 0xFF) == -31.0
    for fmt, f in FORMATS.items():
        half = 1 << (f["width"] - 1)
        pos = [orc.mx_decode(fmt, c) for c in f["finite"] if c < half]
        assert pos == sorted(pos) and len(set(pos)) == len(pos) and pos[0] == 0.0 and pos[-1] == f["max"]
        for c in f["finite"]:
            assert orc.mx_encode(fmt, orc.mx_decode(fmt, c)) == c         # every grid point encodes to itself


def _nearest_even_code(fmt, x):
    """Brute force over the whole grid: nearest value, ties to the code with an even mantissa, sign of x kept."""
    f = FORMATS[fmt]
    half = 1 << (f["width"] - 1)
    best, best_d = None, None
    for c in f["finite"]:
        if c >= half:
            continue
        d = abs(abs(x) - orc.mx_decode(fmt, c))
        if best is None or d < best_d or (d == best_d and c % 2 == 0):
            best, best_d = c, d
    return best | (half if math.copysign(1.0, x) < 0 else 0)


@pytest.mark.parametrize("fmt", [E4M3, E3M2, E3M4])
def test_rounding_is_nearest_even_with_clamping(fmt):
    f = FORMATS[fmt]
    half = 1 << (f["width"] - 1)
    grid = sorted(orc.mx_decode(fmt, c) for c in f["finite"] if c < half)
    xs = [0.0, -0.0, f["max"] * 1.01, f["max"] * 4, -f["max"] * 1e6, grid[1] / 2, grid[1] / 2 * 1.0001, grid[1] / 2 * 0.9999, grid[1] / 4]
    for a, b in zip(grid[:-1], grid[1:]):
        xs += [(a + b) / 2, (a + b) / 2 * (1 + 1e-9), (a + b) / 2 * (1 - 1e-9), a + (b - a) * 0.3, -(a + b) / 2, -(a + (b - a) * 0.7)]
    xs += list(np.random.default_rng(1).normal(0, f["max"] / 3, 2000)) + list(np.random.default_rng(2).normal(0, grid[3], 2000))
    for x in xs:
        want = _nearest_even_code(fmt, x) if abs(x) <= f["max"] else ((half if x < 0 else 0) | max(c for c in f["finite"] if c < half))
        assert orc.mx_encode(fmt, x) == want, x


def test_e4m3_rounding_matches_the_library_cast():
    rng = np.random.default_rng(3)
    x = np.concatenate([rng.normal(0, 100, 20000), rng.normal(0, 0.01, 20000), rng.uniform(-448, 448, 20000),
                        np.ldexp(rng.integers(-15, 16, 5000).astype(np.float64), -10)]).astype(np.float32)
    x = x[np.abs(x) <= 448.0]
    lib = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    mine = np.array([orc.mx_encode(E4M3, float(v)) for v in x], np.uint8)
    assert np.array_equal(mine, lib)


def _w_hat(rows, cols, seed, sigma=0.02):
    g = torch.Generator().manual_seed(seed)
    t = torch.randn(rows, cols, generator=g) * sigma
    t[0, :3] = torch.tensor([0.0, -0.0, sigma * 8])
    return bits_of(t.to(torch.bfloat16))


@pytest.mark.parametrize("fmt", [E4M3, E3M2, E3M4])
@pytest.mark.parametrize("rows,cols,gr,gc", [(4, 128, 1, 32), (3, 256, 1, 128), (5, 96, 1, 0), (64, 64, 32, 32)])
def test_emission_properties(fmt, rows, cols, gr, gc):
    f = FORMATS[fmt]
    w = _w_hat(rows, cols, 11)
    w.reshape(rows, cols)[-1, -32:] = 0                       # an all-zero vector
    codes, scales = orc.mx_emit(w, rows, cols, gr, gc, fmt)
    vals = f32_of_bits(w).astype(np.float64).reshape(rows, cols)
    gcc = cols if gc == 0 else gc
    half = 1 << (f["width"] - 1)
    deq = np.array([orc.mx_decode(fmt, int(c)) for c in codes]).reshape(rows, cols)
    sc = scales.reshape(rows, cols // 32)
    for i0 in range(0, rows, gr):
        for j0 in range(0, cols, gcc):
            blk = vals[i0:i0 + gr, j0:j0 + gcc]
            amax = np.abs(blk).max()
            shared = max(math.floor(math.log2(amax)) - f["emax"], -127) if amax > 0 else -127
            s_blk = sc[i0:i0 + gr, j0 // 32:(j0 + gcc) // 32]
            assert (s_blk == shared + 127).all()                                  # every vector of the group shares it
            scaled = blk / 2.0 ** shared
            d = deq[i0:i0 + gr, j0:j0 + gcc]
            assert np.abs(scaled).max() < 2.0 ** (f["emax"] + 1)
            # nearest grid point unless clamped; half a spacing is at most 2^(e - mbits - 1)
            spacing = 2.0 ** (np.maximum(np.floor(np.log2(np.maximum(np.abs(scaled), 1e-300))), 1 - f["bias"]) - f["mbits"])
            clamped = np.abs(scaled) > f["max"]
            assert (np.abs(d - scaled)[~clamped] <= spacing[~clamped] / 2).all()
            assert (np.abs(d)[clamped] == f["max"]).all()
            assert (np.sign(d) * np.sign(scaled) >= 0).all()
            if amax > 0:
                top = np.abs(d).max()
                assert top >= 2.0 ** f["emax"]                                    # the group's largest element uses the top binade
    assert (codes.reshape(rows, cols)[-1, -32:] & (half - 1) == 0).all()
    assert codes[0] == 0 and codes[1] == half                                    # the sign of zero is kept


def test_square_blocks_commute_with_transposition():
    # the reason Section 3.2 gives for square blocks: W and its transpose must quantize to the same values
    n = 96
    w = _w_hat(n, n, 5)
    wt = np.ascontiguousarray(w.reshape(n, n).T).ravel()
    for fmt in (E4M3, E3M2, E3M4):
        c, s = orc.mx_emit(w, n, n, 32, 32, fmt)
        ct, st = orc.mx_emit(wt, n, n, 32, 32, fmt)
        assert np.array_equal(c.reshape(n, n).T, ct.reshape(n, n))
        blocks = s.reshape(n, n // 32)[::32]            # one row of scales per band of blocks
        blocks_t = st.reshape(n, n // 32)[::32]
        assert np.array_equal(blocks.T, blocks_t)
        # with per-vector (1 x 32) scales the two disagree: the sharing rule is what makes them agree
        c1, _ = orc.mx_emit(w, n, n, 1, 32, fmt)
        c1t, _ = orc.mx_emit(wt, n, n, 1, 32, fmt)
        assert not np.array_equal(c1.reshape(n, n).T, c1t.reshape(n, n))


def test_six_bit_packing_is_a_little_endian_bit_stream():
    codes = np.random.default_rng(4).integers(0, 64, 256).astype(np.uint8)
    packed = orc.mx_pack6(codes)
    assert packed.size == 192
    bits = np.unpackbits(packed, bitorder="little")
    back = (bits.reshape(-1, 6) * (1 << np.arange(6))).sum(axis=1)
    assert np.array_equal(back, codes)
    assert list(orc.mx_pack6(np.array([0x3F, 0, 0, 0], np.uint8))) == [0x3F, 0, 0]
    assert list(orc.mx_pack6(np.array([0, 0x3F, 0, 0], np.uint8))) == [0xC0, 0x0F, 0]
    assert list(orc.mx_pack6(np.array([0, 0, 0, 0x21], np.uint8))) == [0, 0, 0x84]
