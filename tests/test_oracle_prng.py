"""Pins for the oracle's random-bit source: Philox4x32-10 (Section 3.4 names Philox) and the
(seed, step, element index) -> (counter, key) mapping."""
import os

import numpy as np

from oracle import gws_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _kat_rows():
    rows = []
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            v = [int(x, 16) for x in line.split()]
            rows.append((v[0:4], v[4:6], v[6:10]))
    return rows


def test_philox_known_answers():
    rows = _kat_rows()
    assert len(rows) == 3
    for ctr, key, want in rows:
        got = orc.philox4x32_10(ctr, key)
        assert [int(x) for x in got] == want


def test_philox_is_a_bijection_on_small_counter_range():
    # For a fixed key the block function permutes counters: distinct counters, distinct outputs.
    out = orc.philox_words(seed=123, step=0, first_vec=0, n_vec=4096)
    assert len({tuple(r) for r in out.tolist()}) == 4096


def test_counter_key_mapping():
    # counter = (lo(vec), hi(vec), lo(step), hi(step)), key = (lo(seed), hi(seed))
    seed = 0x0123456789ABCDEF
    step = 0xFEDCBA9876543210
    for vec in (0, 1, 7, 0xFFFFFFFF, 0x100000000, 0x123456789A):
        want = orc.philox4x32_10([vec & 0xFFFFFFFF, vec >> 32, step & 0xFFFFFFFF, step >> 32],
                                 [seed & 0xFFFFFFFF, seed >> 32])
        got = orc.philox_words(seed, step, vec, 1)[0]
        assert (got == want).all()
    # golden row 3 read through the mapping: vec = ctr1:ctr0, step = ctr3:ctr2, seed = key1:key0
    ctr, key, want = _kat_rows()[2]
    got = orc.philox_words(key[0] | (key[1] << 32), ctr[2] | (ctr[3] << 32), ctr[0] | (ctr[1] << 32), 1)[0]
    assert [int(x) for x in got] == want


def test_field_order_inside_a_vector():
    # element t of a vector uses bits [16*(t&1), +16) of output word t>>1
    seed, step, vec = 99, 5, 1234
    o = orc.philox_words(seed, step, vec, 1)[0]
    r = orc.noise_r(seed, step, vec * 8, 8)
    for t in range(8):
        field = (int(o[t >> 1]) >> (16 * (t & 1))) & 0xFFFF
        assert int(r[t]) == orc.decode_field(field)


def test_bits_are_balanced_and_streams_differ():
    n = 1 << 16
    a = orc.philox_words(seed=1, step=0, first_vec=0, n_vec=n)
    bits = np.unpackbits(a.view(np.uint8))
    # each bit ~ Bernoulli(1/2): mean within 5 standard errors
    assert abs(bits.mean() - 0.5) < 5 * 0.5 / np.sqrt(bits.size)
    per_position = np.unpackbits(a.view(np.uint8).reshape(n, 16), axis=1).mean(axis=0)
    assert np.all(np.abs(per_position - 0.5) < 5 * 0.5 / np.sqrt(n))
    # another step / another seed gives an unrelated stream (about half the bits differ)
    for other in (orc.philox_words(1, 1, 0, n), orc.philox_words(2, 0, 0, n)):
        diff = np.unpackbits((a ^ other).view(np.uint8)).mean()
        assert abs(diff - 0.5) < 5 * 0.5 / np.sqrt(bits.size)


def test_regeneration_is_exact():
    # forward and backward must see the same R (Section 3.6, "Managing seed")
    a = orc.noise_r(7, 3, 0, 10000)
    b = orc.noise_r(7, 3, 0, 10000)
    assert (a == b).all()
    # a window of the stream equals the same window of a longer run (counter-based, no state)
    c = orc.noise_r(7, 3, 4096, 1000)
    assert (c == a[4096:5096]).all()
