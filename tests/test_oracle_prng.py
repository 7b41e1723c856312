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


def _columns_of(t):
    """Bit columns owned by element t of a vector (j = t >> 1, h = t & 1): c+1, c, c-7, c-8 with c = 16h + 14 - 2j."""
    c = 16 * (t & 1) + 14 - 2 * (t >> 1)
    return c, {c + 1, c, c - 7, c - 8}


def test_fields_partition_the_128_bits_of_a_vector():
    # Flip each of the 128 output bits in turn: exactly one element's field changes, in exactly one bit, and that
    # element is the one that owns the bit's column.  So the eight fields use every random bit exactly once
    # (independent elements, Eq. 9's premise) and the column layout is the stated one.
    rng = np.random.default_rng(3)
    base = rng.integers(0, 1 << 32, 4, dtype=np.uint64).astype(np.uint32)
    f0 = [orc.field_of_element(base, t) for t in range(8)]
    seen = {t: set() for t in range(8)}
    for word in range(4):
        for col in range(32):
            w = base.copy()
            w[word] ^= np.uint32(1 << col)
            changed = [(t, orc.field_of_element(w, t) ^ f0[t]) for t in range(8)]
            changed = [(t, d) for t, d in changed if d]
            assert len(changed) == 1, (word, col, changed)
            t, d = changed[0]
            assert bin(d).count("1") == 1
            assert col in _columns_of(t)[1], (word, col, t)
            seen[t].add(d.bit_length() - 1)
    assert all(seen[t] == set(range(16)) for t in range(8))


def test_field_bits_feed_the_stated_terms():
    # Which word / column feeds which AND / OR term, stated as sets (order inside a term cannot matter):
    #   eight-input AND of |R| = 2: columns c-7 (all four words), c-8 (words 1..3), c+1 (word 0)
    #   its OR: column c+1 of words 1, 2;  sign: column c+1 of word 3
    #   |R| = 1: (word 0 | word 1) & (word 2 | word 3) at column c, and word 0 at column c-8
    for t in range(8):
        c, _ = _columns_of(t)
        def field_with(bits):
            w = np.zeros(4, np.uint32)
            for word, col in bits:
                w[word] |= np.uint32(1 << col)
            return orc.field_of_element(w, t)
        and8 = [(k, c - 7) for k in range(4)] + [(k, c - 8) for k in (1, 2, 3)] + [(0, c + 1)]
        assert field_with(and8) == 0x00FF
        assert {field_with([(1, c + 1)]), field_with([(2, c + 1)])} == {1 << 8, 1 << 9}
        assert field_with([(3, c + 1)]) == 1 << 15
        assert {field_with([(0, c)]), field_with([(1, c)])} == {1 << 10, 1 << 11}
        assert {field_with([(2, c)]), field_with([(3, c)])} == {1 << 12, 1 << 13}
        assert field_with([(0, c - 8)]) == 1 << 14
        # and through the decode: a full |R| = 2 pattern, a |R| = 1 pattern, their negatives
        assert orc.decode_field(field_with(and8 + [(2, c + 1)])) == 2
        assert orc.decode_field(field_with(and8 + [(1, c + 1), (3, c + 1)])) == -2
        assert orc.decode_field(field_with([(1, c), (2, c), (0, c - 8)])) == 1
        assert orc.decode_field(field_with([(0, c), (3, c), (0, c - 8), (3, c + 1)])) == -1
        assert orc.decode_field(field_with([(0, c), (3, c)])) == 0


def test_noise_is_decode_of_the_gathered_field():
    seed, step, vec = 99, 5, 1234
    o = orc.philox_words(seed, step, vec, 1)[0]
    r = orc.noise_r(seed, step, vec * 8, 8)
    for t in range(8):
        assert int(r[t]) == orc.decode_field(orc.field_of_element(o, t))


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
