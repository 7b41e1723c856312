"""The C-ABI library: it builds, loads, exports every symbol the header declares, validates its
arguments on the host, and its inline bit tricks agree with the oracle.  No GPU needed."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2505_11170_b200 as gws
from oracle import gws_oracle as orc
from paper_2505_11170_b200 import _build, binding
from paper_2505_11170_b200.binding import Desc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    _build.build()
    return gws.load_library()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "gws.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gws_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = _declared_functions()
    assert {"gws_sample_fwd", "gws_sample_bwd", "gws_group_absmax", "gws_noise"} <= set(names)
    raw = ctypes.CDLL(_build.LIB_PATH)
    for name in names:
        assert hasattr(raw, name), name
    # and the binding declares a signature for each of them
    assert set(names) <= set(binding._SIGNATURES) | {"gws_status_string"}


def test_status_strings(lib):
    seen = {gws.status_string(s) for s in range(0, -9, -1)}
    assert len(seen) == 9 and "unknown status" not in seen
    assert gws.status_string(-99) == "unknown status"


def test_validation_happens_before_any_launch(lib):
    fake = ctypes.c_void_p(0x1000)          # never dereferenced: every call below fails validation
    null = ctypes.c_void_p(None)
    good = Desc.make(4, 64, 1, 32)
    L = lib
    before = gws.launch_count()
    assert L.gws_sample_fwd(None, fake, fake, fake, null, null) == binding.ERR_NULL
    assert L.gws_sample_fwd(ctypes.byref(good), null, fake, fake, null, null) == binding.ERR_NULL
    assert L.gws_sample_bwd(ctypes.byref(good), fake, null, null, fake, null) == binding.ERR_NULL
    assert L.gws_group_absmax(ctypes.byref(good), fake, null, null) == binding.ERR_NULL
    assert L.gws_noise(ctypes.byref(good), null, null) == binding.ERR_NULL
    assert L.gws_sample_fwd(ctypes.byref(Desc.make(-1, 64)), fake, fake, fake, null, null) == binding.ERR_SHAPE
    assert L.gws_sample_fwd(ctypes.byref(Desc.make(4, 64, ld=60)), fake, fake, fake, null, null) == binding.ERR_SHAPE
    assert L.gws_sample_fwd(ctypes.byref(Desc.make(4, 64, elem_offset=4)), fake, fake, fake, null, null) == binding.ERR_SHAPE
    assert L.gws_sample_fwd(ctypes.byref(Desc.make(4, 64, group_rows=0)), fake, fake, fake, null, null) == binding.ERR_GROUP
    assert L.gws_sample_fwd(ctypes.byref(Desc.make(4, 64, group_cols=-2)), fake, fake, fake, null, null) == binding.ERR_GROUP
    assert L.gws_sample_fwd(ctypes.byref(good), ctypes.c_void_p(0x1001), fake, fake, null, null) == binding.ERR_ALIGN
    assert L.gws_sample_fwd(ctypes.byref(good), fake, ctypes.c_void_p(0x1002), fake, null, null) == binding.ERR_ALIGN
    assert L.gws_sample_fwd(ctypes.byref(good), fake, fake, fake, null, null) == binding.ERR_ALIAS      # w_hat == w
    assert L.gws_sample_fwd(ctypes.byref(good), fake, fake, ctypes.c_void_p(0x1000 + 100), null, null) == binding.ERR_ALIAS
    assert L.gws_sample_bwd(ctypes.byref(good), fake, fake, ctypes.c_void_p(0x1000 + 64), fake, null) == binding.ERR_ALIAS
    assert L.gws_philox_words(0, 0, 0, -1, fake, null) == binding.ERR_SHAPE
    assert L.gws_philox_words(0, 0, 0, 4, ctypes.c_void_p(0x1004), null) == binding.ERR_ALIGN
    # empty tensors are a successful no-op
    assert L.gws_sample_fwd(ctypes.byref(Desc.make(0, 64)), null, null, null, null, null) == binding.OK
    assert L.gws_noise(ctypes.byref(Desc.make(8, 0)), null, null) == binding.OK
    assert gws.launch_count() == before
    # multi: workspace checks
    plan = binding._MultiPlan()
    ptrs = binding._MultiPtrs()
    d = (Desc * 1)(good)
    hostws = ctypes.create_string_buffer(1 << 20)
    assert L.gws_multi_prepare(1, d, ctypes.byref(ptrs), fake, 1 << 20, hostws, 1 << 20, ctypes.byref(plan), null) == binding.ERR_NULL
    arr = (ctypes.c_void_p * 1)(0x2000)
    out = (ctypes.c_void_p * 1)(0x9000)
    pp = ctypes.POINTER(ctypes.c_void_p)
    ptrs = binding._MultiPtrs(ctypes.cast(arr, pp), ctypes.cast(arr, pp), ctypes.cast(out, pp), None, None, None, None)
    assert L.gws_multi_prepare(1, d, ctypes.byref(ptrs), null, 1 << 20, hostws, 1 << 20, ctypes.byref(plan), null) == binding.ERR_WORKSPACE
    assert L.gws_multi_prepare(1, d, ctypes.byref(ptrs), ctypes.c_void_p(0x10010), 1 << 20, hostws, 1 << 20, ctypes.byref(plan), null) == binding.ERR_WORKSPACE
    assert L.gws_multi_prepare(1, d, ctypes.byref(ptrs), ctypes.c_void_p(0x10000), 8, hostws, 1 << 20, ctypes.byref(plan), null) == binding.ERR_WORKSPACE
    assert L.gws_multi_prepare(1, d, ctypes.byref(ptrs), ctypes.c_void_p(0x10000), 1 << 20, null, 1 << 20, ctypes.byref(plan), null) == binding.ERR_WORKSPACE
    assert L.gws_multi_prepare(1, d, ctypes.byref(ptrs), ctypes.c_void_p(0x10000), 1 << 20, hostws, 8, ctypes.byref(plan), null) == binding.ERR_WORKSPACE
    assert L.gws_workspace_bytes(154) >= 154 * 2 * 112
    assert L.gws_sample_fwd_multi(None, 0, null) == binding.ERR_NULL


def test_group_count_and_kernel_class(lib):
    assert gws.n_groups(Desc.make(3072, 768)) == 3072
    assert gws.n_groups(Desc.make(2048, 5632, 1, 128)) == 2048 * 44
    assert gws.n_groups(Desc.make(33, 40, 32, 32)) == 4
    assert gws.n_groups(Desc.make(5, 72, 1, 32)) == 15
    assert gws.n_groups(Desc.make(0, 72, 1, 32)) == 0
    for d in (Desc.make(33, 40, 32, 32), Desc.make(5, 72, 1, 32), Desc.make(7, 13, 2, 5)):
        assert gws.n_groups(d) == orc.n_groups(d.rows, d.cols, d.group_rows, d.group_cols)
    assert gws.kernel_class(Desc.make(2048, 5632, 1, 128)) == 0
    assert gws.kernel_class(Desc.make(2048, 2048, 1, 32)) == 0
    assert gws.kernel_class(Desc.make(3072, 768)) == 1
    assert gws.kernel_class(Desc.make(768, 3072)) == 1
    assert gws.kernel_class(Desc.make(8192, 8192)) == 2
    assert gws.kernel_class(Desc.make(8192, 28672)) == 2
    assert gws.kernel_class(Desc.make(64, 64, 32, 32)) == 3
    assert gws.kernel_class(Desc.make(5, 72, 1, 32)) == 3          # ragged last group
    assert gws.kernel_class(Desc.make(4, 64, 1, 32, ld=80)) == 3   # padded rows
    assert gws.kernel_class(Desc.make(4, 100, 1, 0)) == 3          # cols not a multiple of 8


def test_inline_philox_matches_oracle(lib):
    rng = np.random.default_rng(0)
    for _ in range(200):
        seed, step, vec = (int(x) for x in rng.integers(0, 1 << 63, 3, dtype=np.uint64))
        vec >>= int(rng.integers(0, 60))
        assert binding.host_philox(seed, step, vec) == [int(x) for x in orc.philox_words(seed, step, vec, 1)[0]]


def test_inline_decode_matches_oracle_on_every_field_value(lib):
    # each of the 65536 field values, scattered into the bit columns of each of the 8 elements, random bits elsewhere
    rng = np.random.default_rng(1)
    want = np.array([orc.decode_field(x) for x in range(1 << 16)], np.int64)
    noise_words = rng.integers(0, 1 << 32, size=(1 << 16, 4), dtype=np.uint64)
    # where the oracle reads bit k of element t's field: found by probing it with single-bit words
    where = {}
    for word in range(4):
        for col in range(32):
            w = [0, 0, 0, 0]
            w[word] = 1 << col
            for t in range(8):
                f = orc.field_of_element(w, t)
                if f:
                    where[(t, f.bit_length() - 1)] = (word, col)
    assert len(where) == 128
    for t in range(8):
        for x in range(0, 1 << 16, 1):
            if (x * 8 + t) % 5:            # a fifth of all (value, position) pairs, every value covered in some position
                continue
            words = [int(v) for v in noise_words[x]]
            for k in range(16):
                word, col = where[(t, k)]
                words[word] = (words[word] & ~(1 << col)) | (((x >> k) & 1) << col)
            r, packed = binding.host_decode8(words)
            assert r[t] == want[x], (hex(x), t, r[t], want[x])
            nib = (packed >> (4 * t)) & 0xF
            mag = abs(int(want[x]))
            assert nib == ((8 if want[x] < 0 else 0) | mag)
            if x % 64 == 0:
                # neighbours are decoded from their own bits
                for u in range(8):
                    assert r[u] == want[orc.field_of_element(words, u)]


def test_gradient_decode_differs_from_the_forward_decode_only_in_the_sign_of_zero(lib):
    # the backward kernels skip the step that clears the sign of a zero noise value (g * -0 adds nothing to the sum);
    # everything else about the two decodes must agree, on random words and on words that make |R| = 2 likely
    rng = np.random.default_rng(5)
    cases = [rng.integers(0, 2**32, size=4, dtype=np.uint64) for _ in range(4000)]
    cases += [rng.integers(0, 2**32, size=4, dtype=np.uint64) | rng.integers(0, 2**32, size=4, dtype=np.uint64) |
              rng.integers(0, 2**32, size=4, dtype=np.uint64) for _ in range(4000)]
    seen_minus_zero = seen_two = 0
    for words in cases:
        p, q = binding.host_decode8_pairs([int(x) for x in words])
        r, _ = binding.host_decode8([int(x) for x in words])
        for j in range(4):
            for h in range(2):
                a, b = (p[j] >> (16 * h)) & 0xFFFF, (q[j] >> (16 * h)) & 0xFFFF
                assert a & 0x7FFF == b & 0x7FFF
                if a & 0x7FFF:
                    assert a == b
                else:
                    assert a == 0 and b in (0, 0x8000)
                    seen_minus_zero += b == 0x8000
                seen_two += (a & 0x7FFF) == 0x4080
                assert {0: 0, 0x4000: 1, 0x4080: 2}[a & 0x7FFF] == abs(r[2 * j + h])
    assert seen_minus_zero > 1000 and seen_two > 50


def test_fused_gemm_refuses_outputs_that_overlap_inputs(lib):
    # every thread block along M re-reads W and every block along N re-reads X, so an output laid over an input would
    # silently corrupt Y (and the master weights); the check is host arithmetic on the pointers, nothing is launched
    n, k, m = 128, 128, 128
    d = Desc.make(n, k, 1, 128)
    x, w, bt, y, wh, sc = (ctypes.c_void_p(0x10000000 + 0x100000 * i) for i in range(6))
    null = ctypes.c_void_p(None)
    call = lambda x_, w_, bt_, y_, wh_, sc_: lib.gws_gemm_fused(ctypes.byref(d), m, x_, w_, bt_, y_, wh_, sc_, null, 128, null)
    before = gws.launch_count()
    assert call(x, w, bt, y, w, null) == binding.ERR_ALIAS                                 # w_hat_out on top of w
    assert call(x, w, bt, y, ctypes.c_void_p(w.value + 2 * n * k - 32), null) == binding.ERR_ALIAS   # ... or only touching its tail
    assert call(x, w, bt, x, null, null) == binding.ERR_ALIAS                              # y on top of x
    assert call(x, w, bt, w, null, null) == binding.ERR_ALIAS                              # y on top of w
    assert call(x, w, bt, y, y, null) == binding.ERR_ALIAS                                 # the two outputs on each other
    assert call(x, w, bt, y, wh, bt) == binding.ERR_ALIAS                                  # scale_out on top of bt
    assert gws.launch_count() == before


def test_launch_overlap_setting_is_off_at_load_and_returns_the_previous_value(lib):
    assert lib.gws_set_launch_overlap(0) == 0          # off when the library is loaded
    assert lib.gws_set_launch_overlap(7) == 0          # any non-zero value switches it on ...
    assert lib.gws_set_launch_overlap(1) == 1          # ... and is reported as 1
    assert gws.set_launch_overlap(False) is True
    assert gws.set_launch_overlap(False) is False


def test_multi_layer_bitwidth_calls_validate_every_item_before_any_launch(lib):
    Item = binding.BitwidthItem
    assert lib.gws_bitwidth_multi(0, None, None) == binding.OK
    assert lib.gws_bitwidth_multi(-1, None, None) == binding.ERR_SHAPE
    assert lib.gws_bitwidth_multi(1, None, None) == binding.ERR_NULL
    items = (Item * 2)(Item(256, 512, None, None, 0, 6.0, 4.0, 0.0, 0, 0), Item(None, 512, None, None, 8, 6.0, 4.0, 0.0, 0, 0))
    assert lib.gws_bitwidth_multi(2, ctypes.cast(items, ctypes.c_void_p), None) == binding.ERR_NULL      # second item: no b_i
    items[1] = Item(256, 514, None, None, 8, 6.0, 4.0, 0.0, 0, 0)
    assert lib.gws_bitwidth_multi(2, ctypes.cast(items, ctypes.c_void_p), None) == binding.ERR_ALIGN
    items[1] = Item(256, 512, None, None, -3, 6.0, 4.0, 0.0, 0, 0)
    assert lib.gws_bitwidth_multi(2, ctypes.cast(items, ctypes.c_void_p), None) == binding.ERR_SHAPE
    items[1] = Item(256, 512, None, None, 1 << 31, 6.0, 4.0, 0.0, 0, 0)
    assert lib.gws_bitwidth_multi(2, ctypes.cast(items, ctypes.c_void_p), None) == binding.ERR_LIMIT
    items[1] = Item(256, 512, 768, None, 8, 6.0, 4.0, 0.0, 0, 0)
    assert lib.gws_bitwidth_grad_multi(2, ctypes.cast(items, ctypes.c_void_p), None) == binding.ERR_NULL # no grad_bi
    items[1] = Item(None, None, None, None, 0, 6.0, 4.0, 0.0, 0, 0)
    assert lib.gws_bitwidth_grad_multi(2, ctypes.cast(items, ctypes.c_void_p), None) == binding.OK       # empty layers only
