"""Host logic of the multi-tensor launch: the table image gws_multi_prepare would upload (no GPU needed)."""
import ctypes
from ctypes import POINTER, Structure, c_int32, c_int64, c_uint32, c_uint64, c_void_p

import pytest

import paper_2505_11170_b200 as gws
from paper_2505_11170_b200 import _build, binding
from paper_2505_11170_b200.binding import Desc


class Record(Structure):
    """The 112-byte table record documented with gws_multi_table_image (104 bytes of fields, padded to 16)."""
    _fields_ = [("inp", c_void_p), ("out", c_void_p), ("gin", c_void_p), ("gout", c_void_p), ("rows", c_int64),
                ("cols", c_int64), ("ld", c_int64), ("group_rows", c_int32), ("group_cols", c_int32),
                ("elem_offset", c_uint64), ("n_vec", c_uint64), ("seed_lo", c_uint32), ("seed_hi", c_uint32),
                ("vpr", c_uint32), ("lanes_log2", c_uint32), ("tile_begin", c_int64), ("pad", c_int64)]


def _image(descs, groups):
    _build.build()
    lib = gws.load_library()
    n = len(descs)
    arr = lambda base: ctypes.cast((c_void_p * n)(*[base + 0x1000000 * i for i in range(n)]), POINTER(c_void_p))
    keep = [arr(b) if b else None for b in groups]
    ptrs = binding._MultiPtrs(*keep)
    plan = binding._MultiPlan()
    d = (Desc * n)(*descs)
    ws_bytes = lib.gws_workspace_bytes(n)
    buf = (ctypes.c_char * ws_bytes)()
    size = lib.gws_multi_table_image(n, d, ctypes.byref(ptrs), c_void_p(0x7000000000), ws_bytes, ctypes.byref(plan), buf, ws_bytes)
    assert size >= 0, size
    return plan, bytes(buf[:size]), size


def _records(image, offset, count):
    assert ctypes.sizeof(Record) == 112
    return [Record.from_buffer_copy(image, offset + 112 * k) for k in range(count)]


def test_table_image_layout_and_tile_prefix_sums():
    descs = [Desc.make(40, 256, 1, 128, seed=(7 << 32) | 5), Desc.make(24, 768, 1, 0), Desc.make(3, 8192, 1, 0),
             Desc.make(64, 64, 32, 32), Desc.make(17, 96, 1, 32), Desc.make(9, 3072, 1, 0), Desc.make(1100, 64, 1, 64),
             Desc.make(0, 64, 1, 64), Desc.make(33, 2048, 1, 128, elem_offset=4096)]
    bases = [0x100000000, 0x200000000, 0x300000000, 0x400000000, 0x500000000, 0x600000000, 0x700000000]
    plan, image, size = _image(descs, bases)
    assert list(plan.count) == [4, 2, 1, 1] and plan.n_tensors == 9 and plan.has_fwd == 1 and plan.has_bwd == 1
    assert plan.total_elements == sum(d.rows * d.cols for d in descs)
    offs = list(plan.fwd_offset) + list(plan.bwd_offset)
    assert all(o % 256 == 0 and 0 <= o < size for o in offs) and len(set(offs)) == 8
    # flat class: tensors 0, 4, 6, 8 in order; tiles of 1024 vectors
    fwd = _records(image, plan.fwd_offset[0], 4)
    bwd = _records(image, plan.bwd_offset[0], 4)
    order = [0, 4, 6, 8]
    tiles = [-(-(descs[i].rows * descs[i].cols // 8) // 1024) for i in order]
    assert [r.tile_begin for r in fwd] == [0, tiles[0], tiles[0] + tiles[1], sum(tiles[:3])]
    assert plan.tiles[0] == sum(tiles)
    for k, i in enumerate(order):
        f, b = fwd[k], bwd[k]
        assert f.inp == bases[0] + 0x1000000 * i and f.gin == bases[1] + 0x1000000 * i
        assert f.out == bases[2] + 0x1000000 * i and f.gout == bases[3] + 0x1000000 * i
        assert b.inp == bases[4] + 0x1000000 * i and b.out == bases[5] + 0x1000000 * i
        assert b.gin == bases[3] + 0x1000000 * i and b.gout == bases[6] + 0x1000000 * i       # scale feeds backward
        assert f.n_vec == descs[i].rows * descs[i].cols // 8 and f.rows == descs[i].rows and f.ld == descs[i].cols
        assert (1 << f.lanes_log2) * 8 == descs[i].group_cols
        assert b.tile_begin == f.tile_begin
    assert fwd[0].seed_lo == 5 and fwd[0].seed_hi == 7 and fwd[3].elem_offset == 4096
    # warp-per-row class: 8 rows per tile
    rw = _records(image, plan.fwd_offset[1], 2)
    assert [r.vpr for r in rw] == [96, 384] and [r.tile_begin for r in rw] == [0, 3] and plan.tiles[1] == 3 + 2
    rc = _records(image, plan.fwd_offset[2], 1)
    assert rc[0].vpr == 1024 and plan.tiles[2] == 3
    ge = _records(image, plan.fwd_offset[3], 1)
    assert ge[0].group_rows == 32 and ge[0].group_cols == 32 and ge[0].rows == 64


def test_table_image_forward_only_and_identity_grad():
    descs = [Desc.make(8, 256, 1, 128), Desc.make(8, 768, 1, 0)]
    plan, image, _ = _image(descs, [0x100000000, 0x200000000, 0x300000000, 0, 0, 0, 0])
    assert plan.has_fwd == 1 and plan.has_bwd == 0
    f = _records(image, plan.fwd_offset[0], 1)[0]
    assert f.gout is None                                    # no scale array: forward does not store scales
    # grad_w == grad_w_hat means identity: the record carries no output pointer
    plan, image, _ = _image(descs, [0, 0, 0, 0x400000000, 0x500000000, 0x500000000, 0x700000000])
    b = _records(image, plan.bwd_offset[0], 1)[0]
    assert plan.has_fwd == 0 and plan.has_bwd == 1 and b.out is None and b.inp == 0x500000000
