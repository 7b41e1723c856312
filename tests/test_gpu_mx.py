"""Parity of the MX output of the forward pass (gws_sample_fwd_mx, gws_mx_quantize, gws_sample_fwd_mx_multi) with the
CPU oracle: element codes and scale bytes bit-exact, in every kernel that writes MX."""
import ctypes

import numpy as np
import pytest
import torch

import paper_2505_11170_b200 as gws
from oracle import gws_oracle as orc
from paper_2505_11170_b200 import binding
from paper_2505_11170_b200.binding import Desc
from util import bits_of

pytestmark = pytest.mark.gpu
DEV = "cuda"
FORMATS = [(gws.MX_FP8_E4M3, orc.MX_E4M3), (gws.MX_FP6_E3M2, orc.MX_E3M2), (gws.MX_FP8_E3M4, orc.MX_E3M4)]

# (rows, cols, group_rows, group_cols): flat groups (several tiles, a ragged last tile), rows shared by 1..32 threads and
# rows that take a whole block, square blocks
CASES = [(37, 384, 1, 128), (50, 160, 1, 32), (19, 512, 1, 256), (3, 1024, 1, 64), (131, 2048, 1, 128), (1100, 64, 1, 32),
         (21, 768, 1, 0), (13, 3072, 1, 0), (70, 544, 1, 0), (9, 32, 1, 0), (5, 8192, 1, 0), (3, 28672, 1, 0), (4, 4128, 1, 0),
         (64, 96, 32, 32), (96, 608, 32, 32), (32, 2048, 32, 32), (160, 32, 32, 32)]


def _weights(rows, cols, seed, sigma=0.02):
    g = torch.Generator().manual_seed(seed)
    w = (torch.randn(rows, cols, generator=g) * sigma).to(torch.bfloat16)
    flat = w.view(-1)
    flat.view(torch.int16)[0] = -32768            # -0.0
    flat[1] = 0.0
    flat[flat.numel() // 2] = 8 * sigma           # an outlier
    if rows * cols >= 4096:
        w.view(-1)[1024:1024 + 32] = 0.0          # an all-zero vector
        w.view(-1)[2048:2048 + 32] *= 2.0 ** -125 # a vector deep in the subnormal range
    return w


def _unpack(buf, desc, fmt_gpu):
    codes_bytes, scales_off, total = gws.mx_layout(desc, fmt_gpu)
    raw = buf.cpu().numpy()
    return raw[:codes_bytes], raw[scales_off:scales_off + desc.rows * desc.cols // 32], raw[codes_bytes:scales_off], raw[total:]


def _want(w_hat_bits, rows, cols, gr, gc, fmt_orc):
    codes, scales = orc.mx_emit(w_hat_bits, rows, cols, gr, gc, fmt_orc)
    return (orc.mx_pack6(codes) if fmt_orc == orc.MX_E3M2 else codes), scales


@pytest.mark.parametrize("fmt_gpu,fmt_orc", FORMATS)
@pytest.mark.parametrize("case", CASES)
def test_quantize_bit_exact(case, fmt_gpu, fmt_orc):
    rows, cols, gr, gc = case
    w_hat = _weights(rows, cols, 5)
    d = Desc.make(rows, cols, gr, gc)
    total = gws.mx_layout(d, fmt_gpu)[2]
    buf = torch.full((total + 64,), 0xAB, dtype=torch.uint8, device=DEV)
    gws.mx_quantize(d, fmt_gpu, w_hat.to(DEV), mx_out=buf)
    torch.cuda.synchronize()
    codes, scales, gap, tail = _unpack(buf, d, fmt_gpu)
    want_codes, want_scales = _want(bits_of(w_hat), rows, cols, gr, gc, fmt_orc)
    assert np.array_equal(scales, want_scales)
    assert np.array_equal(codes, want_codes)
    assert (gap == 0xAB).all() and (tail == 0xAB).all()          # nothing outside the two regions is written


@pytest.mark.parametrize("fmt_gpu,fmt_orc", FORMATS)
@pytest.mark.parametrize("case", CASES)
def test_fused_forward_bit_exact(case, fmt_gpu, fmt_orc):
    rows, cols, gr, gc = case
    w = _weights(rows, cols, 7)
    d = Desc.make(rows, cols, gr, gc, seed=0xC0FFEE1234, step=5, elem_offset=1 << 16)
    ng = gws.n_groups(d)
    bt = torch.randint(3, 7, (ng,), generator=torch.Generator().manual_seed(2)).float()
    buf, scale = gws.sample_fwd_mx(d, fmt_gpu, w.to(DEV), bt.to(DEV))
    torch.cuda.synchronize()
    want_hat, want_scale = orc.sample_fwd(bits_of(w), bt.numpy(), rows, cols, gr, gc, seed=d.seed, step=d.step, elem_offset=d.elem_offset)
    want_codes, want_scales = _want(want_hat, rows, cols, gr, gc, fmt_orc)
    codes, scales, _, _ = _unpack(buf, d, fmt_gpu)
    assert np.array_equal(scale.cpu().numpy().view(np.uint32), want_scale.view(np.uint32))
    assert np.array_equal(scales, want_scales)
    assert np.array_equal(codes, want_codes)
    # and it is the conversion of what the BF16 forward pass writes
    w_hat, _ = gws.sample_fwd(d, w.to(DEV), bt.to(DEV))
    codes2, scales2, _, _ = _unpack(gws.mx_quantize(d, fmt_gpu, w_hat), d, fmt_gpu)
    assert np.array_equal(codes2, codes) and np.array_equal(scales2, scales)


@pytest.mark.parametrize("fmt_gpu,fmt_orc", FORMATS)
def test_many_tensors_share_launches(fmt_gpu, fmt_orc):
    shapes = [(64, 256, 1, 128), (33, 768, 1, 0), (64, 64, 32, 32), (20, 512, 1, 32), (7, 8192, 1, 0), (96, 96, 32, 32), (40, 1024, 1, 128)]
    descs = [Desc.make(r, c, gr, gc, seed=100 + k) for k, (r, c, gr, gc) in enumerate(shapes)]
    W = [_weights(r, c, 50 + k).to(DEV) for k, (r, c, gr, gc) in enumerate(shapes)]
    BT = [torch.randint(3, 7, (gws.n_groups(d),), generator=torch.Generator().manual_seed(k)).float().to(DEV) for k, d in enumerate(descs)]
    OUT = [torch.zeros(gws.mx_layout(d, fmt_gpu)[2], dtype=torch.uint8, device=DEV) for d in descs]
    SC = [torch.empty(gws.n_groups(d), device=DEV) for d in descs]
    plan = gws.MultiPlan(descs, w=W, bt=BT, w_hat=OUT, scale=SC, mx_format=fmt_gpu)
    before = gws.launch_count()
    plan.sample_fwd_mx_multi(fmt_gpu, 9)
    launches = gws.launch_count() - before
    torch.cuda.synchronize()
    assert launches <= 5                    # flat, rows shared by a warp (by chunks per thread), block rows, squares
    # a plan is prepared for one kind of output; every other forward call on it is refused before anything is launched
    lib = gws.load_library()
    before = gws.launch_count()
    assert lib.gws_sample_fwd_multi(ctypes.byref(plan.plan), 9, None) == binding.ERR_UNSUPPORTED
    assert lib.gws_sample_fwd_scaled_multi(ctypes.byref(plan.plan), 9, None) == binding.ERR_UNSUPPORTED
    assert lib.gws_sample_fwd_mx_multi(ctypes.byref(plan.plan), (fmt_gpu + 1) % 3, 9, None) == binding.ERR_UNSUPPORTED
    bf16_plan = gws.MultiPlan(descs, w=W, bt=BT, w_hat=[torch.empty_like(t) for t in W], scale=SC)
    assert lib.gws_sample_fwd_mx_multi(ctypes.byref(bf16_plan.plan), fmt_gpu, 9, None) == binding.ERR_UNSUPPORTED
    assert gws.launch_count() == before
    for k, (r, c, gr, gc) in enumerate(shapes):
        want_hat, want_scale = orc.sample_fwd(bits_of(W[k]), BT[k].cpu().numpy(), r, c, gr, gc, seed=100 + k, step=9)
        want_codes, want_scales = _want(want_hat, r, c, gr, gc, fmt_orc)
        codes, scales, _, _ = _unpack(OUT[k], descs[k], fmt_gpu)
        assert np.array_equal(codes, want_codes), k
        assert np.array_equal(scales, want_scales), k
        assert np.array_equal(SC[k].cpu().numpy().view(np.uint32), want_scale.view(np.uint32)), k


@pytest.mark.parametrize("fmt_gpu,fmt_orc", FORMATS)
def test_conversion_alone_over_many_tensors_shares_launches(fmt_gpu, fmt_orc):
    # gws_mx_quantize_multi: the plan's `w` tensors are BF16 w_hat tensors to convert; no bit-widths are needed
    shapes = [(64, 256, 1, 128), (33, 768, 1, 0), (64, 64, 32, 32), (20, 512, 1, 32), (7, 8192, 1, 0), (96, 96, 32, 32), (40, 1024, 1, 128)]
    descs = [Desc.make(r, c, gr, gc, seed=7 + k) for k, (r, c, gr, gc) in enumerate(shapes)]
    WH = [_weights(r, c, 90 + k).to(DEV) for k, (r, c, gr, gc) in enumerate(shapes)]
    OUT = [torch.full((gws.mx_layout(d, fmt_gpu)[2],), 0xAB, dtype=torch.uint8, device=DEV) for d in descs]
    plan = gws.MultiPlan(descs, w=WH, w_hat=OUT, mx_format=fmt_gpu)
    before = gws.launch_count()
    plan.mx_quantize_multi(fmt_gpu)
    launches = gws.launch_count() - before
    torch.cuda.synchronize()
    assert launches <= 5
    for k, (r, c, gr, gc) in enumerate(shapes):
        want_codes, want_scales = _want(bits_of(WH[k]), r, c, gr, gc, fmt_orc)
        codes, scales, gap, tail = _unpack(OUT[k], descs[k], fmt_gpu)
        assert np.array_equal(codes, want_codes), k
        assert np.array_equal(scales, want_scales), k
        assert (gap == 0xAB).all() and (tail == 0xAB).all()
    # without bit-widths the plan cannot sample; with another format it cannot convert
    lib = gws.load_library()
    before = gws.launch_count()
    assert lib.gws_sample_fwd_mx_multi(ctypes.byref(plan.plan), fmt_gpu, 1, None) == binding.ERR_NULL
    assert lib.gws_mx_quantize_multi(ctypes.byref(plan.plan), (fmt_gpu + 1) % 3, None) == binding.ERR_UNSUPPORTED
    assert gws.launch_count() == before


def test_unsupported_shapes_are_refused_before_any_launch():
    lib = gws.load_library()
    w = torch.zeros(64 * 96 + 64, dtype=torch.bfloat16, device=DEV)
    out = torch.zeros(1 << 16, dtype=torch.uint8, device=DEV)
    bt = torch.full((1024,), 4.0, device=DEV)
    before = gws.launch_count()
    for d, w_ptr in [(Desc.make(64, 96, 1, 16), w.data_ptr()),           # groups narrower than an MX vector
                     (Desc.make(64, 96, 1, 48), w.data_ptr()),           # groups that cut vectors
                     (Desc.make(64, 40, 1, 0), w.data_ptr()),            # cols not a multiple of 32
                     (Desc.make(48, 96, 32, 32), w.data_ptr()),          # ragged square blocks
                     (Desc.make(32, 96, 1, 32, ld=128), w.data_ptr()),   # padded rows
                     (Desc.make(64, 96, 1, 32), w.data_ptr() + 16)]:     # not 32-byte aligned
        st = lib.gws_sample_fwd_mx(ctypes.byref(d), 0, w_ptr, bt.data_ptr(), out.data_ptr(), None, None)
        assert st == binding.ERR_UNSUPPORTED, (d.rows, d.cols, d.group_cols, st)
    d = Desc.make(64, 96, 1, 32)
    assert lib.gws_sample_fwd_mx(ctypes.byref(d), 7, w.data_ptr(), bt.data_ptr(), out.data_ptr(), None, None) == binding.ERR_UNSUPPORTED
    assert lib.gws_sample_fwd_mx(ctypes.byref(d), 0, w.data_ptr(), None, out.data_ptr(), None, None) == binding.ERR_NULL
    assert lib.gws_mx_quantize(ctypes.byref(d), 0, w.data_ptr(), w.data_ptr(), None) == binding.ERR_ALIAS
    assert gws.launch_count() == before
    assert gws.mx_layout(Desc.make(64, 96), 0) == (6144, 6144, 6144 + 192)
    assert gws.mx_layout(Desc.make(64, 96), 1) == (4608, 4608, 4608 + 192)
    assert gws.mx_layout(Desc.make(2, 32), 1) == (48, 256, 258)


def test_nan_and_inf_never_fault():
    # unspecified values, but the call must complete and leave the device usable
    w = _weights(64, 256, 3)
    w.view(-1)[5] = float("nan")
    w.view(-1)[300] = float("inf")
    w.view(-1)[9000] = float("-inf")
    d = Desc.make(64, 256, 1, 128, seed=1, step=1)
    bt = torch.full((gws.n_groups(d),), 5.0, device=DEV)
    for fmt in (gws.MX_FP8_E4M3, gws.MX_FP6_E3M2, gws.MX_FP8_E3M4):
        gws.sample_fwd_mx(d, fmt, w.to(DEV), bt)
        gws.mx_quantize(d, fmt, w.to(DEV))
    gws.sample_fwd_scaled(d, w.to(DEV), torch.full((gws.n_groups(d),), float("nan"), device=DEV))
    torch.cuda.synchronize()
    ok, _ = gws.sample_fwd(d, _weights(64, 256, 4).to(DEV), bt)
    assert not torch.isnan(ok.float()).any()
