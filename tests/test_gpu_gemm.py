"""The fused sample-into-GEMM (gws_gemm_fused) against the oracle: the sampled weights it exports are bit-exact, and
Y equals an FP64 GEMM of the oracle's w_hat within the rounding of an FP32-accumulated BF16 GEMM."""
import ctypes

import numpy as np
import pytest
import torch

import paper_2505_11170_b200 as gws
from oracle import gws_oracle as orc
from paper_2505_11170_b200 import binding
from paper_2505_11170_b200.binding import Desc
from util import bits_of, f32_of_bits

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _inputs(m, n, k, seed):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(m, k, generator=g).to(torch.bfloat16)
    w = (torch.randn(n, k, generator=g) * 0.02).to(torch.bfloat16)
    bt = torch.randint(4, 10, (n * k // 128,), generator=g).float()
    return x, w, bt


def _check_y(y_rows, x_rows, w_hat_f64):
    """y_rows: BF16 outputs of some rows; reference in FP64; tolerance: one BF16 rounding of the result (2^-8 relative)
    plus FP32 accumulation error, bounded through the sum of magnitudes."""
    xf = x_rows.double().numpy()
    ref = xf @ w_hat_f64.T
    mag = np.abs(xf) @ np.abs(w_hat_f64).T
    got = y_rows.double().numpy()
    assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-5 * mag)


@pytest.mark.parametrize("m,n,k,rows_per_block", [(128, 128, 128, 128), (256, 256, 384, 128), (512, 128, 256, 256),
                                                  (1024, 384, 512, 512), (512, 256, 1024, 512)])
def test_fused_gemm_matches_the_oracle(m, n, k, rows_per_block):
    x, w, bt = _inputs(m, n, k, m + n + k)
    d = Desc.make(n, k, 1, 128, seed=0xFACE0FF, step=11, elem_offset=1 << 14)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    w_hat_out = torch.zeros(n, k, dtype=torch.bfloat16, device=DEV)
    scale_out = torch.zeros(n * k // 128, device=DEV)
    y = torch.full((m, n), float("nan"), dtype=torch.bfloat16, device=DEV)
    gws.gemm_fused(d, x.to(DEV), w.to(DEV), bt.to(DEV), y=y, w_hat_out=w_hat_out, scale_out=scale_out, status=status,
                   rows_per_block=rows_per_block)
    torch.cuda.synchronize()
    assert status.item() == 0
    want_hat, want_scale = orc.sample_fwd(bits_of(w), bt.numpy(), n, k, 1, 128, seed=d.seed, step=d.step, elem_offset=d.elem_offset)
    assert np.array_equal(bits_of(w_hat_out).ravel(), want_hat)
    assert np.array_equal(scale_out.cpu().numpy().view(np.uint32), want_scale.view(np.uint32))
    assert not torch.isnan(y.float()).any()
    _check_y(y.cpu(), x, f32_of_bits(want_hat).astype(np.float64).reshape(n, k))


@pytest.mark.parametrize("m,n,k,cluster", [(256, 128, 128, 1), (512, 256, 384, 2), (1024, 128, 256, 4), (2048, 384, 512, 4),
                                           (1024, 256, 1024, 2), (768, 128, 640, 1)])
def test_cluster_form_matches_the_oracle(m, n, k, cluster):
    # every block of a cluster samples a share of each W tile and stores it into the shared memory of all of them
    x, w, bt = _inputs(m, n, k, m + n + k + cluster)
    d = Desc.make(n, k, 1, 128, seed=0xC1A57E4, step=3, elem_offset=1 << 12)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    w_hat_out = torch.zeros(n, k, dtype=torch.bfloat16, device=DEV)
    scale_out = torch.zeros(n * k // 128, device=DEV)
    y = torch.full((m, n), float("nan"), dtype=torch.bfloat16, device=DEV)
    gws.gemm_fused(d, x.to(DEV), w.to(DEV), bt.to(DEV), y=y, w_hat_out=w_hat_out, scale_out=scale_out, status=status, cluster=cluster)
    torch.cuda.synchronize()
    assert status.item() == 0
    want_hat, want_scale = orc.sample_fwd(bits_of(w), bt.numpy(), n, k, 1, 128, seed=d.seed, step=d.step, elem_offset=d.elem_offset)
    assert np.array_equal(bits_of(w_hat_out).ravel(), want_hat)
    assert np.array_equal(scale_out.cpu().numpy().view(np.uint32), want_scale.view(np.uint32))
    assert not torch.isnan(y.float()).any()
    _check_y(y.cpu(), x, f32_of_bits(want_hat).astype(np.float64).reshape(n, k))
    # the same sums in the same order as the single-block form: identical bits
    y_single = gws.gemm_fused(d, x.to(DEV), w.to(DEV), bt.to(DEV), rows_per_block=128 if m % 256 else 256)
    torch.cuda.synchronize()
    assert torch.equal(y.view(torch.int16), y_single.view(torch.int16))


@pytest.mark.parametrize("m,n,k,cluster", [(256, 256, 128, 1), (512, 256, 384, 2), (1024, 512, 256, 4), (2048, 256, 512, 4),
                                           (1024, 256, 1024, 2), (768, 512, 640, 1), (512, 768, 2048, 2)])
def test_wide_form_matches_the_oracle(m, n, k, cluster):
    # 256 x 256 tiles of Y per block (MMAs of N = 256), W in stages of 128 along K, X in stages of 64
    x, w, bt = _inputs(m, n, k, m + n + k + cluster + 1)
    d = Desc.make(n, k, 1, 128, seed=0x71DE, step=6, elem_offset=1 << 13)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    w_hat_out = torch.zeros(n, k, dtype=torch.bfloat16, device=DEV)
    scale_out = torch.zeros(n * k // 128, device=DEV)
    y = torch.full((m, n), float("nan"), dtype=torch.bfloat16, device=DEV)
    gws.gemm_fused(d, x.to(DEV), w.to(DEV), bt.to(DEV), y=y, w_hat_out=w_hat_out, scale_out=scale_out, status=status, cluster=cluster, wide=True)
    torch.cuda.synchronize()
    assert status.item() == 0
    want_hat, want_scale = orc.sample_fwd(bits_of(w), bt.numpy(), n, k, 1, 128, seed=d.seed, step=d.step, elem_offset=d.elem_offset)
    assert np.array_equal(bits_of(w_hat_out).ravel(), want_hat)
    assert np.array_equal(scale_out.cpu().numpy().view(np.uint32), want_scale.view(np.uint32))
    assert not torch.isnan(y.float()).any()
    _check_y(y.cpu(), x, f32_of_bits(want_hat).astype(np.float64).reshape(n, k))
    y_single = gws.gemm_fused(d, x.to(DEV), w.to(DEV), bt.to(DEV), rows_per_block=256)
    torch.cuda.synchronize()
    assert torch.equal(y.view(torch.int16), y_single.view(torch.int16))


def test_cluster_form_refuses_other_shapes_before_any_launch():
    lib = gws.load_library()
    buf = torch.zeros(1 << 21, dtype=torch.bfloat16, device=DEV)
    f = torch.ones(1 << 14, device=DEV)
    p, fp = buf.data_ptr(), f.data_ptr()
    call = lambda d, m, c: lib.gws_gemm_fused_cluster(ctypes.byref(d), m, p, p + (1 << 20), fp, p + (1 << 21), None, None, None, c, None)
    assert call(Desc.make(128, 128, 1, 128), 256, 3) == binding.ERR_UNSUPPORTED            # cluster size
    assert call(Desc.make(128, 128, 1, 128), 256, 2) == binding.ERR_UNSUPPORTED            # m not a multiple of 256 * 2
    assert call(Desc.make(128, 128, 1, 128), 128, 1) == binding.ERR_UNSUPPORTED
    assert call(Desc.make(128, 128, 1, 32), 256, 1) == binding.ERR_UNSUPPORTED             # group size
    assert call(Desc.make(128, 128, 1, 128), 0, 4) == binding.OK                           # nothing to do
    wide = lambda d, m, c: lib.gws_gemm_fused_wide(ctypes.byref(d), m, p, p + (1 << 20), fp, p + (1 << 21), None, None, None, c, None)
    assert wide(Desc.make(128, 128, 1, 128), 256, 1) == binding.ERR_UNSUPPORTED            # rows of W not a multiple of 256
    assert wide(Desc.make(256, 128, 1, 128), 256, 2) == binding.ERR_UNSUPPORTED            # m not a multiple of 256 * 2
    assert wide(Desc.make(256, 128, 1, 128), 256, 3) == binding.ERR_UNSUPPORTED
    assert wide(Desc.make(256, 128, 1, 128), 0, 2) == binding.OK


def test_fused_gemm_without_optional_outputs_gives_the_same_y():
    m, n, k = 512, 256, 256
    x, w, bt = _inputs(m, n, k, 5)
    d = Desc.make(n, k, 1, 128, seed=9, step=2)
    args = (d, x.to(DEV), w.to(DEV), bt.to(DEV))
    y1 = gws.gemm_fused(*args, rows_per_block=512)
    y2 = gws.gemm_fused(*args, w_hat_out=torch.empty(n, k, dtype=torch.bfloat16, device=DEV), rows_per_block=128)
    torch.cuda.synchronize()
    assert torch.equal(y1.view(torch.int16), y2.view(torch.int16))          # the tiling does not change the sums


def test_config5_up_projection_on_sampled_rows():
    # X [8 x 2048 tokens, 2048] ~ N(0, 1), W 5632 x 2048 (2048 -> 5632), groups of 128, 6 bits
    from paper_2505_11170_b200 import synthetic as syn
    m, n, k = 16384, 5632, 2048
    spec = syn.TensorSpec("up", n, k, 1, 128)
    w = syn.weights(spec, 0)
    bt = syn.bitwidths(spec, 0, fixed=6.0)
    g = torch.Generator().manual_seed(3 * 1000003)
    x = torch.randn(m, k, generator=g).to(torch.bfloat16)
    d = Desc.make(n, k, 1, 128, seed=syn.layer_seed(0, 0), step=0)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    y = gws.gemm_fused(d, x.to(DEV), w.to(DEV), bt.to(DEV), status=status, rows_per_block=512)
    y_cluster = gws.gemm_fused(d, x.to(DEV), w.to(DEV), bt.to(DEV), status=status, cluster=4)
    y_wide = gws.gemm_fused(d, x.to(DEV), w.to(DEV), bt.to(DEV), status=status, cluster=2, wide=True)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert torch.equal(y.view(torch.int16), y_cluster.view(torch.int16))
    assert torch.equal(y.view(torch.int16), y_wide.view(torch.int16))
    want_hat, _ = orc.sample_fwd(bits_of(w), bt.numpy(), n, k, 1, 128, seed=d.seed, step=0)
    rows = np.concatenate([np.arange(0, 8), np.random.default_rng(1).choice(m, 40, replace=False), np.arange(m - 8, m)])
    rows = torch.from_numpy(np.unique(rows))
    _check_y(y.cpu()[rows], x[rows], f32_of_bits(want_hat).astype(np.float64).reshape(n, k))
    # and against the unfused path: sampled weights, then the library GEMM (both round an FP32 sum to BF16 once)
    w_hat, _ = gws.sample_fwd(d, w.to(DEV), bt.to(DEV))
    y_unfused = x.to(DEV) @ w_hat.t()
    assert (y.float() - y_unfused.float()).abs().max().item() <= 2.0 ** -6 * y_unfused.float().abs().max().item()


def test_fused_gemm_refuses_other_shapes_before_any_launch():
    lib = gws.load_library()
    buf = torch.zeros(1 << 20, dtype=torch.bfloat16, device=DEV)
    f = torch.ones(1 << 14, device=DEV)
    p, fp = buf.data_ptr(), f.data_ptr()
    call = lambda d, m, rpb, x=p, w=p + (1 << 19), y=p + (1 << 20): lib.gws_gemm_fused(ctypes.byref(d), m, x, w, fp, y, None, None, None, rpb, None)
    assert call(Desc.make(128, 128, 1, 128), 128, 64) == binding.ERR_UNSUPPORTED           # rows per block
    assert call(Desc.make(128, 128, 1, 64), 128, 128) == binding.ERR_UNSUPPORTED           # group size
    assert call(Desc.make(96, 128, 1, 128), 128, 128) == binding.ERR_UNSUPPORTED           # n not a multiple of 128
    assert call(Desc.make(128, 192, 1, 128), 128, 128) == binding.ERR_UNSUPPORTED          # k not a multiple of 128
    assert call(Desc.make(128, 128, 1, 128), 200, 128) == binding.ERR_UNSUPPORTED          # m not a multiple of the block rows
    assert call(Desc.make(128, 128, 1, 128), 128, 128, w=p + (1 << 19) + 16) == binding.ERR_ALIGN
    assert call(Desc.make(128, 128, 1, 128), 0, 128) == binding.OK                         # nothing to do
    assert lib.gws_gemm_fused(ctypes.byref(Desc.make(128, 128, 1, 128)), 128, None, p, fp, p, None, None, None, 128, None) == binding.ERR_NULL


def test_a_wait_that_nothing_completes_gives_up_and_reports_it():
    # the GEMM's waits (on the copy of X, on the tensor core) are bounded: the same wait on a barrier that no one
    # will ever complete must return after about a second with the failure recorded, the context still usable
    lib = gws.load_library()
    status = torch.full((2,), -1, dtype=torch.int32, device=DEV)
    assert lib.gws_gemm_wait_probe(status.data_ptr(), None) == binding.OK
    torch.cuda.synchronize()
    gave_up, cycles = status.cpu().tolist()
    assert gave_up == 1
    assert cycles >= 2_000_000_000 // 1024                          # it waited its whole limit first (cycles / 1024)
    y = gws.gemm_fused(Desc.make(128, 128, 1, 128), torch.zeros(128, 128, dtype=torch.bfloat16, device=DEV),
                       torch.zeros(128, 128, dtype=torch.bfloat16, device=DEV), torch.full((128,), 4.0, device=DEV), rows_per_block=128)
    torch.cuda.synchronize()
    assert (y == 0).all()                                           # the device still works
