"""The comparison noises on the GPU against the oracle: the BF16 uniform noise and the forward pass with it bit for bit;
the Box-Muller rounded normal equal to the oracle's FP64 evaluation except where z / 2 sits within FP32 rounding of a
rounding boundary (there either neighbour is a valid answer), and the forward pass with it bit for bit given the GPU's own R."""
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
CASES = [(64, 256, 128), (33, 96, 32), (5, 1280, 256), (130, 512, 64), (1000, 2048, 128)]   # several tiles and a ragged last tile


def _inputs(rows, cols, gc, seed):
    g = torch.Generator().manual_seed(seed)
    w = (torch.randn(rows, cols, generator=g) * 0.02).to(torch.bfloat16)
    w.view(-1)[3] = -0.0
    bt = torch.randint(3, 10, (rows * cols // gc,), generator=g).float()
    return w, bt


def _unpack_nibbles(words: np.ndarray) -> np.ndarray:
    w = words.view(np.uint32)
    nib = (w[:, None] >> (4 * np.arange(8, dtype=np.uint32))[None, :]) & 0xF
    mag = (nib & 7).astype(np.int8)
    return np.where(nib & 8, -mag, mag).astype(np.int8).reshape(-1)


@pytest.mark.parametrize("rows,cols,gc", CASES)
def test_uniform_noise_and_forward_bit_exact(rows, cols, gc):
    w, bt = _inputs(rows, cols, gc, rows + cols)
    d = Desc.make(rows, cols, 1, gc, seed=0xD1FF0123, step=6, elem_offset=64)
    u = gws.noise_compare(d, gws.NOISE_UNIFORM_BF16)
    w_hat, scale = gws.sample_fwd_compare(d, gws.NOISE_UNIFORM_BF16, w.to(DEV), bt.to(DEV))
    torch.cuda.synchronize()
    want_u = orc.noise_uniform(d.seed, d.step, d.elem_offset, rows * cols)
    assert np.array_equal(bits_of(u).ravel(), want_u)
    want_hat, want_scale = orc.sample_fwd_bf16_noise(bits_of(w), bt.numpy(), want_u, rows, cols, 1, gc)
    assert np.array_equal(bits_of(w_hat).ravel(), want_hat)
    assert np.array_equal(scale.cpu().numpy().view(np.uint32), want_scale.view(np.uint32))


@pytest.mark.parametrize("rows,cols,gc", CASES)
def test_box_muller_noise_matches_fp64_away_from_rounding_boundaries_and_forward_is_bit_exact(rows, cols, gc):
    w, bt = _inputs(rows, cols, gc, rows * 3 + cols)
    d = Desc.make(rows, cols, 1, gc, seed=0xB0C5, step=2, elem_offset=32)
    r_gpu = _unpack_nibbles(gws.noise_compare(d, gws.NOISE_BOX_MULLER).cpu().numpy())
    w_hat, scale = gws.sample_fwd_compare(d, gws.NOISE_BOX_MULLER, w.to(DEV), bt.to(DEV))
    torch.cuda.synchronize()
    z = orc.noise_bm_z(d.seed, d.step, d.elem_offset, rows * cols)
    r_orc = orc.noise_bm_r(d.seed, d.step, d.elem_offset, rows * cols)
    differ = r_gpu != r_orc
    # FP32 evaluation of log, sqrt, sin / cos: a few ulp of a number of size <= 6; an R may differ only where z / 2 is that
    # close to k + 1/2, and then only by one
    half = 0.5 * z
    near_boundary = np.abs(half - np.floor(half) - 0.5) < 1e-5
    assert (near_boundary | ~differ).all()
    assert (np.abs(r_gpu.astype(int) - r_orc.astype(int)) <= 1).all()
    assert differ.mean() < 1e-4
    # the forward pass with the R the GPU drew: bit for bit the oracle's Eq. 3 with that R injected
    want_hat, want_scale = orc.sample_fwd(bits_of(w), bt.numpy(), rows, cols, 1, gc, r=r_gpu)
    assert np.array_equal(bits_of(w_hat).ravel(), want_hat)
    assert np.array_equal(scale.cpu().numpy().view(np.uint32), want_scale.view(np.uint32))


def test_comparison_calls_refuse_other_shapes_before_any_launch():
    lib = gws.load_library()
    buf = torch.zeros(1 << 17, dtype=torch.bfloat16, device=DEV)
    f = torch.ones(1 << 12, device=DEV)
    p, fp = buf.data_ptr(), f.data_ptr()
    call = lambda d, kind=0, w=p, out=p + (1 << 16): lib.gws_sample_fwd_compare(ctypes.byref(d), kind, w, fp, out, None, None)
    before = gws.launch_count()
    assert call(Desc.make(16, 256, 1, 16)) == binding.ERR_UNSUPPORTED            # groups narrower than a chunk
    assert call(Desc.make(16, 256, 32, 32)) == binding.ERR_UNSUPPORTED           # square blocks
    assert call(Desc.make(16, 512, 1, 0)) == binding.ERR_UNSUPPORTED             # whole rows longer than the largest group
    assert call(Desc.make(16, 96, 1, 64)) == binding.ERR_UNSUPPORTED             # ragged groups
    assert call(Desc.make(16, 256, 1, 128, elem_offset=8)) == binding.ERR_UNSUPPORTED
    assert call(Desc.make(16, 256, 1, 128), kind=2) == binding.ERR_UNSUPPORTED
    assert call(Desc.make(16, 256, 1, 128), w=p + 16) == binding.ERR_UNSUPPORTED
    assert call(Desc.make(16, 256, 1, 128), out=p) == binding.ERR_ALIAS
    assert gws.launch_count() == before
