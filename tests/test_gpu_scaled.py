"""Parity of gws_scale_from_absmax and gws_sample_fwd_scaled (the forward pass taken apart for tensors
held in parts) with the CPU oracle: bit-exact, in every kernel class."""
import numpy as np
import pytest
import torch

import paper_2505_11170_b200 as gws
from oracle import gws_oracle as orc
from paper_2505_11170_b200.binding import Desc
from test_gpu_parity import ALL, _desc, _make, _plant_special_values
from util import bits_of

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _scales(n, seed):
    # arbitrary positive factors (not derived from the weights), a zero, a tiny one and a large one
    s = np.exp(np.random.default_rng(seed).normal(-6.0, 1.5, n)).astype(np.float32)
    s[0] = 0.0
    if n > 3:
        s[1] = np.float32(2.0 ** -130)
        s[2] = np.float32(3.0e3)
    return s


@pytest.mark.parametrize("case", ALL)
def test_given_scale_forward_bit_exact(case):
    rows, cols, gr, gc, ld = case
    w = _plant_special_values(_make(rows, cols, ld, 31))
    d = _desc(case, elem_offset=1 << 12)
    ng = gws.n_groups(d)
    sc = _scales(ng, rows * 7 + cols)
    canary = torch.full((w.numel() + 512,), 7.0, dtype=torch.bfloat16, device=DEV)
    w_hat_dev = canary[256:256 + w.numel()].view_as(w)
    gws.sample_fwd_scaled(d, w.to(DEV), torch.from_numpy(sc).to(DEV), w_hat=w_hat_dev)
    torch.cuda.synchronize()
    want = orc.sample_fwd_scaled(bits_of(w), sc, rows, cols, gr, gc, seed=d.seed, step=d.step, elem_offset=d.elem_offset,
                                 ld=d.ld).reshape(rows, d.ld)
    got = bits_of(w_hat_dev).reshape(rows, d.ld)
    assert (got[:, :cols] == want[:, :cols]).all()
    if d.ld > cols:
        assert (got[:, cols:] == bits_of(torch.tensor([7.0], dtype=torch.bfloat16))[0]).all()
    assert (canary[:256] == 7.0).all() and (canary[256 + w.numel():] == 7.0).all()


@pytest.mark.parametrize("case", [ALL[0], ALL[8], ALL[15], ALL[19], ALL[23]])
def test_given_the_fused_scale_it_repeats_the_fused_forward(case):
    rows, cols, gr, gc, ld = case
    w = _make(rows, cols, ld, 41).to(DEV)
    d = _desc(case)
    bt = torch.randint(4, 10, (gws.n_groups(d),), generator=torch.Generator().manual_seed(3)).float().to(DEV)
    want, scale = gws.sample_fwd(d, w, bt)
    absmax = gws.group_absmax(d, w)
    scale2 = gws.scale_from_absmax(absmax, bt)
    got = gws.sample_fwd_scaled(d, w, scale2)
    torch.cuda.synchronize()
    assert torch.equal(scale.view(torch.int32), scale2.view(torch.int32))
    view = lambda t: bits_of(t).reshape(rows, d.ld)[:, :cols]
    assert (view(got) == view(want)).all()


def test_scale_from_absmax_bit_exact_integer_and_fractional_bits():
    n = 5000
    rng = np.random.default_rng(9)
    absmax = np.abs(rng.normal(0.0, 0.05, n)).astype(np.float32)
    absmax[:3] = [0.0, np.float32(2.0 ** -126), np.float32(3.0e38)]
    bt = rng.integers(0, 14, n).astype(np.float32)
    bt[n // 2:] = rng.uniform(0.0, 13.0, n - n // 2).astype(np.float32)     # fractional: exp2 in double, rounded once
    got = gws.scale_from_absmax(torch.from_numpy(absmax).to(DEV), torch.from_numpy(bt).to(DEV)).cpu().numpy()
    want = orc.scale(absmax, bt)
    assert (got.view(np.uint32) == want.view(np.uint32)).all()
    # in place
    a = torch.from_numpy(absmax).to(DEV)
    gws.scale_from_absmax(a, torch.from_numpy(bt).to(DEV), scale=a)
    assert (a.cpu().numpy().view(np.uint32) == want.view(np.uint32)).all()


def test_given_scale_forward_rejects_bad_arguments():
    d = Desc.make(4, 64, 1, 32)
    w = torch.zeros(4, 64, dtype=torch.bfloat16, device=DEV)
    sc = torch.ones(8, device=DEV)
    with pytest.raises(gws.GwsError) as e:
        gws.sample_fwd_scaled(d, w, sc, w_hat=w)
    assert e.value.status == gws.binding.ERR_ALIAS
    lib = gws.load_library()
    import ctypes
    assert lib.gws_sample_fwd_scaled(ctypes.byref(d), w.data_ptr(), None, w.data_ptr(), None) == gws.binding.ERR_NULL
    assert lib.gws_scale_from_absmax(-1, sc.data_ptr(), sc.data_ptr(), sc.data_ptr(), None) == gws.binding.ERR_SHAPE
    assert lib.gws_scale_from_absmax(0, None, None, None, None) == gws.binding.OK
    assert lib.gws_scale_from_absmax(4, None, sc.data_ptr(), sc.data_ptr(), None) == gws.binding.ERR_NULL
