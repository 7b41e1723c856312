"""Parity of the CUDA library (through its C ABI) with the CPU oracle, element by element.

Bar: bit-exact for Philox words, packed noise, absmax, scale and sampled BF16 weights; the FP32
gradient reductions within 1e-5 relative (gate A: per group against ln2 * s * sum|g R|; gate B:
per tensor against the largest gradient)."""
import ctypes

import numpy as np
import pytest
import torch

import paper_2505_11170_b200 as gws
from oracle import gws_oracle as orc
from paper_2505_11170_b200 import synthetic as syn
from paper_2505_11170_b200.binding import Desc
from util import bf16_from_bits, bits_of

pytestmark = pytest.mark.gpu
DEV = "cuda"
LN2 = float(np.log(2.0))
REL = 1e-5

# (rows, cols, group_rows, group_cols, ld) - several tiles and a ragged tail in every kernel class
FLAT = [(37, 384, 1, 128, None), (50, 160, 1, 32, None), (1030, 64, 1, 8, None), (19, 512, 1, 256, None),
        (3, 1024, 1, 64, None), (2, 16, 1, 16, None), (131, 2048, 1, 128, None)]
ROW_WARP = [(21, 768, 1, 0, None), (13, 3072, 1, 0, None), (9, 2304, 1, 0, None), (11, 4096, 1, 0, None),
            (70, 520, 1, 0, None), (1, 24, 1, 0, None), (12, 776, 1, 776, None)]
ROW_CTA = [(5, 8192, 1, 0, None), (3, 28672, 1, 0, None), (2, 65536, 1, 0, None), (4, 4104, 1, 0, None)]
SQUARE = [(64, 96, 32, 32, None), (96, 608, 32, 32, None), (32, 2048, 32, 32, None), (160, 32, 32, 32, None)]
GENERAL = [(33, 40, 32, 32, None), (5, 72, 1, 32, None), (6, 64, 1, 32, 80), (7, 13, 2, 5, None),
           (4, 100, 1, 0, None), (3, 66000, 1, 0, None), (40, 48, 8, 48, 56), (300, 8, 1, 0, 8)]
ALL = FLAT + ROW_WARP + ROW_CTA + SQUARE + GENERAL


def _make(rows, cols, ld, seed, sigma=0.02):
    ld = cols if ld is None else ld
    g = torch.Generator().manual_seed(seed)
    buf = (torch.randn(rows, ld, generator=g) * sigma).to(torch.bfloat16)
    return buf


def _desc(case, seed=0x5EED0123456789, step=3, elem_offset=0):
    rows, cols, gr, gc, ld = case
    return Desc.make(rows, cols, gr, gc, seed=seed, step=step, elem_offset=elem_offset, ld=ld)


def _bt(n, seed=1):
    return torch.randint(4, 10, (n,), generator=torch.Generator().manual_seed(seed)).float()


def test_philox_words_bit_exact():
    for seed, step, first, n in [(0, 0, 0, 1000), (0xDEADBEEFCAFEF00D, 0x1122334455667788, 0xFFFFFFF0, 4099),
                                 (7, 9, (1 << 40) + 5, 257)]:
        got = gws.philox_words(seed, step, first, n).cpu().numpy().view(np.uint32)
        assert (got == orc.philox_words(seed, step, first, n)).all()


@pytest.mark.parametrize("rows,cols,off", [(1, 8, 0), (3, 1000, 0), (5, 13, 8), (257, 2048, 1 << 33), (1, 1, 16)])
def test_noise_packed_bit_exact(rows, cols, off):
    d = Desc.make(rows, cols, seed=0xABCDEF, step=12, elem_offset=off)
    got = gws.noise(d).cpu().numpy().view(np.uint32)
    want = orc.noise_packed(0xABCDEF, 12, off, rows * cols)
    assert got.shape == want.shape and (got == want).all()


@pytest.mark.parametrize("case", ALL)
def test_group_absmax_bit_exact(case):
    rows, cols, gr, gc, ld = case
    w = _make(rows, cols, ld, 11)
    d = _desc(case)
    got = gws.group_absmax(d, w.to(DEV)).cpu().numpy()
    want = orc.group_absmax(bits_of(w), rows, cols, gr, gc, ld=d.ld)
    assert (got.view(np.uint32) == want.view(np.uint32)).all()


def _plant_special_values(w):
    flat = w.view(-1)
    n = flat.numel()
    bits = flat.view(torch.int16)
    bits[0] = -32768                       # -0.0
    if n > 40:
        bits[17] = -32768
        flat[23] = 0.0
        flat[n // 2] = 0.16                # an outlier: 8 sigma
        flat[n - 1] = -0.16
    return w


@pytest.mark.parametrize("case", ALL)
def test_sample_fwd_bit_exact(case):
    rows, cols, gr, gc, ld = case
    w = _plant_special_values(_make(rows, cols, ld, 21))
    d = _desc(case)
    ng = gws.n_groups(d)
    bt = _bt(ng)
    canary = torch.full((w.numel() + 512,), 7.0, dtype=torch.bfloat16, device=DEV)
    w_hat_dev = canary[256:256 + w.numel()].view_as(w)
    scale_dev = torch.full((ng + 64,), -5.0, device=DEV)
    gws.sample_fwd(d, w.to(DEV), bt.to(DEV), w_hat=w_hat_dev, scale_out=scale_dev[32:32 + ng])
    torch.cuda.synchronize()
    want_hat, want_scale = orc.sample_fwd(bits_of(w), bt.numpy(), rows, cols, gr, gc, seed=d.seed, step=d.step, ld=d.ld)
    got_hat = bits_of(w_hat_dev).reshape(rows, d.ld)
    assert (scale_dev[32:32 + ng].cpu().numpy().view(np.uint32) == want_scale.view(np.uint32)).all()
    assert (got_hat[:, :cols] == want_hat.reshape(rows, d.ld)[:, :cols]).all()
    # nothing outside the tensor was written: padding columns, the guard bands, the scale guards
    if d.ld > cols:
        assert (got_hat[:, cols:] == bits_of(torch.tensor([7.0], dtype=torch.bfloat16))[0]).all()
    assert (canary[:256] == 7.0).all() and (canary[256 + w.numel():] == 7.0).all()
    assert (scale_dev[:32] == -5.0).all() and (scale_dev[32 + ng:] == -5.0).all()
    # scale_out is optional
    w_hat2, none = gws.sample_fwd(d, w.to(DEV), bt.to(DEV), want_scale=False)
    assert none is None and (bits_of(w_hat2).reshape(rows, d.ld)[:, :cols] == got_hat[:, :cols]).all()


def _check_grad(got, want, scale, g_bits, r, rows, cols, gr, gc, ld):
    """Gates A and B for grad_bt."""
    gf = (g_bits.reshape(rows, ld)[:, :cols].astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    absprod = np.abs(gf * r.reshape(rows, cols))
    gcc = cols if gc == 0 else gc
    nbr, nbc = -(-rows // gr), -(-cols // gcc)
    sums = np.zeros((nbr, nbc))
    for bi in range(nbr):          # small loops: group counts here are modest
        for bj in range(nbc):
            sums[bi, bj] = absprod[bi * gr:(bi + 1) * gr, bj * gcc:(bj + 1) * gcc].sum()
    bound = REL * LN2 * scale.astype(np.float64) * sums.ravel()
    diff = np.abs(got.astype(np.float64) - want.astype(np.float64))
    assert (diff <= bound + 1e-45).all(), float((diff - bound).max())
    assert diff.max() <= REL * np.abs(want).max() + 1e-45


@pytest.mark.parametrize("case", ALL)
def test_sample_bwd_within_tolerance_and_copy_bit_exact(case):
    rows, cols, gr, gc, ld = case
    g = _make(rows, cols, ld, 31, sigma=1e-4)
    d = _desc(case, step=8)
    ng = gws.n_groups(d)
    scale = (torch.rand(ng, generator=torch.Generator().manual_seed(2)) * 1e-2 + 1e-4)
    gw_dev = torch.full_like(g, 3.0, device=DEV)
    gw, gbt = gws.sample_bwd(d, g.to(DEV), scale.to(DEV), grad_w=gw_dev)
    torch.cuda.synchronize()
    want_gw, want_gbt = orc.sample_bwd(bits_of(g), scale.numpy(), rows, cols, gr, gc, seed=d.seed, step=d.step, ld=d.ld)
    assert (bits_of(gw).reshape(rows, d.ld)[:, :cols] == want_gw.reshape(rows, d.ld)[:, :cols]).all()
    if d.ld > cols:
        assert (gw.cpu().view(rows, d.ld)[:, cols:] == 3.0).all()
    r = orc.noise_r(d.seed, d.step, 0, rows * cols).astype(np.float64)
    _check_grad(gbt.cpu().numpy(), want_gbt, scale.numpy(), bits_of(g), r, rows, cols, gr, gc, d.ld)
    # identity mode: no grad_w buffer, same grad_bt bits, and run-to-run identical bits (fixed reduction order)
    g_dev = g.to(DEV)
    same, gbt2 = gws.sample_bwd(d, g_dev, scale.to(DEV))
    assert same is g_dev and (gbt2 == gbt).all()
    _, gbt3 = gws.sample_bwd(d, g_dev, scale.to(DEV), grad_w=g_dev)
    assert (gbt3 == gbt).all()


def test_forward_noise_equals_backward_noise():
    # R seen by forward (recovered from w_hat at b_t = 4) equals R used by backward (one-hot gradients)
    rows, cols = 16, 256
    d = Desc.make(rows, cols, 1, 128, seed=77, step=5)
    w = _make(rows, cols, None, 3)
    bt = torch.full((rows * 2,), 4.0)
    w_hat, sc = gws.sample_fwd(d, w.to(DEV), bt.to(DEV))
    diff = w_hat.float().cpu().double() - w.double()
    r_fwd = torch.round(diff.view(rows * 2, 128) / sc.cpu().double().view(-1, 1)).long()
    for col in (0, 9, 127):
        g = torch.zeros(rows, cols, dtype=torch.bfloat16)
        g.view(rows * 2, 128)[:, col] = 1.0
        _, gbt = gws.sample_bwd(d, g.to(DEV), torch.ones(rows * 2, device=DEV))
        assert (torch.round(gbt.cpu().double() / -LN2).long() == r_fwd[:, col]).all()


def test_fractional_bitwidths():
    rows, cols = 64, 1024
    d = Desc.make(rows, cols, 1, 128, seed=5, step=1)
    w = _make(rows, cols, None, 4)
    bt = torch.rand(rows * 8, generator=torch.Generator().manual_seed(9)) * 8 + 1.5
    w_hat, sc = gws.sample_fwd(d, w.to(DEV), bt.to(DEV))
    want_hat, want_sc = orc.sample_fwd(bits_of(w), bt.numpy(), rows, cols, 1, 128, seed=5, step=1)
    mismatch = sc.cpu().numpy().view(np.uint32) != want_sc.view(np.uint32)
    # 2^(1-b) goes through a double-precision exp2 on both sides; a differently rounded double can flip the
    # float only in a halfway case (about 2^-29 per group)
    assert mismatch.sum() == 0
    assert (bits_of(w_hat).ravel() == want_hat).all()


def test_extreme_scales_and_zero_groups():
    # all-zero groups, subnormal scales, huge bit-widths, b_t = 0
    rows, cols = 8, 256
    w = _make(rows, cols, None, 6)
    w[0] = 0.0
    w[1] = w[1] * 1e-36            # tiny weights: scale goes subnormal
    w[2] = w[2] * 1e30
    bt = torch.tensor([6, 6, 9, 9, 4, 4, 0, 0, 20, 20, 120, 130, 5, 5, 7, 7], dtype=torch.float32)
    d = Desc.make(rows, cols, 1, 128, seed=1, step=2)
    w_hat, sc = gws.sample_fwd(d, w.to(DEV), bt.to(DEV))
    want_hat, want_sc = orc.sample_fwd(bits_of(w), bt.numpy(), rows, cols, 1, 128, seed=1, step=2)
    assert (sc.cpu().numpy().view(np.uint32) == want_sc.view(np.uint32)).all()
    assert (bits_of(w_hat).ravel() == want_hat).all()
    assert (bits_of(w_hat)[0] == 0).all()


@pytest.mark.parametrize("case", [(16, 512, 1, 128, None), (16, 768, 1, 0, None), (64, 64, 32, 32, None), (5, 72, 1, 32, None)])
def test_nan_and_inf_inputs_never_fault(case):
    # Values are unspecified for NaN / Inf inputs, but every call returns 0, the context stays usable and
    # groups without such inputs are unaffected.
    rows, cols, gr, gc, ld = case
    d = _desc(case)
    w, g = _make(rows, cols, ld, 41), _make(rows, cols, ld, 42, sigma=1e-4)
    clean_hat, clean_sc = gws.sample_fwd(d, w.to(DEV), _bt(gws.n_groups(d)).to(DEV))
    w[0, 0], w[0, 1], w[0, 2] = float("nan"), float("inf"), -float("inf")
    g[0, 3] = float("nan")
    bt = _bt(gws.n_groups(d))
    bt[0] = float("inf")
    w_hat, sc = gws.sample_fwd(d, w.to(DEV), bt.to(DEV))
    _, gbt = gws.sample_bwd(d, g.to(DEV), sc)
    am = gws.group_absmax(d, w.to(DEV))
    torch.cuda.synchronize()
    assert am.numel() == gws.n_groups(d) and gbt.numel() == gws.n_groups(d)
    # the last row holds no special value and (for these shapes) shares no group with row 0 unless groups span rows
    if gr == 1:
        assert torch.equal(w_hat[-1].view(torch.int16), clean_hat[-1].view(torch.int16))


@pytest.mark.parametrize("case", [(131, 2048, 1, 128, None), (50, 160, 1, 32, None), (21, 768, 1, 0, None), (5, 8192, 1, 0, None),
                                  (96, 608, 32, 32, None), (70, 520, 1, 0, None), (33, 40, 32, 32, None)])
def test_backward_reductions_repeat_bit_for_bit(case):
    # fixed summation order, no atomics: two runs give identical bits (and a race in a reduction would not)
    rows, cols, gr, gc, ld = case
    d = _desc(case)
    g = _make(rows, cols, ld, 51, sigma=1e-4).to(DEV)
    sc = torch.rand(gws.n_groups(d), device=DEV) * 1e-3
    runs = [gws.sample_bwd(d, g, sc)[1].clone() for _ in range(3)]
    assert torch.equal(runs[0].view(torch.int32), runs[1].view(torch.int32))
    assert torch.equal(runs[0].view(torch.int32), runs[2].view(torch.int32))


def test_elem_offset_reproduces_the_unsharded_tensor():
    rows, cols = 64, 512
    w = _make(rows, cols, None, 8)
    bt = _bt(rows * 4)
    full, _ = gws.sample_fwd(Desc.make(rows, cols, 1, 128, seed=11, step=2), w.to(DEV), bt.to(DEV))
    half = rows // 2
    part, _ = gws.sample_fwd(Desc.make(half, cols, 1, 128, seed=11, step=2, elem_offset=half * cols),
                             w[half:].contiguous().to(DEV), bt[half * 4:].contiguous().to(DEV))
    assert (part == full[half:]).all()


@pytest.mark.parametrize("offset,group_cols,want_class", [
    ((1 << 35) + 8 * 40, 128, 0),          # high counter word 1 for every vector: flat kernel
    ((5 << 35) + 8 * 12, 16, 0),           # narrow groups, high word 5
    ((1 << 35) - 8 * 1000, 128, 3),        # the vectors straddle 2^32: not a flat-kernel tensor
    ((1 << 35) - 8 * 1000, 0, 1),          # whole-row groups keep their 64-bit counters
    (((1 << 64) - (1 << 40)) & ~7, 32, 0),  # the top of the index range
])
def test_large_element_offsets(offset, group_cols, want_class, step=(1 << 40) + 3, seed=0xF00DFACE12345678):
    rows, cols = 48, 512
    d = Desc.make(rows, cols, 1, group_cols, seed=seed, step=step, elem_offset=offset)
    assert gws.kernel_class(d) == want_class
    w, g = _make(rows, cols, None, 21), _make(rows, cols, None, 22, sigma=1e-4)
    bt = _bt(gws.n_groups(d), seed=5)
    w_hat, scale = gws.sample_fwd(d, w.to(DEV), bt.to(DEV))
    _, gbt = gws.sample_bwd(d, g.to(DEV), scale)
    want_hat, want_sc = orc.sample_fwd(bits_of(w), bt.numpy(), rows, cols, 1, group_cols, seed=seed, step=step, elem_offset=offset)
    _, want_gbt = orc.sample_bwd(bits_of(g), want_sc, rows, cols, 1, group_cols, seed=seed, step=step, elem_offset=offset)
    assert (bits_of(w_hat).ravel() == want_hat).all()
    assert (scale.cpu().numpy().view(np.uint32) == want_sc.view(np.uint32)).all()
    err = np.abs(gbt.cpu().numpy().astype(np.float64) - want_gbt)
    assert err.max() <= 1e-5 * np.abs(want_gbt).max()
    packed = gws.noise(d).cpu().numpy().view(np.uint32)
    assert (packed == orc.noise_packed(seed, step, offset, rows * cols)).all()


def test_square_blocks_commute_with_transposition():
    # The paper's 32 x 32 blocks are chosen so that the block maxima of W^T are the transposed block maxima of W
    # (Section 3.1: forward and backward GEMMs see the same scales).
    rows, cols = 96, 160
    w = _make(rows, cols, None, 31)
    a = gws.group_absmax(Desc.make(rows, cols, 32, 32), w.to(DEV)).cpu().view(rows // 32, cols // 32)
    at = gws.group_absmax(Desc.make(cols, rows, 32, 32), w.t().contiguous().to(DEV)).cpu().view(cols // 32, rows // 32)
    assert torch.equal(a.t().contiguous(), at)
    want = w.float().abs().view(rows // 32, 32, cols // 32, 32).amax(dim=(1, 3))
    assert torch.equal(a, want)


def test_arithmetic_probe_runs_and_depends_on_the_stream():
    d = Desc.make(512, 2048, 1, 128, seed=9, step=1)
    a = gws.noise_alu_probe(d).cpu()
    b = gws.noise_alu_probe(d).cpu()
    c = gws.noise_alu_probe(d.with_step(2)).cpu()
    assert a.numel() == 512 * 2048 // 8 // 2048 and torch.equal(a, b) and not torch.equal(a, c)


def test_steps_and_seeds_give_different_noise_and_same_step_repeats():
    rows, cols = 32, 1024
    w = _make(rows, cols, None, 9).to(DEV)
    bt = torch.full((rows * 8,), 6.0, device=DEV)
    a, _ = gws.sample_fwd(Desc.make(rows, cols, 1, 128, seed=1, step=0), w, bt)
    b, _ = gws.sample_fwd(Desc.make(rows, cols, 1, 128, seed=1, step=1), w, bt)
    c, _ = gws.sample_fwd(Desc.make(rows, cols, 1, 128, seed=2, step=0), w, bt)
    a2, _ = gws.sample_fwd(Desc.make(rows, cols, 1, 128, seed=1, step=0), w, bt)
    assert (a == a2).all()
    assert (a != b).float().mean() > 0.2 and (a != c).float().mean() > 0.2


def _run_multi_against_oracle(specs, steps, with_copy):
    descs, W, BT, G, WH, SC, GW, GBT = [], [], [], [], [], [], [], []
    for i, s in enumerate(specs):
        descs.append(Desc.make(s.rows, s.cols, s.group_rows, s.group_cols, seed=syn.layer_seed(0, i)))
        W.append(syn.weights(s, i))
        BT.append(syn.bitwidths(s, i))
        G.append(syn.upstream_grad(s, i))
    dW, dBT, dG = [t.to(DEV) for t in W], [t.to(DEV) for t in BT], [t.to(DEV) for t in G]
    dWH = [torch.empty_like(t) for t in dW]
    dSC = [torch.empty(s.n_groups, device=DEV) for s in specs]
    dGW = [torch.empty_like(t) for t in dG] if with_copy else None
    dGBT = [torch.empty(s.n_groups, device=DEV) for s in specs]
    plan = gws.MultiPlan(descs, w=dW, bt=dBT, w_hat=dWH, scale=dSC, grad_w_hat=dG, grad_w=dGW, grad_bt=dGBT)
    assert plan.total_elements == syn.total_elements(specs)
    for step in steps:
        plan.sample_fwd_multi(step)
        plan.sample_bwd_multi(step)
        torch.cuda.synchronize()
        for i, s in enumerate(specs):
            hat, sc = orc.sample_fwd(bits_of(W[i]), BT[i].numpy(), s.rows, s.cols, s.group_rows, s.group_cols,
                                     seed=descs[i].seed, step=step)
            assert (bits_of(dWH[i]).ravel() == hat).all(), (s.name, step)
            assert (dSC[i].cpu().numpy().view(np.uint32) == sc.view(np.uint32)).all(), (s.name, step)
            gw, gbt = orc.sample_bwd(bits_of(G[i]), sc, s.rows, s.cols, s.group_rows, s.group_cols,
                                     seed=descs[i].seed, step=step)
            if with_copy:
                assert (bits_of(dGW[i]).ravel() == gw).all()
            got = dGBT[i].cpu().numpy()
            assert np.abs(got.astype(np.float64) - gbt).max() <= REL * np.abs(gbt).max(), (s.name, step)
            if i % 3 == 0:
                r = orc.noise_r(descs[i].seed, step, 0, s.numel).astype(np.float64)
                _check_grad(got, gbt, sc, bits_of(G[i]), r, s.rows, s.cols, s.group_rows, s.group_cols, s.cols)
    return plan


def test_multi_tensor_launch_mixed_classes():
    T = syn.TensorSpec
    specs = [T("a", 40, 256, 1, 128), T("b", 24, 768, 1, 0), T("c", 3, 8192, 1, 0), T("d", 64, 64, 32, 32),
             T("e", 17, 96, 1, 32), T("f", 9, 3072, 1, 0), T("g", 1100, 64, 1, 64), T("h", 5, 72, 1, 32),
             T("i", 2, 16384, 1, 0), T("j", 33, 2048, 1, 128)]
    plan = _run_multi_against_oracle(specs, steps=(0, 1, 9), with_copy=True)
    assert list(plan.plan.count) == [4, 2, 2, 2]
    # flat groups (a, e, g, j): 1; short rows b, f (3 chunks per thread): 1; block rows c (1 chunk per thread) and
    # i (2 chunks): 1 each; general d, h: 1 each
    assert plan.launches_per_pass == 6


def test_multi_tensor_plan_larger_than_one_parameter_block():
    # more tensors of a kind than one launch carries in its parameters (192 flat-group, 168 whole-row records):
    # the plan splits them over several launches and every tensor still matches the oracle
    T = syn.TensorSpec
    specs = ([T(f"f{k}", 8 + k % 5, 256, 1, 128) for k in range(200)] + [T(f"n{k}", 3, 48, 1, 16) for k in range(5)] +
             [T(f"r{k}", 4 + k % 3, 96, 1, 0) for k in range(180)] + [T(f"b{k}", 2, 8192, 1, 0) for k in range(3)] +
             [T(f"s{k}", 32, 64, 32, 32) for k in range(6)])
    plan = _run_multi_against_oracle(specs, steps=(5,), with_copy=False)
    assert list(plan.plan.count) == [205, 180, 3, 6]
    # flat 200 -> 2, narrow 5 -> 1, shared rows 180 -> 2, block rows 3 -> 1, squares 6 -> 1
    assert plan.launches_per_pass == 7


def test_multi_tensor_empty_entries_and_forward_only():
    T = syn.TensorSpec
    specs = [T("a", 8, 256, 1, 128), T("z", 0, 256, 1, 128), T("b", 8, 768, 1, 0)]
    descs = [Desc.make(s.rows, s.cols, s.group_rows, s.group_cols, seed=i) for i, s in enumerate(specs)]
    W = [syn.weights(s, i).to(DEV) for i, s in enumerate(specs)]
    BT = [syn.bitwidths(s, i).to(DEV) for i, s in enumerate(specs)]
    WH = [torch.empty_like(t) for t in W]
    plan = gws.MultiPlan(descs, w=W, bt=BT, w_hat=WH)
    plan.sample_fwd_multi(4)
    with pytest.raises(gws.GwsError):
        plan.sample_bwd_multi(4)
    for i in (0, 2):
        s = specs[i]
        hat, _ = orc.sample_fwd(bits_of(W[i]), BT[i].cpu().numpy(), s.rows, s.cols, 1, s.group_cols, seed=i, step=4)
        assert (bits_of(WH[i]).ravel() == hat).all()


def test_host_buffer_step_matches_device_calls():
    rows, cols = 96, 512
    d = Desc.make(rows, cols, 1, 128, seed=21, step=6)
    ng = gws.n_groups(d)
    pin = lambda t: t.pin_memory()
    h_w, h_g, h_bt = pin(_make(rows, cols, None, 1)), pin(_make(rows, cols, None, 2, 1e-4)), pin(_bt(ng))
    h_hat, h_sc, h_gbt = pin(torch.empty_like(h_w)), pin(torch.empty(ng)), pin(torch.empty(ng))
    dev = lambda t: torch.empty_like(t, device=DEV)
    gws.sample_step_host(d, h_w, h_bt, h_g, h_hat, h_sc, h_gbt, dev(h_w), dev(h_w), dev(h_w), dev(h_bt), dev(h_bt), dev(h_bt))
    torch.cuda.synchronize()
    hat, sc = gws.sample_fwd(d, h_w.to(DEV), h_bt.to(DEV))
    _, gbt = gws.sample_bwd(d, h_g.to(DEV), sc)
    assert (h_hat == hat.cpu()).all() and (h_sc == sc.cpu()).all() and (h_gbt == gbt.cpu()).all()
    want_hat, _ = orc.sample_fwd(bits_of(h_w), h_bt.numpy(), rows, cols, 1, 128, seed=21, step=6)
    assert (bits_of(h_hat).ravel() == want_hat).all()


def test_errors_surface_as_exceptions():
    w = torch.zeros(4, 64, dtype=torch.bfloat16, device=DEV)
    bt = torch.full((8,), 6.0, device=DEV)
    with pytest.raises(gws.GwsError) as e:
        gws.sample_fwd(Desc.make(4, 64, 1, 32), w, bt, w_hat=w)
    assert e.value.status == -5
    with pytest.raises(ValueError):
        gws.sample_fwd(Desc.make(4, 64, 1, 32), w.cpu(), bt)


def test_multi_tensor_launches_replay_from_a_cuda_graph():
    # the launches of a plan carry their tensor records in the kernel parameters, so a captured graph replays them
    # as they are: same step, same bits; nothing in the library synchronises or allocates during the capture
    specs = [syn.TensorSpec("a", 64, 1024, 1, 128), syn.TensorSpec("b", 48, 768, 1, 0), syn.TensorSpec("c", 64, 96, 32, 32)]
    descs = [Desc.make(s.rows, s.cols, s.group_rows, s.group_cols, seed=31 + i) for i, s in enumerate(specs)]
    W = [syn.weights(s, i, device=DEV) for i, s in enumerate(specs)]
    BT = [syn.bitwidths(s, i, device=DEV) for i, s in enumerate(specs)]
    G = [syn.upstream_grad(s, i, device=DEV) for i, s in enumerate(specs)]
    WH = [torch.zeros_like(t) for t in W]
    SC = [torch.zeros(s.n_groups, device=DEV) for s in specs]
    GBT = [torch.zeros(s.n_groups, device=DEV) for s in specs]
    plan = gws.MultiPlan(descs, w=W, bt=BT, w_hat=WH, scale=SC, grad_w_hat=G, grad_bt=GBT)
    plan.sample_fwd_multi(5)
    plan.sample_bwd_multi(5)
    torch.cuda.synchronize()
    want = [t.clone() for t in WH + SC + GBT]
    for t in WH + SC + GBT:
        t.zero_()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            plan.sample_fwd_multi(5, stream=side)
            plan.sample_bwd_multi(5, stream=side)
    torch.cuda.synchronize()
    assert all((t == 0).all() for t in WH)            # capture records, it does not run
    graph.replay()
    torch.cuda.synchronize()
    for got, ref in zip(WH + SC + GBT, want):
        assert torch.equal(got.view(torch.int16) if got.dtype == torch.bfloat16 else got.view(torch.int32),
                           ref.view(torch.int16) if ref.dtype == torch.bfloat16 else ref.view(torch.int32))
