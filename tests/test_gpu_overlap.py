"""Overlapping launches (gws_set_launch_overlap): blocks of a launch may become resident while the kernel before it on the
stream drains, and wait there until it has completed.  Nothing but timing may change: every result must be the oracle's,
bit for bit where the pass is exact, also when launches that depend on one another follow each other with no host
synchronisation in between (backward reads the scale its forward wrote; the next forward overwrites it)."""
import numpy as np
import pytest
import torch

import paper_2505_11170_b200 as gws
import test_gpu_parity as par
from oracle import gws_oracle as orc
from paper_2505_11170_b200 import synthetic as syn
from paper_2505_11170_b200.binding import Desc
from util import bits_of

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture
def overlap():
    assert gws.set_launch_overlap(True) is False
    yield
    assert gws.set_launch_overlap(False) is True


def test_mixed_kernel_classes_match_the_oracle_with_overlapping_launches(overlap):
    T = syn.TensorSpec
    specs = [T("a", 40, 256, 1, 128), T("b", 24, 768, 1, 0), T("c", 3, 8192, 1, 0), T("d", 64, 64, 32, 32),
             T("e", 17, 96, 1, 32), T("f", 9, 3072, 1, 0), T("g", 1100, 64, 1, 64), T("h", 5, 72, 1, 32),
             T("i", 2, 16384, 1, 0), T("j", 33, 2048, 1, 128), T("k", 96, 608, 32, 32), T("l", 300, 16, 1, 8)]
    par._run_multi_against_oracle(specs, steps=(0, 4), with_copy=True)


@pytest.mark.parametrize("case", par.FLAT + par.ROW_WARP[:4] + par.ROW_CTA[:2] + par.SQUARE, ids=str)
def test_single_tensor_calls_back_to_back(case, overlap):
    rows, cols, gr, gc, ld = case
    d = par._desc(case)
    n_groups = gws.n_groups(d)
    w, g, bt = par._make(rows, cols, ld, 11), par._make(rows, cols, ld, 12, sigma=1e-4), par._bt(n_groups)
    dw, dg, dbt = w.to(DEV), g.to(DEV), bt.to(DEV)
    w_hat, scale = torch.empty_like(dw), torch.empty(n_groups, device=DEV)
    absmax, grad_bt = torch.empty(n_groups, device=DEV), torch.empty(n_groups, device=DEV)
    # absmax, forward and backward of one tensor follow one another with no synchronisation; twice, so that the second
    # forward overwrites what the first backward reads
    for _ in range(2):
        gws.group_absmax(d, dw, absmax)
        gws.sample_fwd(d, dw, dbt, w_hat, scale)
        gws.sample_bwd(d, dg, scale, None, grad_bt)
    torch.cuda.synchronize()
    hat, sc = orc.sample_fwd(bits_of(w), bt.numpy(), rows, cols, gr, gc, seed=d.seed, step=d.step, ld=d.ld)
    _, gbt = orc.sample_bwd(bits_of(g), sc, rows, cols, gr, gc, seed=d.seed, step=d.step, ld=d.ld)
    assert (bits_of(w_hat).ravel() == hat.ravel()).all()
    assert (scale.cpu().numpy().view(np.uint32) == sc.view(np.uint32)).all()
    assert (absmax.cpu().numpy().view(np.uint32) == orc.group_absmax(bits_of(w), rows, cols, gr, gc, ld=d.ld).view(np.uint32)).all()
    assert np.abs(grad_bt.cpu().numpy().astype(np.float64) - gbt).max() <= par.REL * max(np.abs(gbt).max(), 1e-30)


def test_a_chain_of_dependent_steps_is_bit_identical_with_and_without_overlap():
    # ten steps of forward + backward over one buffer set, enqueued without a single synchronisation: with overlapping
    # launches the blocks of step k + 1 are resident while step k drains, yet must see all of its writes
    specs = [syn.TensorSpec("a", 512, 2048, 1, 128), syn.TensorSpec("b", 768, 768, 1, 0), syn.TensorSpec("c", 128, 3072, 1, 0),
             syn.TensorSpec("d", 256, 256, 32, 32), syn.TensorSpec("e", 6, 8192, 1, 0)]
    descs = [Desc.make(s.rows, s.cols, s.group_rows, s.group_cols, seed=77 + i) for i, s in enumerate(specs)]
    W = [syn.weights(s, i, device=DEV) for i, s in enumerate(specs)]
    BT = [syn.bitwidths(s, i, device=DEV) for i, s in enumerate(specs)]
    G = [syn.upstream_grad(s, i, device=DEV) for i, s in enumerate(specs)]
    WH = [torch.empty_like(t) for t in W]
    SC = [torch.empty(s.n_groups, device=DEV) for s in specs]
    steps = 10
    GBT = [[torch.empty(s.n_groups, device=DEV) for s in specs] for _ in range(steps)]
    plans = [gws.MultiPlan(descs, w=W, bt=BT, w_hat=WH, scale=SC, grad_w_hat=G, grad_bt=GBT[k]) for k in range(steps)]
    results = {}
    for on in (False, True, True):
        previous = gws.set_launch_overlap(on)
        try:
            for t in WH + SC + [x for row in GBT for x in row]:
                t.zero_()
            for k in range(steps):
                plans[k].sample_fwd_multi(k)
                plans[k].sample_bwd_multi(k)
            torch.cuda.synchronize()
        finally:
            gws.set_launch_overlap(previous)
        snap = [t.view(torch.int16).clone() for t in WH] + [t.view(torch.int32).clone() for t in SC] + \
               [x.view(torch.int32).clone() for row in GBT for x in row]
        if on in results:
            assert all(torch.equal(a, b) for a, b in zip(results[on], snap))
        results[on] = snap
    assert all(torch.equal(a, b) for a, b in zip(results[False], results[True]))
    # and the last step is the oracle's
    for i, s in enumerate(specs):
        hat, sc = orc.sample_fwd(bits_of(W[i]), BT[i].cpu().numpy(), s.rows, s.cols, s.group_rows, s.group_cols, seed=descs[i].seed,
                                 step=steps - 1)
        assert (bits_of(WH[i]).ravel() == hat.ravel()).all()
        for k in (0, steps - 1):
            _, sck = orc.sample_fwd(bits_of(W[i]), BT[i].cpu().numpy(), s.rows, s.cols, s.group_rows, s.group_cols, seed=descs[i].seed,
                                    step=k)
            _, gbt = orc.sample_bwd(bits_of(G[i]), sck, s.rows, s.cols, s.group_rows, s.group_cols, seed=descs[i].seed, step=k)
            assert np.abs(GBT[k][i].cpu().numpy().astype(np.float64) - gbt).max() <= par.REL * np.abs(gbt).max()


def test_captured_launches_are_ordinary_ones(overlap):
    # inside stream capture the library launches as it does with the overlap off; the replayed graph gives the same bits
    specs = [syn.TensorSpec("a", 64, 1024, 1, 128), syn.TensorSpec("b", 48, 768, 1, 0)]
    descs = [Desc.make(s.rows, s.cols, s.group_rows, s.group_cols, seed=31 + i) for i, s in enumerate(specs)]
    W = [syn.weights(s, i, device=DEV) for i, s in enumerate(specs)]
    BT = [syn.bitwidths(s, i, device=DEV) for i, s in enumerate(specs)]
    WH = [torch.zeros_like(t) for t in W]
    SC = [torch.zeros(s.n_groups, device=DEV) for s in specs]
    plan = gws.MultiPlan(descs, w=W, bt=BT, w_hat=WH, scale=SC)
    plan.sample_fwd_multi(2)
    torch.cuda.synchronize()
    want = [t.clone() for t in WH]
    for t in WH:
        t.zero_()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            plan.sample_fwd_multi(2, stream=side)
            plan.sample_fwd_multi(2, stream=side)
    graph.replay()
    torch.cuda.synchronize()
    assert all(torch.equal(a.view(torch.int16), b.view(torch.int16)) for a, b in zip(WH, want))
