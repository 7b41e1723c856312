"""gws_sample_fwd_multi_static: the forward pass for callers that cannot allocate device memory.

Code that runs inside an allocator hook or an out-of-memory handler, or in a process whose device memory
all belongs to a pool, cannot provide the table workspace gws_multi_prepare wants.  The static entry point
keeps that table in an array built into the library instead.  It must give exactly the bits of the
workspace-based path, on the first call and on every later one (the array keeps the previous call's
table, so the second call here uses a different tensor set, order and step on purpose).

Collected last (file name), so a run that stops at the first failure has seen every other test first.
"""
import ctypes

import pytest
import torch

import paper_2505_11170_b200 as gws
from paper_2505_11170_b200 import binding
from paper_2505_11170_b200 import synthetic as syn
from paper_2505_11170_b200.binding import Desc

DEV = "cuda"


def _tensor_set(specs, base):
    descs = [Desc.make(s.rows, s.cols, s.group_rows, s.group_cols, seed=syn.layer_seed(0, base + i)) for i, s in enumerate(specs)]
    W = [syn.weights(s, base + i, device=DEV) for i, s in enumerate(specs)]
    BT = [syn.bitwidths(s, base + i, device=DEV) for i, s in enumerate(specs)]
    return descs, W, BT


def _outputs(specs, W):
    # poisoned, so an element the kernels skip cannot pass by accident
    WH = [torch.full_like(t, float("nan")) for t in W]
    SC = [torch.full((s.n_groups,), float("nan"), device=DEV) for s in specs]
    return WH, SC


def _same_bits(a, b):
    return torch.equal(a.view(torch.int16), b.view(torch.int16)) if a.dtype == torch.bfloat16 else \
        torch.equal(a.view(torch.int32), b.view(torch.int32))


@pytest.mark.gpu
def test_static_table_forward_matches_workspace_forward_on_two_calls_in_a_row():
    first = [syn.TensorSpec("q", 96, 2048, 1, 128), syn.TensorSpec("fc", 40, 768, 1, 0), syn.TensorSpec("wide", 3, 8192, 1, 0),
             syn.TensorSpec("g32", 33, 96, 1, 32), syn.TensorSpec("ragged", 10, 100, 1, 48)]
    # "odd" (groups of 24 that do not divide the row) and "tall" (2-D groups that are not whole 32 x 32 blocks) run on
    # the kernel class that reads its tensor records from the built-in array on the device: the second call must
    # find its own records there, at other positions than the first call's "ragged" one had
    second = [syn.TensorSpec("odd", 7, 200, 1, 24), syn.TensorSpec("row", 70, 3072, 1, 0), syn.TensorSpec("down", 64, 5632, 1, 128),
              syn.TensorSpec("sq", 64, 64, 32, 32), syn.TensorSpec("tall", 20, 40, 4, 8)]
    for call, (specs, base, step) in enumerate([(first, 0, 5), (second, 100, 6)]):
        descs, W, BT = _tensor_set(specs, base)
        want_hat, want_sc = _outputs(specs, W)
        plan = gws.MultiPlan(descs, w=W, bt=BT, w_hat=want_hat, scale=want_sc)
        plan.sample_fwd_multi(step)
        got_hat, got_sc = _outputs(specs, W)
        gws.sample_fwd_multi_static(descs, W, BT, got_hat, got_sc, step=step)
        torch.cuda.synchronize()
        for i, s in enumerate(specs):
            assert _same_bits(got_hat[i], want_hat[i]), (call, s.name)
            assert _same_bits(got_sc[i], want_sc[i]), (call, s.name)
            assert not torch.isnan(got_hat[i].float()).any()


@pytest.mark.gpu
def test_static_table_scale_is_optional():
    specs = [syn.TensorSpec("q", 16, 256, 1, 128)]
    descs, W, BT = _tensor_set(specs, 7)
    want_hat, _ = gws.sample_fwd(descs[0].with_step(2), W[0], BT[0])
    got_hat = [torch.empty_like(W[0])]
    gws.sample_fwd_multi_static(descs, W, BT, got_hat, None, step=2)
    torch.cuda.synchronize()
    assert _same_bits(got_hat[0], want_hat)


def test_static_table_rejects_more_tensors_than_it_holds():
    # validation happens on the host before anything touches the GPU, so this runs anywhere
    lib = gws.load_library()
    n = binding.STATIC_MAX_TENSORS + 1
    descs = (Desc * n)(*[Desc.make(8, 8, 1, 8) for _ in range(n)])
    import ctypes
    arr = ctypes.cast((ctypes.c_void_p * n)(*[0x10000 * (k + 1) for k in range(n)]), ctypes.POINTER(ctypes.c_void_p))
    ptrs = binding._MultiPtrs(arr, arr, arr, None, None, None, None)
    assert lib.gws_sample_fwd_multi_static(n, descs, ctypes.byref(ptrs), 0, None) == binding.ERR_LIMIT
    assert "maximum" in gws.status_string(binding.ERR_LIMIT)
    assert lib.gws_sample_fwd_multi_static(-1, descs, ctypes.byref(ptrs), 0, None) == binding.ERR_SHAPE
    assert lib.gws_sample_fwd_multi_static(1, None, ctypes.byref(ptrs), 0, None) == binding.ERR_NULL
    # MX outputs belong to gws_sample_fwd_mx_multi: refused here before the array is touched
    mx = binding._MultiPtrs(arr, arr, arr, None, None, None, None, 1)
    assert lib.gws_sample_fwd_multi_static(1, descs, ctypes.byref(mx), 0, None) == binding.ERR_UNSUPPORTED


@pytest.mark.gpu
@pytest.mark.filterwarnings("ignore:The CUDA Graph is empty")
def test_static_table_call_is_refused_while_the_stream_is_recording():
    # the table upload reads host memory that is gone when the call returns, so the call declines to become
    # part of a recorded graph; an ordinary call right afterwards is unaffected
    specs = [syn.TensorSpec("q", 16, 256, 1, 128), syn.TensorSpec("ragged", 10, 100, 1, 48)]
    descs, W, BT = _tensor_set(specs, 3)
    want_hat, want_sc = _outputs(specs, W)
    gws.MultiPlan(descs, w=W, bt=BT, w_hat=want_hat, scale=want_sc).sample_fwd_multi(4)
    got_hat, got_sc = _outputs(specs, W)
    gws.sample_fwd_multi_static(descs, W, BT, got_hat, got_sc, step=4)     # the device's first call: outside capture
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        graph.capture_begin()
        try:
            with pytest.raises(binding.GwsError) as err:
                gws.sample_fwd_multi_static(descs, W, BT, got_hat, got_sc, step=4, stream=side)
            assert err.value.status == binding.ERR_UNSUPPORTED
        finally:
            graph.capture_end()
    torch.cuda.synchronize()
    got_hat, got_sc = _outputs(specs, W)
    gws.sample_fwd_multi_static(descs, W, BT, got_hat, got_sc, step=4)
    torch.cuda.synchronize()
    for i, s in enumerate(specs):
        assert _same_bits(got_hat[i], want_hat[i]) and _same_bits(got_sc[i], want_sc[i]), s.name
