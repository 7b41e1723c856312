"""Host logic of sharded sampling: the shard plan, and the exchange step between two gloo ranks on CPU.

The device work of a rank is the CUDA library's and is tested on the GPU; here the oracle does a rank's local
arithmetic so that the plan (pieces, slots) and the all-reduce can be checked end to end against the uncut tensor."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

from paper_2505_11170_b200.sharding import all_reduce_slots, even_bounds, plan_flat_shard  # noqa: E402


def test_even_bounds_are_multiples_of_eight_and_cover_the_tensor():
    assert even_bounds(1000, 3) == [0, 352, 704, 1000]
    assert even_bounds(1000, 3, align=8) == [0, 336, 672, 1000]
    assert even_bounds(16, 4, align=8) == [0, 8, 16, 16, 16]
    assert even_bounds(0, 2) == [0, 0, 0]
    b = even_bounds(2048 * 5632, 8)
    assert b[0] == 0 and b[-1] == 2048 * 5632 and all(x % 8 == 0 for x in b)


def _covered(plan):
    runs = [(p.local_begin, p.n_elements, p.elem_offset) for p in plan.pieces]
    if plan.body is not None:
        runs.append((plan.body.local_begin, plan.body.n_groups * plan.group, plan.body.elem_offset))
    return sorted(runs)


@pytest.mark.parametrize("n_groups,group,world,bounds", [
    (11, 128, 4, None), (11, 128, 4, [0, 8, 520, 1280, 1408]), (3, 4096, 8, None), (6, 32, 3, [0, 64, 64, 192]),
    (5, 256, 1, None), (2, 64, 6, None), (4, 1024, 4, [0, 1000, 1008, 3072, 4096]), (7, 8, 3, None)])
def test_plans_tile_every_shard_and_agree_on_the_slots(n_groups, group, world, bounds):
    n = n_groups * group
    plans = [plan_flat_shard(n, group, r, world, bounds, elem_offset=group * 5) for r in range(world)]
    cuts = even_bounds(n, world) if bounds is None else bounds
    for r, plan in enumerate(plans):
        assert (plan.begin, plan.end) == (cuts[r], cuts[r + 1])
        # pieces and body tile the shard exactly, in order, with the right global indices
        at = 0
        for begin, count, offset in _covered(plan):
            assert begin == at and count > 0 and offset == group * 5 + plan.begin + begin and begin % 8 == 0
            at += count
        assert at == plan.n_elements
        if plan.n_elements:
            assert plan.first_group == plan.begin // group
            assert plan.n_local_groups == (plan.end - 1) // group - plan.first_group + 1
        for p in plan.pieces:
            g = (p.elem_offset - group * 5) // group
            assert p.n_elements < group and (p.elem_offset - group * 5 + p.n_elements - 1) // group == g   # inside one group
            assert p.local_group == g - plan.first_group
            assert p.read_slot in p.slots and p.read_slot in (r, r + 1)
            assert p.slots == tuple(k for k in range(1, world) if cuts[k] % group and cuts[k] // group == g)
        if plan.body is not None:
            assert (plan.body.elem_offset - group * 5) % group == 0
    # every group held in parts is seen, through the same slots, by every rank that holds a part of it
    by_group = {}
    for plan in plans:
        for p in plan.pieces:
            by_group.setdefault((p.elem_offset - group * 5) // group, []).append(p)
    for g, parts in by_group.items():
        assert len({p.slots for p in parts}) == 1
        assert sum(p.n_elements for p in parts) == group


def test_plan_rejects_what_it_cannot_cut():
    with pytest.raises(ValueError):
        plan_flat_shard(100, 32, 0, 2)            # not whole groups
    with pytest.raises(ValueError):
        plan_flat_shard(128, 12, 0, 2)            # group not a multiple of 8
    with pytest.raises(ValueError):
        plan_flat_shard(128, 32, 0, 2, [0, 60, 128])
    with pytest.raises(ValueError):
        plan_flat_shard(128, 32, 2, 2)
    with pytest.raises(ValueError):
        plan_flat_shard(128, 32, 0, 2, [0, 64, 120])


# ---- two gloo ranks: plan + exchange, the oracle doing each rank's local arithmetic ------------------------

def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _global_inputs(n, n_groups):
    from util import bits_of
    g = torch.Generator().manual_seed(77)
    w = bits_of((torch.randn(n, generator=g) * 0.02).to(torch.bfloat16))
    grad = bits_of((torch.randn(n, generator=g) * 1e-4).to(torch.bfloat16))
    bt = torch.randint(4, 10, (n_groups,), generator=g).float().numpy()
    return w, grad, bt


def _rank_pass(plan, w, grad, bt, seed, step):
    """One rank's forward and backward with the oracle as its arithmetic; the two reductions over gloo."""
    from oracle import gws_oracle as orc
    lo, hi, G = plan.begin, plan.end, plan.group
    w_loc, g_loc = w[lo:hi], grad[lo:hi]
    bt_loc = bt[plan.first_group:plan.first_group + plan.n_local_groups]
    w_hat = np.zeros_like(w_loc)
    scale = np.zeros(plan.n_local_groups, np.float32)
    gbt = np.zeros(plan.n_local_groups, np.float32)
    buf = torch.zeros(plan.n_slots)
    if plan.body is not None:
        b = plan.body
        sl = slice(b.local_begin, b.local_begin + b.n_groups * G)
        gs = slice(b.local_group, b.local_group + b.n_groups)
        w_hat[sl], scale[gs] = orc.sample_fwd(w_loc[sl], bt_loc[gs], b.n_groups, G, seed=seed, step=step, elem_offset=b.elem_offset)
    for p in plan.pieces:
        part = orc.group_absmax(w_loc[p.local_begin:p.local_begin + p.n_elements], 1, p.n_elements)[0]
        for s in p.slots:
            buf[s] = float(part)
    all_reduce_slots(buf, "max")
    for p in plan.pieces:
        k = p.local_group
        scale[k] = orc.scale(np.array([buf[p.read_slot].item()], np.float32), bt_loc[k:k + 1])[0]
        sl = slice(p.local_begin, p.local_begin + p.n_elements)
        w_hat[sl] = orc.sample_fwd_scaled(w_loc[sl], scale[k:k + 1], 1, p.n_elements, seed=seed, step=step, elem_offset=p.elem_offset)
    buf = torch.zeros(plan.n_slots)
    if plan.body is not None:
        b = plan.body
        sl = slice(b.local_begin, b.local_begin + b.n_groups * G)
        gs = slice(b.local_group, b.local_group + b.n_groups)
        _, gbt[gs] = orc.sample_bwd(g_loc[sl], scale[gs], b.n_groups, G, seed=seed, step=step, elem_offset=b.elem_offset)
    for p in plan.pieces:
        k = p.local_group
        sl = slice(p.local_begin, p.local_begin + p.n_elements)
        _, part = orc.sample_bwd(g_loc[sl], scale[k:k + 1], 1, p.n_elements, seed=seed, step=step, elem_offset=p.elem_offset)
        for s in p.slots:
            buf[s] = float(part[0])
    all_reduce_slots(buf, "sum")
    for p in plan.pieces:
        gbt[p.local_group] = buf[p.read_slot].item()
    return w_hat, scale, gbt


def _worker(rank, world, port, n_groups, group, bounds, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        n = n_groups * group
        w, grad, bt = _global_inputs(n, n_groups)
        plan = plan_flat_shard(n, group, rank, world, bounds)
        w_hat, scale, gbt = _rank_pass(plan, w, grad, bt, seed=99, step=6)
        out.put((rank, plan.begin, plan.first_group, w_hat, scale, gbt))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("n_groups,group,bounds", [(9, 128, [0, 600, 1152]), (1, 4096, None), (6, 32, [0, 96, 192])])
def test_two_ranks_reproduce_the_uncut_tensor(n_groups, group, bounds):
    from oracle import gws_oracle as orc
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.SimpleQueue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, n_groups, group, bounds, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = [out.get() for _ in range(world)]
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    n = n_groups * group
    w, grad, bt = _global_inputs(n, n_groups)
    want_hat, want_scale = orc.sample_fwd(w, bt, n_groups, group, seed=99, step=6)
    _, want_gbt = orc.sample_bwd(grad, want_scale, n_groups, group, seed=99, step=6)
    for rank, begin, first_group, w_hat, scale, gbt in results:
        assert np.array_equal(w_hat, want_hat[begin:begin + w_hat.size]), rank
        assert np.array_equal(scale, want_scale[first_group:first_group + scale.size]), rank
        ref = want_gbt[first_group:first_group + gbt.size]
        assert np.allclose(gbt, ref, rtol=1e-5, atol=1e-5 * np.abs(want_gbt).max()), rank
    # a group held by both ranks gets the same gradient on both
    by_group = {}
    for rank, begin, first_group, w_hat, scale, gbt in results:
        for k, v in enumerate(gbt):
            by_group.setdefault(first_group + k, []).append(v)
    assert all(len(set(np.float32(x).tobytes() for x in v)) == 1 for v in by_group.values())
