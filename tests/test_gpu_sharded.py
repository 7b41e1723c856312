"""Sharded sampling on the GPU: every rank's shard, sampled by the CUDA library, must carry the bits the oracle
gives for the uncut tensor.

One GPU stands in for all ranks: their local halves run one after the other, the two reductions (NCCL all-reduces
in a real job) are taken over the stacked slot buffers here, then the finishing halves run.  No kernel waits on
another, so the order is immaterial."""
import numpy as np
import pytest
import torch

from oracle import gws_oracle as orc
from paper_2505_11170_b200.sharding import ShardedSampler, plan_flat_shard
from util import bits_of, f32_of_bits

pytestmark = pytest.mark.gpu
DEV = "cuda"
LN2 = float(np.log(2.0))

CASES = [
    # n_groups, group, world, bounds
    (40, 128, 4, [0, 8, 1800, 3336, 5120]),        # cuts inside groups, a shard of one vector
    (300, 128, 8, None),                           # even cuts, some on group boundaries
    (3, 4096, 8, None),                            # row groups wider than a shard: several cuts inside one group
    (64, 32, 3, [0, 680, 680, 2048]),              # an empty shard
    (5, 256, 1, None),                             # one rank: nothing to exchange
    (2, 64, 6, None),                              # more ranks than work
    (24, 3072, 4, [0, 10000, 40000, 60008, 73728]),  # whole rows, body on the row kernels
    (513, 8, 2, None),                             # the smallest group
]


def _inputs(n, n_groups, seed):
    g = torch.Generator().manual_seed(seed)
    w = (torch.randn(n, generator=g) * 0.02).to(torch.bfloat16)
    grad = (torch.randn(n, generator=g) * 1e-4).to(torch.bfloat16)
    bt = torch.randint(4, 10, (n_groups,), generator=g).float()
    return w, grad, bt


@pytest.mark.parametrize("n_groups,group,world,bounds", CASES)
def test_shards_carry_the_bits_of_the_uncut_tensor(n_groups, group, world, bounds):
    n = n_groups * group
    seed, step, base = 0xFEED5EED, 12, group * 1024
    w, grad, bt = _inputs(n, n_groups, n_groups + group)
    want_hat, want_scale = orc.sample_fwd(bits_of(w), bt.numpy(), n_groups, group, seed=seed, step=step, elem_offset=base)
    _, want_gbt = orc.sample_bwd(bits_of(grad), want_scale, n_groups, group, seed=seed, step=step, elem_offset=base)

    ranks = []
    for r in range(world):
        plan = plan_flat_shard(n, group, r, world, bounds, elem_offset=base)
        gs = slice(plan.first_group, plan.first_group + plan.n_local_groups)
        ranks.append(dict(
            plan=plan, sampler=ShardedSampler(plan, seed),
            w=w[plan.begin:plan.end].to(DEV), grad=grad[plan.begin:plan.end].to(DEV), bt=bt[gs].to(DEV),
            w_hat=torch.full((plan.n_elements,), float("nan"), dtype=torch.bfloat16, device=DEV),
            scale=torch.full((plan.n_local_groups,), float("nan"), device=DEV),
            gbt=torch.full((plan.n_local_groups,), float("nan"), device=DEV)))

    bufs = [k["sampler"].forward_local(step, k["w"], k["bt"], k["w_hat"], k["scale"]) for k in ranks]
    reduced = torch.stack(bufs).max(dim=0).values
    for k in ranks:
        k["sampler"].forward_finish(step, reduced.clone(), k["w"], k["bt"], k["w_hat"], k["scale"])
    bufs = [k["sampler"].backward_local(step, k["grad"], k["scale"], k["gbt"]) for k in ranks]
    reduced = torch.stack(bufs).sum(dim=0)
    for k in ranks:
        k["sampler"].backward_finish(reduced.clone(), k["gbt"])
    torch.cuda.synchronize()

    # gate A of the gradient: 1e-5 of ln2 * s * sum |g R| per group (one more rounding per part than the uncut sum)
    r_all = orc.noise_r(seed, step, base, n).astype(np.float64)
    absprod = np.abs(f32_of_bits(bits_of(grad)).astype(np.float64) * r_all).reshape(n_groups, group).sum(axis=1)
    tol = 1e-5 * LN2 * want_scale.astype(np.float64) * absprod + 1e-45
    for k in ranks:
        plan = k["plan"]
        gs = slice(plan.first_group, plan.first_group + plan.n_local_groups)
        assert np.array_equal(bits_of(k["w_hat"]), want_hat[plan.begin:plan.end]), plan.rank
        assert np.array_equal(k["scale"].cpu().numpy().view(np.uint32), want_scale[gs].view(np.uint32)), plan.rank
        got = k["gbt"].cpu().numpy().astype(np.float64)
        assert np.all(np.abs(got - want_gbt[gs].astype(np.float64)) <= tol[gs]), plan.rank
    assert np.abs(want_gbt).max() > 0


def test_single_rank_sampler_runs_without_a_process_group():
    n_groups, group = 12, 128
    w, grad, bt = _inputs(n_groups * group, n_groups, 5)
    plan = plan_flat_shard(n_groups * group, group, 0, 1)
    s = ShardedSampler(plan, seed=3)
    w_hat = torch.empty_like(w, device=DEV)
    scale = torch.empty(n_groups, device=DEV)
    gbt = torch.empty(n_groups, device=DEV)
    s.forward(2, w.to(DEV), bt.to(DEV), w_hat, scale)
    s.backward(2, grad.to(DEV), scale, gbt)
    want_hat, want_scale = orc.sample_fwd(bits_of(w), bt.numpy(), n_groups, group, seed=3, step=2)
    assert np.array_equal(bits_of(w_hat), want_hat)
    assert np.array_equal(scale.cpu().numpy().view(np.uint32), want_scale.view(np.uint32))


def test_sampler_rejects_buffers_of_the_wrong_size():
    plan = plan_flat_shard(1024, 128, 0, 2)
    s = ShardedSampler(plan, seed=1)
    w = torch.zeros(plan.n_elements, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(ValueError):
        s.forward_local(0, w, torch.zeros(plan.n_local_groups + 1, device=DEV), torch.empty_like(w),
                        torch.zeros(plan.n_local_groups, device=DEV))
    with pytest.raises(ValueError):
        s.forward_local(0, w[:-8], torch.zeros(plan.n_local_groups, device=DEV), torch.empty_like(w),
                        torch.zeros(plan.n_local_groups, device=DEV))


def _set_inputs(shapes, seed):
    out = []
    for k, (n_groups, group) in enumerate(shapes):
        out.append(_inputs(n_groups * group, n_groups, seed + k))
    return out


@pytest.mark.parametrize("world,align", [(4, 32), (3, 8), (1, 32), (8, 32)])
def test_tensor_set_sampler_carries_the_bits_of_the_uncut_tensors(world, align):
    from paper_2505_11170_b200.sharding import ShardedSetSampler, even_bounds
    # (groups, group size): groups of 128, of 32, whole rows of 2048 and 4096 + 32, narrow groups, a tensor smaller than the world
    shapes = [(90, 128), (77, 32), (10, 2048), (3, 4128), (200, 8), (1, 64), (50, 256)]
    step, user_seed = 21, 0xABCDEF12345
    inputs = _set_inputs(shapes, 300)
    seeds = [user_seed + 977 * k for k in range(len(shapes))]
    want = []
    for (n_groups, group), (w, grad, bt), seed in zip(shapes, inputs, seeds):
        hat, scale = orc.sample_fwd(bits_of(w), bt.numpy(), n_groups, group, seed=seed, step=step)
        _, gbt = orc.sample_bwd(bits_of(grad), scale, n_groups, group, seed=seed, step=step)
        r = orc.noise_r(seed, step, 0, n_groups * group).astype(np.float64)
        absprod = np.abs(f32_of_bits(bits_of(grad)).astype(np.float64) * r).reshape(n_groups, group).sum(axis=1)
        want.append((hat, scale, gbt, 1e-5 * LN2 * scale.astype(np.float64) * absprod + 1e-45))

    ranks = []
    for r in range(world):
        plans = [plan_flat_shard(ng * g, g, r, world, even_bounds(ng * g, world, align)) for ng, g in shapes]
        loc = lambda p, t: t[p.begin:p.end].to(DEV)
        grp = lambda p, t: t[p.first_group:p.first_group + p.n_local_groups].to(DEV)
        w = [loc(p, x[0]) for p, x in zip(plans, inputs)]
        grad = [loc(p, x[1]) for p, x in zip(plans, inputs)]
        bt = [grp(p, x[2]) for p, x in zip(plans, inputs)]
        w_hat = [torch.full_like(t, float("nan")) for t in w]
        ranks.append(dict(plans=plans, w_hat=w_hat, sampler=ShardedSetSampler(plans, seeds, w, bt, w_hat, grad)))

    bufs = [k["sampler"].forward_local(step) for k in ranks]
    reduced = torch.stack(bufs).max(dim=0).values
    for k in ranks:
        k["sampler"].forward_finish(step, reduced.clone())
    bufs = [k["sampler"].backward_local(step) for k in ranks]
    reduced = torch.stack(bufs).sum(dim=0)
    for k in ranks:
        k["sampler"].backward_finish(reduced.clone())
    torch.cuda.synchronize()

    for k in ranks:
        for t, p in enumerate(k["plans"]):
            hat, scale, gbt, tol = want[t]
            gs = slice(p.first_group, p.first_group + p.n_local_groups)
            assert np.array_equal(bits_of(k["w_hat"][t]), hat[p.begin:p.end]), (p.rank, t)
            assert np.array_equal(k["sampler"].scale[t].cpu().numpy().view(np.uint32), scale[gs].view(np.uint32)), (p.rank, t)
            got = k["sampler"].grad_bt[t].cpu().numpy().astype(np.float64)
            assert np.all(np.abs(got - gbt[gs].astype(np.float64)) <= tol[gs]), (p.rank, t)
    if world > 1 and align == 32:
        # whole groups share one launch; the end pieces (rows of 64-byte chunks) a few more, twice
        assert max(k["sampler"].launches_per_forward for k in ranks) <= 20
