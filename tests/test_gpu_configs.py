"""The benchmark configurations at full size, in the launch configuration the benchmark times
(one multi-tensor launch per kernel class), against the oracle.  Whole weight sets and whole matrices are
compared element by element and group by group: the oracle runs as one single-threaded process per host
core over disjoint tensors or row bands (oracle/pool.py; a row band with elem_offset = first_row * cols
reproduces the noise stream of the full tensor).  Only the intermediate step counters of the ten-step run and the MX
outputs are checked on row slices."""
import numpy as np
import pytest
import torch

import paper_2505_11170_b200 as gws
from oracle import gws_oracle as orc
from paper_2505_11170_b200 import synthetic as syn
from paper_2505_11170_b200.binding import Desc
from oracle.pool import OraclePool
from util import bits_of

pytestmark = pytest.mark.gpu
DEV = "cuda"
REL = 1e-5


def _slice_check(spec, desc_seed, step, w, bt, w_hat, scale, g, gbt, r0, nrows):
    """Oracle on rows [r0, r0+nrows) of one tensor (groups must not straddle the slice)."""
    cols = spec.cols
    gc = cols if spec.group_cols == 0 else spec.group_cols
    gpr = cols // gc
    sl = slice(r0, r0 + nrows)
    gsl = slice(r0 * gpr, (r0 + nrows) * gpr)
    hat, sc = orc.sample_fwd(bits_of(w[sl]), bt[gsl].cpu().numpy(), nrows, cols, 1, spec.group_cols, seed=desc_seed,
                             step=step, elem_offset=r0 * cols)
    assert (bits_of(w_hat[sl]).ravel() == hat).all(), (spec.name, step, r0)
    assert (scale[gsl].cpu().numpy().view(np.uint32) == sc.view(np.uint32)).all()
    if g is not None:
        _, want = orc.sample_bwd(bits_of(g[sl]), sc, nrows, cols, 1, spec.group_cols, seed=desc_seed, step=step,
                                 elem_offset=r0 * cols)
        got = gbt[gsl].cpu().numpy().astype(np.float64)
        r = orc.noise_r(desc_seed, step, r0 * cols, nrows * cols).astype(np.float64)
        gf = g[sl].float().cpu().numpy().astype(np.float64).reshape(-1)
        sums = np.abs(gf * r).reshape(nrows * gpr, gc).sum(axis=1)
        bound = REL * np.log(2.0) * sc.astype(np.float64) * sums
        assert (np.abs(got - want) <= bound + 1e-45).all(), (spec.name, step, r0)
        assert np.abs(got - want).max() <= REL * np.abs(want).max() + 1e-45


def _bands(rows, want):
    """Splits `rows` into about `want` bands of whole rows: (first row, number of rows)."""
    per = max(1, -(-rows // want))
    return [(r0, min(per, rows - r0)) for r0 in range(0, rows, per)]


def _whole_check(pool, specs, seeds, step, W, BT, WH, SC, G, GBT, min_tasks=32):
    """Every element of w_hat, every scale and every grad_bt of a tensor set against the oracle."""
    host = lambda t: t.cpu()
    tasks, where = [], []
    per_tensor = max(1, min_tasks // len(specs))
    for i, s in enumerate(specs):
        assert s.group_rows == 1
        gc = s.group_cols or s.cols
        gpr = s.cols // gc
        w, bt, g = bits_of(host(W[i])).reshape(s.rows, s.cols), host(BT[i]).numpy(), bits_of(host(G[i])).reshape(s.rows, s.cols)
        for r0, nr in _bands(s.rows, per_tensor):
            tasks.append(dict(rows=nr, cols=s.cols, group_rows=1, group_cols=s.group_cols, seed=seeds[i], step=step,
                              elem_offset=r0 * s.cols, w=w[r0:r0 + nr], bt=bt[r0 * gpr:(r0 + nr) * gpr], g=g[r0:r0 + nr]))
            where.append((i, r0, nr, gpr))
    res = pool.run(tasks, bound=True)
    got_hat = [bits_of(host(t)).reshape(s.rows, s.cols) for t, s in zip(WH, specs)]
    got_sc = [host(t).numpy() for t in SC]
    got_gbt = [host(t).numpy().astype(np.float64) for t in GBT]
    worst = {}
    for k, (i, r0, nr, gpr) in enumerate(where):
        name = specs[i].name
        assert np.array_equal(got_hat[i][r0:r0 + nr].ravel(), np.asarray(res["w_hat"][k]).ravel()), (name, step, r0)
        gsl = slice(r0 * gpr, (r0 + nr) * gpr)
        assert np.array_equal(got_sc[i][gsl].view(np.uint32), np.asarray(res["scale"][k]).view(np.uint32)), (name, step, r0)
        want = np.asarray(res["grad_bt"][k]).astype(np.float64)
        err = np.abs(got_gbt[i][gsl] - want)
        assert (err <= REL * np.asarray(res["grad_bt_bound"][k]) + 1e-45).all(), (name, step, r0)
        e, m = worst.get(i, (0.0, 0.0))
        worst[i] = (max(e, float(err.max())), max(m, float(np.abs(want).max())))
    for i, (e, m) in worst.items():
        assert e <= REL * m + 1e-45, (specs[i].name, step)
    return res["elements"]


@pytest.mark.parametrize("literal", [False, True])
def test_config1_gpt2_single_mlp_weight(literal):
    spec = syn.gpt2_124m_single(literal)[0]
    w = syn.weights(spec, 0)
    bt = syn.bitwidths(spec, 0, fixed=6.0)
    d = Desc.make(spec.rows, spec.cols, 1, 0, seed=syn.layer_seed(0, 0), step=0)
    w_hat, sc = gws.sample_fwd(d, w.to(DEV), bt.to(DEV))
    hat, want_sc = orc.sample_fwd(bits_of(w), bt.numpy(), spec.rows, spec.cols, 1, 0, seed=d.seed, step=0)
    assert (bits_of(w_hat).ravel() == hat).all()
    assert (sc.cpu().numpy().view(np.uint32) == want_sc.view(np.uint32)).all()
    packed = gws.noise(d).cpu().numpy().view(np.uint32)
    assert (packed == orc.noise_packed(d.seed, 0, 0, spec.numel)).all()


def _device_set(specs, device=DEV):
    W = [syn.weights(s, i, device=device) for i, s in enumerate(specs)]
    BT = [syn.bitwidths(s, i, device=device) for i, s in enumerate(specs)]
    G = [syn.upstream_grad(s, i, device=device) for i, s in enumerate(specs)]
    WH = [torch.empty_like(t) for t in W]
    SC = [torch.empty(s.n_groups, device=device) for s in specs]
    GBT = [torch.empty(s.n_groups, device=device) for s in specs]
    descs = [Desc.make(s.rows, s.cols, s.group_rows, s.group_cols, seed=syn.layer_seed(0, i)) for i, s in enumerate(specs)]
    return descs, W, BT, G, WH, SC, GBT


def test_config2_gpt2_all_linear_weights_forward_backward_whole_set():
    specs = syn.gpt2_124m_all()
    assert syn.total_elements(specs) == 84934656 and sum(s.n_groups for s in specs) == 82944
    descs, W, BT, G, WH, SC, GBT = _device_set(specs)
    plan = gws.MultiPlan(descs, w=W, bt=BT, w_hat=WH, scale=SC, grad_w_hat=G, grad_bt=GBT)
    assert plan.launches_per_pass == 1                     # every tensor is a warp-per-row tensor
    plan.sample_fwd_multi(0)
    plan.sample_bwd_multi(0)
    torch.cuda.synchronize()
    with OraclePool() as pool:
        assert _whole_check(pool, specs, [d.seed for d in descs], 0, W, BT, WH, SC, G, GBT) == 84934656


def test_config3_llama2_1b_ten_steps_whole_set_at_steps_0_and_9():
    specs = syn.llama2_1b()
    assert syn.total_elements(specs) == 1130364928 and sum(s.n_groups for s in specs) == 8830976
    descs, W, BT, G, WH, SC, GBT = _device_set(specs)
    plan = gws.MultiPlan(descs, w=W, bt=BT, w_hat=WH, scale=SC, grad_w_hat=G, grad_bt=GBT)
    assert plan.launches_per_pass == 1
    rng = np.random.default_rng(3)
    seeds = [d.seed for d in descs]
    for step in range(10):
        plan.sample_fwd_multi(step)
        plan.sample_bwd_multi(step)
        torch.cuda.synchronize()
        if step in (0, 9):
            # all 1,130,364,928 elements and all 8,830,976 groups
            with OraclePool() as pool:
                assert _whole_check(pool, specs, seeds, step, W, BT, WH, SC, G, GBT) == 1130364928
        else:
            for i in rng.choice(len(specs), 6, replace=False):
                s = specs[int(i)]
                r0 = int(rng.integers(0, s.rows - 8))
                _slice_check(s, descs[int(i)].seed, step, W[int(i)], BT[int(i)], WH[int(i)], SC[int(i)], G[int(i)],
                             GBT[int(i)], r0, 8)


@pytest.mark.parametrize("shape", syn.STRESS_SHAPES)
def test_config4_stress_sweep(shape):
    rows, cols = shape
    case = 0
    for sigma in syn.STRESS_SIGMAS:
        base = syn.TensorSpec("stress", rows, cols, 1, 0)
        w = syn.add_outliers(syn.weights(base, case, sigma=sigma, device=DEV), case, sigma)
        g = syn.upstream_grad(base, case, device=DEV)
        w_hat = torch.empty_like(w)
        for gc in syn.STRESS_GROUPS:
            spec = syn.stress_case(rows, cols, gc)
            for bits in syn.STRESS_BITS:
                case += 1
                d = Desc.make(rows, cols, 1, gc, seed=syn.layer_seed(4, case), step=case)
                bt = syn.bitwidths(spec, 0, fixed=bits, device=DEV)
                _, sc = gws.sample_fwd(d, w, bt, w_hat=w_hat)
                _, gbt = gws.sample_bwd(d, g, sc)
                torch.cuda.synchronize()
                # the whole matrix (up to 234,881,024 elements), cut into row bands for the oracle processes
                with OraclePool() as pool:
                    assert _whole_check(pool, [spec], [d.seed], case, [w], [bt], [w_hat], [sc], [g], [gbt]) == rows * cols
                # the outliers are there and the absmax sees them
                am = gws.group_absmax(d, w)
                assert float(am.max()) >= 7.9 * sigma


def test_config5_sample_then_gemm_unfused():
    # Up-projection of the Llama2-1B shape: W 5632 x 2048 (rows = outputs), groups of 128, 6 bits; X 16384 x 2048.
    # The sampled weight is checked bit for bit, whole; Y = X W_hat^T (the stock BF16 GEMM the paper keeps) is
    # checked on sampled outputs against a float64 dot product with the oracle's W_hat.
    spec = syn.TensorSpec("up", 5632, 2048, 1, 128)
    w = syn.weights(spec, 0, device=DEV)
    bt = syn.bitwidths(spec, 0, fixed=6.0, device=DEV)
    d = Desc.make(spec.rows, spec.cols, 1, 128, seed=syn.layer_seed(5, 0), step=0)
    w_hat, sc = gws.sample_fwd(d, w, bt)
    x = torch.randn(16384, 2048, generator=torch.Generator().manual_seed(3)).to(torch.bfloat16).to(DEV)
    y = torch.matmul(x, w_hat.t())
    torch.cuda.synchronize()
    rng = np.random.default_rng(5)
    hat_all, sc_all = orc.sample_fwd(bits_of(w), bt.cpu().numpy(), spec.rows, spec.cols, 1, 128, seed=d.seed, step=0)
    assert np.array_equal(bits_of(w_hat).ravel(), hat_all)                      # all 11,534,336 elements
    assert np.array_equal(sc.cpu().numpy().view(np.uint32), sc_all.view(np.uint32))
    rows = sorted({0, spec.rows - 1, *[int(v) for v in rng.integers(0, spec.rows, 6)]})
    for n in rows:
        hat, _ = orc.sample_fwd(bits_of(w[n:n + 1]), bt[n * 16:(n + 1) * 16].cpu().numpy(), 1, spec.cols, 1, 128, seed=d.seed,
                                step=0, elem_offset=n * spec.cols)
        wn = (hat.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        for m in (0, 16383, int(rng.integers(0, 16384))):
            want = float(x[m].double().cpu().numpy() @ wn)
            got = float(y[m, n])
            # BF16 output rounding (2^-8 relative, with margin) plus FP32 accumulation error relative to sum |x||w|
            budget = 2.0 ** -8 * abs(want) + 1e-5 * float(np.abs(x[m].double().cpu().numpy()) @ np.abs(wn)) + 1e-30
            assert abs(got - want) <= budget, (m, n, got, want)


@pytest.mark.parametrize("fmt_gpu,fmt_orc", [(gws.MX_FP8_E4M3, orc.MX_E4M3), (gws.MX_FP6_E3M2, orc.MX_E3M2), (gws.MX_FP8_E3M4, orc.MX_E3M4)])
def test_config3_with_mx_output_on_row_slices(fmt_gpu, fmt_orc):
    # the whole Llama2-1B-shaped set in one launch with w_hat written as MX; the oracle on a slice of every tensor
    specs = syn.llama2_1b()
    descs = [Desc.make(s.rows, s.cols, 1, s.group_cols, seed=syn.layer_seed(0, i)) for i, s in enumerate(specs)]
    W = [syn.weights(s, i, device=DEV) for i, s in enumerate(specs)]
    BT = [syn.bitwidths(s, i, device=DEV) for i, s in enumerate(specs)]
    SC = [torch.empty(s.n_groups, device=DEV) for s in specs]
    MX = [torch.empty(gws.mx_layout(d, fmt_gpu)[2], dtype=torch.uint8, device=DEV) for d in descs]
    plan = gws.MultiPlan(descs, w=W, bt=BT, w_hat=MX, scale=SC, mx_format=fmt_gpu)
    assert plan.launches_per_pass == 1
    step = 4
    plan.sample_fwd_mx_multi(fmt_gpu, step)
    torch.cuda.synchronize()
    rng = np.random.default_rng(11)
    code_bytes_per_row = lambda cols: cols * 3 // 4 if fmt_orc == orc.MX_E3M2 else cols
    for i, s in enumerate(specs):
        nrows = 4
        r0 = int(rng.integers(0, s.rows - nrows)) if i % 7 else s.rows - nrows      # the last rows of some tensors
        gpr = s.cols // s.group_cols
        hat, _ = orc.sample_fwd(bits_of(W[i][r0:r0 + nrows]), BT[i][r0 * gpr:(r0 + nrows) * gpr].cpu().numpy(), nrows, s.cols, 1,
                                s.group_cols, seed=descs[i].seed, step=step, elem_offset=r0 * s.cols)
        codes, scales = orc.mx_emit(hat, nrows, s.cols, 1, s.group_cols, fmt_orc)
        want_codes = orc.mx_pack6(codes) if fmt_orc == orc.MX_E3M2 else codes
        codes_bytes, scales_off, _ = gws.mx_layout(descs[i], fmt_gpu)
        cb = code_bytes_per_row(s.cols)
        got_codes = MX[i][r0 * cb:(r0 + nrows) * cb].cpu().numpy()
        got_scales = MX[i][scales_off + r0 * s.cols // 32:scales_off + (r0 + nrows) * s.cols // 32].cpu().numpy()
        assert np.array_equal(got_codes, want_codes), (s.name, r0)
        assert np.array_equal(got_scales, scales), (s.name, r0)


def test_config3_cut_into_six_flat_shards_carries_the_bits_of_the_uncut_set():
    # one rank's share of every tensor (6 does not divide them: every shard has a partial group at each end), the other
    # ranks' partial results for those groups supplied from the uncut tensors; forward and backward of the rank
    from paper_2505_11170_b200.sharding import ShardedSetSampler, plan_flat_shard
    specs = syn.llama2_1b(n_blocks=4)
    world, rank, step = 6, 2, 7
    descs, W, BT, G, WH, SC, GBT = _device_set(specs)
    full = gws.MultiPlan(descs, w=W, bt=BT, w_hat=WH, scale=SC, grad_w_hat=G, grad_bt=GBT)
    full.sample_fwd_multi(step)
    full.sample_bwd_multi(step)
    plans = [plan_flat_shard(s.numel, s.group_cols, rank, world) for s in specs]
    cut = lambda t, p: t.view(-1)[p.begin:p.end]
    grp = lambda t, p: t[p.first_group:p.first_group + p.n_local_groups]
    w_hat = [torch.full((p.n_elements,), float("nan"), dtype=torch.bfloat16, device=DEV) for p in plans]
    sh = ShardedSetSampler(plans, [d.seed for d in descs], [cut(W[i], p) for i, p in enumerate(plans)],
                           [grp(BT[i], p) for i, p in enumerate(plans)], w_hat, [cut(G[i], p) for i, p in enumerate(plans)])
    assert sh.n_pieces == sum(len(p.pieces) for p in plans) >= len(specs) and sh.launches_per_forward <= 8
    # forward: what the MAX all-reduce would deliver is the uncut tensor's factor of each shared group
    buf = sh.forward_local(step)
    reduced = buf.clone()
    n_slots = world + 1
    for t, p in enumerate(plans):
        for piece in p.pieces:
            reduced[t * n_slots + piece.read_slot] = SC[t][p.first_group + piece.local_group]
    assert (reduced >= buf).all()                                  # a part's factor never exceeds the group's
    sh.forward_finish(step, reduced)
    # backward: the SUM all-reduce delivers the uncut group's gradient; this rank's share must not exceed it in magnitude
    # by more than rounding, and what it keeps for whole groups must match outright
    buf = sh.backward_local(step)
    reduced = buf.clone()
    for t, p in enumerate(plans):
        for piece in p.pieces:
            reduced[t * n_slots + piece.read_slot] = GBT[t][p.first_group + piece.local_group]
    sh.backward_finish(reduced)
    torch.cuda.synchronize()
    for t, p in enumerate(plans):
        assert torch.equal(w_hat[t].view(torch.int16), cut(WH[t], p).view(torch.int16)), specs[t].name
        assert torch.equal(sh.scale[t].view(torch.int32), grp(SC[t], p).view(torch.int32)), specs[t].name
        assert torch.equal(sh.grad_bt[t].view(torch.int32), grp(GBT[t], p).view(torch.int32)), specs[t].name
