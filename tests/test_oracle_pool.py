"""The process pool that spreads the oracle over host cores returns exactly what the oracle returns when called
directly, tensor by tensor and row band by row band (a band with elem_offset = first_row * cols carries the noise of
the uncut tensor), and its gradient bound is the sum it says it is."""
import numpy as np

from oracle import gws_oracle as orc
from oracle.pool import OraclePool


def _tensor(rng, rows, cols):
    return (rng.integers(0, 2 ** 16, size=(rows, cols), dtype=np.uint16) & 0xBFFF).astype(np.uint16)   # no Inf / NaN patterns


def test_pool_outputs_equal_direct_oracle_calls():
    rng = np.random.default_rng(0)
    tasks = []
    for i, (r, c, gc) in enumerate([(64, 256, 128), (33, 96, 32), (10, 100, 48), (8, 512, 0)]):
        ng = orc.n_groups(r, c, 1, gc)
        tasks.append(dict(rows=r, cols=c, group_rows=1, group_cols=gc, seed=123 + i, step=7, w=_tensor(rng, r, c),
                          bt=rng.integers(4, 10, size=ng).astype(np.float32), g=_tensor(rng, r, c) if i != 1 else None))
    with OraclePool(3) as pool:
        res = pool.run(tasks)
        assert res["processes"] == 3 and res["elements"] == sum(t["rows"] * t["cols"] for t in tasks)
        for i, t in enumerate(tasks):
            hat, sc = orc.sample_fwd(t["w"], t["bt"], t["rows"], t["cols"], 1, t["group_cols"], seed=t["seed"], step=7)
            assert np.array_equal(np.asarray(res["w_hat"][i]).ravel(), hat.ravel())
            assert np.array_equal(np.asarray(res["scale"][i]).view(np.uint32), sc.view(np.uint32))
            if t["g"] is None:
                assert res["grad_bt"][i] is None
            else:
                _, gbt = orc.sample_bwd(t["g"], sc, t["rows"], t["cols"], 1, t["group_cols"], seed=t["seed"], step=7)
                assert np.array_equal(np.asarray(res["grad_bt"][i]).view(np.uint32), gbt.view(np.uint32))


def test_row_bands_reproduce_the_uncut_tensor_and_the_bound_is_the_sum_of_magnitudes():
    rng = np.random.default_rng(1)
    rows, cols, gc = 24, 256, 64
    w, g = _tensor(rng, rows, cols), _tensor(rng, rows, cols)
    bt = rng.integers(4, 10, size=rows * cols // gc).astype(np.float32)
    hat, sc = orc.sample_fwd(w, bt, rows, cols, 1, gc, seed=9, step=2)
    _, gbt = orc.sample_bwd(g, sc, rows, cols, 1, gc, seed=9, step=2)
    gpr = cols // gc
    bands = [(0, 7), (7, 9), (16, 8)]
    tasks = [dict(rows=n, cols=cols, group_rows=1, group_cols=gc, seed=9, step=2, elem_offset=r0 * cols, w=w[r0:r0 + n],
                  bt=bt[r0 * gpr:(r0 + n) * gpr], g=g[r0:r0 + n]) for r0, n in bands]
    with OraclePool(2) as pool:
        res = pool.run(tasks, bound=True)
        r = orc.noise_r(9, 2, 0, rows * cols).astype(np.float64)
        gf = (g.astype(np.uint32) << 16).view(np.float32).astype(np.float64).ravel()
        den = np.log(2.0) * sc.astype(np.float64) * np.abs(gf * r).reshape(-1, gc).sum(axis=1)
        for k, (r0, n) in enumerate(bands):
            assert np.array_equal(np.asarray(res["w_hat"][k]).reshape(n, cols), hat.reshape(rows, cols)[r0:r0 + n])
            gsl = slice(r0 * gpr, (r0 + n) * gpr)
            assert np.array_equal(np.asarray(res["scale"][k]).view(np.uint32), sc[gsl].view(np.uint32))
            assert np.array_equal(np.asarray(res["grad_bt"][k]).view(np.uint32), gbt[gsl].view(np.uint32))
            assert np.allclose(np.asarray(res["grad_bt_bound"][k]), den[gsl], rtol=1e-12, atol=0)
