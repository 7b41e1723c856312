"""Runs the CPU oracle over many tensors at once: one single-threaded oracle process per host core, disjoint tensors.

TEST INFRASTRUCTURE ONLY, like the rest of this directory.  The oracle itself is untouched: every worker process calls
``gws_oracle.sample_fwd`` / ``gws_oracle.sample_bwd`` exactly as a test would, on the tensors it was given.  The pool
only spreads whole tensors over processes so that a weight set of a billion elements is checked (and timed) in seconds
instead of minutes.  Arrays travel as ``.npy`` files in a scratch directory (shared memory if it has the room), which
the workers map instead of copying.

    with OraclePool() as pool:
        res = pool.run(tasks)          # tasks: dicts with rows, cols, group_rows, group_cols, seed, step, w, bt, g
        res["w_hat"][i], res["scale"][i], res["grad_bt"][i]     # read-only arrays, valid inside the with block
        res["grad_bt_bound"][i]        # with bound=True: ln2 * s_g * sum_group |g * R| per group (float64), the quantity
                                       # a relative tolerance on the gradient sum is relative to; 1 x G groups only

Worker entry point: ``python -m oracle.pool <scratch directory> <worker index>``.
"""
from __future__ import annotations

import json
import os
import shutil
import subprocess
import sys
import tempfile
import time

import numpy as np

_ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _scratch_parent(need_bytes: int) -> str:
    for cand in ("/dev/shm", tempfile.gettempdir()):
        try:
            st = os.statvfs(cand)
            if st.f_bavail * st.f_frsize > need_bytes * 1.2 + (64 << 20):
                return cand
        except OSError:
            continue
    return tempfile.gettempdir()


class OraclePool:
    def __init__(self, procs: int | None = None):
        self.procs = procs or os.cpu_count() or 1
        self.dir = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def close(self):
        if self.dir is not None:
            shutil.rmtree(self.dir, ignore_errors=True)
            self.dir = None

    def run(self, tasks, keep_outputs: bool = True, bound: bool = False) -> dict:
        """Forward (and, where a task has ``g``, backward) of every task.  Returns the outputs (lists parallel to
        ``tasks``; None where not produced), the wall time from the first oracle call of any worker to the last
        one's return, the summed in-call time, the element count and the number of worker processes used."""
        from oracle import gws_oracle
        gws_oracle.build()                 # once, here, not in every worker
        self.close()
        need = sum(int(t["w"].nbytes) * (2 + (1 if t.get("g") is not None else 0)) for t in tasks)
        self.dir = tempfile.mkdtemp(prefix="gws_oracle_pool_", dir=_scratch_parent(need))
        meta = []
        for i, t in enumerate(tasks):
            np.save(os.path.join(self.dir, f"w_{i}.npy"), np.ascontiguousarray(t["w"], dtype=np.uint16))
            np.save(os.path.join(self.dir, f"bt_{i}.npy"), np.ascontiguousarray(t["bt"], dtype=np.float32))
            if t.get("g") is not None:
                np.save(os.path.join(self.dir, f"g_{i}.npy"), np.ascontiguousarray(t["g"], dtype=np.uint16))
            meta.append({k: int(t[k]) for k in ("rows", "cols", "group_rows", "group_cols", "seed", "step")} |
                        {"elem_offset": int(t.get("elem_offset", 0)), "bwd": t.get("g") is not None, "index": i, "bound": bool(bound)})
        # longest tensors first, each to the least loaded worker
        n_workers = max(1, min(self.procs, len(tasks)))
        load, share = [0] * n_workers, [[] for _ in range(n_workers)]
        for m in sorted(meta, key=lambda m: -m["rows"] * m["cols"]):
            k = load.index(min(load))
            share[k].append(m)
            load[k] += m["rows"] * m["cols"]
        with open(os.path.join(self.dir, "tasks.json"), "w") as f:
            json.dump({"share": share, "keep_outputs": keep_outputs}, f)
        env = dict(os.environ, OMP_NUM_THREADS="1", OPENBLAS_NUM_THREADS="1", MKL_NUM_THREADS="1")
        workers = [subprocess.Popen([sys.executable, "-m", "oracle.pool", self.dir, str(k)], cwd=_ROOT, env=env)
                   for k in range(n_workers)]
        codes = [w.wait() for w in workers]
        if any(codes):
            raise RuntimeError(f"oracle worker processes failed: exit codes {codes}")
        results = []
        for k in range(n_workers):
            with open(os.path.join(self.dir, f"result_{k}.json")) as f:
                results.append(json.load(f))
        load_out = lambda name, i: np.load(os.path.join(self.dir, f"{name}_{i}.npy"), mmap_mode="r")
        out = {"w_hat": [None] * len(tasks), "scale": [None] * len(tasks), "grad_bt": [None] * len(tasks),
               "grad_bt_bound": [None] * len(tasks)}
        if keep_outputs:
            for m in meta:
                i = m["index"]
                out["w_hat"][i], out["scale"][i] = load_out("what", i), load_out("scale", i)
                if m["bwd"]:
                    out["grad_bt"][i] = load_out("gbt", i)
                    if m["bound"]:
                        out["grad_bt_bound"][i] = load_out("den", i)
        out.update({"seconds": max(r["end"] for r in results) - min(r["start"] for r in results),
                    "seconds_in_calls": sum(r["in_calls"] for r in results),
                    "elements": sum(m["rows"] * m["cols"] for m in meta), "processes": n_workers, "threads_per_process": 1})
        return out


def _worker(scratch: str, k: int) -> None:
    from oracle import gws_oracle as orc
    with open(os.path.join(scratch, "tasks.json")) as f:
        spec = json.load(f)
    mine, keep = spec["share"][k], spec["keep_outputs"]
    orc.lib()
    load = lambda name, i: np.load(os.path.join(scratch, f"{name}_{i}.npy"), mmap_mode="r")
    start, in_calls = time.time(), 0.0
    for m in mine:
        i = m["index"]
        w, bt = load("w", i), load("bt", i)
        geo = dict(rows=m["rows"], cols=m["cols"], group_rows=m["group_rows"], group_cols=m["group_cols"], seed=m["seed"],
                   step=m["step"], elem_offset=m["elem_offset"])
        t0 = time.perf_counter()
        w_hat, scale = orc.sample_fwd(w, bt, **geo)
        in_calls += time.perf_counter() - t0
        gbt = None
        if m["bwd"]:
            g = load("g", i)
            t0 = time.perf_counter()
            _, gbt = orc.sample_bwd(g, scale, **geo)
            in_calls += time.perf_counter() - t0
        if keep:
            np.save(os.path.join(scratch, f"what_{i}.npy"), w_hat)
            np.save(os.path.join(scratch, f"scale_{i}.npy"), scale)
            if gbt is not None:
                np.save(os.path.join(scratch, f"gbt_{i}.npy"), gbt)
                if m["bound"]:
                    gc = m["group_cols"] or m["cols"]
                    assert m["group_rows"] == 1 and m["cols"] % gc == 0
                    n = m["rows"] * m["cols"]
                    r = orc.noise_r(m["seed"], m["step"], m["elem_offset"], n).astype(np.float64)
                    gf = (np.asarray(g, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)
                    sums = np.abs(gf.reshape(-1)[:n] * r).reshape(-1, gc).sum(axis=1)
                    np.save(os.path.join(scratch, f"den_{i}.npy"), np.log(2.0) * scale.astype(np.float64) * sums)
    end = time.time()
    with open(os.path.join(scratch, f"result_{k}.json"), "w") as f:
        json.dump({"start": start, "end": end, "in_calls": in_calls, "tensors": len(mine)}, f)


if __name__ == "__main__":
    _worker(sys.argv[1], int(sys.argv[2]))
