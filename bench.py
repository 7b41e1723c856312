#!/usr/bin/env python
"""Benchmark of the GaussWS weight-sampling pass on B200.

One "step" = the workload's ten consecutive gradient-update counters: ten times one forward pass
(Eq. 3 + BF16 cast) plus one backward pass (Eq. 4, noise regenerated) over the whole Llama2-1B-shaped
linear weight set (154 tensors, 1,130,364,928 BF16 elements, groups of 128 along the input dimension,
b_t uniform on {4..9}), each pass one launch.  Inputs are synthetic (seeded N(0, 0.02^2) weights,
N(0, 1e-4^2) upstream gradients) and resident in HBM when the timed region starts; every pass streams
2.26 GB per tensor set, far beyond L2.  `value` comes from exactly --steps steps; the roofline
fractions are reported twice: over the first 20 launches of each kernel (a burst at full clocks) and
sustained (everything after the first 0.3 s, the run extended to at least 1.5 s of device time).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle on a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "sampling fwd+bwd GB/s and Gelem/s at 1 B200; fraction of HBM peak"
WORKLOAD = "llama2_1b_linear_set_g128"
PASSES_PER_STEP = 10                       # the workload names ten consecutive step counters
SUSTAIN_MS = 1500.0                        # device time the launch stream is extended to for the sustained figures
BURST_LAUNCHES = 20
FWD_BYTES_PER_ELEM = 2 + 2 + 8 / 128      # read w, write w_hat, read b_t + write scale per 128 elements
BWD_BYTES_PER_ELEM = 2 + 8 / 128          # read dL/dw_hat, read scale + write dL/db_t per 128 elements
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0                   # B200 HBM3e data-sheet figure, for context beside the measured copy peak


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return FALLBACK_HBM_GBS, "fallback"


PROFILE = os.path.join(ROOT, "profiles", "k_flat_llama2_1b_g128.md")
CSRC = os.path.join(ROOT, "paper_2505_11170_b200", "csrc")


def kernel_source_hash() -> str:
    """Hash of the device code (comments and white space removed) and of the tile-shape macros of the host file:
    what has to be unchanged for ncu counters to still describe the kernels."""
    import hashlib
    import re
    h = hashlib.sha256()
    for name in ("gws_kernels.cuh", "gws_math.cuh"):
        with open(os.path.join(CSRC, name)) as f:
            text = f.read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        text = re.sub(r"//[^\n]*", "", text)
        h.update(re.sub(r"\s+", " ", text).encode())
    with open(os.path.join(CSRC, "gws_api.cu")) as f:
        h.update(" ".join(sorted(re.findall(r"#define\s+GWS_FLAT_CPT_\w+\s+\d+", f.read()))).encode())
    return h.hexdigest()[:16]


def ncu_traffic():
    """Per-launch DRAM bytes from the committed ncu summary: its line
    ``bench: fwd_bytes_per_launch=<n> bwd_bytes_per_launch=<n> sources=<hash>``.
    Empty (traffic null) if there is no summary or the kernel sources changed since the counters were taken."""
    if not os.path.exists(PROFILE):
        return {}
    with open(PROFILE) as f:
        for line in f:
            if line.startswith("bench:"):
                kv = dict(item.split("=", 1) for item in line.split()[1:])
                if kv.get("sources") != kernel_source_hash():
                    return {}
                return {k: int(v) for k, v in kv.items() if k.endswith("_bytes_per_launch")}
    return {}


def max_over_ranks(values, dist, device):
    """Element-wise maximum of a list of per-rank numbers over all ranks (the values themselves if not distributed)."""
    t = torch.tensor([float(v) for v in values], device=device, dtype=torch.float64)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def whole_job_throughput(units_per_rank: float, world: int, ms_per_step: float) -> float:
    """Units per second of the whole job: every rank processes ``units_per_rank`` per step (replicas, weak scaling)
    and a step takes as long as the slowest rank."""
    return world * units_per_rank / (ms_per_step * 1e-3)


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.samples = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.QUERY,
                                          "--format=csv,noheader,nounits", "-lms", "20"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append((time.time(), line.strip()))

    def stop(self):
        if self.proc is None:
            return
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()

    def window(self, t0: float, t1: float):
        """Median SM clock and the throttle reasons seen between two wall-clock times."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        rows = [s for (t, s) in self.samples if t0 - 0.03 <= t <= t1 + 0.03]
        if not rows:      # a window shorter than the sampling period: the nearest sample
            mid = 0.5 * (t0 + t1)
            rows = [min(self.samples, key=lambda ts: abs(ts[0] - mid))[1]] if self.samples else []
        mhz, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            f = [x.strip() for x in r.split(",")]
            try:
                mhz.append(float(f[0]))
                mx = float(f[1])
            except Exception:
                continue
            for name, val in zip(names, f[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        mhz.sort()
        return {"sm_mhz": mhz[len(mhz) // 2] if mhz else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(mhz)}


def run_reference(args, rank: int, world: int):
    """The CPU oracle, as it stands, on a bounded sample of the workload (rank 0 only)."""
    if rank != 0:
        return
    import numpy as np
    from oracle import gws_oracle as orc
    from paper_2505_11170_b200 import synthetic as syn
    specs = syn.llama2_1b()
    sample = [0, 4]                       # l0.q (2048x2048) and l0.gate (5632x2048): 15.7 M elements
    data = []
    for i in sample:
        s = specs[i]
        as_bits = lambda t: t.view(torch.int16).numpy().view(np.uint16)
        data.append((s, syn.layer_seed(0, i), as_bits(syn.weights(s, i)), syn.bitwidths(s, i).numpy(),
                     as_bits(syn.upstream_grad(s, i))))
    elems = sum(d[0].numel for d in data)

    def step(k):
        for s, seed, w, bt, g in data:
            _, sc = orc.sample_fwd(w, bt, s.rows, s.cols, 1, s.group_cols, seed=seed, step=k)
            orc.sample_bwd(g, sc, s.rows, s.cols, 1, s.group_cols, seed=seed, step=k)

    for k in range(args.warmup):
        step(k)
    t0 = time.perf_counter()
    for k in range(args.steps):
        step(args.warmup + k)
    dt = time.perf_counter() - t0
    gbs = elems * (FWD_BYTES_PER_ELEM + BWD_BYTES_PER_ELEM) * args.steps / dt / 1e9
    sample_text = ("tensors l0.q and l0.gate of the 154 (15,728,640 of 1,130,364,928 elements), one forward + backward pass "
                   "(one step counter of the ten) per step")
    line = {"impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16 storage, f32 arithmetic (f64 gradient sum)", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sample": sample_text},
            "gelem_per_s": elems * args.steps / dt / 1e9,
            "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample_text},
            "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# Instructions the backward kernel k_flat<bwd> executes per 8-element vector and thread, by kind: the Philox4x32-10 and
# decode counts follow from the source (18 multiplies 32x32->64 and 19 XORs after hoisting; 13 logic operations, 1 right
# and 6 left shifts for the gradient decode; 8 mixed-precision FMAs), `other` is what ncu counts beyond them
# (sm__inst_executed_pipe_alu minus the above: index arithmetic, predicates, the tile lookup), see profiles/.
BWD_INSTRUCTIONS_PER_VECTOR = {"mul_wide": 18, "xor3": 19, "logic": 14, "shl": 6, "fma_bf16": 8, "other_alu": 5}


def arithmetic_budget(gws, dev):
    """Cost of each instruction kind on this chip (gws_issue_probe, cycles per warp instruction and SM sub-partition,
    from an additive fit that the mixed probes confirm), the cycles per 8-element vector they add up to for the backward
    pass, and the element rate that budget allows at the measured SM clock."""
    sink = torch.zeros(8, dtype=torch.int32, device=dev)

    clock = {}

    def cycles(mix, iterations):
        steps, _ = gws.issue_probe_mix(mix)
        for _ in range(2):
            blocks, sms = gws.issue_probe(mix, iterations, sink)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(5):
            gws.issue_probe(mix, iterations, sink)
        b.record()
        torch.cuda.synchronize()
        # the SM clock comes from the first (longest) probe: cycle counter over nanosecond timer of one of its warps
        ghz = clock.setdefault("ghz", int(sink[0].item()) / max(int(sink[1].item()), 1))
        warp_steps = blocks * 8 / (sms * 4) * iterations * steps
        return a.elapsed_time(b) / 5 * 1e-3 * ghz * 1e9 / warp_steps, ghz, sms

    c_round, ghz, sms = cycles(0, 1024)
    c_logic = cycles(10, 1024)[0]
    c_round_2logic = cycles(2, 1024)[0]
    c_fma = (cycles(8, 1024)[0] - c_round) / 2.0     # the cost of an FMA next to integer work, which is how the pass runs it
    c_add = (cycles(9, 1024)[0] - c_round) / 2.0
    c_mul = (c_round - 2.0 * c_logic) / 2.0          # additive: a round is 2 multiplies + 2 XORs
    n = BWD_INSTRUCTIONS_PER_VECTOR
    terms = {"mul_wide": n["mul_wide"] * c_mul, "xor3": n["xor3"] * c_logic, "logic": n["logic"] * c_logic,
             "shl": n["shl"] * c_add, "fma_bf16": n["fma_bf16"] * c_fma, "other_alu": n["other_alu"] * c_logic}
    budget = sum(terms.values())
    body = cycles(107, 2048)[0]
    rate = lambda cyc: sms * 4 * ghz * 1e9 / cyc * 32 * 8 / 1e9            # Gelem/s at `cyc` cycles per warp-vector
    return {"cycles_per_warp_instruction": {"philox_round_2mul_2xor": c_round, "logic_op": c_logic, "mul_wide_from_round": c_mul,
                                            "fma_f32_bf16_beside_a_round": c_fma, "integer_add_beside_a_round": c_add,
                                            "philox_round_plus_2_logic_ops": c_round_2logic,
                                            "additive_prediction_of_that": c_round + 2.0 * c_logic},
            "bwd_instructions_per_vector": n, "bwd_cycles_per_vector_terms": terms, "bwd_cycles_per_vector_budget": budget,
            "bwd_cycles_per_vector_arithmetic_only_measured": body, "sm_clock_ghz": ghz, "sms": sms,
            "bwd_ceiling_gelem_per_s": rate(budget),
            "bwd_arithmetic_only_gelem_per_s": rate(body),
            "bwd_ceiling_is": "sum over instruction kinds of (instructions per 8-element vector) x (measured cycles per warp "
                              "instruction), at the SM clock the probes measured"}


def sharded_step_leg(make_sampler, specs, rank, world, dist, device, timer, reps=10):
    """The one form of the pass that has an exchange step: every tensor cut into `world` flat shards (ZeRO / FSDP style),
    each rank sampling its shard; groups that reach across a cut go through a MAX all-reduce (forward) and a SUM all-reduce
    (backward) of world + 1 floats per tensor.  `make_sampler(plans)` returns an object with forward(step) / backward(step)
    that does the rank's local work and the all-reduces; `timer(fn, reps)` returns milliseconds per call on this rank.
    Returns the whole-job figures (maximum over ranks of the time, sum over ranks of the elements)."""
    from paper_2505_11170_b200.sharding import plan_flat_shard
    plans = [plan_flat_shard(s.rows * s.cols, s.group_cols or s.cols, rank, world) for s in specs]
    sampler = make_sampler(plans)
    fwd_ms = timer(lambda k: sampler.forward(k), reps)
    bwd_ms = timer(lambda k: sampler.backward(k), reps)
    mine = float(sum(p.n_elements for p in plans))
    fwd_ms, bwd_ms = max_over_ranks([fwd_ms, bwd_ms], dist, device)
    t = torch.tensor([mine, float(sum(len(p.pieces) for p in plans))], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
    elems, pieces = float(t[0]), int(t[1])
    return {"world": world, "elements": int(elems), "end_pieces_all_ranks": pieces, "fwd_ms": fwd_ms, "bwd_ms": bwd_ms,
            "fwd_GB/s": elems * FWD_BYTES_PER_ELEM / (fwd_ms * 1e-3) / 1e9, "bwd_GB/s": elems * BWD_BYTES_PER_ELEM / (bwd_ms * 1e-3) / 1e9,
            "all_reduce_floats_per_pass": len(specs) * (world + 1),
            "note": "whole job: every rank samples 1/world of every tensor; times are the slowest rank's, all-reduces included"}


def cpu_baseline(specs, descs, W, BT, G):
    """The oracle, as it stands, on one full forward + backward pass of the whole weight set (one step counter):
    one single-threaded oracle process per host core, each with its own tensors (oracle/pool.py)."""
    import numpy as np
    from oracle.pool import OraclePool
    as_bits = lambda t: t.cpu().view(torch.int16).numpy().view(np.uint16)
    tasks = [dict(rows=s.rows, cols=s.cols, group_rows=1, group_cols=s.group_cols, seed=descs[i].seed, step=0, w=as_bits(W[i]),
                  bt=BT[i].cpu().numpy(), g=as_bits(G[i])) for i, s in enumerate(specs)]
    with OraclePool() as pool:
        res = pool.run(tasks, keep_outputs=False)
    elems, t = res["elements"], res["seconds"]
    return {"value": elems * (FWD_BYTES_PER_ELEM + BWD_BYTES_PER_ELEM) / t / 1e9, "unit": "GB/s", "cores": res["processes"],
            "kind": "oracle", "gelem_per_s": elems / t / 1e9, "seconds": t, "host_cores": os.cpu_count(),
            "processes": res["processes"], "threads_per_process": 1,
            "single_thread_gelem_per_s": elems / res["seconds_in_calls"] / 1e9,
            "sample": "the whole set: %d tensors, %d elements, one forward + backward pass (one step counter of the ten)"
                      % (len(specs), elems)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None, help="timed steps (default 100; 3 for --impl reference)")
    ap.add_argument("--warmup", type=int, default=None, help="untimed steps (default 5, at least 3; 1 for --impl reference)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--blocks", type=int, default=22, help="Llama blocks in the set (22 = the full workload)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the side measurements (per-layer launches, copy mode, ALU ceiling)")
    ap.add_argument("--no-sustain", action="store_true", help="do not extend the launch stream beyond --steps (profiler runs)")
    ap.add_argument("--source-hash", action="store_true", help="print the hash an ncu summary records with its counters")
    args = ap.parse_args()
    if args.impl == "ours":
        args.steps = 100 if args.steps is None else args.steps            # ~1.3 s of device time at N = 1
        args.warmup = 3 if args.warmup is None else max(args.warmup, 3)
    else:
        args.steps = 3 if args.steps is None else args.steps              # ~2.4 s of CPU time per step
        args.warmup = 1 if args.warmup is None else args.warmup

    if args.source_hash:
        print(kernel_source_hash())
        return
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    import paper_2505_11170_b200 as gws
    from paper_2505_11170_b200 import synthetic as syn
    from paper_2505_11170_b200.binding import Desc

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the sampling pass has no CPU path")
    gws.load_library()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    # Every rank holds a full replica of the weight set (the pass has no exchange step): weak scaling.
    specs = syn.llama2_1b(n_blocks=args.blocks)
    n_elem = syn.total_elements(specs)
    descs = [Desc.make(s.rows, s.cols, 1, s.group_cols, seed=syn.layer_seed(rank, i)) for i, s in enumerate(specs)]
    W = [syn.weights(s, i, device=dev) for i, s in enumerate(specs)]
    BT = [syn.bitwidths(s, i, device=dev) for i, s in enumerate(specs)]
    G = [syn.upstream_grad(s, i, device=dev) for i, s in enumerate(specs)]
    WH = [torch.empty_like(t) for t in W]
    SC = [torch.empty(s.n_groups, device=dev) for s in specs]
    GBT = [torch.empty(s.n_groups, device=dev) for s in specs]
    plan = gws.MultiPlan(descs, w=W, bt=BT, w_hat=WH, scale=SC, grad_w_hat=G, grad_bt=GBT)
    stream = torch.cuda.current_stream()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def one_step(counter0, events=None):
        """The ten step counters of one step; with `events`, an event after every launch."""
        for j in range(PASSES_PER_STEP):
            if events is not None:
                e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
                e[0].record(stream)
            plan.sample_fwd_multi(counter0 + j, stream)
            if events is not None:
                e[1].record(stream)
            plan.sample_bwd_multi(counter0 + j, stream)
            if events is not None:
                e[2].record(stream)
                events.append(e)

    counter = 0
    for _ in range(args.warmup):
        one_step(counter)
        counter += PASSES_PER_STEP
    barrier()

    # ---- device-resident timing: K steps, an event after every launch; the same launch stream then runs on until
    # ---- it has covered SUSTAIN_MS, which is where the sustained roofline fractions come from
    ev = []
    sampler = ClockSampler(local_rank) if rank == 0 else None
    launches0 = gws.launch_count()
    barrier()
    t_wall0 = time.time()
    for k in range(args.steps):
        one_step(counter, ev)
        counter += PASSES_PER_STEP
    n_timed = len(ev)
    launches = gws.launch_count() - launches0
    while True:      # extension: whole steps, decided from the measured time of what has run so far
        ev[-1][2].synchronize()
        done_ms = ev[0][0].elapsed_time(ev[-1][2])
        if done_ms >= SUSTAIN_MS or args.no_sustain:
            break
        per_step = done_ms / (len(ev) / PASSES_PER_STEP)
        for _ in range(max(1, int((SUSTAIN_MS - done_ms) / per_step) + 1)):
            one_step(counter, ev)
            counter += PASSES_PER_STEP
    barrier()
    if sampler:
        sampler.stop()
    total_ms = ev[0][0].elapsed_time(ev[n_timed - 1][2])
    fwd_all = [e[0].elapsed_time(e[1]) for e in ev]
    bwd_all = [e[1].elapsed_time(e[2]) for e in ev]
    offset = [ev[0][0].elapsed_time(e[0]) for e in ev]                   # ms from the start of the timed region
    mean = lambda xs: sum(xs) / max(len(xs), 1)
    sustained = [i for i, t in enumerate(offset) if t >= 300.0] or list(range(len(ev)))
    burst = list(range(min(BURST_LAUNCHES, len(ev))))
    fwd_ms, bwd_ms = mean(fwd_all[:n_timed]), mean(bwd_all[:n_timed])
    fwd_burst, bwd_burst = mean([fwd_all[i] for i in burst]), mean([bwd_all[i] for i in burst])
    fwd_sus, bwd_sus = mean([fwd_all[i] for i in sustained]), mean([bwd_all[i] for i in sustained])
    total_ms, fwd_ms, bwd_ms, fwd_burst, bwd_burst, fwd_sus, bwd_sus = max_over_ranks(
        [total_ms, fwd_ms, bwd_ms, fwd_burst, bwd_burst, fwd_sus, bwd_sus], dist, dev)
    clocks = None
    if sampler:
        wall = lambda i, j=0: t_wall0 + ev[0][0].elapsed_time(ev[i][j]) * 1e-3
        clocks = sampler.window(t_wall0, wall(n_timed - 1, 2))
        clocks["burst"] = sampler.window(t_wall0, wall(burst[-1], 2))
        clocks["sustained"] = sampler.window(wall(sustained[0]), wall(sustained[-1], 2))
        clocks["sustained"]["device_ms"] = ev[sustained[0]][0].elapsed_time(ev[sustained[-1]][2])
    ms_per_step = total_ms / args.steps
    bytes_per_pass = n_elem * (FWD_BYTES_PER_ELEM + BWD_BYTES_PER_ELEM)
    bytes_per_step = bytes_per_pass * PASSES_PER_STEP
    value = whole_job_throughput(bytes_per_step, world, ms_per_step) / 1e9
    gelem = whole_job_throughput(n_elem * PASSES_PER_STEP, world, ms_per_step) / 1e9

    # ---- end to end through the host-buffer entry point: pinned host tensors in, results out ----
    e2e = None
    if not args.no_e2e:
        pin = lambda x: x.cpu().pin_memory()
        block = list(range(min(7, len(specs))))            # one transformer block of pinned host buffers, reused
        hW, hBT, hG = [pin(W[i]) for i in block], [pin(BT[i]) for i in block], [pin(G[i]) for i in block]
        hWH = [torch.empty_like(x).pin_memory() for x in hW]
        hSC = [torch.empty_like(x).pin_memory() for x in hBT]
        hGBT = [torch.empty_like(x).pin_memory() for x in hBT]

        # One stream per set of pinned buffers: the upload of one tensor overlaps the download of another (the two copy
        # directions use different engines), and tensors that share pinned buffers share a stream, which orders them.
        side = [torch.cuda.Stream(device=dev) for _ in range(len(block))]

        def host_step(k):
            for st in side:
                st.wait_stream(stream)
            for i in range(len(specs)):
                j = i % len(block)
                gws.sample_step_host(descs[i].with_step(k), hW[j], hBT[j], hG[j], hWH[j], hSC[j], hGBT[j], W[i], WH[i], G[i],
                                     BT[i], SC[i], GBT[i], side[j % len(side)])
            for st in side:
                stream.wait_stream(st)

        host_step(0)
        barrier()
        e2e_steps = 1                                      # one step = ten passes, about a second behind the host link
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for k in range(e2e_steps * PASSES_PER_STEP):
            host_step(1 + k)
        e1.record(stream)
        barrier()
        e2e_ms = max_over_ranks([e0.elapsed_time(e1) / e2e_steps], dist, dev)[0]
        n_groups = sum(s.n_groups for s in specs)
        e2e = {"value": whole_job_throughput(bytes_per_step, world, e2e_ms) / 1e9, "unit": "GB/s",
               "h2d_bytes_per_step": int(n_elem * 4 + n_groups * 4) * PASSES_PER_STEP,
               "d2h_bytes_per_step": int(n_elem * 2 + n_groups * 8) * PASSES_PER_STEP,
               "ms_per_step": float(e2e_ms), "steps": e2e_steps,
               "note": "gws_sample_step_host per tensor on seven streams; pinned host buffers of one transformer block reused "
                       "for all 22; bound by the host link (6.9 GB cross it per step)"}

    # ---- side measurements (one GPU only; not part of `value`) ----
    extras = None
    if world == 1 and not args.no_extras:
        def timed(fn, reps):
            fn(0)
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for k in range(reps):
                fn(1 + k)
            b.record(stream)
            torch.cuda.synchronize()
            return a.elapsed_time(b) / reps

        def per_layer(k):
            for i in range(len(specs)):
                d = descs[i].with_step(k)
                gws.sample_fwd(d, W[i], BT[i], WH[i], SC[i], stream=stream)
                gws.sample_bwd(d, G[i], SC[i], None, GBT[i], stream=stream)

        per_layer_ms = timed(per_layer, 5)
        previous_overlap = gws.set_launch_overlap(True)     # the same 308 launches, each allowed to start while the one before drains
        try:
            per_layer_overlap_ms = timed(per_layer, 5)
        finally:
            gws.set_launch_overlap(previous_overlap)
        GW = [torch.empty_like(t) for t in G]
        copy_plan = gws.MultiPlan(descs, scale=SC, grad_w_hat=G, grad_w=GW, grad_bt=GBT)
        bwd_copy_ms = timed(lambda k: copy_plan.sample_bwd_multi(k), 10)
        del copy_plan, GW
        alu = arithmetic_budget(gws, dev)
        # one rank's share of the same set with every tensor cut into 6 flat shards (6 does not divide the tensors, so
        # every shard has a partial group at each end): the local work of a sharded step, without the two small
        # all-reduces a real job adds
        from paper_2505_11170_b200.sharding import ShardedSetSampler, plan_flat_shard
        shard_world, shard_rank = 6, 2
        sh_plans = [plan_flat_shard(s_.rows * s_.cols, s_.group_cols or s_.cols, shard_rank, shard_world) for s_ in specs]
        cut = lambda t, p_: t.view(-1)[p_.begin:p_.end]
        sh = ShardedSetSampler(sh_plans, [d.seed for d in descs], [cut(W[i], p_) for i, p_ in enumerate(sh_plans)],
                               [BT[i][p_.first_group:p_.first_group + p_.n_local_groups] for i, p_ in enumerate(sh_plans)],
                               [cut(WH[i], p_) for i, p_ in enumerate(sh_plans)], [cut(G[i], p_) for i, p_ in enumerate(sh_plans)])
        sh_elems = sum(p_.n_elements for p_ in sh_plans)
        sh_fwd_ms = timed(lambda k: sh.forward_finish(k, sh.forward_local(k)), 20)
        sh_bwd_ms = timed(lambda k: sh.backward_finish(sh.backward_local(k)), 20)
        # forward pass with w_hat written as MX floating point instead of BF16 (Table C.1's datatypes for w_hat)
        fwd_mx = {}
        for name, fmt, code_bytes in (("fp8_e4m3", gws.MX_FP8_E4M3, 1.0), ("fp6_e3m2", gws.MX_FP6_E3M2, 0.75)):
            MX = [torch.empty(gws.mx_layout(d, fmt)[2], dtype=torch.uint8, device=dev) for d in descs]
            mx_plan = gws.MultiPlan(descs, w=W, bt=BT, w_hat=MX, scale=SC, mx_format=fmt)
            ms = timed(lambda k: mx_plan.sample_fwd_mx_multi(fmt, k), 20)
            per_elem = 2 + code_bytes + 1 / 32 + 8 / 128
            fwd_mx[name] = {"ms_per_launch": ms, "bytes_per_element": per_elem, "GB/s": n_elem * per_elem / (ms * 1e-3) / 1e9,
                            "gelem_per_s": n_elem / (ms * 1e-3) / 1e9}
            # the conversion alone, from the BF16 w_hat of the last forward pass: one launch over the whole set
            q_plan = gws.MultiPlan(descs, w=WH, w_hat=MX, mx_format=fmt)
            q_ms = timed(lambda k: q_plan.mx_quantize_multi(fmt), 10)
            q_gbs = n_elem * (2 + code_bytes + 1 / 32) / (q_ms * 1e-3) / 1e9
            fwd_mx[name]["quantize_only"] = {"ms": q_ms, "launches": q_plan.launches_per_pass, "GB/s": q_gbs,
                                             "frac_of_measured_hbm": q_gbs / measured_peaks()[0]}
            del mx_plan, q_plan, MX
        extras = {
            "fwd_mx_output": fwd_mx,
            "sharded_rank_local_work": {"world": shard_world, "rank": shard_rank, "elements": sh_elems, "end_pieces": sh.n_pieces,
                                        "fwd_ms": sh_fwd_ms, "bwd_ms": sh_bwd_ms, "launches_per_forward": sh.launches_per_forward,
                                        "fwd_GB/s": sh_elems * FWD_BYTES_PER_ELEM / (sh_fwd_ms * 1e-3) / 1e9,
                                        "bwd_GB/s": sh_elems * BWD_BYTES_PER_ELEM / (sh_bwd_ms * 1e-3) / 1e9,
                                        "note": "each pass reads %.2f GB, more than L2; a real job adds two all-reduces of %d floats" % (sh_elems * 2 / 1e9, len(specs) * (shard_world + 1))},
            "per_layer_launches": {"ms_per_pass": per_layer_ms, "launches_per_pass": 2 * len(specs),
                                   "GB/s": bytes_per_pass / (per_layer_ms * 1e-3) / 1e9,
                                   "ms_per_pass_overlapping_launches": per_layer_overlap_ms,
                                   "GB/s_overlapping_launches": bytes_per_pass / (per_layer_overlap_ms * 1e-3) / 1e9},
            "bwd_with_grad_w_copy": {"ms_per_launch": bwd_copy_ms, "GB/s": n_elem * (4 + 8 / 128) / (bwd_copy_ms * 1e-3) / 1e9,
                                     "bytes_per_element": 4 + 8 / 128},
            "arithmetic_budget": alu,
        }

    # ---- N > 1 only: the sharded form of the step, the one place where ranks exchange anything ----
    sharded = None
    if world > 1 and not args.no_extras:
        from paper_2505_11170_b200.sharding import ShardedSetSampler
        cut = lambda t, p_: t.view(-1)[p_.begin:p_.end]

        def make_sampler(plans):
            return ShardedSetSampler(plans, [d.seed for d in descs], [cut(W[i], p_) for i, p_ in enumerate(plans)],
                                     [BT[i][p_.first_group:p_.first_group + p_.n_local_groups].contiguous() for i, p_ in enumerate(plans)],
                                     [cut(WH[i], p_) for i, p_ in enumerate(plans)], [cut(G[i], p_) for i, p_ in enumerate(plans)])

        def rank_timer(fn, reps):
            fn(0)
            barrier()
            a_, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a_.record(stream)
            for k in range(reps):
                fn(1 + k)
            b_.record(stream)
            barrier()
            return a_.elapsed_time(b_) / reps

        sharded = sharded_step_leg(make_sampler, specs, rank, world, dist, dev, rank_timer)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peaks()
    traffic = ncu_traffic()
    fwd_bytes = n_elem * FWD_BYTES_PER_ELEM
    bwd_bytes = n_elem * BWD_BYTES_PER_ELEM
    gbs = lambda nbytes, ms: nbytes / (ms * 1e-3) / 1e9
    fwd_gbs, bwd_gbs = gbs(fwd_bytes, fwd_sus), gbs(bwd_bytes, bwd_sus)
    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 storage, f32 arithmetic", "data": "synthetic",
        "config": {"workload": WORKLOAD, "tensors": len(specs), "elements": n_elem, "group": "1x128",
                   "bits": "uniform integers 4..9", "passes": "forward + backward (identity grad_w), one launch each",
                   "step": "%d consecutive step counters = %d forward + %d backward launches" % (PASSES_PER_STEP, PASSES_PER_STEP, PASSES_PER_STEP),
                   "l2": "inputs larger than L2: each pass streams %.2f GB" % (n_elem * 2 / 1e9),
                   "multi_gpu": "replicas only (no exchange step in the path)"},
        "gelem_per_s": gelem, "hbm_frac": value / world / peak, "hbm_frac_of_nominal_8000": value / world / NOMINAL_HBM_GBS,
        "roofline": {"bound": "hbm", "kernel": "k_flat<fwd> (gws_sample_fwd_multi)", "achieved": fwd_gbs, "peak": peak,
                     "peak_kind": peak_kind, "unit": "GB/s", "frac": fwd_gbs / peak, "frac_of_nominal_8000": fwd_gbs / NOMINAL_HBM_GBS,
                     "frac_is": "sustained: launches after the first 0.3 s of a launch stream of at least %.1f s" % (SUSTAIN_MS * 1e-3),
                     "ms_per_launch": fwd_sus, "frac_burst": gbs(fwd_bytes, fwd_burst) / peak, "ms_per_launch_burst": fwd_burst,
                     "frac_timed_steps": gbs(fwd_bytes, fwd_ms) / peak, "ms_per_launch_timed_steps": fwd_ms,
                     "algorithmic_bytes_per_launch": fwd_bytes, "traffic": traffic.get("fwd_bytes_per_launch")},
        "roofline_bwd": {"bound": "hbm", "kernel": "k_flat<bwd> (gws_sample_bwd_multi)", "achieved": bwd_gbs, "peak": peak,
                         "unit": "GB/s", "frac": bwd_gbs / peak, "ms_per_launch": bwd_sus,
                         "frac_burst": gbs(bwd_bytes, bwd_burst) / peak, "ms_per_launch_burst": bwd_burst,
                         "frac_timed_steps": gbs(bwd_bytes, bwd_ms) / peak, "ms_per_launch_timed_steps": bwd_ms,
                         "algorithmic_bytes_per_launch": bwd_bytes, "traffic": traffic.get("bwd_bytes_per_launch")},
        "clocks": clocks, "gpu_launches": int(launches), "e2e": e2e,
    }
    if sharded is not None:
        line["extras"] = {"sharded_step": sharded}
    if extras is not None:
        line["extras"] = extras
        # the backward pass is bound by integer instruction issue, not by HBM: also report it against the ceiling that
        # follows from the instructions it executes per 8 elements and what each kind costs on this chip
        alu = extras["arithmetic_budget"]
        ceiling = alu["bwd_ceiling_gelem_per_s"]
        line["roofline_bwd"].update({"arithmetic_ceiling_gelem_per_s": ceiling,
                                     "frac_of_arithmetic_ceiling": n_elem / (bwd_sus * 1e-3) / 1e9 / ceiling,
                                     "frac_of_arithmetic_ceiling_burst": n_elem / (bwd_burst * 1e-3) / 1e9 / ceiling,
                                     "arithmetic_ceiling_is": alu["bwd_ceiling_is"]})
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(specs, descs, W, BT, G)
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
