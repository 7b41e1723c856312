"""Throughput of the sampling pass on the other workload shapes of the paper (one JSON line each).

    python throughput.py [gpt2] [gpt2_single] [stress] [square] [llama] [mx] [gemm] [issue] [compare] [module] [overhead] [--reps N] [--blocks B]

gpt2         all GPT2-124M linear weights, one group per row (and the same set with groups of 128)
gpt2_single  one GPT2-124M MLP weight, both orientations
stress       4096^2, 8192^2, 28672 x 8192 with groups of 32, 128 and whole rows
square       Llama2-1B-shaped blocks with the paper's 32 x 32 groups (Eq. 3, b_l = 32)
llama        the Llama2-1B-shaped set with groups of 128 (the benchmark's workload; --blocks limits it)
mx           the same set with w_hat written as MX FP8 / FP6 instead of BF16
gemm         sampling fused into a tcgen05 GEMM against sampling + library GEMM against the plain library GEMM
compare      forward pass with the method's noise against the same kernel shape with Box-Muller and with BF16 uniform noise
             (the series "ours", "bm" and the DiffQ-style noise of the paper's forward benchmark), matrices of its range
module       the sampling part of an update through the module wrappers: layer by layer against all layers at once (GaussWSSet)
overhead     the three GEMMs of every linear layer for one micro-batch, with and without the sampling pass around them
issue        cycles per warp instruction of the instruction kinds the passes are made of, and of the passes' arithmetic
             without memory traffic (gws_issue_probe): the terms of the arithmetic ceiling of the backward pass

Every timed pass is one multi-tensor launch set over the whole workload, timed with CUDA events on the launching
stream after three warm-up passes; a 256 MiB buffer is written between passes so that no pass finds its inputs in L2.
Bytes are the algorithmic ones (read W, write w_hat, read b_t, write scale; read grad, read scale, write grad_bt).
With more than one repetition every workload line also times forward + backward as a pair (no event between the two)
and as ten pairs in a row, with ordinary launches and with overlapping ones (gws_set_launch_overlap).
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import torch

_ROOT = os.path.dirname(os.path.abspath(__file__))
if _ROOT not in sys.path:
    sys.path.insert(0, _ROOT)

from paper_2505_11170_b200 import binding as gws       # noqa: E402
from paper_2505_11170_b200 import synthetic as syn     # noqa: E402
from paper_2505_11170_b200.binding import Desc         # noqa: E402


def _peak_gbs() -> float:
    try:
        with open(os.path.join(_ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"])
    except (OSError, KeyError, ValueError):
        return 6650.0


def run(name: str, specs, reps: int, dev, mx_format=None) -> dict:
    n = syn.total_elements(specs)
    descs = [Desc.make(s.rows, s.cols, s.group_rows, s.group_cols, seed=syn.layer_seed(0, i)) for i, s in enumerate(specs)]
    W = [syn.weights(s, i, device=dev) for i, s in enumerate(specs)]
    BT = [syn.bitwidths(s, i, device=dev) for i, s in enumerate(specs)]
    G = [syn.upstream_grad(s, i, device=dev) for i, s in enumerate(specs)]
    if mx_format is None:
        WH = [torch.empty_like(t) for t in W]
        out_bytes = 2.0
    else:
        WH = [torch.empty(gws.mx_layout(d, mx_format)[2], dtype=torch.uint8, device=dev) for d in descs]
        out_bytes = (0.75 if mx_format == gws.MX_FP6_E3M2 else 1.0) + 1.0 / 32.0
    SC = [torch.empty(s.n_groups, device=dev) for s in specs]
    GBT = [torch.empty(s.n_groups, device=dev) for s in specs]
    fwd_plan = gws.MultiPlan(descs, w=W, bt=BT, w_hat=WH, scale=SC, mx_format=mx_format)
    bwd_plan = gws.MultiPlan(descs, scale=SC, grad_w_hat=G, grad_bt=GBT)
    forward = (lambda k: fwd_plan.sample_fwd_multi(k)) if mx_format is None else (lambda k: fwd_plan.sample_fwd_mx_multi(mx_format, k))
    n_groups = sum(s.n_groups for s in specs)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    t_fwd = t_bwd = 0.0
    for k in range(3 + reps):
        flush.zero_()
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        e[0].record()
        forward(k)
        e[1].record()
        bwd_plan.sample_bwd_multi(k)
        e[2].record()
        torch.cuda.synchronize()
        if k >= 3:
            t_fwd += e[0].elapsed_time(e[1])
            t_bwd += e[1].elapsed_time(e[2])
    t_fwd, t_bwd = t_fwd / reps, t_bwd / reps

    # forward + backward as a pair (no event between them) and as ten pairs in a row (after a flush; inside the ten the
    # L2 holds what it can), with ordinary launches and with overlapping ones (gws_set_launch_overlap)
    def pairs(chain: int, overlap: bool) -> float:
        previous = gws.set_launch_overlap(overlap)
        try:
            total = 0.0
            for k in range(3 + reps):
                flush.zero_()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                for c in range(chain):
                    forward(k * chain + c)
                    bwd_plan.sample_bwd_multi(k * chain + c)
                b.record()
                torch.cuda.synchronize()
                if k >= 3:
                    total += a.elapsed_time(b)
        finally:
            gws.set_launch_overlap(previous)
        return total / reps / chain
    pair = {}
    for c in ((1, 10) if reps > 1 else ()):   # --reps 1 is what the profiler commands use: the two timed launches only
        for o in (False, True, False, True):  # off, on, off, on: a drift of the clocks falls on both settings alike
            pair[c, o] = pair.get((c, o), 0.0) + 0.5 * pairs(c, o)
    fwd_bytes = n * (2.0 + out_bytes) + n_groups * 8
    bwd_bytes = n * 2.0 + n_groups * 8
    peak = _peak_gbs()
    line = {"workload": name, "elements": n, "tensors": len(specs), "output": "bf16" if mx_format is None else ("mx_fp8_e4m3", "mx_fp6_e3m2", "mx_fp8_e3m4")[mx_format],
            "fwd_us": t_fwd * 1e3, "fwd_GB/s": fwd_bytes / t_fwd / 1e6, "fwd_frac_of_measured_hbm": fwd_bytes / t_fwd / 1e6 / peak,
            "bwd_us": t_bwd * 1e3, "bwd_GB/s": bwd_bytes / t_bwd / 1e6, "bwd_frac_of_measured_hbm": bwd_bytes / t_bwd / 1e6 / peak,
            "launches_fwd": fwd_plan.launches_per_pass, "launches_bwd": bwd_plan.launches_per_pass, "reps": reps, "l2": "flushed between passes"}
    if pair:
        line.update({"pair_us": pair[1, False] * 1e3, "pair_overlap_us": pair[1, True] * 1e3,
                     "pair_in_chain_of_10_us": pair[10, False] * 1e3, "pair_in_chain_of_10_overlap_us": pair[10, True] * 1e3,
                     "pair_frac_of_measured_hbm": (fwd_bytes + bwd_bytes) / pair[1, False] / 1e6 / peak,
                     "pair_overlap_frac_of_measured_hbm": (fwd_bytes + bwd_bytes) / pair[1, True] / 1e6 / peak})
    print(json.dumps(line), flush=True)
    return line


def run_gemm(reps: int, dev) -> dict:
    """Llama2-1B-shaped up-projection: X [8 x 2048 tokens, 2048] times w_hat^T (W 5632 x 2048, groups of 128, 6 bits):
    sampling fused into the GEMM, against sampling followed by the library GEMM, against the library GEMM on W alone."""
    m, n, k = 16384, 5632, 2048
    spec = syn.TensorSpec("up", n, k, 1, 128)
    w = syn.weights(spec, 0, device=dev)
    bt = syn.bitwidths(spec, 0, fixed=6.0, device=dev)
    x = torch.randn(m, k, generator=torch.Generator(device=dev).manual_seed(3 * 1000003), device=dev).to(torch.bfloat16)
    d = Desc.make(n, k, 1, 128, seed=syn.layer_seed(0, 0))
    y = torch.empty(m, n, dtype=torch.bfloat16, device=dev)
    w_hat = torch.empty_like(w)
    scale = torch.empty(spec.n_groups, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def timed(fn):
        total = 0.0
        for i in range(3 + reps):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn(i)
            b.record()
            torch.cuda.synchronize()
            if i >= 3:
                total += a.elapsed_time(b)
        return total / reps * 1e3

    def unfused(i):
        gws.sample_fwd(d.with_step(i), w, bt, w_hat, scale)
        torch.matmul(x, w_hat.t(), out=y)

    line = {"workload": "up-projection 16384 x 2048 by 5632 x 2048 (groups of 128, 6 bits)", "flops": 2.0 * m * n * k, "reps": reps,
            "plain_gemm_us": timed(lambda i: torch.matmul(x, w.t(), out=y)), "sample_then_gemm_us": timed(unfused)}
    for rpb in (128, 256, 512):
        line[f"fused_{rpb}_rows_per_block_us"] = timed(lambda i: gws.gemm_fused(d.with_step(i), x, w, bt, y=y, status=status, rows_per_block=rpb))
    for c in (1, 2, 4):
        line[f"fused_cluster_of_{c}_us"] = timed(lambda i: gws.gemm_fused(d.with_step(i), x, w, bt, y=y, status=status, cluster=c))
    for c in (1, 2, 4):
        line[f"fused_wide_cluster_of_{c}_us"] = timed(lambda i: gws.gemm_fused(d.with_step(i), x, w, bt, y=y, status=status, cluster=c, wide=True))
    best_wide = min(line[f"fused_wide_cluster_of_{c}_us"] for c in (1, 2, 4))
    line["fused_wide_best_TFLOP/s"] = line["flops"] / (best_wide * 1e-6) / 1e12
    line["overhead_fused_wide_best_pct"] = 100.0 * (best_wide / line["plain_gemm_us"] - 1.0)
    line["status"] = int(status.item())
    line["fused_TFLOP/s"] = line["flops"] / (line["fused_512_rows_per_block_us"] * 1e-6) / 1e12
    line["fused_cluster_of_4_TFLOP/s"] = line["flops"] / (line["fused_cluster_of_4_us"] * 1e-6) / 1e12
    line["overhead_fused_cluster_of_4_pct"] = 100.0 * (line["fused_cluster_of_4_us"] / line["plain_gemm_us"] - 1.0)
    line["overhead_unfused_pct"] = 100.0 * (line["sample_then_gemm_us"] / line["plain_gemm_us"] - 1.0)
    line["overhead_fused_pct"] = 100.0 * (line["fused_512_rows_per_block_us"] / line["plain_gemm_us"] - 1.0)
    print(json.dumps(line), flush=True)
    return line


COMPARE_SHAPES = [(2048, 512), (2048, 2048), (2048, 8192), (4096, 4096), (8192, 8192), (16384, 4096), (16384, 16384)]


def run_compare(reps: int, dev) -> list:
    """Forward pass (Eq. 3 + cast, groups of 128, 6 bits) in 10^9 elements per second with three noises: the method's AND / OR
    generation, the rounded normal from Box-Muller, and BF16 uniform noise; L2 flushed between passes."""
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    lines = []
    for rows, cols in COMPARE_SHAPES:
        spec = syn.TensorSpec("m", rows, cols, 1, 128)
        w, bt = syn.weights(spec, 0, device=dev), syn.bitwidths(spec, 0, fixed=6.0, device=dev)
        d = Desc.make(rows, cols, 1, 128, seed=syn.layer_seed(0, 0))
        w_hat, scale = torch.empty_like(w), torch.empty(spec.n_groups, device=dev)
        calls = {"ours": lambda k: gws.sample_fwd(d.with_step(k), w, bt, w_hat, scale),
                 "bm": lambda k: gws.sample_fwd_compare(d.with_step(k), gws.NOISE_BOX_MULLER, w, bt, w_hat, scale),
                 "uniform_bf16": lambda k: gws.sample_fwd_compare(d.with_step(k), gws.NOISE_UNIFORM_BF16, w, bt, w_hat, scale),
                 "copy": lambda k: w_hat.copy_(w)}
        line = {"workload": f"forward {rows}x{cols}, groups of 128, 6 bits", "elements": rows * cols, "reps": reps}
        for name, fn in calls.items():
            total = 0.0
            for k in range(3 + reps):
                flush.zero_()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                fn(k)
                b.record()
                torch.cuda.synchronize()
                if k >= 3:
                    total += a.elapsed_time(b)
            us = total / reps * 1e3
            line[name + "_us"] = us
            line[name + "_gelem_per_s"] = rows * cols / us / 1e3
        print(json.dumps(line), flush=True)
        lines.append(line)
    return lines


ISSUE_MIXES = list(range(20)) + [101, 103, 107, 109]
_KINDS = ("mul 32x32->64", "xor3 fed by it", "lop3", "ffma", "fma.f32.bf16", "iadd", "prmt")
_BODY = {101: "Philox4x32-10 (hoisted), per 8-element vector", 103: "Philox + gradient decode, per vector",
         107: "Philox + gradient decode + 8 FMAs = backward arithmetic, per vector",
         109: "Philox + forward decode + Eq. 3 add + BF16 packing = forward arithmetic, per vector"}


def run_issue(reps: int, dev) -> list:
    """Cycles per step (or per 8-element vector) and SM sub-partition for every mix of gws_issue_probe.  The SM clock is
    the one the probe measures itself (cycle counter over the nanosecond timer of one warp)."""
    sink = torch.zeros(8, dtype=torch.int32, device=dev)
    lines = []
    ghz = None
    for mix in ISSUE_MIXES:
        steps, counts = gws.issue_probe_mix(mix)
        iterations = 1024 if mix < 100 else 2048
        for _ in range(3):
            blocks, sms = gws.issue_probe(mix, iterations, sink)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            gws.issue_probe(mix, iterations, sink)
        b.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / reps
        if ghz is None:      # from the first probe, which runs for more than a millisecond
            ghz = int(sink[0].item()) / int(sink[1].item())
        warp_steps = blocks * 8 / (sms * 4) * iterations * steps            # per sub-partition
        line = {"mix": mix, "what": _BODY.get(mix) or " + ".join(f"{c} {k}" for c, k in zip(counts, _KINDS) if c),
                "ms": ms, "sm_clock_ghz": ghz, "cycles_per_step_per_subpartition": ms * 1e-3 * ghz * 1e9 / warp_steps}
        print(json.dumps(line), flush=True)
        lines.append(line)
    return lines


def run_module(reps: int, dev, n_blocks: int) -> dict:
    """The module wrappers on the Llama2-1B-shaped layer set (the paper's 32 x 32 groups): the sampling part of an update
    (Eq. 11, Eq. 3 forward; Eq. 4, Eq. 11 / Eq. 12 backward) layer by layer, as GaussWSLinear does on its own, against all
    layers at once through GaussWSSet.  No GEMMs: weight.grad is filled with synthetic gradients.  Host time included (events
    on the stream around the Python calls)."""
    from paper_2505_11170_b200.module import GaussWSLinear, GaussWSSet
    specs = syn.llama2_1b(n_blocks=n_blocks)

    def build():
        layers = [GaussWSLinear(s.cols, s.rows, bias=False, group=(32, 32), lam=0.1, layer_index=k, device=dev) for k, s in enumerate(specs)]
        for k, (layer, s) in enumerate(zip(layers, specs)):
            layer.weight.grad = syn.upstream_grad(s, k, device=dev)
        return layers
    alone, together = build(), build()
    sampler = GaussWSSet(together)

    def timed(fn):
        total = 0.0
        for i in range(3 + reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize()
            if i >= 3:
                total += a.elapsed_time(b)
        return total / reps

    def alone_fwd():
        for layer in alone:
            layer.sampled_weight()

    saved = []
    for layer in alone:                                   # what a layer's forward pass keeps for its backward pass
        bt = layer.bitwidth()
        saved.append((bt, gws.sample_fwd(layer._desc(), layer.weight.detach(), bt)[1]))

    def alone_bwd():
        for layer, (bt, scale) in zip(alone, saved):
            _, grad_bt = gws.sample_bwd(layer._desc(), layer.weight.grad, scale)
            gws.bitwidth_grad(grad_bt, bt, layer.b_init, layer.b_target, layer.lam)
    n = syn.total_elements(specs)
    with torch.no_grad():
        fwd_alone = timed(alone_fwd)
    bwd_alone = timed(alone_bwd)
    fwd_set = timed(sampler.sample)
    bwd_set = timed(sampler.finish_backward)
    line = {"workload": f"module wrappers, llama2_1b {n_blocks} blocks, 32x32 groups", "layers": len(specs), "elements": n,
            "forward_layer_by_layer_ms": fwd_alone, "forward_set_ms": fwd_set, "backward_layer_by_layer_ms": bwd_alone, "backward_set_ms": bwd_set,
            "launches_per_pass_set": sampler.launches_per_pass, "reps": reps}
    print(json.dumps(line), flush=True)
    return line


def run_overhead(reps: int, dev, n_blocks: int, tokens: int = 16384) -> dict:
    """What the sampling pass adds to the linear layers of a training step (the kind of number Table 1 of the paper gives for
    whole steps): for every Llama2-1B-shaped linear layer the three BF16 GEMMs of a micro-batch of `tokens` tokens (y = x W^T,
    dx = dy W, dW = dy^T x; torch's GEMMs on synthetic activations), once on the master weights and once on weights sampled
    by GaussWSSet with Eq. 4 / Eq. 11 / Eq. 12 at the end of the step.  No attention, norms or optimizer: the percentage is
    an upper bound on the overhead of a full step."""
    from paper_2505_11170_b200.module import GaussWSLinear, GaussWSSet
    specs = syn.llama2_1b(n_blocks=n_blocks)
    layers = [GaussWSLinear(s.cols, s.rows, bias=False, group=(32, 32), lam=0.1, layer_index=k, device=dev) for k, s in enumerate(specs)]
    sampler = GaussWSSet(layers)
    gen = torch.Generator(device=dev).manual_seed(1)
    xs = {c: torch.randn(tokens, c, generator=gen, device=dev).to(torch.bfloat16) for c in {s.cols for s in specs}}
    dys = {r: (torch.randn(tokens, r, generator=gen, device=dev) * 1e-2).to(torch.bfloat16) for r in {s.rows for s in specs}}
    ys = {r: torch.empty(tokens, r, dtype=torch.bfloat16, device=dev) for r in dys}
    dxs = {c: torch.empty(tokens, c, dtype=torch.bfloat16, device=dev) for c in xs}
    for layer in layers:
        layer.weight.grad = torch.empty_like(layer.weight)

    def gemms(weights):
        for layer, s, w in zip(layers, specs, weights):
            torch.mm(xs[s.cols], w.t(), out=ys[s.rows])
            torch.mm(dys[s.rows], w, out=dxs[s.cols])
            torch.mm(dys[s.rows].t(), xs[s.cols], out=layer.weight.grad)

    def plain():
        gemms([l.weight.detach() for l in layers])

    def sampled():
        sampler.sample()
        gemms([sampler.w_hat_of(l) for l in layers])
        sampler.finish_backward()
        sampler.advance()

    def timed(fn):
        total = 0.0
        for i in range(2 + reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize()
            if i >= 2:
                total += a.elapsed_time(b)
        return total / reps
    with torch.no_grad():
        t_plain, t_sampled, t_plain2 = timed(plain), timed(sampled), timed(plain)
    base = 0.5 * (t_plain + t_plain2)
    flops = 6.0 * syn.total_elements(specs) * tokens
    line = {"workload": f"linear layers of llama2_1b ({n_blocks} blocks), one micro-batch of {tokens} tokens, 32x32 groups",
            "gemms_only_ms": base, "gemms_with_sampling_ms": t_sampled, "overhead_pct": 100.0 * (t_sampled / base - 1.0),
            "gemm_TFLOP/s": flops / (base * 1e-3) / 1e12, "reps": reps}
    print(json.dumps(line), flush=True)
    return line


def main(argv=None) -> None:
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("which", nargs="*", default=["gpt2", "stress"])
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--blocks", type=int, default=22, help="transformer blocks of the Llama-shaped sets")
    args = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise SystemExit("a CUDA device is needed: the sampling pass has no CPU path")
    gws.load_library()
    dev = torch.device("cuda", 0)
    for w in args.which:
        if w == "gpt2":
            run("gpt2_124m all linear weights, row groups", syn.gpt2_124m_all(), args.reps, dev)
            run("gpt2_124m all linear weights, groups of 128", syn.gpt2_124m_all(128), args.reps, dev)
        elif w == "gpt2_single":
            run("gpt2_124m fc 3072x768, row groups", syn.gpt2_124m_single(), args.reps, dev)
            run("gpt2_124m fc 768x3072 (literal orientation), row groups", syn.gpt2_124m_single(True), args.reps, dev)
        elif w == "stress":
            for rows, cols in syn.STRESS_SHAPES:
                for g in syn.STRESS_GROUPS:
                    run(f"{rows}x{cols}, groups of {g or 'one row'}", [syn.stress_case(rows, cols, g)], args.reps, dev)
        elif w == "square":
            specs = [syn.TensorSpec(s.name, s.rows, s.cols, 32, 32) for s in syn.llama2_1b(n_blocks=min(args.blocks, 4))]
            run(f"llama2_1b blocks 0-{min(args.blocks, 4) - 1}, 32x32 groups", specs, args.reps, dev)
        elif w == "llama":
            run(f"llama2_1b {args.blocks} blocks, groups of 128", syn.llama2_1b(n_blocks=args.blocks), args.reps, dev)
        elif w == "gemm":
            run_gemm(args.reps, dev)
        elif w == "overhead":
            run_overhead(max(1, args.reps // 4), dev, args.blocks)
        elif w == "module":
            run_module(args.reps, dev, args.blocks)
        elif w == "issue":
            run_issue(args.reps, dev)
        elif w == "compare":
            run_compare(args.reps, dev)
        elif w == "mx":
            for fmt in (gws.MX_FP8_E4M3, gws.MX_FP6_E3M2, gws.MX_FP8_E3M4):
                run(f"llama2_1b {args.blocks} blocks, groups of 128", syn.llama2_1b(n_blocks=args.blocks), args.reps, dev, mx_format=fmt)
        else:
            raise SystemExit(f"unknown workload {w!r}")


if __name__ == "__main__":
    main(sys.argv[1:])
