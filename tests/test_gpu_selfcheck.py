"""The self-checking build (-DGWS_SELF_CHECK): every kernel access is tested against a declared window.

With the window set to the arena that holds all tensors, a full forward + backward of every kernel class must report
no violation: no kernel touches memory outside the tensors it was given.  With the window set to the inputs only, the
stores are reported (and skipped) instead of performed.  Runs in a child process because it loads a second build of the
library."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import json, sys
sys.path.insert(0, %(root)r)
import torch
from paper_2505_11170_b200 import _build, binding
from paper_2505_11170_b200.binding import Desc
import os
# the build made with the main library travels with the tree; compiled here only if it is missing or older than its sources
binding.load_library(_build.build(self_check=True))
assert binding.selfcheck_enabled()
dev = "cuda"
arena = torch.zeros(128 << 20, dtype=torch.uint8, device=dev)
cursor = [0]
def carve(nbytes, dtype):
    start = (cursor[0] + 255) // 256 * 256
    cursor[0] = start + nbytes
    assert cursor[0] <= arena.numel()
    return arena[start:start + nbytes].view(dtype)
cases = [(300, 2048, 1, 128), (64, 48, 1, 16), (77, 768, 1, 0), (9, 8192, 1, 0), (5, 28672, 1, 0), (96, 608, 32, 32),
         (33, 40, 32, 32), (21, 520, 1, 0), (3, 65536, 1, 0), (7, 13, 2, 5)]
report = {}
def run_all(window_inputs_only):
    cursor[0] = 0
    ins, outs = [], []
    for k, (rows, cols, gr, gc) in enumerate(cases):
        d = Desc.make(rows, cols, gr, gc, seed=k + 1, step=3)
        ng = binding.n_groups(d)
        w = carve(rows * cols * 2, torch.bfloat16).view(rows, cols); w.copy_((torch.randn(rows, cols, device=dev) * 0.02).to(torch.bfloat16))
        g = carve(rows * cols * 2, torch.bfloat16).view(rows, cols); g.copy_((torch.randn(rows, cols, device=dev) * 1e-4).to(torch.bfloat16))
        bt = carve(ng * 4, torch.float32); bt.fill_(6.0)
        ins.append((d, w, g, bt, ng))
    split = cursor[0]
    for d, w, g, bt, ng in ins:
        mx_ok = d.cols %% 32 == 0 and (d.group_rows, d.group_cols) in ((1, 128), (1, 0), (32, 32)) and d.rows %% d.group_rows == 0 \
            and d.cols <= 32768
        mx = [carve(binding.mx_layout(d, f)[2], torch.uint8) for f in (0, 1)] if mx_ok else None
        outs.append((carve(w.numel() * 2, torch.bfloat16).view_as(w), carve(ng * 4, torch.float32), carve(ng * 4, torch.float32),
                     carve(ng * 4, torch.float32), carve(w.numel() * 2, torch.bfloat16).view_as(w), mx))
    window = arena[:split] if window_inputs_only else arena[:cursor[0]]
    binding.selfcheck_set_window(window)
    for (d, w, g, bt, ng), (w_hat, sc, gbt, am, gw, mx) in zip(ins, outs):
        binding.sample_fwd(d, w, bt, w_hat, sc)
        binding.sample_bwd(d, g, sc, gw, gbt)
        binding.group_absmax(d, w, am)
        binding.scale_from_absmax(am, bt, scale=am)
        binding.sample_fwd_scaled(d, w, am, w_hat)
        if mx is not None:
            for f in (0, 1):
                binding.sample_fwd_mx(d, f, w, bt, mx_out=mx[f], scale_out=sc)
                binding.mx_quantize(d, f, w_hat, mx_out=mx[f])
    torch.cuda.synchronize()
    return binding.selfcheck_report()
report["inside"] = run_all(False)
report["inputs_only"] = run_all(True)
print(json.dumps(report))
"""


@pytest.mark.gpu
def test_no_kernel_leaves_its_tensors_and_outside_accesses_are_skipped_not_performed():
    r = subprocess.run([sys.executable, "-c", CHILD % {"root": ROOT}], capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stderr[-3000:]
    rep = json.loads(r.stdout.strip().splitlines()[-1])
    assert rep["inside"][0] == 0, rep["inside"]                       # violations, kind, address, block, thread
    violations, kind = rep["inputs_only"][0], rep["inputs_only"][1]
    assert violations > 0 and kind in (2, 4, 6)                       # the first access outside the window was a store
