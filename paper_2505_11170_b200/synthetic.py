"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws numbers and lists shapes; it contains none of the
sampling method's arithmetic, so both the CUDA tests and the CPU oracle may be
fed from it.  The paper trains GPT2-124M and Llama2 models (Section 4); their
trained weights need its datasets, so weights here are BF16 N(0, sigma^2) in
the same layer shapes, upstream gradients BF16 N(0, (1e-4)^2), and per-group
bit-widths integers uniform on {4..9} (the range Section 3.3 and Figure 5
motivate) stored as FP32.

Storage convention: a linear layer "in x out" is allocated as rows = out,
cols = in (the layout of ``torch.nn.Linear.weight``), so groups of contiguous
elements run along the input dimension.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

import torch

BASE_W, BASE_G, BASE_BT, BASE_X, BASE_OUTLIER = 0, 1, 2, 3, 4


@dataclass(frozen=True)
class TensorSpec:
    name: str
    rows: int
    cols: int
    group_rows: int
    group_cols: int  # 0 = whole row

    @property
    def numel(self) -> int:
        return self.rows * self.cols

    @property
    def n_groups(self) -> int:
        gc = self.cols if self.group_cols == 0 else self.group_cols
        return -(-self.rows // self.group_rows) * -(-self.cols // gc)


def _gen(base: int, index: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(base * 1000003 + index)
    return g


def weights(spec: TensorSpec, index: int, sigma: float = 0.02, device="cpu", base: int = BASE_W) -> torch.Tensor:
    """BF16 [rows, cols] ~ N(0, sigma^2), rounded from FP32 draws."""
    x = torch.randn(spec.rows, spec.cols, generator=_gen(base, index, device), device=device, dtype=torch.float32)
    return (x * sigma).to(torch.bfloat16)


def upstream_grad(spec: TensorSpec, index: int, sigma: float = 1e-4, device="cpu") -> torch.Tensor:
    return weights(spec, index, sigma=sigma, device=device, base=BASE_G)


def bitwidths(spec: TensorSpec, index: int, lo: int = 4, hi: int = 9, fixed: Optional[float] = None,
              device="cpu") -> torch.Tensor:
    """FP32 [n_groups]: integers uniform on {lo..hi}, or the constant ``fixed``."""
    if fixed is not None:
        return torch.full((spec.n_groups,), float(fixed), dtype=torch.float32, device=device)
    b = torch.randint(lo, hi + 1, (spec.n_groups,), generator=_gen(BASE_BT, index, device), device=device)
    return b.to(torch.float32)


def add_outliers(w: torch.Tensor, index: int, sigma: float, fraction: float = 1e-3, magnitude: float = 8.0):
    """Overwrite ``fraction`` of the entries, at seeded positions, with +-magnitude*sigma (in place)."""
    n = w.numel()
    k = max(1, int(round(n * fraction)))
    g = _gen(BASE_OUTLIER, index, w.device)
    pos = torch.randint(0, n, (k,), generator=g, device=w.device)
    sign = torch.randint(0, 2, (k,), generator=g, device=w.device).to(torch.float32) * 2.0 - 1.0
    w.view(-1)[pos] = (sign * (magnitude * sigma)).to(w.dtype)
    return w


def layer_seed(user_seed: int, layer_index: int) -> int:
    """A 64-bit per-layer seed (stands in for the per-layer host PRNG of Section 3.6).

    A splitmix-style integer hash; any injective-looking map would do."""
    z = (user_seed * 0x9E3779B97F4A7C15 + (layer_index + 1) * 0xBF58476D1CE4E5B9) & 0xFFFFFFFFFFFFFFFF
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & 0xFFFFFFFFFFFFFFFF
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & 0xFFFFFFFFFFFFFFFF
    return z ^ (z >> 31)


# ---- workloads -----------------------------------------------------------------

def gpt2_124m_single(literal_orientation: bool = False) -> List[TensorSpec]:
    """One GPT2-124M MLP weight (768 -> 3072), one group per storage row."""
    if literal_orientation:
        return [TensorSpec("fc_literal", 768, 3072, 1, 0)]
    return [TensorSpec("fc", 3072, 768, 1, 0)]


def gpt2_124m_all(group_cols: int = 0) -> List[TensorSpec]:
    """All linear weights of GPT2-124M: 12 blocks x {qkv, attn-proj, fc, mlp-proj}; 84,934,656 elements."""
    out = []
    for b in range(12):
        out += [TensorSpec(f"h{b}.qkv", 2304, 768, 1, group_cols), TensorSpec(f"h{b}.attn_proj", 768, 768, 1, group_cols),
                TensorSpec(f"h{b}.fc", 3072, 768, 1, group_cols), TensorSpec(f"h{b}.mlp_proj", 768, 3072, 1, group_cols)]
    return out


def llama2_1b(group_cols: int = 128, n_blocks: int = 22) -> List[TensorSpec]:
    """Llama2-style ~1B linear weights: 22 blocks, d_model 2048, d_ff 5632; 1,130,364,928 elements."""
    out = []
    for b in range(n_blocks):
        out += [TensorSpec(f"l{b}.{n}", 2048, 2048, 1, group_cols) for n in ("q", "k", "v", "o")]
        out += [TensorSpec(f"l{b}.gate", 5632, 2048, 1, group_cols), TensorSpec(f"l{b}.up", 5632, 2048, 1, group_cols),
                TensorSpec(f"l{b}.down", 2048, 5632, 1, group_cols)]
    return out


STRESS_SHAPES = [(4096, 4096), (8192, 8192), (28672, 8192)]
STRESS_SIGMAS = [0.002, 0.02, 0.2]
STRESS_GROUPS = [32, 128, 0]
STRESS_BITS = [4.0, 9.0]


def stress_case(rows: int, cols: int, group_cols: int) -> TensorSpec:
    return TensorSpec(f"stress_{rows}x{cols}_g{group_cols or 'row'}", rows, cols, 1, group_cols)


def total_elements(specs: List[TensorSpec]) -> int:
    return sum(s.numel for s in specs)


def shard(specs: List[TensorSpec], rank: int, world: int) -> List[int]:
    """Indices of the tensors rank ``rank`` of ``world`` owns: round-robin over the list.

    Every group is independent, so a data-parallel split needs no exchange step; for the
    benchmark at N GPUs each rank instead holds a full replica of the set (weak scaling)."""
    return [i for i in range(len(specs)) if i % world == rank]
