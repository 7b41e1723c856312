"""The paper's "single PyTorch module" (Section 3.5, last paragraph) on top of the C ABI.

``GaussWSLinear`` is a linear layer whose weight is sampled at every forward pass:

    b_t  = b_target + b_i * (b_init - b_target)                      Eq. 11, one b_i per group
    w_hat = bf16( w + R * max_group|w| * 2^(1 - b_t) )               Eq. 3 + cast   (gws_sample_fwd)
    y    = x @ w_hat^T + bias                                        stock BF16 GEMM, as in the paper

and whose backward pass returns dL/dw = dL/dw_hat, dL/db_i through Eq. 4 (gws_sample_bwd, R regenerated from
the same (seed, step)) and Eq. 11 / Eq. 12 (gws_bitwidth_grad).  The module only wires tensors to the library:
every step of the sampling pass runs in its kernels.  The GEMMs are torch's, exactly as the paper keeps them.
"""
from __future__ import annotations

from typing import Optional

import torch

from . import binding
from .binding import Desc


class _SampledWeight(torch.autograd.Function):
    """(w, b_i) -> w_hat with the gradients of Eq. 4 and Eq. 11 / Eq. 12."""

    @staticmethod
    def forward(ctx, w, bi, desc, b_init, b_target, lam, update):
        bt = binding.bitwidth(bi.detach(), b_init, b_target)
        w_hat, scale = binding.sample_fwd(desc, w.detach(), bt)
        ctx.save_for_backward(scale, bt)
        ctx.desc, ctx.hyper, ctx.update = desc, (b_init, b_target, lam), update
        return w_hat

    @staticmethod
    def backward(ctx, grad_w_hat):
        scale, bt = ctx.saved_tensors
        b_init, b_target, lam = ctx.hyper
        g = grad_w_hat.contiguous()
        _, grad_bt = binding.sample_bwd(ctx.desc, g, scale)                 # dL/dw is dL/dw_hat itself (Eq. 4)
        # Eq. 12 adds its term once per gradient update, however many micro-batches are accumulated into b_i.grad:
        # the first backward pass of an update carries it, the others are the plain chain rule.
        first = ctx.update["lambda_term_due"]
        ctx.update["lambda_term_due"] = False
        grad_bi = binding.bitwidth_grad(grad_bt, bt, b_init, b_target, lam if first else 0.0)
        return g, grad_bi, None, None, None, None, None


class GaussWSLinear(torch.nn.Module):
    """Linear layer trained with Gaussian weight sampling.

    ``group`` is (group_rows, group_cols); the paper's choice is the 32 x 32 square block.  ``layer_index`` and
    ``user_seed`` give the layer its own noise stream (Section 3.6); call :meth:`advance` once per gradient update
    (not per micro-batch) so that forward and backward of one update see the same noise and the next update a new one.
    ``lam`` > 0 adds this layer's term of Eq. 12 to the gradient of ``b_i``, once per update: the first backward pass
    after construction or :meth:`advance` carries it, so accumulating k micro-batches does not multiply lambda by k;
    :meth:`bitwidth_loss` returns the term's value.
    """

    def __init__(self, in_features: int, out_features: int, bias: bool = True, group=(32, 32), b_init: float = 6.0,
                 b_target: float = 4.0, lam: float = 0.0, user_seed: int = 0, layer_index: int = 0, device="cuda"):
        super().__init__()
        self.in_features, self.out_features = in_features, out_features
        self.group, self.b_init, self.b_target, self.lam = tuple(group), float(b_init), float(b_target), float(lam)
        self.weight = torch.nn.Parameter(torch.empty(out_features, in_features, dtype=torch.bfloat16, device=device))
        torch.nn.init.normal_(self.weight, std=0.02)
        self.bias = torch.nn.Parameter(torch.zeros(out_features, dtype=torch.bfloat16, device=device)) if bias else None
        self.seed = binding.layer_seed(user_seed, layer_index)
        self.step = 0
        self._update = {"lambda_term_due": True}
        n_groups = binding.n_groups(self._desc())
        self.b_i = torch.nn.Parameter(torch.ones(n_groups, dtype=torch.float32, device=device))   # Eq. 11: starts at 1

    def _desc(self) -> Desc:
        return Desc.make(self.out_features, self.in_features, self.group[0], self.group[1], seed=self.seed, step=self.step)

    def advance(self) -> None:
        """One gradient update has been applied: the next forward pass draws new noise."""
        self.step += 1
        self._update["lambda_term_due"] = True

    def sampled_weight(self) -> torch.Tensor:
        return _SampledWeight.apply(self.weight, self.b_i, self._desc(), self.b_init, self.b_target, self.lam, self._update)

    def bitwidth(self) -> torch.Tensor:
        return binding.bitwidth(self.b_i.detach(), self.b_init, self.b_target)

    def bitwidth_loss(self) -> torch.Tensor:
        """This layer's term of Eq. 12 without lambda (a one-element tensor; its gradient is folded into ``b_i.grad``)."""
        return binding.bitwidth_loss(self.bitwidth(), self.b_target)

    def forward(self, x: torch.Tensor) -> torch.Tensor:
        return torch.nn.functional.linear(x, self.sampled_weight(), self.bias)
