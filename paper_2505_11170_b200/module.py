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


class _PresampledWeight(torch.autograd.Function):
    """w -> the w_hat a GaussWSSet has already written for this update; dL/dw = dL/dw_hat (Eq. 4).  The gradient of b_i is
    formed once per update by GaussWSSet.finish_backward from the accumulated dL/dw."""

    @staticmethod
    def forward(ctx, w, w_hat):
        return w_hat.view_as(w_hat)

    @staticmethod
    def backward(ctx, grad_w_hat):
        return grad_w_hat, None


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
        self._set = None
        n_groups = binding.n_groups(self._desc())
        self.b_i = torch.nn.Parameter(torch.ones(n_groups, dtype=torch.float32, device=device))   # Eq. 11: starts at 1

    def _desc(self) -> Desc:
        return Desc.make(self.out_features, self.in_features, self.group[0], self.group[1], seed=self.seed, step=self.step)

    def advance(self) -> None:
        """One gradient update has been applied: the next forward pass draws new noise."""
        self.step += 1
        self._update["lambda_term_due"] = True

    def sampled_weight(self) -> torch.Tensor:
        if self._set is not None:                       # sampled together with the other layers of a GaussWSSet
            return _PresampledWeight.apply(self.weight, self._set.w_hat_of(self))
        return _SampledWeight.apply(self.weight, self.b_i, self._desc(), self.b_init, self.b_target, self.lam, self._update)

    def bitwidth(self) -> torch.Tensor:
        return binding.bitwidth(self.b_i.detach(), self.b_init, self.b_target)

    def bitwidth_loss(self) -> torch.Tensor:
        """This layer's term of Eq. 12 without lambda (a one-element tensor; its gradient is folded into ``b_i.grad``)."""
        return binding.bitwidth_loss(self.bitwidth(), self.b_target)

    def forward(self, x: torch.Tensor) -> torch.Tensor:
        return torch.nn.functional.linear(x, self.sampled_weight(), self.bias)


class GaussWSSet:
    """All GaussWSLinear layers of a model sampled together: the whole sampling pass of an update is one multi-tensor
    launch set forward (gws_sample_fwd_multi) and one backward (gws_sample_bwd_multi) instead of two launches per layer.

        layers = [m for m in model.modules() if isinstance(m, GaussWSLinear)]
        sampler = GaussWSSet(layers)
        for each update:
            sampler.sample()                    # Eq. 11, then Eq. 3 + cast, for every layer at once
            for each micro-batch: loss(model(x)).backward()      # dL/dw accumulates in weight.grad (dL/dw = dL/dw_hat)
            sampler.finish_backward()           # Eq. 4 for every layer at once, then Eq. 11 / Eq. 12 into b_i.grad
            optimizer.step(); optimizer.zero_grad(); sampler.advance()

    Eq. 4's sum is linear in dL/dw_hat and all micro-batches of an update share R and the scale, so dL/db_t is taken once,
    from the accumulated weight.grad, instead of once per micro-batch (with one micro-batch the two are the same numbers; with
    several, weight.grad carries the BF16 rounding of its accumulation).  The Eq. 12 term is added once per
    update.  The layers keep their parameters; the set owns the sampled weights, bit-widths, scales and dL/db_t buffers.
    Every step of the pass runs in the library's kernels; this class only holds tensors and the launch plans.
    """

    def __init__(self, layers):
        self.layers = list(layers)
        if not self.layers:
            raise ValueError("gws: a GaussWSSet needs at least one layer")
        for layer in self.layers:
            if layer._set is not None:
                raise ValueError("gws: a layer belongs to one GaussWSSet at most")
        dev = self.layers[0].weight.device
        self._w_hat = [torch.empty_like(l.weight) for l in self.layers]
        self._bt = [torch.empty(l.b_i.numel(), dtype=torch.float32, device=dev) for l in self.layers]
        self._scale = [torch.empty_like(t) for t in self._bt]
        self._grad_bt = [torch.empty_like(t) for t in self._bt]
        self._index = {id(l): k for k, l in enumerate(self.layers)}
        self._fwd_plan = None
        self._fwd_key = None
        self._bwd_plan = None
        self._bwd_key = None
        self._sampled_step = None
        for layer in self.layers:
            layer._set = self

    def _descs(self):
        return [l._desc() for l in self.layers]

    def w_hat_of(self, layer) -> torch.Tensor:
        if self._sampled_step != self._step():
            raise RuntimeError("gws: call GaussWSSet.sample() once per update before the forward passes")
        return self._w_hat[self._index[id(layer)]]

    def _step(self) -> int:
        steps = {l.step for l in self.layers}
        if len(steps) != 1:
            raise RuntimeError("gws: the layers of a GaussWSSet advance together (GaussWSSet.advance)")
        return steps.pop()

    def sample(self, stream=None) -> None:
        """Eq. 11 for every layer (one launch per 64 layers), then Eq. 3 + the BF16 cast for all of them in one launch per kernel
        class."""
        step = self._step()
        binding.bitwidth_multi([dict(bi=l.b_i.detach(), bt=bt, b_init=l.b_init, b_target=l.b_target) for l, bt in zip(self.layers, self._bt)],
                               stream=stream)
        key = tuple(l.weight.data_ptr() for l in self.layers)
        if key != self._fwd_key:                        # the plan holds the addresses of the weights
            self._fwd_plan = binding.MultiPlan(self._descs(), w=[l.weight.detach() for l in self.layers], bt=self._bt, w_hat=self._w_hat,
                                               scale=self._scale, stream=stream)
            self._fwd_key = key
        self._fwd_plan.sample_fwd_multi(step, stream=stream)
        self._sampled_step = step

    def finish_backward(self, stream=None) -> None:
        """Eq. 4 for every layer from the accumulated dL/dw (one launch per kernel class), then Eq. 11 / Eq. 12: adds
        dL'/db_i of this update to every layer's ``b_i.grad``.  Call once per update, after the last backward pass."""
        step = self._step()
        if self._sampled_step != step:
            raise RuntimeError("gws: finish_backward() belongs to the update that sample() started")
        grads = []
        for layer in self.layers:
            g = layer.weight.grad
            if g is None or not g.is_contiguous() or g.dtype != torch.bfloat16:
                raise RuntimeError("gws: every layer needs a contiguous BF16 weight.grad before finish_backward()")
            grads.append(g)
        key = tuple(g.data_ptr() for g in grads)
        if key != self._bwd_key:                        # the plan holds the addresses of the gradients
            self._bwd_plan = binding.MultiPlan(self._descs(), scale=self._scale, grad_w_hat=grads, grad_bt=self._grad_bt, stream=stream)
            self._bwd_key = key
        self._bwd_plan.sample_bwd_multi(step, stream=stream)
        items = []
        for layer, bt, grad_bt in zip(self.layers, self._bt, self._grad_bt):
            fresh = layer.b_i.grad is None
            if fresh:
                layer.b_i.grad = torch.empty_like(layer.b_i)
            items.append(dict(grad_bt=grad_bt, bt=bt, grad_bi=layer.b_i.grad, b_init=layer.b_init, b_target=layer.b_target, lam=layer.lam,
                              accumulate=not fresh))
        binding.bitwidth_grad_multi(items, stream=stream)

    def advance(self) -> None:
        """One gradient update has been applied to every layer: the next sample() draws new noise."""
        for layer in self.layers:
            layer.advance()

    @property
    def launches_per_pass(self) -> int:
        return self._fwd_plan.launches_per_pass if self._fwd_plan is not None else 0

