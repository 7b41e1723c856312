"""GaussWSSet: the layers of a model sampled in one launch set per update, against the same layers sampled one by one
(which tests/test_gpu_bitwidth.py holds against the oracle chain) and against the oracle directly."""
import numpy as np
import pytest
import torch

from oracle import gws_oracle as orc
from paper_2505_11170_b200.module import GaussWSLinear, GaussWSSet
from util import bits_of

pytestmark = pytest.mark.gpu
DEV = "cuda"

# (in, out, group): the paper's square blocks, groups of 128, whole rows, and a shape only the general kernel takes
SHAPES = [(256, 96, (32, 32)), (384, 128, (1, 128)), (768, 64, (1, 0)), (96, 160, (32, 32)), (72, 40, (1, 24))]


def _model(lam):
    torch.manual_seed(5)
    layers = [GaussWSLinear(i, o, bias=(k % 2 == 0), group=g, b_init=6.0 + 0.5 * (k % 2), b_target=4.0, lam=lam, user_seed=11, layer_index=k)
              for k, (i, o, g) in enumerate(SHAPES)]
    with torch.no_grad():
        for k, layer in enumerate(layers):
            layer.b_i.uniform_(0.0, 1.3, generator=None)
    return layers


def _clone_into(dst_layers, src_layers):
    with torch.no_grad():
        for d, s in zip(dst_layers, src_layers):
            d.weight.copy_(s.weight)
            d.b_i.copy_(s.b_i)
            if d.bias is not None:
                d.bias.copy_(s.bias)


def _run(layers, xs, ups):
    for k, layer in enumerate(layers):
        y = layer(xs[k])
        y.backward(ups[k])


def _inputs(seed, scale=1e-2):
    g = torch.Generator().manual_seed(seed)
    xs = [torch.randn(24, i, generator=g).to(torch.bfloat16).to(DEV) for i, _, _ in SHAPES]
    ups = [(torch.randn(24, o, generator=g) * scale).to(torch.bfloat16).to(DEV) for _, o, _ in SHAPES]
    return xs, ups


def test_one_micro_batch_per_update_matches_layer_by_layer_sampling():
    one_by_one, together = _model(0.25), _model(0.25)
    _clone_into(together, one_by_one)
    sampler = GaussWSSet(together)
    for update in range(3):
        xs, ups = _inputs(100 + update)
        _run(one_by_one, xs, ups)
        sampler.sample()
        _run(together, xs, ups)
        sampler.finish_backward()
        torch.cuda.synchronize()
        for a, b in zip(one_by_one, together):
            assert torch.equal(a.sampled_weight().detach().view(torch.int16), b.sampled_weight().detach().view(torch.int16))
            assert torch.equal(a.weight.grad.view(torch.int16), b.weight.grad.view(torch.int16))
            # Eq. 4, Eq. 11 and the Eq. 12 term, once: the same numbers up to the order of the FP32 sums
            ga, gb = a.b_i.grad.double(), b.b_i.grad.double()
            assert float((ga - gb).abs().max()) <= 1e-5 * float(ga.abs().max())
        for layer in one_by_one + together:
            layer.weight.grad = None
            layer.b_i.grad = None
        for layer in one_by_one:
            layer.advance()
        sampler.advance()
    # flat groups + whole rows + square blocks + general: one launch per kernel class, not two per layer
    assert 1 <= sampler.launches_per_pass <= 4


def test_sampled_weights_and_bitwidth_gradients_match_the_oracle():
    layers = _model(0.1)
    sampler = GaussWSSet(layers)
    sampler.advance()
    sampler.sample()
    xs, ups = _inputs(7)
    _run(layers, xs, ups)
    sampler.finish_backward()
    torch.cuda.synchronize()
    for k, (layer, (i, o, (gr, gc))) in enumerate(zip(layers, SHAPES)):
        seed = orc.layer_seed(11, k)
        bt = orc.bitwidth(layer.b_i.detach().cpu().numpy(), layer.b_init, 4.0)
        want_hat, want_scale = orc.sample_fwd(bits_of(layer.weight.detach()), bt, o, i, gr, gc, seed=seed, step=1)
        assert (bits_of(layer.sampled_weight().detach()).ravel() == want_hat).all()
        _, want_gbt = orc.sample_bwd(bits_of(layer.weight.grad), want_scale, o, i, gr, gc, seed=seed, step=1)
        want_gbi = orc.bitwidth_grad(want_gbt, bt, layer.b_init, 4.0, 0.1)
        got = layer.b_i.grad.cpu().numpy().astype(np.float64)
        assert np.abs(got - want_gbi).max() <= 1e-5 * np.abs(want_gbi).max()


def test_micro_batches_accumulate_and_the_eq12_term_is_added_once():
    layers = _model(0.3)
    sampler = GaussWSSet(layers)
    sampler.sample()
    for micro in range(3):
        xs, ups = _inputs(40 + micro)
        _run(layers, xs, ups)                       # every pass sees the same sampled weights
    sampler.finish_backward()
    torch.cuda.synchronize()
    for k, (layer, (i, o, (gr, gc))) in enumerate(zip(layers, SHAPES)):
        seed = orc.layer_seed(11, k)
        bt = orc.bitwidth(layer.b_i.detach().cpu().numpy(), layer.b_init, 4.0)
        _, want_scale = orc.sample_fwd(bits_of(layer.weight.detach()), bt, o, i, gr, gc, seed=seed, step=0)
        # Eq. 4 on the accumulated gradient (linear in it), then the Eq. 12 term exactly once
        _, want_gbt = orc.sample_bwd(bits_of(layer.weight.grad), want_scale, o, i, gr, gc, seed=seed, step=0)
        want_gbi = orc.bitwidth_grad(want_gbt, bt, layer.b_init, 4.0, 0.3)
        got = layer.b_i.grad.cpu().numpy().astype(np.float64)
        assert np.abs(got - want_gbi).max() <= 1e-5 * np.abs(want_gbi).max()


def test_misuse_is_reported():
    layers = _model(0.0)
    sampler = GaussWSSet(layers)
    x = torch.randn(4, SHAPES[0][0], device=DEV, dtype=torch.bfloat16)
    with pytest.raises(RuntimeError):
        layers[0](x)                                # no sample() yet for this update
    sampler.sample()
    layers[0](x)
    layers[0].advance()                             # one layer ahead of the others
    with pytest.raises(RuntimeError):
        sampler.sample()
    with pytest.raises(ValueError):
        GaussWSSet(layers)                          # already in a set
    with pytest.raises(ValueError):
        GaussWSSet([])
