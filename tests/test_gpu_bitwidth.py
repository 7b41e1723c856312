"""Eq. 11 / Eq. 12 kernels and the module wrapper against the oracle (GPU)."""
import numpy as np
import pytest
import torch

import paper_2505_11170_b200 as gws
from oracle import gws_oracle as orc
from paper_2505_11170_b200.binding import Desc
from paper_2505_11170_b200.module import GaussWSLinear
from util import bits_of

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("n", [1, 255, 4096, 100003])
def test_eq11_bit_exact_and_in_place(n):
    bi = torch.empty(n).uniform_(-0.5, 1.5, generator=torch.Generator().manual_seed(n))
    for b_init, b_target in ((6.0, 4.0), (6.3, 3.9), (8.0, 0.0)):
        want = orc.bitwidth(bi.numpy(), b_init, b_target)
        got = gws.bitwidth(bi.to(DEV), b_init, b_target)
        assert (got.cpu().numpy().view(np.uint32) == want.view(np.uint32)).all()
    x = bi.to(DEV)
    gws.bitwidth(x, 6.0, 4.0, bt=x)
    assert (x.cpu().numpy().view(np.uint32) == orc.bitwidth(bi.numpy(), 6.0, 4.0).view(np.uint32)).all()


@pytest.mark.parametrize("m", [1, 31, 1024, 90112])
def test_eq12_loss_and_gradient(m):
    g = torch.Generator().manual_seed(m)
    bt = torch.empty(m).uniform_(2, 9, generator=g)
    bt[::7] = 4.0                                                    # exactly on target: sign = 0
    grad_bt = torch.randn(m, generator=g) * 1e-3
    want_loss = orc.bitwidth_loss(bt.numpy(), 4.0)
    got_loss = float(gws.bitwidth_loss(bt.to(DEV), 4.0).cpu())
    assert abs(got_loss - want_loss) <= 1e-5 * want_loss
    for lam in (0.0, 0.37):
        want = orc.bitwidth_grad(grad_bt.numpy(), bt.numpy(), 6.0, 4.0, lam)
        got = gws.bitwidth_grad(grad_bt.to(DEV), bt.to(DEV), 6.0, 4.0, lam).cpu().numpy().astype(np.float64)
        assert np.abs(got - want).max() <= 1e-6 * np.abs(want).max()
    assert float(gws.bitwidth_loss(torch.empty(0, device=DEV), 4.0).cpu()) == 0.0


def test_layer_seed_matches_oracle():
    for user in (0, 12345, (1 << 64) - 1):
        for layer in (0, 1, 153, 1 << 35):
            assert gws.layer_seed(user, layer) == orc.layer_seed(user, layer)


@pytest.mark.parametrize("group", [(32, 32), (1, 128), (1, 0)])
def test_module_forward_backward_match_the_oracle_chain(group):
    torch.manual_seed(0)
    layer = GaussWSLinear(256, 96, bias=True, group=group, b_init=6.0, b_target=4.0, lam=0.25, user_seed=7, layer_index=3)
    with torch.no_grad():
        layer.b_i.uniform_(0.0, 1.3)
    layer.advance()
    layer.advance()
    x = torch.randn(40, 256, device=DEV, dtype=torch.bfloat16, requires_grad=True)
    y = layer(x)
    upstream = torch.randn_like(y) * 1e-2
    y.backward(upstream)

    seed, step, (gr, gc) = orc.layer_seed(7, 3), 2, group
    assert layer.seed == seed and layer.step == step
    bt = orc.bitwidth(layer.b_i.detach().cpu().numpy(), 6.0, 4.0)
    w_bits = bits_of(layer.weight.detach())
    want_hat, want_scale = orc.sample_fwd(w_bits, bt, 96, 256, gr, gc, seed=seed, step=step)
    got_hat = layer.sampled_weight().detach()
    assert (bits_of(got_hat).ravel() == want_hat).all()
    # y is the stock GEMM of x with the sampled weight
    ref_y = torch.nn.functional.linear(x.detach(), got_hat, layer.bias.detach())
    assert torch.equal(y.detach(), ref_y)
    # dL/dw = dL/dw_hat = upstream^T x (torch's GEMM), passed through unchanged
    grad_w_hat = (upstream.float().t() @ x.detach().float()).to(torch.bfloat16)
    assert torch.allclose(layer.weight.grad.float(), grad_w_hat.float(), rtol=2e-2, atol=1e-4)
    # dL/db_i: Eq. 4 on the gradient the module actually saw, then Eq. 11 / Eq. 12
    _, want_gbt = orc.sample_bwd(bits_of(layer.weight.grad), want_scale, 96, 256, gr, gc, seed=seed, step=step)
    want_gbi = orc.bitwidth_grad(want_gbt, bt, 6.0, 4.0, 0.25)
    got_gbi = layer.b_i.grad.cpu().numpy().astype(np.float64)
    assert np.abs(got_gbi - want_gbi).max() <= 1e-5 * np.abs(want_gbi).max()
    assert abs(float(layer.bitwidth_loss().cpu()) - orc.bitwidth_loss(bt, 4.0)) <= 1e-5


def test_module_noise_changes_only_when_advanced():
    layer = GaussWSLinear(128, 64, bias=False, group=(32, 32), user_seed=1, layer_index=0)
    a, b = layer.sampled_weight().detach().clone(), layer.sampled_weight().detach().clone()
    layer.advance()
    c = layer.sampled_weight().detach()
    assert torch.equal(a, b) and not torch.equal(a, c)
    other = GaussWSLinear(128, 64, bias=False, group=(32, 32), user_seed=1, layer_index=1)
    with torch.no_grad():
        other.weight.copy_(layer.weight)
    assert not torch.equal(other.sampled_weight().detach(), c) and other.seed != layer.seed


def test_module_adds_the_bitwidth_loss_term_once_per_update():
    # Eq. 12's term belongs to the update, not to the micro-batch: two accumulated backward passes at one step give
    # twice the Eq. 4 gradient but the lambda term once; after advance() the next backward pass carries it again
    torch.manual_seed(1)
    lam = 0.5
    layer = GaussWSLinear(128, 64, bias=False, group=(1, 128), b_init=6.0, b_target=4.0, lam=lam, user_seed=2, layer_index=5)
    with torch.no_grad():
        layer.b_i.uniform_(0.2, 1.2)
    x = torch.randn(16, 128, device=DEV, dtype=torch.bfloat16)
    upstream = torch.randn(16, 64, device=DEV, dtype=torch.bfloat16) * 1e-2

    def one_backward():
        layer.b_i.grad = None
        layer.weight.grad = None
        layer(x).backward(upstream)
        return layer.b_i.grad.detach().cpu().numpy().astype(np.float64)

    bt = orc.bitwidth(layer.b_i.detach().cpu().numpy(), 6.0, 4.0)
    with_term = one_backward()            # first backward pass of the update: chain rule + lambda term
    without_term = one_backward()         # second one of the same update: chain rule only
    m = bt.size
    term = (6.0 - 4.0) * lam / m * np.sign(bt.astype(np.float64) - 4.0)
    assert np.abs(with_term - without_term - term).max() <= 1e-6 * np.abs(term).max() + 1e-12
    # accumulated over the two micro-batches
    layer.advance()
    layer.b_i.grad = None
    layer(x).backward(upstream)
    layer(x).backward(upstream)
    acc = layer.b_i.grad.detach().cpu().numpy().astype(np.float64)
    layer.advance()
    layer.step -= 1                        # same noise, a fresh update
    layer.b_i.grad = None
    layer(x).backward(upstream)
    single = layer.b_i.grad.detach().cpu().numpy().astype(np.float64)
    assert np.abs(acc - (2.0 * single - term)).max() <= 1e-5 * np.abs(single).max()


def test_multi_layer_calls_give_the_bits_of_the_layer_by_layer_calls():
    # 150 layers (more than one launch carries), sizes from 1 to 100003, different hyper-parameters, one empty layer
    g = torch.Generator().manual_seed(9)
    sizes = [1, 255, 1024, 1025, 4096, 100003, 0] + [int(v) for v in torch.randint(1, 5000, (143,), generator=g)]
    layers = []
    for k, n in enumerate(sizes):
        layers.append(dict(bi=torch.empty(n).uniform_(-0.5, 1.5, generator=g).to(DEV), bt=torch.empty(n, device=DEV),
                           grad_bt=(torch.randn(n, generator=g) * 1e-3).to(DEV), grad_bi=torch.full((n,), 0.5, device=DEV),
                           b_init=6.0 + 0.25 * (k % 5), b_target=4.0 - 0.5 * (k % 3), lam=0.1 * (k % 4), accumulate=(k % 2 == 1)))
    gws.bitwidth_multi(layers)
    gws.bitwidth_grad_multi(layers)
    torch.cuda.synchronize()
    for it in layers:
        want_bt = gws.bitwidth(it["bi"], it["b_init"], it["b_target"])
        assert torch.equal(it["bt"].view(torch.int32), want_bt.view(torch.int32))
        want = gws.bitwidth_grad(it["grad_bt"], want_bt, it["b_init"], it["b_target"], it["lam"])
        if it["accumulate"]:
            want = torch.full_like(want, 0.5) + want
        assert torch.equal(it["grad_bi"].view(torch.int32), want.view(torch.int32))
    # and one layer against the oracle
    it = layers[5]
    want = orc.bitwidth(it["bi"].cpu().numpy(), it["b_init"], it["b_target"])
    assert (it["bt"].cpu().numpy().view(np.uint32) == want.view(np.uint32)).all()
