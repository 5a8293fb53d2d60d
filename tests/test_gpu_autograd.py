"""The autograd wrapper: its gradients are the library's Algorithm-3 outputs, and they estimate the true gradients."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def torch_gpu():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no GPU")
    return torch


def test_backward_is_the_library_call_and_estimates_the_gradient(torch_gpu):
    torch = torch_gpu
    from paper_2502_20586_b200 import binding as mx
    from paper_2502_20586_b200.autograd import MxFp4Linear
    gen = torch.Generator(device="cuda").manual_seed(3)
    layer = MxFp4Linear(256, 384, bias=True, g=64, seed=11)
    x = torch.randn(4, 128, 256, device="cuda", generator=gen).to(torch.bfloat16).requires_grad_(True)
    dy = (torch.randn(4, 128, 384, device="cuda", generator=gen) * 1e-3).to(torch.bfloat16)
    y = layer(x)
    assert y.shape == (4, 128, 384) and y.dtype == torch.bfloat16
    y.backward(dy)
    # identical to calling the library directly with the same seed
    dx_lib, dw_lib = mx.mxfp4_linear_backward(dy.reshape(-1, 384), x.detach().reshape(-1, 256), layer.weight.detach(), 64, 11)
    assert torch.equal(x.grad.reshape(-1, 256), dx_lib) and torch.equal(layer.weight.grad, dw_lib)
    # and a reasonable one-sample estimate of the exact gradients
    dx_ref = dy.double().reshape(-1, 384) @ layer.weight.detach().double()
    dw_ref = dy.double().reshape(-1, 384).t() @ x.detach().double().reshape(-1, 256)
    ex = float((x.grad.double().reshape(-1, 256) - dx_ref).norm() / dx_ref.norm())
    ew = float((layer.weight.grad.double() - dw_ref).norm() / dw_ref.norm())
    assert ex < 0.5 and ew < 0.5
    # the bias gradient is the plain column sum (bf16-rounded for the bf16 parameter)
    db_ref = dy.double().reshape(-1, 384).sum(0)
    assert float((layer.bias.grad.double() - db_ref).abs().max()) <= 2.0 ** -8 * float(db_ref.abs().max()) + 1e-12
    assert mx.mxfp4_device_status() == 0


def test_seeds_advance_and_the_mean_gradient_converges(torch_gpu):
    """SR makes the backward unbiased (Lemma 3.1): the mean over T calls approaches the exact gradient like T^-1/2."""
    torch = torch_gpu
    from paper_2502_20586_b200.autograd import MxFp4Linear
    gen = torch.Generator(device="cuda").manual_seed(5)
    layer = MxFp4Linear(128, 128, g=32, seed=100)
    x = torch.randn(256, 128, device="cuda", generator=gen).to(torch.bfloat16)
    dy = (torch.randn(256, 128, device="cuda", generator=gen) * 1e-2).to(torch.bfloat16)
    dw_ref = dy.double().t() @ x.double()
    T = 64
    acc = torch.zeros_like(dw_ref)
    first = None
    for _ in range(T):
        layer.weight.grad = None
        layer(x).backward(dy)
        acc += layer.weight.grad.double()
        if first is None:
            first = float((layer.weight.grad.double() - dw_ref).norm() / dw_ref.norm())
    mean_err = float((acc / T - dw_ref).norm() / dw_ref.norm())
    assert layer.calls == T
    assert mean_err < first / 4          # ideal: first / 8


@pytest.mark.parametrize("rounding", ["SR", "SR16"])
def test_a_small_network_trains_like_its_bf16_twin(torch_gpu, rounding):
    """The recipe of Section 4 in miniature: bf16 forward, Algorithm-3 backward, fp32 master weights.  A two-layer
    network fitted to a random teacher reaches the loss of the same network trained with exact bf16 gradients
    (unbiased gradients with bounded variance only add noise that averages out over steps)."""
    torch = torch_gpu
    from paper_2502_20586_b200 import binding as mx
    from paper_2502_20586_b200.autograd import MxFp4LinearFunction
    gen = torch.Generator(device="cuda").manual_seed(9)
    d_in, d_h, d_out, tokens = 256, 512, 256, 1024
    teacher = torch.randn(d_in, d_out, device="cuda", generator=gen) / d_in ** 0.5
    rnd = getattr(mx, "ROUND_" + rounding)

    def run(mxfp4: bool):
        g2 = torch.Generator(device="cuda").manual_seed(1)
        w1 = (torch.randn(d_h, d_in, device="cuda", generator=g2) * 0.05).requires_grad_(True)      # fp32 master weights
        w2 = (torch.randn(d_out, d_h, device="cuda", generator=g2) * 0.05).requires_grad_(True)
        opt = torch.optim.SGD([w1, w2], lr=0.5, momentum=0.9)
        data = torch.Generator(device="cuda").manual_seed(2)
        losses = []
        for step in range(120):
            x = torch.randn(tokens, d_in, device="cuda", generator=data)
            target = x @ teacher
            xb = x.to(torch.bfloat16)
            if mxfp4:
                h = MxFp4LinearFunction.apply(xb, w1.to(torch.bfloat16), None, 64, 1000 + 2 * step, rnd)
                y = MxFp4LinearFunction.apply(torch.relu(h), w2.to(torch.bfloat16), None, 64, 1001 + 2 * step, rnd)
            else:
                y = torch.relu(xb @ w1.to(torch.bfloat16).t()) @ w2.to(torch.bfloat16).t()
            loss = ((y.float() - target) ** 2).mean()
            opt.zero_grad()
            loss.backward()
            opt.step()
            losses.append(float(loss.detach()))
        return losses

    ref = run(False)
    ours = run(True)
    assert mx.mxfp4_device_status() == 0
    assert ref[-1] < 0.2 * ref[0]                                    # the task is learnable in 120 steps
    tail_ref, tail_ours = np.mean(ref[-10:]), np.mean(ours[-10:])
    assert tail_ours < 0.2 * ours[0]
    assert tail_ours < 1.25 * tail_ref                         # close to the exact-gradient run
