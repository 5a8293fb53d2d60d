"""Failure detection without a fault: a bounded device-side wait that runs out is reported, and the context stays usable."""
import pytest

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_once_and_the_library_keeps_working():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no GPU")
    from paper_2502_20586_b200 import binding as mx
    assert mx.mxfp4_device_status() == 0
    mx.mxfp4_selftest_wait_expiry()                  # one thread waits ~2 s on a barrier nothing signals, then returns
    assert mx.mxfp4_device_status() == 9             # MXFP4_ERR_TIMEOUT, read from the kernel's status word
    assert mx.mxfp4_device_status() == 0             # reading clears it
    gen = torch.Generator(device="cuda").manual_seed(0)
    dY = (torch.randn(256, 256, device="cuda", generator=gen) * 1e-3).to(torch.bfloat16)
    X = torch.randn(256, 128, device="cuda", generator=gen).to(torch.bfloat16)
    W = (torch.randn(256, 128, device="cuda", generator=gen) * 0.02).to(torch.bfloat16)
    dX, dW = mx.mxfp4_linear_backward(dY, X, W, 64, 1)
    assert mx.mxfp4_device_status() == 0
    ref = dY.double() @ W.double()
    assert float((dX.double() - ref).norm() / ref.norm()) < 0.5
