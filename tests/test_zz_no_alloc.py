"""The allocation-free backward entry point against the ordinary one.

mxfp4_linear_backward_static serves callers that cannot ask anyone for device scratch memory (a hook running while
its framework's pool is locked or spent, a plug-in barred from the CUDA allocator): it keeps the quantised operands
in a fixed array inside the library.  Same inputs and seed must give the same gradients as mxfp4_linear_backward,
on two calls in a row (the array keeps the first call's bytes), and oversized shapes must be refused.
This file is collected last so that a failure here cannot hide any other test under `pytest -x`.
"""
import numpy as np
import pytest

from paper_2502_20586_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _dev(bits):
    import torch
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def test_static_workspace_backward_matches_workspace_backward():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no GPU")
    from paper_2502_20586_b200 import binding as mx

    rng = np.random.default_rng(21)
    cases = [((256, 512, 512), 64, mx.ROUND_SR, 5), ((384, 256, 640), 128, mx.ROUND_SR, 6), ((256, 512, 512), 64, mx.ROUND_RN, 7)]
    for (b, n, m), g, rounding, seed in cases:                       # back to back: the array keeps the previous call's bytes
        dY = _dev(wl.grad_like(rng, (b, m), 1e-3, outlier_rate=1e-3))
        X = _dev(wl.activation_like(rng, (b, n), n_outlier_channels=4))
        W = _dev(wl.weight_like(rng, (m, n)))
        assert mx.mxfp4_linear_backward_workspace(b, m, n) <= mx.STATIC_WORKSPACE_BYTES
        dX = torch.empty((b, n), dtype=torch.float32, device="cuda")
        dW = torch.empty((m, n), dtype=torch.float32, device="cuda")
        mx.mxfp4_linear_backward_static(dY, X, W, g, seed, rounding, mx.OUT_FP32, dX=dX, dW=dW)
        rX, rW = mx.mxfp4_linear_backward(dY, X, W, g, seed, rounding, mx.OUT_FP32)
        assert mx.mxfp4_device_status() == 0
        for got, want in ((dX, rX), (dW, rW)):
            got = got.cpu().numpy().astype(np.float64); want = want.cpu().numpy().astype(np.float64)
            assert np.isfinite(got).all()
            assert np.linalg.norm(got - want) <= 1e-5 * np.linalg.norm(want)      # the GEMM tolerance of the parity tests

    # a shape whose quantised operands do not fit the fixed array is refused, and nothing is enqueued
    b, n, m = 4096, 4096, 4096
    assert mx.mxfp4_linear_backward_workspace(b, m, n) > mx.STATIC_WORKSPACE_BYTES
    big = torch.zeros((4096, 4096), dtype=torch.bfloat16, device="cuda")
    out = torch.empty((4096, 4096), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(mx.MxFp4Error) as err:
        mx.mxfp4_linear_backward_static(big, big, big, 64, 0, dX=out, dW=out.clone())
    assert err.value.code == 6
