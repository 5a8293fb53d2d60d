"""The allocation-free backward entry point against the ordinary one.

mxfp4_linear_backward_static serves callers that cannot ask anyone for device scratch memory (a hook running while
its framework's pool is locked or spent, a plug-in barred from the CUDA allocator): it keeps the quantised operands
in a fixed array inside the library.  Same inputs and seed must give the SAME gradients, bit for bit, as
mxfp4_linear_backward, on two calls in a row (the array keeps the first call's bytes, here deliberately bad ones),
the call must take no device memory from anyone, and oversized shapes must be refused.
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
    inf = lambda shape: torch.full(shape, float("-inf"), dtype=torch.bfloat16, device="cuda")

    def scale_regions(b, m, n):
        """Byte ranges of the four operands' scale tiles inside the scratch, from the library's own layout call."""
        offs = mx.mxfp4_operand_layout(b, m, n)
        R, K = (b, n, m, n), (m, m, b, b)
        return [(offs[i][1], offs[i][1] + mx.mxfp4_scale_bytes(R[i], K[i])) for i in range(4)]

    # n = 264 and 136 are not multiples of 128: the last scale tile of the two n-row operands has rows that no call
    # writes but the GEMM loads.  Each case names the layers whose all-infinite inputs leave the NaN scale byte 0xFF
    # on exactly those tiles beforehand (shapes found by searching the layout; the cover is re-checked below).
    cases = [((256, 512, 512), 64, mx.ROUND_SR, 5, [(256, 512, 512)]),
             ((384, 264, 640), 128, mx.ROUND_SR, 6, [(128, 704, 512), (128, 896, 768)]),
             ((256, 136, 512), 64, mx.ROUND_RN, 7, [(128, 192, 640), (128, 320, 640), (128, 640, 128)]),
             ((256, 512, 512), 64, mx.ROUND_RN, 8, [])]
    for (b, n, m), g, rounding, seed, poison in cases:              # back to back: the array keeps the previous call's bytes
        dY = _dev(wl.grad_like(rng, (b, m), 1e-3, outlier_rate=1e-3))
        X = _dev(wl.activation_like(rng, (b, n), n_outlier_channels=4))
        W = _dev(wl.weight_like(rng, (m, n)))
        assert mx.mxfp4_linear_backward_workspace(b, m, n) <= mx.STATIC_WORKSPACE_BYTES
        dX = torch.empty((b, n), dtype=torch.float32, device="cuda")
        dW = torch.empty((m, n), dtype=torch.float32, device="cuda")
        if n % 128 != 0:
            for t0, t1 in (scale_regions(b, m, n)[i] for i in (1, 3)):
                covered = np.zeros(t1 - t0, bool)
                for (pb, pn, pm) in poison:
                    for s0, s1 in scale_regions(pb, pm, pn):
                        lo, hi = max(s0, t0), min(s1, t1)
                        if lo < hi:
                            covered[lo - t0:hi - t0] = True
                assert covered.all()
        for (pb, pn, pm) in poison:                                  # (the first of these is also the warm-up call of the device)
            mx.mxfp4_linear_backward_static(inf((pb, pm)), inf((pb, pn)), inf((pm, pn)), 0, seed, mx.ROUND_RN, mx.OUT_FP32)
        torch.cuda.synchronize()
        # the call proper: outputs passed in, so nothing may be taken from torch's pool or from the device
        pool_before, free_before = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
        mx.mxfp4_linear_backward_static(dY, X, W, g, seed, rounding, mx.OUT_FP32, dX=dX, dW=dW)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == pool_before
        assert torch.cuda.mem_get_info()[0] == free_before
        rX, rW = mx.mxfp4_linear_backward(dY, X, W, g, seed, rounding, mx.OUT_FP32)
        assert mx.mxfp4_device_status() == 0
        for got, want in ((dX, rX), (dW, rW)):
            assert torch.isfinite(got).all()
            assert torch.equal(got, want)                             # the library's contract: the same bits

    # a shape whose quantised operands do not fit the fixed array is refused, and nothing is enqueued
    b, n, m = 4096, 4096, 4096
    assert mx.mxfp4_linear_backward_workspace(b, m, n) > mx.STATIC_WORKSPACE_BYTES
    big = torch.zeros((4096, 4096), dtype=torch.bfloat16, device="cuda")
    out = torch.empty((4096, 4096), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(mx.MxFp4Error) as err:
        mx.mxfp4_linear_backward_static(big, big, big, 64, 0, dX=out, dW=out.clone())
    assert err.value.code == 6
