"""The small-footprint builds of the pair GEMM and of the tensor-core quantiser, and the overlapped form of the
backward call that uses them.

Both kernels exist in a second build sized so that one CTA of each fits on an SM together (fewer pipeline stages, part
of the tensor memory, fewer registers): the library can then quantise the operands of one product while the other
product's GEMM runs on the same SMs (MXFP4_OVERLAP=1).  The arithmetic, the draws and the accumulation order are those
of the full-size builds, so every output must be the SAME BITS; here that is checked on ragged and tiny shapes through
MXFP4_FORCE_LITE=1 (which routes every eligible launch to the small builds), against the oracle on the quantiser
side, and on a layer large enough for the overlapped form to engage.
"""
import os

import numpy as np
import pytest

from paper_2502_20586_b200 import workloads as wl
from tests import helpers as hp

pytestmark = pytest.mark.gpu


@pytest.fixture()
def env():
    saved = {k: os.environ.get(k) for k in ("MXFP4_FORCE_LITE", "MXFP4_OVERLAP", "MXFP4_DUAL_DY")}
    yield os.environ
    for k, v in saved.items():
        if v is None:
            os.environ.pop(k, None)
        else:
            os.environ[k] = v


def _dev(bits):
    import torch
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


@pytest.mark.parametrize("b,n,m,g", [(384, 264, 640, 128), (256, 136, 512, 64), (1280, 1032, 2176, 32), (2048, 512, 256, 128)])
@pytest.mark.parametrize("rounding", [0, 1, 2])
def test_small_builds_give_the_same_bits(env, ref, b, n, m, g, rounding):
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no GPU")
    from paper_2502_20586_b200 import binding as mx
    rng = np.random.default_rng(b + n + m)
    dY = _dev(wl.grad_like(rng, (b, m), 1e-3, outlier_rate=1e-3))
    X = _dev(wl.activation_like(rng, (b, n), n_outlier_channels=4))
    W = _dev(wl.weight_like(rng, (m, n)))
    env["MXFP4_OVERLAP"] = "0"
    out, ops = {}, {}
    for lite in ("0", "1"):
        env["MXFP4_FORCE_LITE"] = lite
        ws = torch.zeros(mx.mxfp4_linear_backward_workspace(b, m, n), dtype=torch.uint8, device="cuda")
        q = mx.mxfp4_quantize_operands(dY, X, W, g, 9, rounding, workspace=ws)
        ops[lite] = [(c.clone(), s.clone()) for c, s in q]
        out[lite] = mx.mxfp4_linear_backward(dY, X, W, g, 9, rounding, mx.OUT_FP32)
        assert mx.mxfp4_device_status() == 0
    for (c0, s0), (c1, s1) in zip(ops["0"], ops["1"]):
        assert torch.equal(c0, c1) and torch.equal(s0, s1)
    assert torch.equal(out["0"][0], out["1"][0]) and torch.equal(out["0"][1], out["1"][1])
    # and the small quantiser against the oracle directly (Q4 = X^T, a transposing view with a ragged row count)
    codes = hp.unpack_codes(ops["1"][3][0].cpu().numpy())
    scales = hp.sf_native_to_linear(ops["1"][3][1].cpu().numpy(), n, b)
    xb = X.view(torch.int16).cpu().numpy().view(np.uint16)
    _, oc, os_ = ref.rht_quantize(xb, g, rounding, 9, 4, transpose=True)
    hp.compare_quantised_rows(codes, scales, oc, os_)


@pytest.mark.parametrize("mode", ["1", "2", "3"])
def test_overlapped_backward_gives_the_same_bits(env, mode):
    """A layer large enough for the side stream (>= 74 pair tiles per product): the overlapped form against the serial one."""
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no GPU")
    from paper_2502_20586_b200 import binding as mx
    layer = [l for l in wl.CONFIGS["gpt_1p3b"][0] if l.name == "attn_out"][0]
    dY, X, W = wl.layer_inputs_device("gpt_1p3b", layer, seed=1)
    env["MXFP4_FORCE_LITE"] = "0"
    res = {}
    for ov in ("0", mode):
        env["MXFP4_OVERLAP"] = ov
        for _ in range(2):                                        # twice: the second call reuses the side stream and events
            res[ov] = mx.mxfp4_linear_backward(dY, X, W, 128, 5, mx.ROUND_SR, mx.OUT_BF16)
        assert mx.mxfp4_device_status() == 0
    assert torch.equal(res["0"][0], res[mode][0]) and torch.equal(res["0"][1], res[mode][1])


@pytest.mark.parametrize("b,m,g,rounding", [(384, 640, 128, 0), (1280, 2176, 32, 2), (256, 128, 64, 1), (2048, 4096, 128, 0)])
def test_one_read_of_dy_gives_the_same_codes_as_two(env, b, m, g, rounding):
    """Algorithm 3 lines 3 and 5 quantise two views of the same dL/dy; by default every 128 x 128 tile of it is loaded
    once and transformed twice (as the K-major and as the MN-major operand).  Same codes and scales as separate passes."""
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no GPU")
    from paper_2502_20586_b200 import binding as mx
    rng = np.random.default_rng(b + m)
    n = 264
    dY = _dev(wl.grad_like(rng, (b, m), 1e-3, outlier_rate=1e-3))
    X = _dev(wl.activation_like(rng, (b, n)))
    W = _dev(wl.weight_like(rng, (m, n)))
    env["MXFP4_FORCE_LITE"] = "0"
    ops = {}
    for dual in ("1", "0"):
        env["MXFP4_DUAL_DY"] = "2" if dual == "1" else "0"          # 2: one read whatever the size (the default decides by size)
        ws = torch.zeros(mx.mxfp4_linear_backward_workspace(b, m, n), dtype=torch.uint8, device="cuda")
        ops[dual] = [(c.clone(), s.clone()) for c, s in mx.mxfp4_quantize_operands(dY, X, W, g, 3, rounding, workspace=ws)]
        assert mx.mxfp4_device_status() == 0
    for (c0, s0), (c1, s1) in zip(ops["0"], ops["1"]):
        assert torch.equal(c0, c1) and torch.equal(s0, s1)
    # and view by view against the stand-alone call
    for i, (t, rd) in enumerate(((dY, 1), (W, 0), (dY, 0), (X, 0))):
        c, s = mx.mxfp4_rht_sr_quantize(t, rd, g, 3, i + 1, rounding, mx.SF_NATIVE)
        R, K = c.shape[0], 2 * c.shape[1]
        valid = torch.from_numpy(hp.sf_native_offsets(R, K)).cuda()        # padding rows of the last scale tile are never written
        assert torch.equal(c, ops["1"][i][0]) and torch.equal(s[valid], ops["1"][i][1][valid])


def test_bias_sums_from_the_quantiser_launch_agree_with_the_separate_pass(env, ref):
    """The bias gradient's first pass (column sums of every 128-row band of dL/dy) rides along in the dual-view quantiser
    launch, which has every tile in shared memory anyway; with MXFP4_DUAL_DY=0 a stand-alone kernel reads dL/dy again.
    Both against the fp64 oracle within the fp32 summation bound; dX and dW are the same bits either way."""
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no GPU")
    from paper_2502_20586_b200 import binding as mx
    rng = np.random.default_rng(77)
    b, m, n = 2048, 1152, 264
    dYb = wl.grad_like(rng, (b, m), 1e-3, outlier_rate=1e-3)
    dY, X, W = _dev(dYb), _dev(wl.activation_like(rng, (b, n))), _dev(wl.weight_like(rng, (m, n)))
    want = ref.bias_grad(dYb)
    bound = 64 * np.sqrt(b) * 2.0 ** -24 * np.abs(wl.bf16_bits_to_f64(dYb)).sum(axis=0)
    env["MXFP4_FORCE_LITE"] = "0"
    res = {}
    for dual in ("1", "0"):
        env["MXFP4_DUAL_DY"] = dual
        res[dual] = mx.mxfp4_linear_backward_ex(dY, X, W, 128, 5, mx.ROUND_SR, mx.OUT_FP32, with_bias=True)
        assert mx.mxfp4_device_status() == 0
        assert np.all(np.abs(res[dual][2].cpu().numpy().astype(np.float64) - want) <= bound)
    assert torch.equal(res["0"][0], res["1"][0]) and torch.equal(res["0"][1], res["1"][1])
