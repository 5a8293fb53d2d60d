"""Fused-producer variant: the GEMM kernel that transforms and quantises its A operand itself.

The codes it derives must be those of the stand-alone quantiser (same Philox draws, keyed on the element index), so
the product is compared (a) with the library's own GEMM on the stand-alone quantiser's output and (b) with the
oracle's fp64 product of the oracle-checked codes.
"""
import numpy as np
import pytest

from paper_2502_20586_b200 import workloads as wl
from tests import helpers as hp

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no GPU")
    from paper_2502_20586_b200 import binding
    return binding


def _dev(bits):
    import torch
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


@pytest.mark.parametrize("rounding", [0, 1, 2])
@pytest.mark.parametrize("g", [32, 64, 128])
@pytest.mark.parametrize("reduce_dim,shape,N", [(1, (200, 512), 264), (0, (768, 136), 128), (1, (384, 1024), 520), (0, (256, 128), 8)])
def test_fused_gemm_equals_quantise_then_gemm(gpu, ref, rounding, g, reduce_dim, shape, N):
    """Ragged M and N, several K-steps and tiles; both majornesses of A."""
    rng = np.random.default_rng(5)
    x = wl.grad_like(rng, shape, 1e-3, outlier_rate=1e-3)
    K = shape[1] if reduce_dim == 1 else shape[0]
    bsrc = wl.weight_like(rng, (N, K))
    seed = 91
    cb, sb = gpu.mxfp4_rht_sr_quantize(_dev(bsrc), 1, g, seed, 2, rounding, gpu.SF_NATIVE)
    ca, sa = gpu.mxfp4_rht_sr_quantize(_dev(x), reduce_dim, g, seed, 1, rounding, gpu.SF_NATIVE)
    want = gpu.mxfp4_gemm(ca, sa, cb, sb, 1.0, gpu.OUT_FP32).cpu().numpy()
    got = gpu.mxfp4_gemm_fused(_dev(x), reduce_dim, g, seed, 1, rounding, cb, sb, 1.0, gpu.OUT_FP32).cpu().numpy()
    assert gpu.mxfp4_device_status() == 0
    # same codes, same fp32 accumulation order along K: equal up to the fp32 rounding of differently shaped tiles
    assert np.linalg.norm(got - want) <= 1e-6 * np.linalg.norm(want)
    # against the oracle's product of the codes the stand-alone quantiser wrote (themselves checked against the oracle elsewhere)
    M = got.shape[0]
    A = (hp.unpack_codes(ca.cpu().numpy()), hp.sf_native_to_linear(sa.cpu().numpy(), M, K))
    B = (hp.unpack_codes(cb.cpu().numpy()), hp.sf_native_to_linear(sb.cpu().numpy(), N, K))
    exact = ref.gemm(*A, *B, alpha=1.0)
    assert np.linalg.norm(got - exact) <= 1e-5 * np.linalg.norm(exact)
    # bf16 output
    gb = gpu.mxfp4_gemm_fused(_dev(x), reduce_dim, g, seed, 1, rounding, cb, sb, 1.0, gpu.OUT_BF16).float().cpu().numpy()
    assert np.linalg.norm(gb - exact) <= 2.0 ** -8 * np.linalg.norm(exact)


@pytest.mark.parametrize("rounding", [0, 2])
def test_fused_linear_backward_against_oracle(gpu, ref, rounding):
    """Algorithm 3 through the fused kernels: every output element against the oracle and against the unfused call."""
    layer = wl.CONFIGS["single_256x512"][0][0]
    dY, X, W = wl.layer_inputs("single_256x512", layer, seed=0)
    dX, dW = gpu.mxfp4_linear_backward_fused(_dev(dY), _dev(X), _dev(W), 64, 3, rounding, gpu.OUT_FP32)
    assert gpu.mxfp4_device_status() == 0
    uX, uW = gpu.mxfp4_linear_backward(_dev(dY), _dev(X), _dev(W), 64, 3, rounding, gpu.OUT_FP32)
    dX, dW, uX, uW = (t.cpu().numpy().astype(np.float64) for t in (dX, dW, uX, uW))
    assert np.linalg.norm(dX - uX) <= 1e-6 * np.linalg.norm(uX)
    assert np.linalg.norm(dW - uW) <= 1e-6 * np.linalg.norm(uW)
    rdX, rdW = ref.linear_backward(dY, X, W, 64, rounding, 3)
    assert np.linalg.norm(dX - rdX) / np.linalg.norm(rdX) <= 2e-2
    assert np.linalg.norm(dW - rdW) / np.linalg.norm(rdW) <= 2e-2


def test_fused_full_size_layer_sampled(gpu, ref):
    """The 6.7B attention-output layer at full size: sampled entries against the unfused path."""
    import torch
    layers, g = wl.CONFIGS["gpt_6p7b"]
    layer = [l for l in layers if l.name == "attn_out"][0]
    dY, X, W = wl.layer_inputs_device("gpt_6p7b", layer, seed=0)
    fX, fW = gpu.mxfp4_linear_backward_fused(dY, X, W, g, 3, gpu.ROUND_SR, gpu.OUT_BF16)
    assert gpu.mxfp4_device_status() == 0
    uX, uW = gpu.mxfp4_linear_backward(dY, X, W, g, 3, gpu.ROUND_SR, gpu.OUT_BF16)
    idx = torch.randint(0, fX.numel(), (200000,), device="cuda", generator=torch.Generator(device="cuda").manual_seed(1))
    a, b = fX.flatten()[idx].float(), uX.flatten()[idx].float()
    assert (a - b).norm() <= 2.0 ** -7 * b.norm()
    idx = torch.randint(0, fW.numel(), (200000,), device="cuda", generator=torch.Generator(device="cuda").manual_seed(2))
    a, b = fW.flatten()[idx].float(), uW.flatten()[idx].float()
    assert (a - b).norm() <= 2.0 ** -7 * b.norm()
