"""Parity of the two extensions (FP8 E4M3 forward pass, MXINT4 elements) against the oracle, through the C ABI.

Tolerances as for the main path: quantised codes and scales bit for bit where both sides see the same fp32 values,
GEMM outputs within 1e-5 relative Frobenius of the fp64 product of the same codes (fp32 output), bf16 output within
the unit roundoff of bf16.
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


# ------------------------------------------------------------------------------------------------ FP8 forward
@pytest.mark.parametrize("shape", [(200, 1184), (3, 8), (1024, 1024)])
def test_fp8_quantiser_bit_exact(gpu, ref, shape):
    rng = np.random.default_rng(shape[0])
    x = wl.activation_like(rng, shape, n_outlier_channels=min(4, shape[1]))
    codes, scale = gpu.mxfp4_fp8_quantize(_dev(x))
    oc, osf = ref.fp8_quantize(x)
    sc = scale.cpu().numpy()
    assert sc[0] == np.float32(osf) and sc[1] == np.float32(np.abs(wl.bf16_bits_to_f32(x)).max())
    assert np.array_equal(codes.cpu().numpy(), oc)
    assert gpu.mxfp4_device_status() == 0
    # an all-zero tensor: scale 1, codes +0 / -0
    z = np.zeros((8, 64), np.uint16); z[0, 1] = 0x8000
    codes, scale = gpu.mxfp4_fp8_quantize(_dev(z))
    assert scale.cpu().numpy()[0] == 1.0 and codes.cpu().numpy()[0, 1] == 0x80 and codes.cpu().numpy().sum() == 0x80


@pytest.mark.parametrize("M,N,K", [(128, 256, 128), (200, 264, 640), (1, 8, 128), (384, 1032, 2176), (512, 512, 4096)])
def test_fp8_gemm_matches_fp64_product_of_the_codes(gpu, ref, M, N, K):
    import torch
    rng = np.random.default_rng(M + N + K)
    A = rng.integers(0, 256, (M, K)).astype(np.uint8); A[(A & 0x7F) == 0x7F] = 0x30          # no NaN codes
    B = rng.integers(0, 256, (N, K)).astype(np.uint8); B[(B & 0x7F) == 0x7F] = 0x30
    A[(A & 0x78) > 0x58] &= 0xDF; B[(B & 0x78) > 0x58] &= 0xDF                               # keep magnitudes moderate
    sa = torch.tensor([3.5, 0.0], dtype=torch.float32, device="cuda"); sb = torch.tensor([0.125, 0.0], dtype=torch.float32, device="cuda")
    C = gpu.mxfp4_fp8_gemm(torch.from_numpy(A).cuda(), sa, torch.from_numpy(B).cuda(), sb, gpu.OUT_FP32).cpu().numpy().astype(np.float64)
    assert gpu.mxfp4_device_status() == 0
    Cref = ref.fp8_gemm(A, B, alpha=1.0 / (3.5 * 0.125))
    assert np.linalg.norm(C - Cref) <= 1e-5 * np.linalg.norm(Cref)
    Cb = gpu.mxfp4_fp8_gemm(torch.from_numpy(A).cuda(), sa, torch.from_numpy(B).cuda(), sb, gpu.OUT_BF16).float().cpu().numpy()
    assert np.linalg.norm(Cb - Cref) <= 2.0 ** -8 * np.linalg.norm(Cref)


@pytest.mark.parametrize("b,n,m", [(256, 512, 512), (384, 640, 264), (2048, 1024, 3072)])
def test_fp8_linear_forward(gpu, ref, b, n, m):
    rng = np.random.default_rng(b + n + m)
    x = wl.activation_like(rng, (b, n), n_outlier_channels=4); W = wl.weight_like(rng, (m, n))
    y = gpu.mxfp4_linear_forward_fp8(_dev(x), _dev(W), gpu.OUT_FP32).cpu().numpy().astype(np.float64)
    assert gpu.mxfp4_device_status() == 0
    rows = np.unique(np.concatenate([hp.band_rows(b), [0, b - 1]])); cols = np.unique(np.concatenate([hp.chunk_cols(m), [0, m - 1]]))
    yo = ref.linear_forward_fp8(x, W, rows=rows, cols=cols)
    assert np.linalg.norm(y[rows][:, cols] - yo) <= 1e-5 * np.linalg.norm(yo)
    exact = wl.bf16_bits_to_f64(x[rows]) @ wl.bf16_bits_to_f64(W[cols]).T
    assert np.linalg.norm(y[rows][:, cols] - exact) < 0.1 * np.linalg.norm(exact)             # and it is the product it claims to be
    yb = gpu.mxfp4_linear_forward_fp8(_dev(x), _dev(W), gpu.OUT_BF16).float().cpu().numpy()
    assert np.linalg.norm(yb - y) <= 2.0 ** -8 * np.linalg.norm(y)


def test_autograd_layer_with_fp8_forward(gpu, ref):
    import torch
    from paper_2502_20586_b200.autograd import MxFp4Linear
    gen = torch.Generator(device="cuda").manual_seed(3)
    layer = MxFp4Linear(256, 384, g=64, seed=11, forward="fp8")
    x = torch.randn(4, 128, 256, device="cuda", generator=gen).to(torch.bfloat16).requires_grad_(True)
    y = layer(x)
    xb = x.detach().reshape(-1, 256).view(torch.int16).cpu().numpy().view(np.uint16)
    wb = layer.weight.detach().view(torch.int16).cpu().numpy().view(np.uint16)
    yo = ref.linear_forward_fp8(xb, wb)
    assert np.linalg.norm(y.detach().float().cpu().numpy().reshape(-1, 384) - yo) <= 2.0 ** -8 * np.linalg.norm(yo)
    dy = (torch.randn(4, 128, 384, device="cuda", generator=gen) * 1e-3).to(torch.bfloat16)
    y.backward(dy)
    dx_lib, dw_lib = gpu.mxfp4_linear_backward(dy.reshape(-1, 384), x.detach().reshape(-1, 256), layer.weight.detach(), 64, 11)
    assert torch.equal(x.grad.reshape(-1, 256), dx_lib) and torch.equal(layer.weight.grad, dw_lib)    # the backward is Algorithm 3 unchanged


# ------------------------------------------------------------------------------------------------ MXINT4
def _int4_codes_from_e4m3(codes):
    """E4M3 container bytes -> the oracle's code byte (bit 3 sign, bits 0-2 magnitude), through the library's decode."""
    import torch
    v = torch.from_numpy(codes).view(torch.float8_e4m3fn).to(torch.float32).numpy()
    assert np.all(v == np.round(v)) and np.abs(v).max() <= 7
    return (np.abs(v).astype(np.uint8) | (np.signbit(v).astype(np.uint8) << 3))


@pytest.mark.parametrize("g", [0, 64, 128])
@pytest.mark.parametrize("reduce_dim,shape", [(1, (130, 1280)), (0, (768, 136)), (1, (3, 32))])
@pytest.mark.parametrize("rounding", [0, 1])
def test_int4_quantiser_bit_exact_on_gpu_values(gpu, ref, g, reduce_dim, shape, rounding):
    K = shape[1] if reduce_dim == 1 else shape[0]
    if g and K % g:
        pytest.skip("reduce length not a multiple of g")
    rng = np.random.default_rng(7 + g)
    x = wl.grad_like(rng, shape, 1e-3, outlier_rate=1e-3)
    x[0, 0] = 0x8000
    codes, scales, y = gpu.mxfp4_int4_quantize(_dev(x), reduce_dim, g, 55, 3, rounding)
    assert gpu.mxfp4_device_status() == 0
    y = y.cpu().numpy()
    R, Kk = y.shape
    y_ref = ref.rht(x, g, 55, transpose=(reduce_dim == 0)).astype(np.float64) if g else wl.bf16_bits_to_f64(x if reduce_dim == 1 else np.ascontiguousarray(x.T))
    if g:
        d = (y.astype(np.float64) - y_ref).reshape(R, Kk // g, g)
        rel = np.linalg.norm(d, axis=2) / np.maximum(np.linalg.norm(y_ref.reshape(R, Kk // g, g), axis=2), 1e-300)
        assert rel.max() <= 1e-5
    else:
        assert np.array_equal(y.astype(np.float64), y_ref)
    oc, os_ = ref.mxint4_quantize(y, rounding, 55, 3)
    assert np.array_equal(hp.sf_native_to_linear(scales.cpu().numpy(), R, Kk), os_)
    assert np.array_equal(_int4_codes_from_e4m3(codes.cpu().numpy()), oc)


@pytest.mark.parametrize("M,N,K", [(128, 256, 128), (200, 264, 640), (1, 8, 128), (384, 1032, 2176)])
def test_int4_gemm_matches_fp64_product(gpu, ref, M, N, K):
    import torch
    rng = np.random.default_rng(M + N + K)
    ca = rng.integers(0, 16, (M, K)).astype(np.uint8); sa = rng.integers(120, 134, (M, K // 32)).astype(np.uint8)
    cb = rng.integers(0, 16, (N, K)).astype(np.uint8); sb = rng.integers(120, 134, (N, K // 32)).astype(np.uint8)
    lut = np.array([0x00, 0x38, 0x40, 0x44, 0x48, 0x4A, 0x4C, 0x4E], np.uint8)                # E4M3 bytes of 0..7
    enc = lambda c: (lut[c & 7] | ((c & 8) << 4)).astype(np.uint8)
    assert np.array_equal(_int4_codes_from_e4m3(enc(ca)) & 7, ca & 7)
    SA = torch.from_numpy(hp.sf_linear_to_native(sa, fill=255)).cuda(); SB = torch.from_numpy(hp.sf_linear_to_native(sb, fill=255)).cuda()
    C = gpu.mxfp4_int4_gemm(torch.from_numpy(enc(ca)).cuda(), SA, torch.from_numpy(enc(cb)).cuda(), SB, 16 / 9, gpu.OUT_FP32)
    assert gpu.mxfp4_device_status() == 0
    Cref = ref.mxint4_gemm(ca, sa, cb, sb, alpha=16 / 9)
    assert np.linalg.norm(C.cpu().numpy().astype(np.float64) - Cref) <= 1e-5 * np.linalg.norm(Cref)


def test_int4_backward_products_estimate_the_gradients(gpu, ref):
    """Algorithm 3 with MXINT4 elements, composed from the two calls: against the oracle's products of the same codes,
    and (mean over seeds) against the exact gradient."""
    import torch
    layer = wl.CONFIGS["single_256x512"][0][0]
    dY, X, W = wl.layer_inputs("single_256x512", layer, seed=0)
    exact = wl.bf16_bits_to_f64(dY) @ wl.bf16_bits_to_f64(W)
    acc = np.zeros_like(exact)
    T = 24
    for t in range(T):
        qa = gpu.mxfp4_int4_quantize(_dev(dY), 1, 64, 200 + t, 1)             # dY  [b, K = m]
        qb = gpu.mxfp4_int4_quantize(_dev(W), 0, 64, 200 + t, 2)              # W^T [n, K = m]
        dX = gpu.mxfp4_int4_gemm(qa[0], qa[1], qb[0], qb[1], 16 / 9, gpu.OUT_FP32).cpu().numpy().astype(np.float64)
        if t == 0:
            oa = ref.mxint4_quantize(qa[2].cpu().numpy(), 0, 200, 1); ob = ref.mxint4_quantize(qb[2].cpu().numpy(), 0, 200, 2)
            want = ref.mxint4_gemm(*oa, *ob, alpha=16 / 9)
            assert np.linalg.norm(dX - want) <= 1e-5 * np.linalg.norm(want)
            e1 = np.linalg.norm(dX - exact) / np.linalg.norm(exact)
        acc += dX
    eT = np.linalg.norm(acc / T - exact) / np.linalg.norm(exact)
    assert gpu.mxfp4_device_status() == 0
    assert eT < e1 / 3                                                         # unbiased: the mean converges like T^-1/2
