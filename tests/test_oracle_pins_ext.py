"""Pins of the oracle's extensions: the FP8 (E4M3) forward pass and MXINT4 elements.

As for the main path, every function is tied to something other than itself: the E4M3 codec to a library's
independent implementation of the same format (torch's float8_e4m3fn casts on the CPU), the rounding rules to
numpy's round-half-even and to full enumeration of the draws, the products to integer arithmetic and to numpy,
Algorithm 2's unbiasedness to convergence over seeds.
"""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2502_20586_b200 import workloads as wl


# ------------------------------------------------------------------------------------------------ E4M3
def _torch_e4m3_decode(codes):
    return torch.from_numpy(np.asarray(codes, np.uint8)).view(torch.float8_e4m3fn).to(torch.float64).numpy()


def test_e4m3_decode_matches_the_library_format():
    codes = np.arange(256, dtype=np.uint8)
    want = _torch_e4m3_decode(codes)
    got = np.array([ref.e4m3_value(int(c)) for c in codes])
    assert np.array_equal(np.isnan(got), np.isnan(want))
    assert np.isnan(got).sum() == 2                                  # 0x7F and 0xFF only: no infinities in this format
    assert np.array_equal(got[~np.isnan(got)], want[~np.isnan(want)])
    assert np.nanmax(got) == 448.0 and ref.e4m3_value(0x01) == 2.0 ** -9 and ref.e4m3_value(0x08) == 2.0 ** -6


def test_e4m3_round_matches_the_library_cast_and_handles_ties_and_saturation():
    rng = np.random.default_rng(0)
    v = np.concatenate([np.exp(rng.uniform(np.log(1e-4), np.log(460.0), 200000)) * rng.choice([-1.0, 1.0], 200000),
                        rng.uniform(-0.02, 0.02, 20000)]).astype(np.float32)
    grid = np.array([ref.e4m3_value(c) for c in range(0x7F)])
    mid = ((grid[:-1] + grid[1:]) / 2).astype(np.float32)            # exact ties (representable in fp32)
    v = np.concatenate([v, mid, -mid, np.nextafter(mid, np.float32(0)), np.nextafter(mid, np.float32(1e9))])
    got = np.array([ref.e4m3_round(float(x)) for x in v], np.uint8)
    want = torch.from_numpy(v).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(got, want)
    # ties go to the even code
    tie_codes = np.array([ref.e4m3_round(float(x)) for x in mid])
    assert np.all(tie_codes % 2 == 0)
    # saturation (the library cast turns overflow into NaN; here the quantiser must clamp) and signed zero
    assert ref.e4m3_round(448.0) == 0x7E and ref.e4m3_round(1e9) == 0x7E and ref.e4m3_round(-465.0) == 0xFE
    assert ref.e4m3_round(0.0) == 0x00 and ref.e4m3_round(-0.0) == 0x80
    # relative error of a normal value is at most half a unit in the 3-bit mantissa
    vn = v[(np.abs(v) >= 2.0 ** -6) & (np.abs(v) <= 448)]
    back = np.array([ref.e4m3_value(ref.e4m3_round(float(x))) for x in vn[:20000]])
    assert np.max(np.abs(back - vn[:20000]) / np.abs(vn[:20000])) <= 2.0 ** -4


def test_fp8_tensor_scale_and_quantise():
    rng = np.random.default_rng(1)
    x = wl.to_bf16_bits(rng.standard_normal((64, 96)) * 3.0)
    xf = wl.bf16_bits_to_f64(x)
    s = ref.fp8_tensor_scale(x)
    assert s == np.float32(448.0) / np.float32(np.abs(xf).max())
    assert ref.fp8_tensor_scale(np.zeros((4, 32), np.uint16)) == 1.0
    codes, _ = ref.fp8_quantize(x)
    i = np.unravel_index(np.abs(xf).argmax(), xf.shape)
    assert codes[i] & 0x7F == 0x7E                                   # the largest element lands on +-448
    # the whole tensor against the library cast of the same fp32 products
    v = (wl.bf16_bits_to_f32(x) * np.float32(s)).astype(np.float32)
    want = torch.from_numpy(v).clamp(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(codes, want)


def test_fp8_gemm_is_exact_on_integers_and_matches_numpy():
    rng = np.random.default_rng(2)
    ia, ib = rng.integers(-8, 9, (24, 64)), rng.integers(-8, 9, (40, 64))
    enc = lambda a: np.array([[ref.e4m3_round(float(v)) for v in row] for row in a], np.uint8)
    A, B = enc(ia), enc(ib)
    assert np.array_equal(ref.fp8_gemm(A, B), (ia @ ib.T).astype(np.float64))
    assert np.array_equal(ref.fp8_gemm(A, B, alpha=0.25, rows=[3, 5], cols=[0, 7, 9]), 0.25 * (ia @ ib.T)[[3, 5]][:, [0, 7, 9]])
    codes_a = rng.integers(0, 256, (16, 96)).astype(np.uint8); codes_a[codes_a % 128 == 127] = 0
    codes_b = rng.integers(0, 256, (8, 96)).astype(np.uint8); codes_b[codes_b % 128 == 127] = 0
    want = _torch_e4m3_decode(codes_a) @ _torch_e4m3_decode(codes_b).T
    assert np.allclose(ref.fp8_gemm(codes_a, codes_b), want, rtol=1e-13, atol=0)


def test_fp8_forward_is_the_library_cast_pipeline_and_has_the_expected_error():
    rng = np.random.default_rng(3)
    b, n, m = 96, 256, 80
    x = wl.activation_like(rng, (b, n)); W = wl.weight_like(rng, (m, n))
    y = ref.linear_forward_fp8(x, W)
    sx, sw = ref.fp8_tensor_scale(x), ref.fp8_tensor_scale(W)
    q = lambda bits, s: torch.from_numpy((wl.bf16_bits_to_f32(bits) * np.float32(s)).astype(np.float32)).clamp(-448, 448) \
        .to(torch.float8_e4m3fn).to(torch.float64).numpy()
    want = q(x, sx) @ q(W, sw).T / (float(sx) * float(sw))
    assert np.allclose(y, want, rtol=1e-12, atol=0)
    exact = wl.bf16_bits_to_f64(x) @ wl.bf16_bits_to_f64(W).T
    err = np.linalg.norm(y - exact) / np.linalg.norm(exact)
    assert 0.015 < err < 0.06                                        # two operands with 3 mantissa bits each
    rows, cols = [0, 17, 95], [3, 79]
    assert np.array_equal(ref.linear_forward_fp8(x, W, rows=rows, cols=cols), y[rows][:, cols])


# ------------------------------------------------------------------------------------------------ MXINT4
def test_int4_codes_and_nearest_rounding():
    assert [ref.int4_value(c) for c in range(16)] == [0, 1, 2, 3, 4, 5, 6, 7, -0.0, -1, -2, -3, -4, -5, -6, -7]
    rng = np.random.default_rng(4)
    w = np.concatenate([rng.uniform(-9, 9, 5000), np.arange(-8, 8.5, 0.5)])
    got = np.array([ref.int4_value(ref.int4_rn_round(float(v))) for v in w])
    want = np.clip(np.rint(w), -7, 7)                                # numpy's rint rounds half to even
    assert np.array_equal(got, want)
    assert ref.int4_rn_round(-0.2) == 8                               # the sign of the input is kept


def test_int4_stochastic_rounding_is_eq_2_and_unbiased():
    rng = np.random.default_rng(5)
    r = np.arange(256)
    delta = 0.5 - (r + 0.5) / 256.0                                   # the dither of Eq. 1, discretised to 8 bits
    for w in list(rng.uniform(0, 6, 300)) + [5.25, 0.75, 1.0, 3.0, 0.001, 5.999]:
        got = np.array([ref.int4_value(ref.int4_sr_round(float(w), int(k))) for k in r])
        want = np.where(w + delta < np.floor(w) + 0.5, np.floor(w), np.ceil(w))      # Eq. 2 as printed
        assert np.array_equal(got, want)
        assert set(got) <= {np.floor(w), np.ceil(w)}
        frac = w - np.floor(w)
        assert abs(got.mean() - w) <= 2.0 ** -9                      # unbiased up to the dither's resolution
        if (256 * frac) % 1 == 0:
            assert got.mean() == w                                    # exactly unbiased when 256 frac is an integer
            assert np.isclose(got.var(), (np.ceil(w) - w) * (w - np.floor(w)))
    # hand-worked: 5.25 -> {5: 3/4, 6: 1/4};  -1.5 -> {-1: 1/2, -2: 1/2}
    v = np.array([ref.int4_value(ref.int4_sr_round(5.25, int(k))) for k in r])
    assert (v == 6).sum() == 64 and (v == 5).sum() == 192
    v = np.array([ref.int4_value(ref.int4_sr_round(-1.5, int(k))) for k in r])
    assert (v == -2).sum() == 128 and (v == -1).sum() == 128


def test_mxint4_blocks_scale_rule_and_clipping():
    y = np.zeros((1, 64), np.float32)
    y[0, :4] = [7.0, 1.0, -2.2, 0.3]; y[0, 32:36] = [7.9, -3.5, 0.5, 0.0]
    c, s = ref.mxint4_quantize(y, ref.ROUND_RN, 0, 0)
    assert list(s[0]) == [127, 127]                                   # amax in [4, 8): X = 1
    assert [ref.int4_value(int(k)) for k in c[0, :4]] == [7, 1, -2, 0]
    assert [ref.int4_value(int(k)) for k in c[0, 32:35]] == [7, -4, 0]          # 7.9 clips to 7; -3.5 and 0.5 tie to even
    # Algorithm 1 clips only values in (7.5, 8) X here; Algorithm 2 clips nothing and never exceeds 6
    rng = np.random.default_rng(6)
    g = rng.standard_normal((256, 1024)).astype(np.float32)
    crn, srn = ref.mxint4_quantize(g, ref.ROUND_RN, 1, 1)
    X = np.exp2(srn.astype(np.float64) - 127).repeat(32, axis=1)
    clipped = (np.abs(g) / X > 7.5).mean()
    assert 0 < clipped < 0.01
    csr, ssr = ref.mxint4_quantize(g, ref.ROUND_SR, 1, 1)
    assert np.array_equal(ssr, srn) and (csr & 7).max() <= 6
    w = 0.75 * g / X
    q = np.array([ref.int4_value(int(k)) for k in csr.ravel()]).reshape(g.shape)
    assert np.all((q == np.floor(w)) | (q == np.ceil(w)))
    assert abs((q - w).mean()) < 5 * np.sqrt(0.25 / g.size)


def test_mxint4_gemm_matches_numpy_and_the_estimate_is_unbiased_with_16_over_9():
    rng = np.random.default_rng(7)
    A = rng.standard_normal((24, 128)).astype(np.float32); B = rng.standard_normal((16, 128)).astype(np.float32)
    ca, sa = ref.mxint4_quantize(A, ref.ROUND_SR, 9, 1); cb, sb = ref.mxint4_quantize(B, ref.ROUND_SR, 9, 2)
    deq = lambda c, s: np.where(c & 8, -1.0, 1.0) * (c & 7) * np.exp2(s.astype(np.float64) - 127).repeat(32, axis=1)
    assert np.allclose(ref.mxint4_gemm(ca, sa, cb, sb, alpha=16 / 9), 16 / 9 * deq(ca, sa) @ deq(cb, sb).T, rtol=1e-13)
    exact = A.astype(np.float64) @ B.astype(np.float64).T
    errs = []
    for T in (16, 256):
        acc = np.zeros_like(exact)
        for t in range(T):
            ca, sa = ref.mxint4_quantize(A, ref.ROUND_SR, 100 + t, 1); cb, sb = ref.mxint4_quantize(B, ref.ROUND_SR, 100 + t, 2)
            acc += ref.mxint4_gemm(ca, sa, cb, sb, alpha=16 / 9)
        errs.append(np.linalg.norm(acc / T - exact) / np.linalg.norm(exact))
    assert errs[1] < errs[0] / 2.5                                    # T^-1/2: 16 times the samples, about a quarter of the error
    # nearest rounding without the pre-scale is biased: its error does not average out (one deterministic result)
    ca, sa = ref.mxint4_quantize(A, ref.ROUND_RN, 0, 1); cb, sb = ref.mxint4_quantize(B, ref.ROUND_RN, 0, 2)
    assert np.linalg.norm(ref.mxint4_gemm(ca, sa, cb, sb) - exact) / np.linalg.norm(exact) > errs[1]
