"""Parity of the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs.

Tolerances (stated by the benchmark spec):
  - codes and scales bit-exact when both sides see the same fp32 pre-quantisation values;
  - RHT output within 1e-5 relative (2-norm per g-chunk) of the fp64 transform;
  - end to end, at most 1e-4 of the codes differ, each by one grid step (blocks whose amax sits within fp32
    rounding of a power of two may pick a neighbouring scale; they are counted separately);
  - GEMM within 1e-5 relative Frobenius of the fp64 product of the same dequantised operands (fp32 output).
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


def _dev(bits: np.ndarray):
    import torch
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def _quant_gpu(gpu, x_bits, reduce_dim, g, seed, tag, rounding, layout):
    codes, scales = gpu.mxfp4_rht_sr_quantize(_dev(x_bits), reduce_dim, g, seed, tag, rounding, layout)
    assert gpu.mxfp4_device_status() == 0
    codes = hp.unpack_codes(codes.cpu().numpy())
    R, K = codes.shape
    s = scales.cpu().numpy()
    s = hp.sf_native_to_linear(s, R, K) if layout == gpu.SF_NATIVE else s.reshape(R, K // 32)
    return codes, s


def _inputs(kind, shape, seed):
    rng = np.random.default_rng(seed)
    if kind == "grad":
        return wl.grad_like(rng, shape, 1e-3, outlier_rate=1e-3)
    if kind == "act":
        return wl.activation_like(rng, shape, n_outlier_channels=4)
    if kind == "int":
        return wl.small_integer_like(rng, shape)
    raise ValueError(kind)


# ------------------------------------------------------------------------------------------- quantiser

@pytest.mark.parametrize("rounding", [0, 1, 2])
@pytest.mark.parametrize("reduce_dim,shape", [(1, (200, 1184)), (1, (3, 32)), (0, (544, 200)), (0, (32, 8)),
                                              (1, (200, 1280)), (0, (640, 200))])   # the last two: reduce length a multiple of 128
def test_quantizer_bit_exact_without_rht(gpu, ref, rounding, reduce_dim, shape):
    """g = 0: both sides quantise the same fp32 values (the bf16 inputs), so everything is bit-exact.
    Shapes span several tiles and a ragged tail in both dimensions."""
    x = _inputs("grad", shape, 1)
    x[0, :8] = 0                                            # some zeros, a negative zero
    x[0, 1] = 0x8000
    for layout in (gpu.SF_LINEAR, gpu.SF_NATIVE):
        codes, scales = _quant_gpu(gpu, x, reduce_dim, 0, 77, 5, rounding, layout)
        _, rc, rs = ref.rht_quantize(x, 0, rounding, 77, 5, transpose=(reduce_dim == 0))
        assert np.array_equal(scales, rs)
        assert np.array_equal(codes, rc)


@pytest.mark.parametrize("g", [64, 256])
@pytest.mark.parametrize("reduce_dim,shape", [(1, (130, 1024)), (0, (768, 136))])
def test_quantizer_bit_exact_on_integer_inputs(gpu, ref, g, reduce_dim, shape):
    """Small-integer inputs make every +-sum exact in fp32 in any order and 1/sqrt(g) is a power of two, so the
    fp32 transform is identical on both sides and the whole quantiser (RHT included) must match bit for bit."""
    x = _inputs("int", shape, 2)
    for rounding in (0, 1, 2):
        codes, scales = _quant_gpu(gpu, x, reduce_dim, g, 1234, 2, rounding, gpu.SF_NATIVE)
        y, rc, rs = ref.rht_quantize(x, g, rounding, 1234, 2, transpose=(reduce_dim == 0))
        ygpu = gpu.mxfp4_rht(_dev(x), reduce_dim, g, 1234).cpu().numpy()
        assert np.array_equal(ygpu, y)
        assert np.array_equal(scales, rs)
        assert np.array_equal(codes, rc)


@pytest.mark.parametrize("g", [32, 64, 128, 256])
@pytest.mark.parametrize("reduce_dim,shape,kind", [(1, (96, 1280), "grad"), (0, (1024, 72), "act"), (0, (512, 264), "grad")])
def test_rht_within_tolerance_and_quantiser_exact_on_gpu_values(gpu, ref, g, reduce_dim, shape, kind):
    x = _inputs(kind, shape, 3)
    seed = 4321
    y_ref = ref.rht(x, g, seed, transpose=(reduce_dim == 0)).astype(np.float64)
    y_gpu = gpu.mxfp4_rht(_dev(x), reduce_dim, g, seed).cpu().numpy()
    R, K = y_ref.shape
    d = (y_gpu.astype(np.float64) - y_ref).reshape(R, K // g, g)
    rel = np.linalg.norm(d, axis=2) / np.maximum(np.linalg.norm(y_ref.reshape(R, K // g, g), axis=2), 1e-300)
    assert rel.max() <= 1e-5
    # feed the GPU's own fp32 values to the oracle quantiser: codes and scales must then be bit-exact
    for rounding in (0, 1, 2):
        codes, scales = _quant_gpu(gpu, x, reduce_dim, g, seed, 9, rounding, gpu.SF_LINEAR)
        rc, rs = ref.quantize(y_gpu, rounding, seed, 9)
        assert np.array_equal(scales, rs)
        assert np.array_equal(codes, rc)


@pytest.mark.parametrize("rounding", [0, 2])
@pytest.mark.parametrize("g", [64, 128])
def test_quantizer_end_to_end_mismatch_rate(gpu, ref, g, rounding):
    """Against the oracle's own fp64 transform: <= 1e-4 of codes differ, each by one grid step."""
    for reduce_dim, shape in ((1, (512, 2048)), (0, (2048, 512))):
        x = _inputs("act", shape, 5)
        codes, scales = _quant_gpu(gpu, x, reduce_dim, g, 99, 1, rounding, gpu.SF_NATIVE)
        _, rc, rs = ref.rht_quantize(x, g, rounding, 99, 1, transpose=(reduce_dim == 0))
        assert (scales != rs).mean() <= 1e-5                      # amax within rounding of a power of two
        hp.compare_quantised_rows(codes, scales, rc, rs)          # such blocks are compared by their dequantised values


@pytest.mark.parametrize("rounding", [0, 2])
def test_quantiser_exact_on_four_million_gpu_values(gpu, ref, rounding):
    """A sample large enough to meet the rare decisions: with full fp32 mantissas about one element in 2^17 sits
    within one dither step of its threshold, where a rounded (instead of truncated) fraction or an off-by-one in the
    comparison would flip the code.  The GPU's own fp32 transform is fed to the oracle, so codes must be bit-exact."""
    x = _inputs("grad", (2048, 2048), 41)
    seed = 77
    for reduce_dim in (1, 0):
        y_gpu = gpu.mxfp4_rht(_dev(x), reduce_dim, 128, seed).cpu().numpy()
        codes, scales = _quant_gpu(gpu, x, reduce_dim, 128, seed, 4, rounding, gpu.SF_NATIVE)
        rc, rs = ref.quantize(y_gpu, rounding, seed, 4)
        assert np.array_equal(scales, rs)
        assert np.array_equal(codes, rc)
        mag = codes & 7
        assert all((mag == i).any() for i in range(8))


def test_quantizer_is_deterministic_and_tags_differ(gpu):
    x = _inputs("grad", (256, 512), 6)
    a = _quant_gpu(gpu, x, 0, 64, 5, 1, 0, gpu.SF_NATIVE)
    b = _quant_gpu(gpu, x, 0, 64, 5, 1, 0, gpu.SF_NATIVE)
    c = _quant_gpu(gpu, x, 0, 64, 5, 2, 0, gpu.SF_NATIVE)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    assert not np.array_equal(a[0], c[0]) and np.array_equal(a[1], c[1])


def test_quantizer_huge_and_tiny_magnitudes(gpu, ref):
    """Scale clamps and the wide-exponent path: blocks near 2^100 and near the subnormals."""
    rng = np.random.default_rng(8)
    x = rng.standard_normal((64, 256)).astype(np.float32)
    x[:16] *= 2.0 ** 100
    x[16:32] *= 2.0 ** -120
    x[32:48] *= 2.0 ** 30
    x[48:, :32] = 0
    xb = wl.to_bf16_bits(x)
    for rounding in (0, 1, 2):
        codes, scales = _quant_gpu(gpu, xb, 1, 0, 3, 1, rounding, gpu.SF_LINEAR)
        _, rc, rs = ref.rht_quantize(xb, 0, rounding, 3, 1)
        assert np.array_equal(scales, rs)
        assert np.array_equal(codes, rc)


# ------------------------------------------------------------------------------------------------ GEMM

def _rand_operand(rng, R, K, scale_lo=118, scale_hi=136):
    codes = rng.integers(0, 16, (R, K)).astype(np.uint8)
    scales = rng.integers(scale_lo, scale_hi, (R, K // 32)).astype(np.uint8)
    return codes, scales


def _gemm_gpu(gpu, ca, sa, cb, sb, alpha=1.0, out=None):
    import torch
    from oracle import ref as _ref
    A = torch.from_numpy(_ref.pack(ca)).cuda()
    Bm = torch.from_numpy(_ref.pack(cb)).cuda()
    SA = torch.from_numpy(hp.sf_linear_to_native(sa, fill=255)).cuda()     # padding bytes are NaN scales on purpose
    SB = torch.from_numpy(hp.sf_linear_to_native(sb, fill=255)).cuda()
    Cm = gpu.mxfp4_gemm(A, SA, Bm, SB, alpha, gpu.OUT_FP32 if out is None else out)
    assert gpu.mxfp4_device_status() == 0
    return Cm.float().cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("M,N,K", [(128, 256, 256), (128, 256, 128), (256, 512, 1024), (200, 264, 640), (1, 8, 128), (384, 1032, 2176)])
def test_gemm_matches_fp64_product_of_dequantised_operands(gpu, ref, M, N, K):
    rng = np.random.default_rng(M + N + K)
    ca, sa = _rand_operand(rng, M, K)
    cb, sb = _rand_operand(rng, N, K)
    C = _gemm_gpu(gpu, ca, sa, cb, sb)
    Cref = ref.gemm(ca, sa, cb, sb)
    assert np.linalg.norm(C - Cref) / np.linalg.norm(Cref) <= 1e-5
    # alpha and the bf16 epilogue
    Cb = _gemm_gpu(gpu, ca, sa, cb, sb, alpha=16 / 9, out=gpu.OUT_BF16)
    assert np.linalg.norm(Cb - 16 / 9 * Cref) / np.linalg.norm(Cref) <= 2.0 ** -8


def test_gemm_special_cases(gpu):
    M, N, K = 128, 256, 512
    ones = np.full((M, K), 2, np.uint8)
    C = _gemm_gpu(gpu, ones, np.full((M, K // 32), 127, np.uint8), np.full((N, K), 2, np.uint8), np.full((N, K // 32), 127, np.uint8))
    assert np.all(C == K)
    # a single nonzero block with distinct scales: exact power-of-two scaling, correct (row, col, k-block)
    rng = np.random.default_rng(0)
    for _ in range(8):
        i, j, kb = rng.integers(0, M), rng.integers(0, N), rng.integers(0, K // 32)
        ca = np.zeros((M, K), np.uint8); cb = np.zeros((N, K), np.uint8)
        sa = np.full((M, K // 32), 127, np.uint8); sb = np.full((N, K // 32), 127, np.uint8)
        ca[i, 32 * kb:32 * kb + 32] = 7; cb[j, 32 * kb:32 * kb + 32] = 0xD
        ea, eb = int(rng.integers(-20, 20)), int(rng.integers(-20, 20))
        sa[i, kb] = 127 + ea; sb[j, kb] = 127 + eb
        C = _gemm_gpu(gpu, ca, sa, cb, sb)
        expect = np.zeros((M, N)); expect[i, j] = 32 * 6 * -3 * 2.0 ** (ea + eb)
        assert np.array_equal(C, expect)


def test_gemm_long_k_accumulation(gpu, ref):
    """K = 16384 (the wgrad reduction length of the GPT shapes): fp32 accumulation stays within 1e-5."""
    rng = np.random.default_rng(11)
    M, N, K = 128, 256, 16384
    ca, sa = _rand_operand(rng, M, K, 125, 130)
    cb, sb = _rand_operand(rng, N, K, 125, 130)
    C = _gemm_gpu(gpu, ca, sa, cb, sb)
    Cref = ref.gemm(ca, sa, cb, sb)
    assert np.linalg.norm(C - Cref) / np.linalg.norm(Cref) <= 1e-5


# ------------------------------------------------------------------------------------- Algorithm 3 end to end

@pytest.mark.parametrize("rounding", [0, 1, 2])
def test_linear_backward_single_layer(gpu, ref, rounding):
    """256 tokens x 512 -> 512, g = 64, seed 0: every output element against the oracle."""
    import torch
    layer = wl.CONFIGS["single_256x512"][0][0]
    dY, X, W = wl.layer_inputs("single_256x512", layer, seed=0)
    dX, dW = gpu.mxfp4_linear_backward(_dev(dY), _dev(X), _dev(W), 64, 0, rounding, gpu.OUT_FP32)
    assert gpu.mxfp4_device_status() == 0
    dX = dX.cpu().numpy().astype(np.float64); dW = dW.cpu().numpy().astype(np.float64)
    rdX, rdW = ref.linear_backward(dY, X, W, 64, rounding, 0)
    # strict: the GEMMs reproduce the fp64 product of the operands the GPU itself quantised
    tags = {1: (dY, 1), 2: (W, 0), 3: (dY, 0), 4: (X, 0)}
    q, rate = {}, {}
    for tag, (t, rd) in tags.items():
        q[tag] = _quant_gpu(gpu, t, rd, 64, 0, tag, rounding, gpu.SF_NATIVE)
        _, oc, os_ = ref.rht_quantize(t, 64, rounding, 0, tag, transpose=(rd == 0))
        rate[tag] = hp.compare_quantised_rows(q[tag][0], q[tag][1], oc, os_)
    # codes may differ in <= 1e-4 of the elements by one step, so the end-to-end outputs agree closely, not bitwise:
    # the bound follows from the differences actually counted (1e-5 when there are none)
    assert np.linalg.norm(dX - rdX) / np.linalg.norm(rdX) <= hp.product_tolerance(rate[1], rate[2])
    assert np.linalg.norm(dW - rdW) / np.linalg.norm(rdW) <= hp.product_tolerance(rate[3], rate[4])
    alpha = 16 / 9 if rounding != 1 else 1.0
    assert np.linalg.norm(dX - ref.gemm(*q[1], *q[2], alpha=alpha)) / np.linalg.norm(rdX) <= 1e-5
    assert np.linalg.norm(dW - ref.gemm(*q[3], *q[4], alpha=alpha)) / np.linalg.norm(rdW) <= 1e-5
    # and the result is a sane estimate of the true gradients
    ex = wl.bf16_bits_to_f64(dY) @ wl.bf16_bits_to_f64(W)
    assert np.linalg.norm(dX - ex) / np.linalg.norm(ex) < 0.5
    # bf16 outputs
    dXb, dWb = gpu.mxfp4_linear_backward(_dev(dY), _dev(X), _dev(W), 64, 0, rounding, gpu.OUT_BF16)
    assert np.linalg.norm(dXb.float().cpu().numpy() - dX) / np.linalg.norm(dX) <= 2.0 ** -8
    assert np.linalg.norm(dWb.float().cpu().numpy() - dW) / np.linalg.norm(dW) <= 2.0 ** -8


# ------------------------------------------------------------------------------------- measurement aid

def test_fp4_ceiling_kernel_runs_and_reports_its_work(gpu):
    """The tensor-pipe ceiling kernel: flop count = pairs x MMAs (rounded up to 32) x 2*256*256*64, no timeout."""
    import torch
    pairs = torch.cuda.get_device_properties(0).multi_processor_count // 2
    assert gpu.mxfp4_fp4_ceiling(40) == pairs * 64 * 2 * 256 * 256 * 64
    assert gpu.mxfp4_fp4_ceiling(1) == pairs * 32 * 2 * 256 * 256 * 64
    assert gpu.mxfp4_device_status() == 0
    with pytest.raises(gpu.MxFp4Error):
        gpu.mxfp4_fp4_ceiling(0)


# ------------------------------------------------------------------------------------- bias gradient, accumulation

@pytest.mark.parametrize("b,m,n", [(256, 512, 512), (384, 640, 264), (2048, 1152, 128), (256, 128, 64)])
def test_bias_grad_and_accumulation(gpu, ref, b, m, n):
    """dL/db = 1 dL/dy in fp32 against the fp64 oracle; accumulate adds a second micro-batch into fp32 dW and db."""
    import torch
    rng = np.random.default_rng(b + m)
    m = (m // 128) * 128
    dY = wl.to_bf16_bits(rng.standard_t(3, (b, m)) * 1e-3)
    X = wl.to_bf16_bits(rng.standard_normal((b, n)))
    W = wl.to_bf16_bits(rng.standard_normal((m, n)) * 0.02)
    dX, dW, db = gpu.mxfp4_linear_backward_ex(_dev(dY), _dev(X), _dev(W), 64, 5, gpu.ROUND_SR, gpu.OUT_FP32, with_bias=True)
    assert gpu.mxfp4_device_status() == 0
    # fp32 sums of b terms: error bounded by b 2^-24 sum|dY| per column; typical sqrt(b) 2^-24
    want = ref.bias_grad(dY)
    bound = 64 * np.sqrt(b) * 2.0 ** -24 * np.abs(wl.bf16_bits_to_f64(dY)).sum(axis=0) + 1e-30
    assert np.all(np.abs(db.cpu().numpy().astype(np.float64) - want) <= bound)
    # the other outputs equal the plain call's
    dX0, dW0 = gpu.mxfp4_linear_backward(_dev(dY), _dev(X), _dev(W), 64, 5, gpu.ROUND_SR, gpu.OUT_FP32)
    assert torch.equal(dX, dX0) and torch.equal(dW, dW0)
    # second micro-batch with another seed, accumulated
    dY2 = wl.to_bf16_bits(rng.standard_t(3, (b, m)) * 1e-3)
    X2 = wl.to_bf16_bits(rng.standard_normal((b, n)))
    _, dW1, _ = gpu.mxfp4_linear_backward_ex(_dev(dY2), _dev(X2), _dev(W), 64, 6, gpu.ROUND_SR, gpu.OUT_FP32)
    dWa, dba = dW.clone(), db.clone()
    dX2, dWa, dba = gpu.mxfp4_linear_backward_ex(_dev(dY2), _dev(X2), _dev(W), 64, 6, gpu.ROUND_SR, gpu.OUT_FP32,
                                                  dW=dWa, db=dba, accumulate=True)
    assert gpu.mxfp4_device_status() == 0
    assert torch.equal(dWa, dW + dW1)                      # one fp32 add per element, same operands: exact
    want2 = want + ref.bias_grad(dY2)
    bound2 = bound + 64 * np.sqrt(b) * 2.0 ** -24 * np.abs(wl.bf16_bits_to_f64(dY2)).sum(axis=0)
    assert np.all(np.abs(dba.cpu().numpy().astype(np.float64) - want2) <= bound2)
    # bf16 output cannot accumulate
    with pytest.raises(gpu.MxFp4Error):
        gpu.mxfp4_linear_backward_ex(_dev(dY), _dev(X), _dev(W), 64, 5, gpu.ROUND_SR, gpu.OUT_BF16,
                                     dW=torch.zeros((m, n), dtype=torch.bfloat16, device="cuda"), accumulate=True)


def test_linear_backward_captures_into_a_cuda_graph(gpu):
    """A shape large enough for the fork / join of the two GEMMs: the captured graph replays to the same bits."""
    import torch
    gen = torch.Generator(device="cuda").manual_seed(1)
    b, n, m, g = 4096, 2048, 4096, 128
    dY = (torch.randn((b, m), generator=gen, device="cuda") * 1e-3).to(torch.bfloat16)
    X = torch.randn((b, n), generator=gen, device="cuda").to(torch.bfloat16)
    W = (torch.randn((m, n), generator=gen, device="cuda") * 0.02).to(torch.bfloat16)
    dX = torch.empty((b, n), dtype=torch.bfloat16, device="cuda")
    dW = torch.empty((m, n), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(gpu.mxfp4_linear_backward_workspace(b, m, n), dtype=torch.uint8, device="cuda")
    gpu.mxfp4_linear_backward(dY, X, W, g, 7, gpu.ROUND_SR, gpu.OUT_BF16, dX=dX, dW=dW, workspace=ws)
    torch.cuda.synchronize()
    want_x, want_w = dX.clone(), dW.clone()
    dX.zero_(); dW.zero_()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            gpu.mxfp4_linear_backward(dY, X, W, g, 7, gpu.ROUND_SR, gpu.OUT_BF16, dX=dX, dW=dW, workspace=ws)
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(dX, want_x) and torch.equal(dW, want_w)
    assert gpu.mxfp4_device_status() == 0


def test_linear_backward_is_bitwise_reproducible(gpu):
    """Same inputs, same seed: the same bits, call after call (fixed MMA order, fixed summation order of the bias sums)."""
    import torch
    gen = torch.Generator(device="cuda").manual_seed(9)
    b, n, m, g = 4096, 2048, 4096, 128
    dY = (torch.randn((b, m), generator=gen, device="cuda") * 1e-3).to(torch.bfloat16)
    X = torch.randn((b, n), generator=gen, device="cuda").to(torch.bfloat16)
    W = (torch.randn((m, n), generator=gen, device="cuda") * 0.02).to(torch.bfloat16)
    first = gpu.mxfp4_linear_backward_ex(dY, X, W, g, 21, gpu.ROUND_SR, gpu.OUT_FP32, with_bias=True)
    for _ in range(3):
        again = gpu.mxfp4_linear_backward_ex(dY, X, W, g, 21, gpu.ROUND_SR, gpu.OUT_FP32, with_bias=True)
        assert all(torch.equal(a, c) for a, c in zip(first, again))
    other = gpu.mxfp4_linear_backward_ex(dY, X, W, g, 22, gpu.ROUND_SR, gpu.OUT_FP32, with_bias=True)
    assert not torch.equal(first[0], other[0]) and torch.equal(first[2], other[2])      # the seed moves dX, not the bias sums
    assert gpu.mxfp4_device_status() == 0


def test_split_form_equals_the_one_call_form(gpu):
    """mxfp4_quantize_operands + two mxfp4_gemm calls give bit for bit what mxfp4_linear_backward gives."""
    import torch
    gen = torch.Generator(device="cuda").manual_seed(13)
    b, m, n, g = 512, 384, 264, 128
    dY = (torch.randn(b, m, device="cuda", generator=gen) * 1e-3).to(torch.bfloat16)
    X = torch.randn(b, n, device="cuda", generator=gen).to(torch.bfloat16)
    W = (torch.randn(m, n, device="cuda", generator=gen) * 0.02).to(torch.bfloat16)
    for rounding, alpha, g in ((gpu.ROUND_SR, 16 / 9, 128), (gpu.ROUND_RN, 1.0, 128), (gpu.ROUND_SR16, 16 / 9, 128), (gpu.ROUND_SR, 16 / 9, 0)):
        q = gpu.mxfp4_quantize_operands(dY, X, W, g, 17, rounding)      # g = 0: the views go through the CUDA-core quantiser one by one
        dX = gpu.mxfp4_gemm(q[0][0], q[0][1], q[1][0], q[1][1], alpha, gpu.OUT_FP32)
        dW = gpu.mxfp4_gemm(q[2][0], q[2][1], q[3][0], q[3][1], alpha, gpu.OUT_FP32)
        rX, rW = gpu.mxfp4_linear_backward(dY, X, W, g, 17, rounding, gpu.OUT_FP32)
        assert torch.equal(dX, rX) and torch.equal(dW, rW)
        # and each view equals the single-operand call with its stream tag
        for i, (t, rd) in enumerate(((dY, 1), (W, 0), (dY, 0), (X, 0))):
            c, s = gpu.mxfp4_rht_sr_quantize(t, rd, g, 17, i + 1, rounding, gpu.SF_NATIVE)
            R, K = c.shape[0], 2 * c.shape[1]                 # padding bytes of the tiled scale layout are not written: compare the decoded scales
            assert torch.equal(c, q[i][0])
            assert np.array_equal(hp.sf_native_to_linear(s.cpu().numpy(), R, K), hp.sf_native_to_linear(q[i][1].cpu().numpy(), R, K))
    assert gpu.mxfp4_device_status() == 0


@pytest.mark.parametrize("reduce_dim,shape", [(1, (200, 1280)), (0, (640, 136))])
def test_quantiser_with_a_given_transform_matrix(gpu, ref, reduce_dim, shape):
    """Section 3.2: any orthogonal matrix may replace the RHT.  (a) Given T = diag(S) H_64 / 8 (exact in bf16) the call
    reproduces the RHT quantiser bit for bit; (b) with a random orthogonal matrix (bf16-rounded) the transform matches
    the oracle's explicit product to 1e-5 per chunk and the codes are the oracle's on the GPU's own fp32 values."""
    import torch
    x = _inputs("grad", shape, 23)
    seed = 1234
    S = ref.sign_vector(seed, 64).astype(np.float64)
    T = wl.to_bf16_bits(((S[:, None] * ref.hadamard(64)) / 8.0).astype(np.float32))
    for rounding in (0, 2):
        c, s = gpu.mxfp4_transform_quantize(_dev(x), reduce_dim, _dev(T), seed, 3, rounding, gpu.SF_LINEAR)
        c0, s0 = gpu.mxfp4_rht_sr_quantize(_dev(x), reduce_dim, 64, seed, 3, rounding, gpu.SF_LINEAR)
        assert torch.equal(c, c0) and torch.equal(s, s0)
    rng = np.random.default_rng(29)
    for g in (32, 128):
        Q, _ = np.linalg.qr(rng.standard_normal((g, g)))
        Qb = wl.to_bf16_bits(Q.astype(np.float32))
        y_gpu = gpu.mxfp4_transform_quantize(_dev(x), reduce_dim, _dev(Qb), seed, 5, dump=True).cpu().numpy()
        y_ref = ref.transform(x, Qb, transpose=(reduce_dim == 0)).astype(np.float64)
        R, K = y_ref.shape
        d = (y_gpu.astype(np.float64) - y_ref).reshape(R, K // g, g)
        rel = np.linalg.norm(d, axis=2) / np.maximum(np.linalg.norm(y_ref.reshape(R, K // g, g), axis=2), 1e-300)
        assert rel.max() <= 1e-5
        for rounding in (0, 1, 2):
            c, s = gpu.mxfp4_transform_quantize(_dev(x), reduce_dim, _dev(Qb), seed, 5, rounding, gpu.SF_LINEAR)
            rc, rs = ref.quantize(y_gpu, rounding, seed, 5)
            assert np.array_equal(hp.unpack_codes(c.cpu().numpy()), rc)
            assert np.array_equal(s.cpu().numpy().reshape(R, K // 32), rs)
    assert gpu.mxfp4_device_status() == 0
