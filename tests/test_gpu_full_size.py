"""Parity at full sizes (GPT 345M / 1.3B / 6.7B layer shapes with their g, and the ablation GEMM), in the launch
configuration bench.py times.

The oracle cannot run whole 16384 x 16384 operands in seconds, so outputs are SAMPLED: every dX / dW entry depends
on one row of each quantised operand, and the oracle quantises exactly those rows (their SR draws are keyed on the
row index in the full operand).  Checked per layer:
  - codes and scales of the sampled operand rows against the oracle (<= 1e-4 mismatches, one grid step; blocks with
    neighbouring scale bytes are compared by their dequantised values),
  - the GPU GEMM on its own codes against the fp64 product of those codes (<= 1e-5, fp32 output),
  - mxfp4_linear_backward's bf16 outputs at the sampled entries against the oracle's Algorithm 3, within a bound
    derived from the counted code differences.
The benchmark's layers and one layer of each smaller config are sampled so that no output tile can be missed: one
row in every 128-row band (rotating through the epilogue quadrants) and one column in every 32-column chunk.
"""
import numpy as np
import pytest

from paper_2502_20586_b200 import workloads as wl
from tests import helpers as hp

pytestmark = pytest.mark.gpu


def _bits(t):
    import torch
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


# (config, layer, rounding, dense): dense = band / chunk sampling that touches every output tile
DENSE = {("gpt_6p7b", "attn_out"), ("gpt_6p7b", "fc1"), ("gpt_6p7b", "qkv"), ("gpt_6p7b", "fc2"), ("gpt_1p3b", "fc2"), ("gpt_345m", "attn_out")}
CASES = [("gpt_6p7b", "attn_out"), ("gpt_6p7b", "fc1"), ("gpt_6p7b", "qkv"), ("gpt_6p7b", "fc2"),
         ("gpt_1p3b", "qkv"), ("gpt_1p3b", "attn_out"), ("gpt_1p3b", "fc1"), ("gpt_1p3b", "fc2"),
         ("gpt_345m", "qkv"), ("gpt_345m", "attn_out"), ("gpt_345m", "fc1"), ("gpt_345m", "fc2")]
# rounding mode per case: the 8-bit SR reading everywhere, the 16-bit one on the benchmark's layers and one small layer
CASES = [c + (0,) for c in CASES] + [("gpt_6p7b", l, 2) for l in ("attn_out", "fc1", "qkv", "fc2")] + [("gpt_345m", "fc1", 2)]


@pytest.mark.parametrize("config,layer_name,rounding", CASES)
def test_sampled_parity_at_full_shapes(ref, config, layer_name, rounding):
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no GPU")
    from paper_2502_20586_b200 import binding as mx

    layers, g = wl.CONFIGS[config]
    layer = [l for l in layers if l.name == layer_name][0]
    b, n, m = layer.b, layer.n, layer.m
    seed = 3
    dY, X, W = wl.layer_inputs_device(config, layer, seed=0)
    if (config, layer_name) in DENSE and rounding == 0:
        I, J = hp.band_rows(b), hp.chunk_cols(n)                                                      # dX[I, J]
        P, Q = hp.band_rows(m), hp.chunk_cols(n)                                                      # dW[P, Q]
    else:
        rng = np.random.default_rng(17)
        I = np.sort(rng.choice(b, 12, replace=False)); J = np.sort(rng.choice(n, 10, replace=False))
        P = np.sort(rng.choice(m, 12, replace=False)); Q = np.sort(rng.choice(n, 10, replace=False))
    It, Jt, Pt, Qt = (torch.from_numpy(a).cuda() for a in (I, J, P, Q))

    # operand views of Algorithm 3: (tensor, reduce_dim, tag, sampled output rows, host slice with those rows as rows)
    views = {
        1: (dY, 1, I, _bits(dY[It, :])),              # Q1 rows I      = dY[I, :]        K = m
        2: (W, 0, J, _bits(W[:, Jt].t())),            # Q2 rows J      = W[:, J]^T       K = m
        3: (dY, 0, P, _bits(dY[:, Pt].t())),          # Q3 rows P      = dY[:, P]^T      K = b
        4: (X, 0, Q, _bits(X[:, Qt].t())),            # Q4 rows Q      = X[:, Q]^T       K = b
    }
    gpu_q, ora_q, rate = {}, {}, {}
    for tag, (t, rd, rows, host_rows) in views.items():
        codes, scales = mx.mxfp4_rht_sr_quantize(t, rd, g, seed, tag, rounding, mx.SF_NATIVE)
        R, K = codes.shape[0], codes.shape[1] * 2
        rt = torch.from_numpy(rows).cuda()
        c = hp.unpack_codes(codes[rt, :].cpu().numpy())
        offs = torch.from_numpy(hp.sf_native_offsets(R, K)[rows, :]).cuda()
        s = scales[offs].cpu().numpy()
        gpu_q[tag] = (c, s, codes, scales)
        _, oc, os_ = ref.rht_quantize(host_rows, g, rounding, seed, tag, row_ids=rows)
        ora_q[tag] = (oc, os_)
        rate[tag] = hp.compare_quantised_rows(c, s, oc, os_)
    assert mx.mxfp4_device_status() == 0

    # GEMMs on the GPU's own codes, fp32 output, against the fp64 product of the same codes
    alpha = 16.0 / 9.0
    Cx = mx.mxfp4_gemm(gpu_q[1][2], gpu_q[1][3], gpu_q[2][2], gpu_q[2][3], alpha, mx.OUT_FP32)
    Cw = mx.mxfp4_gemm(gpu_q[3][2], gpu_q[3][3], gpu_q[4][2], gpu_q[4][3], alpha, mx.OUT_FP32)
    assert mx.mxfp4_device_status() == 0
    gx = Cx[It][:, Jt].cpu().numpy().astype(np.float64); gw = Cw[Pt][:, Qt].cpu().numpy().astype(np.float64)
    rx = ref.gemm(gpu_q[1][0], gpu_q[1][1], gpu_q[2][0], gpu_q[2][1], alpha=alpha)
    rw = ref.gemm(gpu_q[3][0], gpu_q[3][1], gpu_q[4][0], gpu_q[4][1], alpha=alpha)
    assert np.linalg.norm(gx - rx) <= 1e-5 * np.linalg.norm(rx)
    assert np.linalg.norm(gw - rw) <= 1e-5 * np.linalg.norm(rw)
    # entry by entry as well: a tile that was skipped or misplaced shows up as entries that are plainly wrong
    assert np.all(np.abs(gx - rx) <= 1e-4 * np.abs(rx) + 1e-5 * np.sqrt(np.mean(rx ** 2)))
    assert np.all(np.abs(gw - rw) <= 1e-4 * np.abs(rw) + 1e-5 * np.sqrt(np.mean(rw ** 2)))
    del Cx, Cw

    # the one-call path, bf16 outputs as in the benchmark, against the oracle's own Algorithm 3 on the sampled rows
    dX, dW = mx.mxfp4_linear_backward(dY, X, W, g, seed, rounding, mx.OUT_BF16)
    assert mx.mxfp4_device_status() == 0
    ox = ref.gemm(*ora_q[1], *ora_q[2], alpha=alpha); ow = ref.gemm(*ora_q[3], *ora_q[4], alpha=alpha)
    bx = dX[It][:, Jt].float().cpu().numpy().astype(np.float64); bw = dW[Pt][:, Qt].float().cpu().numpy().astype(np.float64)
    assert np.linalg.norm(bx - ox) <= hp.product_tolerance(rate[1], rate[2], out_bits=8) * np.linalg.norm(ox)
    assert np.linalg.norm(bw - ow) <= hp.product_tolerance(rate[3], rate[4], out_bits=8) * np.linalg.norm(ow)
    # against the product of the GPU's own codes only bf16 rounding is left, entry by entry (unit roundoff 2^-8)
    assert np.all(np.abs(bx - rx) <= 2.0 ** -8 * np.abs(rx) + 1e-5 * np.sqrt(np.mean(rx ** 2)))
    assert np.all(np.abs(bw - rw) <= 2.0 ** -8 * np.abs(rw) + 1e-5 * np.sqrt(np.mean(rw ** 2)))
    # and it is a sane estimate of the true gradient entries (fp64 product of the bf16 inputs)
    tx = wl.bf16_bits_to_f64(views[1][3]) @ wl.bf16_bits_to_f64(views[2][3]).T
    assert np.linalg.norm(bx - tx) < 0.6 * np.linalg.norm(tx)


@pytest.mark.parametrize("g", [32, 256])
@pytest.mark.parametrize("reduce_dim", [1, 0])
def test_full_size_operand_through_g32_and_g256(ref, g, reduce_dim):
    """One 16384 x 16384 operand through the block sizes the GPT configs do not use (g = 256 runs its own kernel
    instantiation: two half-transforms per chunk, accumulator pairs).  A row of every 128-row band is checked: the
    transform within 1e-5 per chunk, and codes and scales bit for bit on the GPU's own fp32 values."""
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no GPU")
    from paper_2502_20586_b200 import binding as mx

    n = 16384
    gen = torch.Generator(device="cuda"); gen.manual_seed(5 + g + reduce_dim)
    x = (torch.randn((n, n), generator=gen, device="cuda") * 1e-2).to(torch.bfloat16)
    seed, tag = 11, 3
    rows = hp.band_rows(n)
    rt = torch.from_numpy(rows).cuda()
    host_rows = _bits(x[rt, :]) if reduce_dim == 1 else _bits(x[:, rt].t())
    y_gpu = mx.mxfp4_rht(x, reduce_dim, g, seed)[rt, :].cpu().numpy()
    y_ref = ref.rht(host_rows, g, seed).astype(np.float64)
    d = (y_gpu.astype(np.float64) - y_ref).reshape(len(rows), n // g, g)
    rel = np.linalg.norm(d, axis=2) / np.maximum(np.linalg.norm(y_ref.reshape(len(rows), n // g, g), axis=2), 1e-300)
    assert rel.max() <= 1e-5
    offs = torch.from_numpy(hp.sf_native_offsets(n, n)[rows, :]).cuda()
    for rounding in (0, 1, 2):
        codes, scales = mx.mxfp4_rht_sr_quantize(x, reduce_dim, g, seed, tag, rounding, mx.SF_NATIVE)
        c = hp.unpack_codes(codes[rt, :].cpu().numpy())
        s = scales[offs].cpu().numpy()
        rc, rs = ref.quantize(y_gpu, rounding, seed, tag, row_ids=rows)
        assert np.array_equal(s, rs)
        assert np.array_equal(c, rc)
        del codes, scales
    assert mx.mxfp4_device_status() == 0


@pytest.mark.parametrize("rate", [0.0, 1e-3, 1e-2])
def test_ablation_gemm_at_its_stated_shape(ref, rate):
    """The ablation GEMM at 16384 x 8192 x 2048 for g in {32, 64, 128, 256} x {RHT + SR, RHT + nearest}: the error
    against the fp64 product of the bf16 inputs, on a row of every 128-row band and a column of every 64-column
    chunk, must be the oracle's (same rows, same columns, the oracle's own quantisation and products)."""
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no GPU")
    from paper_2502_20586_b200 import ablation, binding as mx

    M, N, K = 16384, 8192, 2048
    A, B = ablation._operands(M, N, K, rate, 1, torch.device("cuda", 0))
    I, J = hp.band_rows(M), hp.chunk_cols(N, 64)
    It, Jt = torch.from_numpy(I).cuda(), torch.from_numpy(J).cuda()
    a_rows, b_rows = _bits(A[It, :]), _bits(B[Jt, :])
    exact = ref.gemm_bf16(a_rows, b_rows)
    offs_a = torch.from_numpy(hp.sf_native_offsets(M, K)[I, :]).cuda()
    offs_b = torch.from_numpy(hp.sf_native_offsets(N, K)[J, :]).cuda()
    errs = {}
    for g in (32, 64, 128, 256):
        for name, rounding in (("RHT+SR", mx.ROUND_SR), ("RHT+RN", mx.ROUND_RN)):
            alpha = 16 / 9 if rounding != ref.ROUND_RN else 1.0
            qa = mx.mxfp4_rht_sr_quantize(A, 1, g, 5, 1, rounding, mx.SF_NATIVE)
            qb = mx.mxfp4_rht_sr_quantize(B, 1, g, 5, 2, rounding, mx.SF_NATIVE)
            C = mx.mxfp4_gemm(*qa, *qb, alpha, mx.OUT_FP32)[It][:, Jt].cpu().numpy().astype(np.float64)
            _, ca, sa = ref.rht_quantize(a_rows, g, rounding, 5, 1, row_ids=I)
            _, cb, sb = ref.rht_quantize(b_rows, g, rounding, 5, 2, row_ids=J)
            ra = hp.compare_quantised_rows(hp.unpack_codes(qa[0][It, :].cpu().numpy()), qa[1][offs_a].cpu().numpy(), ca, sa)
            rb = hp.compare_quantised_rows(hp.unpack_codes(qb[0][Jt, :].cpu().numpy()), qb[1][offs_b].cpu().numpy(), cb, sb)
            Co = ref.gemm(ca, sa, cb, sb, alpha=alpha)
            e_gpu = np.linalg.norm(C - exact) / np.linalg.norm(exact)
            e_ora = np.linalg.norm(Co - exact) / np.linalg.norm(exact)
            assert abs(e_gpu - e_ora) <= 0.02 * e_ora + 1e-4, (g, name, e_gpu, e_ora)
            assert np.linalg.norm(C - Co) <= hp.product_tolerance(ra, rb) * np.linalg.norm(Co), (g, name)
            errs[(g, name)] = e_gpu
    assert mx.mxfp4_device_status() == 0
    for g in (32, 64, 128, 256):
        assert errs[(g, "RHT+RN")] < errs[(g, "RHT+SR")]          # SR buys unbiasedness, not one-shot error
        assert 0.03 < errs[(g, "RHT+SR")] < 0.6
