"""Parity at full sizes (GPT 345M / 1.3B / 6.7B layer shapes with their g), in the launch configuration bench.py times.

The oracle cannot run whole 16384 x 16384 operands in seconds, so outputs are SAMPLED: every dX / dW entry depends
on one row of each quantised operand, and the oracle quantises exactly those rows (their SR draws are keyed on the
row index in the full operand).  Checked per layer:
  - codes and scales of the sampled operand rows against the oracle (<= 1e-4 mismatches, one grid step),
  - the GPU GEMM on its own codes against the fp64 product of those codes (<= 1e-5, fp32 output),
  - mxfp4_linear_backward's bf16 outputs at the sampled entries against the oracle's Algorithm 3.
"""
import numpy as np
import pytest

from paper_2502_20586_b200 import workloads as wl
from tests import helpers as hp

pytestmark = pytest.mark.gpu


def _bits(t):
    import torch
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


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
    rng = np.random.default_rng(17)
    I = np.sort(rng.choice(b, 12, replace=False)); J = np.sort(rng.choice(n, 10, replace=False))       # dX[I, J]
    P = np.sort(rng.choice(m, 12, replace=False)); Q = np.sort(rng.choice(n, 10, replace=False))       # dW[P, Q]
    It, Jt, Pt, Qt = (torch.from_numpy(a).cuda() for a in (I, J, P, Q))

    # operand views of Algorithm 3: (tensor, reduce_dim, tag, sampled output rows, host slice with those rows as rows)
    views = {
        1: (dY, 1, I, _bits(dY[It, :])),              # Q1 rows I      = dY[I, :]        K = m
        2: (W, 0, J, _bits(W[:, Jt].t())),            # Q2 rows J      = W[:, J]^T       K = m
        3: (dY, 0, P, _bits(dY[:, Pt].t())),          # Q3 rows P      = dY[:, P]^T      K = b
        4: (X, 0, Q, _bits(X[:, Qt].t())),            # Q4 rows Q      = X[:, Q]^T       K = b
    }
    gpu_q, ora_q = {}, {}
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
        same = (s == os_).repeat(32, axis=1)
        assert (s != os_).mean() <= 1e-4
        diff = (c != oc) & same
        assert diff.mean() <= 1e-4, (tag, diff.mean())
        assert np.all(np.abs(hp.E2M1_STEP_INDEX[c[diff]] - hp.E2M1_STEP_INDEX[oc[diff]]) <= 1)
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
    del Cx, Cw

    # the one-call path, bf16 outputs as in the benchmark, against the oracle's own Algorithm 3 on the sampled rows
    dX, dW = mx.mxfp4_linear_backward(dY, X, W, g, seed, rounding, mx.OUT_BF16)
    assert mx.mxfp4_device_status() == 0
    ox = ref.gemm(*ora_q[1], *ora_q[2], alpha=alpha); ow = ref.gemm(*ora_q[3], *ora_q[4], alpha=alpha)
    bx = dX[It][:, Jt].float().cpu().numpy().astype(np.float64); bw = dW[Pt][:, Qt].float().cpu().numpy().astype(np.float64)
    assert np.linalg.norm(bx - ox) <= 2e-2 * np.linalg.norm(ox)       # bf16 rounding + <= 1e-4 differing codes
    assert np.linalg.norm(bw - ow) <= 2e-2 * np.linalg.norm(ow)
    # and it is a sane estimate of the true gradient entries (fp64 product of the bf16 inputs)
    tx = wl.bf16_bits_to_f64(views[1][3]) @ wl.bf16_bits_to_f64(views[2][3]).T
    assert np.linalg.norm(bx - tx) < 0.6 * np.linalg.norm(tx)
