"""Error ablation on one GEMM (the g x {RHT+SR, SR, RHT+RN, RN, RHT+SR16} sweep), checked against the oracle on a reduced shape."""
import numpy as np
import pytest

from paper_2502_20586_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def test_ablation_errors_match_oracle_and_have_the_expected_order(ref):
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no GPU")
    from paper_2502_20586_b200 import ablation, binding as mx

    M, N, K = 256, 192, 2048
    A, B = wl.ablation_inputs(M, N, K, outlier_rate=0.01, seed=1)
    dev = lambda bits: torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    exact = ref.gemm_bf16(A, B)                                   # fp64 product of the bf16 inputs (oracle)
    errs = {}
    for g in (32, 64, 128, 256):
        for name, use_rht, rounding in ablation.MODES:
            geff = g if use_rht else 0
            C = ablation.mxfp4_product(dev(A), dev(B), geff, rounding, 5).cpu().numpy().astype(np.float64)
            _, ca, sa = ref.rht_quantize(A, geff, rounding, 5, 1)
            _, cb, sb = ref.rht_quantize(B, geff, rounding, 5, 2)
            Co = ref.gemm(ca, sa, cb, sb, alpha=16 / 9 if rounding != ref.ROUND_RN else 1.0)
            e_gpu = np.linalg.norm(C - exact) / np.linalg.norm(exact)
            e_ora = np.linalg.norm(Co - exact) / np.linalg.norm(exact)
            assert abs(e_gpu - e_ora) <= 0.02 * e_ora + 1e-4, (g, name, e_gpu, e_ora)
            errs[(g, name)] = e_gpu
    assert mx.mxfp4_device_status() == 0
    for g in (32, 64, 128, 256):
        assert errs[(g, "RHT+RN")] < errs[(g, "RN")]              # with 1 % outliers the RHT lowers the error
        assert errs[(g, "RHT+SR")] < errs[(g, "SR")]
        assert errs[(g, "RN")] < errs[(g, "SR")]                  # SR buys unbiasedness, not one-shot error
        assert 0.03 < errs[(g, "RHT+SR")] < 0.6
        assert abs(errs[(g, "RHT+SR16")] - errs[(g, "RHT+SR")]) < 0.1 * errs[(g, "RHT+SR")]     # the two SR readings differ only in their noise
