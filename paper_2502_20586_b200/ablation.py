"""Ablation of the quantisation recipe on one GEMM (Table 4 / Section 3 of the paper, on synthetic operands).

    python -m paper_2502_20586_b200.ablation [--M 16384 --N 8192 --K 2048] [--json out.json]

C = A B^T with a gradient-like A [M, K] (Student-t, std 1e-4, outlier rate in {0, 0.1 %, 1 %} at x50) and a
weight-like B [N, K] (N(0, 0.02^2)), reduce K.  For g in {32, 64, 128, 256} and the modes
{RHT + SR, SR only, RHT + nearest, nearest, RHT + SR with the 16-bit dither} it reports the relative Frobenius error of the MXFP4 product against the
fp64 product of the bf16 inputs, and the throughput of quantise(A) + quantise(B) + GEMM.  Without the RHT the block
size g has no effect; those cells are repeated so the table is complete.
"""
import argparse
import json

import torch

from . import binding as mx
from . import workloads as wl


def _operands(M, N, K, rate, seed, dev):
    gen = torch.Generator(device=dev); gen.manual_seed(7919 * seed + int(rate * 1e6))
    def normal(shape):
        return torch.randn(shape, generator=gen, device=dev, dtype=torch.float32)
    chi2 = normal((M, K)).square_() + normal((M, K)).square_() + normal((M, K)).square_()
    A = normal((M, K)) / (chi2 / 3.0).sqrt_() * (1e-4 / 3.0 ** 0.5)
    if rate > 0:
        A = torch.where(torch.rand((M, K), generator=gen, device=dev) < rate, A * 50.0, A)
    B = normal((N, K)) * 0.02
    return A.to(torch.bfloat16), B.to(torch.bfloat16)


def mxfp4_product(A, B, g, rounding, seed, out=None):
    """quantise(A) quantise(B)^T through the C ABI; alpha = 16/9 with SR (Algorithm 3 lines 10-11)."""
    ca, sa = mx.mxfp4_rht_sr_quantize(A, 1, g, seed, 1, rounding, mx.SF_NATIVE)
    cb, sb = mx.mxfp4_rht_sr_quantize(B, 1, g, seed, 2, rounding, mx.SF_NATIVE)
    return mx.mxfp4_gemm(ca, sa, cb, sb, 16.0 / 9.0 if rounding != mx.ROUND_RN else 1.0, mx.OUT_FP32, C_out=out)


MODES = (("RHT+SR", True, mx.ROUND_SR), ("SR", False, mx.ROUND_SR), ("RHT+RN", True, mx.ROUND_RN), ("RN", False, mx.ROUND_RN),
         ("RHT+SR16", True, mx.ROUND_SR16))          # the last: the 16-bit-dither reading of SR (hardware convert)


def run(M, N, K, rates=(0.0, 1e-3, 1e-2), gs=(32, 64, 128, 256), seed=0, iters=5):
    dev = torch.device("cuda", 0)
    rows = []
    for rate in rates:
        A, B = _operands(M, N, K, rate, seed, dev)
        ref = A.double() @ B.double().t()
        ref_norm = ref.norm().item()
        out = torch.empty((M, N), dtype=torch.float32, device=dev)
        for g in gs:
            for name, use_rht, rounding in MODES:
                geff = g if use_rht else 0
                C = mxfp4_product(A, B, geff, rounding, seed, out)
                err = (C.double() - ref).norm().item() / ref_norm
                torch.cuda.synchronize()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                for _ in range(iters):
                    mxfp4_product(A, B, geff, rounding, seed, out)
                b.record(); torch.cuda.synchronize()
                ms = a.elapsed_time(b) / iters
                rows.append({"outlier_rate": rate, "g": g, "mode": name, "rel_error": err, "ms": ms,
                             "tflops_incl_quantize": 2.0 * M * N * K / ms / 1e9})
        del ref
    if mx.mxfp4_device_status() != 0:
        raise RuntimeError("device-side wait timed out")
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--M", type=int, default=16384)
    ap.add_argument("--N", type=int, default=8192)
    ap.add_argument("--K", type=int, default=2048)
    ap.add_argument("--json", default=None)
    args = ap.parse_args()
    rows = run(args.M, args.N, args.K)
    print(f"# C = A B^T, M={args.M} N={args.N} K={args.K}; relative Frobenius error vs fp64 product of the bf16 inputs")
    print("| outlier rate | g | " + " | ".join(m[0] for m in MODES) + " | TFLOP/s incl. quantise (RHT+SR) | (RHT+SR16) | (RN, no RHT) |")
    print("|---|---|" + "---|" * (len(MODES) + 3))
    for rate in sorted({r["outlier_rate"] for r in rows}):
        for g in sorted({r["g"] for r in rows}):
            cell = {r["mode"]: r for r in rows if r["outlier_rate"] == rate and r["g"] == g}
            print(f"| {rate:g} | {g} | " + " | ".join(f"{cell[m[0]]['rel_error']:.4f}" for m in MODES) +
                  f" | {cell['RHT+SR']['tflops_incl_quantize']:.0f} | {cell['RHT+SR16']['tflops_incl_quantize']:.0f} | {cell['RN']['tflops_incl_quantize']:.0f} |")
    if args.json:
        with open(args.json, "w") as fh:
            json.dump(rows, fh, indent=1)


if __name__ == "__main__":
    main()
