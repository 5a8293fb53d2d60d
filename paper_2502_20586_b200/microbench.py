"""Time one kernel of the library on one shape (CUDA events), for tuning and for small ncu captures.

    python -m paper_2502_20586_b200.microbench gemm  M N K            [--iters 20] [--out fp32]
    python -m paper_2502_20586_b200.microbench quant ROWS COLS REDUCE_DIM G [--rounding 0] [--iters 20]
    python -m paper_2502_20586_b200.microbench backward B N M G       [--iters 20] [--bias] [--accumulate --out fp32]
    python -m paper_2502_20586_b200.microbench forward B N M          [--iters 20]      (E4M3 forward pass)

Operands are random codes/scales (gemm) or N(0,1) bf16 (quant, backward).  Between timed launches a buffer
larger than L2 is rewritten so every launch starts with a cold L2.  Prints one JSON line.
"""
import argparse
import json
import sys

import torch

from . import binding as mx


def _flush_l2(buf):
    buf.add_(1)


def _time(fn, iters, flush_buf):
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    times = []
    for _ in range(iters):
        if flush_buf is not None:
            _flush_l2(flush_buf)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda._sleep(400000)        # keep the GPU busy while the host enqueues, so host latency is not timed
        a.record(); fn(); b.record()
        torch.cuda.synchronize()
        times.append(a.elapsed_time(b))
    times.sort()
    return times[len(times) // 2], times[0]


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("kind", choices=["gemm", "quant", "backward", "forward"])
    ap.add_argument("dims", type=int, nargs="+")
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--rounding", type=int, default=0)
    ap.add_argument("--out", default="bf16")
    ap.add_argument("--no-flush", action="store_true")
    ap.add_argument("--bias", action="store_true", help="backward: also the bias gradient (extended entry point)")
    ap.add_argument("--accumulate", action="store_true", help="backward: accumulate into fp32 dW / db")
    ap.add_argument("--fused", action="store_true", help="backward: the fused-producer variant (dY quantised inside the GEMM kernels)")
    args = ap.parse_args(argv)
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    gen = torch.Generator(device=dev); gen.manual_seed(0)
    flush = None if args.no_flush else torch.zeros(192 * 1024 * 1024, dtype=torch.uint8, device=dev)
    out_dtype = mx.OUT_FP32 if args.out == "fp32" else mx.OUT_BF16
    res = {"kind": args.kind, "dims": args.dims}
    if args.kind == "gemm":
        M, N, K = args.dims
        A = torch.randint(0, 256, (M, K // 2), generator=gen, device=dev, dtype=torch.uint8)
        B = torch.randint(0, 256, (N, K // 2), generator=gen, device=dev, dtype=torch.uint8)
        SA = torch.randint(120, 134, (mx.mxfp4_scale_bytes(M, K),), generator=gen, device=dev, dtype=torch.uint8)
        SB = torch.randint(120, 134, (mx.mxfp4_scale_bytes(N, K),), generator=gen, device=dev, dtype=torch.uint8)
        C = torch.empty((M, N), dtype=torch.float32 if out_dtype == mx.OUT_FP32 else torch.bfloat16, device=dev)
        med, best = _time(lambda: mx.mxfp4_gemm(A, SA, B, SB, 1.0, out_dtype, C_out=C), args.iters, flush)
        fl = 2.0 * M * N * K
        res.update(ms=med, ms_best=best, tflops=fl / med / 1e9, tflops_best=fl / best / 1e9)
    elif args.kind == "quant":
        rows, cols, rd, g = args.dims
        x = torch.randn((rows, cols), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
        R, K = (rows, cols) if rd == 1 else (cols, rows)
        codes = torch.empty((R, K // 2), dtype=torch.uint8, device=dev)
        scales = torch.empty(mx.mxfp4_scale_bytes(R, K), dtype=torch.uint8, device=dev)
        med, best = _time(lambda: mx.mxfp4_rht_sr_quantize(x, rd, g, 0, 1, args.rounding, mx.SF_NATIVE, codes=codes, scales=scales),
                          args.iters, flush)
        by = rows * cols * (2.0 + 0.5 + 1.0 / 32.0)
        res.update(ms=med, ms_best=best, gbs=by / med / 1e6, gbs_best=by / best / 1e6)
    elif args.kind == "forward":
        b, n, m = args.dims
        x = torch.randn((b, n), generator=gen, device=dev).to(torch.bfloat16)
        W = (torch.randn((m, n), generator=gen, device=dev) * 0.02).to(torch.bfloat16)
        y = torch.empty((b, m), dtype=torch.float32 if out_dtype == mx.OUT_FP32 else torch.bfloat16, device=dev)
        ws = torch.empty(int(mx.lib().mxfp4_linear_forward_fp8_workspace(b, n, m)), dtype=torch.uint8, device=dev)
        med, best = _time(lambda: mx.mxfp4_linear_forward_fp8(x, W, out_dtype, y=y, workspace=ws), args.iters, flush)
        fl = 2.0 * b * m * n
        res.update(ms=med, ms_best=best, tflops=fl / med / 1e9, tflops_best=fl / best / 1e9)
    else:
        b, n, m, g = args.dims
        dY = torch.randn((b, m), generator=gen, device=dev).to(torch.bfloat16)
        X = torch.randn((b, n), generator=gen, device=dev).to(torch.bfloat16)
        W = torch.randn((m, n), generator=gen, device=dev).to(torch.bfloat16)
        dt = torch.float32 if out_dtype == mx.OUT_FP32 else torch.bfloat16
        dX = torch.empty((b, n), dtype=dt, device=dev)
        dW = torch.zeros((m, n), dtype=dt, device=dev)
        if args.bias or args.accumulate:
            db = torch.zeros((m,), dtype=torch.float32, device=dev) if args.bias else None
            ws = torch.empty(mx.mxfp4_linear_backward_ex_workspace(b, m, n, args.bias), dtype=torch.uint8, device=dev)
            fn = lambda: mx.mxfp4_linear_backward_ex(dY, X, W, g, 0, args.rounding, out_dtype, dX=dX, dW=dW, db=db,
                                                     accumulate=args.accumulate, workspace=ws)
        elif args.fused:
            ws = torch.empty(mx.mxfp4_linear_backward_workspace(b, m, n), dtype=torch.uint8, device=dev)
            fn = lambda: mx.mxfp4_linear_backward_fused(dY, X, W, g, 0, args.rounding, out_dtype, dX=dX, dW=dW, workspace=ws)
        else:
            ws = torch.empty(mx.mxfp4_linear_backward_workspace(b, m, n), dtype=torch.uint8, device=dev)
            fn = lambda: mx.mxfp4_linear_backward(dY, X, W, g, 0, args.rounding, out_dtype, dX=dX, dW=dW, workspace=ws)
        med, best = _time(fn, args.iters, flush)
        fl = 4.0 * b * m * n
        res.update(ms=med, ms_best=best, tflops=fl / med / 1e9, tflops_best=fl / best / 1e9)
    status = mx.mxfp4_device_status()
    res["device_status"] = status
    print(json.dumps(res))
    return 0 if status == 0 else 1


if __name__ == "__main__":
    sys.exit(main())
