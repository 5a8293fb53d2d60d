"""A linear layer whose backward pass is Algorithm 3 (MXFP4 GEMMs with blockwise RHT and stochastic rounding).

The forward product is bf16 (the paper's main recipe: BF16 forward, MXFP4 backward, Section 4) or, with forward="fp8", the
E4M3 forward pass the paper combines it with (Section 4.1; ``mxfp4_linear_forward_fp8``); the backward calls
``mxfp4_linear_backward_ex`` of the C-ABI library, so dX, dW and the bias gradient all come from the library's kernels.
"""
import torch

from . import binding as mx


class MxFp4LinearFunction(torch.autograd.Function):
    """y = x W^T (+ b);  dX = dY W, dW = dY^T X through Algorithm 3, db = 1 dY."""

    @staticmethod
    def forward(ctx, x, weight, bias, g, seed, rounding, fp8_forward=False):
        ctx.save_for_backward(x, weight)
        ctx.g, ctx.seed, ctx.rounding, ctx.has_bias = g, seed, rounding, bias is not None
        if fp8_forward:     # Section 4.1: E4M3 forward pass (one scale per tensor), the library's own kernels
            y = mx.mxfp4_linear_forward_fp8(x.reshape(-1, x.shape[-1]).contiguous(), weight.contiguous(), mx.OUT_BF16)
            y = y.view(*x.shape[:-1], weight.shape[0])
        else:
            y = x @ weight.t()
        return y if bias is None else y + bias

    @staticmethod
    def backward(ctx, dy):
        x, weight = ctx.saved_tensors
        n = x.shape[-1]
        m = weight.shape[0]
        dy2 = dy.reshape(-1, m).contiguous()
        x2 = x.reshape(-1, n).contiguous()
        dx, dw, db = mx.mxfp4_linear_backward_ex(dy2, x2, weight.contiguous(), ctx.g, ctx.seed, ctx.rounding, mx.OUT_BF16,
                                                 with_bias=ctx.has_bias)
        return dx.view_as(x), dw, (db.to(torch.bfloat16) if ctx.has_bias else None), None, None, None, None


class MxFp4Linear(torch.nn.Module):
    """bf16 linear layer with the MXFP4 backward.  Tokens (all leading dimensions of the input) and out_features
    must be multiples of 128 and of g, in_features a multiple of 8.  Every backward call uses a fresh seed (base seed
    + number of calls so far), so successive steps draw independent signs and rounding noise."""

    def __init__(self, in_features: int, out_features: int, bias: bool = False, g: int = 64, seed: int = 0,
                 rounding: int = mx.ROUND_SR, device="cuda", forward: str = "bf16"):
        super().__init__()
        assert forward in ("bf16", "fp8")            # fp8: in_features a multiple of 128
        self.g, self.seed, self.rounding, self.fp8_forward = g, seed, rounding, forward == "fp8"
        self.calls = 0
        w = torch.empty(out_features, in_features, device=device, dtype=torch.float32).normal_(0.0, 0.02)
        self.weight = torch.nn.Parameter(w.to(torch.bfloat16))
        self.bias = torch.nn.Parameter(torch.zeros(out_features, device=device, dtype=torch.bfloat16)) if bias else None

    def forward(self, x):
        seed = self.seed + self.calls
        self.calls += 1
        return MxFp4LinearFunction.apply(x, self.weight, self.bias, self.g, seed, self.rounding, self.fp8_forward)
