"""A linear layer whose backward pass is Algorithm 3 (MXFP4 GEMMs with blockwise RHT and stochastic rounding).

The forward product stays in bf16 (the paper's recipe: BF16 forward, MXFP4 backward, Section 4); the backward calls
``mxfp4_linear_backward`` of the C-ABI library, so both gradients come from the library's kernels.  The layer has
no bias: the path computes dX and dW only.
"""
import torch

from . import binding as mx


class MxFp4LinearFunction(torch.autograd.Function):
    """y = x W^T;  dX = dY W and dW = dY^T X through Algorithm 3."""

    @staticmethod
    def forward(ctx, x, weight, g, seed, rounding):
        ctx.save_for_backward(x, weight)
        ctx.g, ctx.seed, ctx.rounding = g, seed, rounding
        return x @ weight.t()

    @staticmethod
    def backward(ctx, dy):
        x, weight = ctx.saved_tensors
        n = x.shape[-1]
        m = weight.shape[0]
        dy2 = dy.reshape(-1, m).contiguous()
        x2 = x.reshape(-1, n).contiguous()
        dx, dw = mx.mxfp4_linear_backward(dy2, x2, weight.contiguous(), ctx.g, ctx.seed, ctx.rounding, mx.OUT_BF16)
        return dx.view_as(x), dw, None, None, None


class MxFp4Linear(torch.nn.Module):
    """bf16 linear layer (no bias) with the MXFP4 backward.  Tokens (all leading dimensions of the input) and
    out_features must be multiples of 128 and of g, in_features a multiple of 8.  Every backward call uses a fresh
    seed (base seed + number of calls so far), so successive steps draw independent signs and rounding noise."""

    def __init__(self, in_features: int, out_features: int, g: int = 64, seed: int = 0, rounding: int = mx.ROUND_SR,
                 device="cuda"):
        super().__init__()
        self.g, self.seed, self.rounding = g, seed, rounding
        self.calls = 0
        w = torch.empty(out_features, in_features, device=device, dtype=torch.float32).normal_(0.0, 0.02)
        self.weight = torch.nn.Parameter(w.to(torch.bfloat16))

    def forward(self, x):
        seed = self.seed + self.calls
        self.calls += 1
        return MxFp4LinearFunction.apply(x, self.weight, self.g, seed, self.rounding)
