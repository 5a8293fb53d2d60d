"""Seeded synthetic inputs and layer shapes for the MXFP4 backward path.

This module holds none of the method's arithmetic: it only draws tensors with
the value distributions the paper describes for LLM training (activation and
weight outliers, heavy-tailed sparse gradients; Section 3.2) in the shapes of
its GPT 345M / 1.3B / 6.7B models (appendix hyper-parameter table), rounds
them to bf16 and hands the same bits to the CUDA library and to the test
oracle.  It imports numpy only.
"""
from dataclasses import dataclass

import numpy as np


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32/fp64 values to bf16 (nearest, ties to even); returns uint16 bit patterns."""
    f = np.ascontiguousarray(a, np.float32)
    u = f.view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


@dataclass(frozen=True)
class Linear:
    """One linear layer y = x W^T with x [b, n], W [m, n], dY [b, m]."""
    name: str
    b: int   # tokens
    n: int   # in features
    m: int   # out features

    @property
    def flops(self) -> int:
        """dgrad 2bmn + wgrad 2bmn."""
        return 4 * self.b * self.m * self.n


def gpt_layers(hidden: int, ffn: int, tokens: int):
    return [
        Linear("qkv", tokens, hidden, 3 * hidden),
        Linear("attn_out", tokens, hidden, hidden),
        Linear("fc1", tokens, hidden, ffn),
        Linear("fc2", tokens, ffn, hidden),
    ]


# config id -> (layers, RHT block size g)
CONFIGS = {
    "single_256x512": ([Linear("single", 256, 512, 512)], 64),
    "gpt_345m": (gpt_layers(1024, 4096, 8 * 1024), 64),
    "gpt_1p3b": (gpt_layers(2048, 8192, 8 * 2048), 128),
    "gpt_6p7b": (gpt_layers(4096, 16384, 8 * 2048), 128),
}
CONFIG_IDS = {name: i for i, name in enumerate(CONFIGS)}


def _rng(seed: int, *path: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, *path])))


def grad_like(rng, shape, std: float, outlier_rate: float = 0.0, outlier_gain: float = 50.0):
    """Student-t (nu = 3) scaled to the given std, with i.i.d. Bernoulli entries multiplied by a gain."""
    a = rng.standard_t(3.0, size=shape) * (std / np.sqrt(3.0))
    if outlier_rate > 0.0:
        mask = rng.random(size=shape) < outlier_rate
        a = np.where(mask, a * outlier_gain, a)
    return to_bf16_bits(a)


def activation_like(rng, shape, n_outlier_channels: int = 0, gain: float = 20.0):
    """N(0, 1) with a seeded choice of feature columns multiplied by a gain."""
    a = rng.standard_normal(size=shape)
    if n_outlier_channels > 0:
        cols = rng.choice(shape[1], size=n_outlier_channels, replace=False)
        a[:, cols] *= gain
    return to_bf16_bits(a)


def weight_like(rng, shape, std: float = 0.02):
    return to_bf16_bits(rng.standard_normal(size=shape) * std)


def small_integer_like(rng, shape, lo: int = -8, hi: int = 8):
    """Small integers: every +-sum of up to 256 of them is exact in fp32 in any order."""
    return to_bf16_bits(rng.integers(lo, hi + 1, size=shape).astype(np.float32))


def layer_inputs(config: str, layer: Linear, seed: int = 0):
    """(dY [b, m], X [b, n], W [m, n]) as bf16 bit patterns for one layer of a named config."""
    cid = CONFIG_IDS[config]
    lid = [l.name for l in CONFIGS[config][0]].index(layer.name)
    r = [_rng(seed, cid, lid, k) for k in range(3)]
    if config == "single_256x512":
        dY = grad_like(r[0], (layer.b, layer.m), 1e-3, outlier_rate=1e-3, outlier_gain=50.0)
        X = activation_like(r[1], (layer.b, layer.n))
    else:
        dY = grad_like(r[0], (layer.b, layer.m), 1e-4)
        X = activation_like(r[1], (layer.b, layer.n), n_outlier_channels=8, gain=20.0)
    W = weight_like(r[2], (layer.m, layer.n))
    return dY, X, W


def layer_inputs_device(config: str, layer: Linear, seed: int = 0, device="cuda"):
    """Same distributions as layer_inputs, drawn on the GPU with torch's seeded generator (the full-size
    tensors have up to 2.7e8 entries; numpy would take minutes).  Returns bf16 torch tensors (dY, X, W)."""
    import torch
    cid = CONFIG_IDS[config]
    lid = [l.name for l in CONFIGS[config][0]].index(layer.name)
    gen = torch.Generator(device=device)
    gen.manual_seed(1_000_003 * seed + 1009 * cid + lid)

    def normal(shape):
        return torch.randn(shape, generator=gen, device=device, dtype=torch.float32)

    def student_t3(shape):
        chi2 = normal(shape).square_()
        chi2 += normal(shape).square_()
        chi2 += normal(shape).square_()
        return normal(shape).div_(chi2.div_(3.0).sqrt_())

    std = 1e-3 if config == "single_256x512" else 1e-4
    dY = student_t3((layer.b, layer.m)).mul_(std / 3.0 ** 0.5)
    if config == "single_256x512":
        mask = torch.rand((layer.b, layer.m), generator=gen, device=device) < 1e-3
        dY = torch.where(mask, dY * 50.0, dY)
    X = normal((layer.b, layer.n))
    if config != "single_256x512":
        cols = torch.randperm(layer.n, generator=gen, device=device)[:8]
        X[:, cols] *= 20.0
    W = normal((layer.m, layer.n)).mul_(0.02)
    return dY.to(torch.bfloat16), X.to(torch.bfloat16), W.to(torch.bfloat16)


def ablation_inputs(M: int, N: int, K: int, outlier_rate: float, seed: int = 0):
    """One GEMM C = A B^T with a gradient-like A [M, K] and a weight-like B [N, K]."""
    ra, rb = _rng(seed, 100, 0), _rng(seed, 100, 1)
    A = grad_like(ra, (M, K), 1e-4, outlier_rate=outlier_rate, outlier_gain=50.0)
    B = weight_like(rb, (N, K))
    return A, B
