"""Seeded synthetic inputs shared by the tests, the benchmark and the smoke check.

This module only draws random tensors with the shapes and value distributions of
the paper's Llama workloads (Section 5 setup); it contains none of the method's
arithmetic.  Real activations, weights and gradients from the paper's training
runs are not available, so these stand in for them.
"""
import math

import torch

# (name, in_features K, out_features N) of one Llama block's linear layers.
LLAMA_350M = dict(tokens=16384, hidden=1024,
                  linears=[("qkv", 1024, 3072), ("o", 1024, 1024), ("gate", 1024, 2816),
                           ("up", 1024, 2816), ("down", 2816, 1024)])
LLAMA_7B = dict(tokens=16384, hidden=4096,
                linears=[("qkv", 4096, 12288), ("o", 4096, 4096), ("gate", 4096, 11008),
                         ("up", 4096, 11008), ("down", 11008, 4096)])
LONG_DW = dict(tokens=65536, K=4096, N=11008)          # long token axis weight-gradient GEMM
TINY_LINEAR = dict(tokens=256, K=512, N=512)           # single small layer


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def normal(shape, std: float, seed: int, device="cpu", dtype=torch.bfloat16) -> torch.Tensor:
    """N(0, std^2) rounded to `dtype` (round-to-nearest-even)."""
    x = torch.randn(shape, generator=_gen(seed, device), device=device, dtype=torch.float32)
    return (x * std).to(dtype)


def heavy_tailed(shape, seed: int, device="cpu", dtype=torch.bfloat16) -> torch.Tensor:
    """0.05 * Student-t(df=3), with 0.1% of the elements multiplied by 100."""
    g = _gen(seed, device)
    z = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
    chi2 = torch.zeros(shape, device=device, dtype=torch.float32)
    for _ in range(3):
        chi2 += torch.randn(shape, generator=g, device=device, dtype=torch.float32) ** 2
    t = z / torch.sqrt(chi2 / 3.0)
    del z, chi2
    outlier = torch.rand(shape, generator=g, device=device, dtype=torch.float32) < 1e-3
    t = 0.05 * t
    t = torch.where(outlier, t * 100.0, t)
    return t.to(dtype)


def linear_inputs(tokens: int, K: int, N: int, seed: int, device="cpu", grad_std: float = 1e-4):
    """X[tokens,K] ~ N(0,1), W[N,K] ~ N(0,0.02^2), dY[tokens,N] ~ N(0,grad_std^2), all bf16."""
    X = normal((tokens, K), 1.0, seed * 3 + 0, device)
    W = normal((N, K), 0.02, seed * 3 + 1, device)
    dY = normal((tokens, N), grad_std, seed * 3 + 2, device)
    return X, W, dY


def square_shape(n_elements: int):
    """Shape used for the quantizer sweep: the squarest power-of-two factorisation."""
    e = int(round(math.log2(n_elements)))
    assert 1 << e == n_elements
    return (1 << (e - e // 2), 1 << (e // 2))
