"""Seeded synthetic inputs shaped like the paper's edge-LLM linear layers.

This module holds no arithmetic of the method: it only draws tensors.  The
same tensors are handed to the CUDA library and (by the tests and the bench)
to the CPU oracle.  The recipes stand in for the activations, weights and
output gradients of the fine-tuning runs in the paper's experiments section
(Llama-3.2-3B, BERT-base, WideResNet-16-4), of which only layer shapes and
value distributions are used:
    activations        A  ~ N(0, 1)
    weights            W  ~ N(0, 0.02^2)
    output gradients   dY ~ N(0, std_dy^2), std_dy = 1 or 1e-3
    quantizer sweep    x  ~ N(0, 1) with an independent 1 % of the entries
                           replaced by N(0, 10^2) outliers
"""
from __future__ import annotations

import torch


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def normal(shape, std: float, seed: int, dtype=torch.float32, device="cpu") -> torch.Tensor:
    """N(0, std^2) tensor drawn in fp32 from a seeded generator, then cast to dtype."""
    x = torch.randn(*shape, generator=_gen(seed, device), device=device, dtype=torch.float32)
    if std != 1.0:
        x.mul_(std)
    return x.to(dtype)


def with_outliers(shape, seed: int, dtype=torch.float32, device="cpu", frac: float = 0.01,
                  std: float = 1.0, outlier_std: float = 10.0) -> torch.Tensor:
    """N(0, std^2) with an independent Bernoulli(frac) mask of N(0, outlier_std^2) entries."""
    g = _gen(seed, device)
    x = torch.randn(*shape, generator=g, device=device, dtype=torch.float32)
    if std != 1.0:
        x.mul_(std)
    mask = torch.rand(*shape, generator=g, device=device, dtype=torch.float32) < frac
    o = torch.randn(*shape, generator=g, device=device, dtype=torch.float32)
    x = torch.where(mask, o * outlier_std, x)
    return x.to(dtype)


def layer_inputs(T: int, N: int, K: int, seed: int, dtype=torch.float32, device="cpu",
                 std_a: float = 1.0, std_w: float = 0.02, std_dy: float = 1.0):
    """A[T,K], W[N,K], dY[T,N] of one linear layer."""
    A = normal((T, K), std_a, 3 * seed + 0, dtype, device)
    W = normal((N, K), std_w, 3 * seed + 1, dtype, device)
    dY = normal((T, N), std_dy, 3 * seed + 2, dtype, device)
    return A, W, dY


# Layer shapes (K_in -> N_out) of the two model families the configurations name.
GPT2_SMALL_LAYERS = {"qkv": (768, 2304), "proj": (768, 768), "fc1": (768, 3072), "fc2": (3072, 768)}
LLAMA_1B_LAYERS = {"qkv": (2048, 2560), "o": (2048, 2048), "gate": (2048, 5632),
                   "up": (2048, 5632), "down": (5632, 2048)}
