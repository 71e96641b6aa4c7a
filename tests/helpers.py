"""Shared test helpers: small input builders (no arithmetic of the method)."""
import numpy as np
import torch

from paper_2609_34272_b200.workloads import bits


def randn_bf16(shape, seed, scale=1.0, offset=None):
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    x = torch.randn(shape, generator=g, dtype=torch.float32) * scale
    if offset is not None:
        x = x + offset
    return x.to(torch.bfloat16)


def grid_bf16(shape, seed, step=0.125, span=16):
    """Values on a coarse grid k*step, |k|<=span: sums with small integers stay exactly BF16."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    k = torch.randint(-span, span + 1, shape, generator=g)
    return (k.to(torch.float32) * step).to(torch.bfloat16)


def as_bits(t):
    return bits(t)


def f64(t):
    return t.to(torch.float64)


def np64(t):
    return t.to(torch.float64).numpy()
