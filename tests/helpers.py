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


def load_values(name):
    """Parse a tests/golden text fixture: one 'key value ...' entry per line, '#' starts a comment."""
    import os
    vals = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", name)) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if line:
                key, *rest = line.split()
                vals[key] = np.array([float(x) for x in rest])
    return vals


def witness128_arrays():
    """The four-key witness laid out as the 128 x 128, d = 64 non-causal problem that
    tests/golden/witness128_key_pass.txt describes (FP64 arrays of BF16-exact values)."""
    gold = load_values("witness_minus24.txt")
    N, d = 128, 64
    Q = np.zeros((N, d)); K = np.zeros((N, d)); V = np.zeros((N, d)); U = np.zeros((N, d))
    Q[:, 2] = 256.0
    Q[:121, 3] = 253.0
    K[4:, 2] = -256.0
    for j in range(4):
        K[j, :2] = gold[f"k{j + 1}"]
        V[j, :2] = gold[f"v{j + 1}"]
    U[:, :2] = gold["u"]
    return Q, K, V, U
