"""Seeded synthetic attention inputs (no arithmetic of the method lives here).

The five workloads stand in for the paper's captured activations (one causal
4096-token sequence per layer, BF16, head dimension 64, scale 1/8; Appendix
"Accuracy and Cost", "Captured inputs"), which are not available.  Keys (and, for
workload 4, queries) carry a common per-head offset, the structure the paper's
offset sweep uses (k_j = z_j + b, Appendix "Gauge Projection: Proofs", "Synthetic
offset sweep").

Recipe: a CPU ``torch.Generator`` seeded with ``BASE_SEED + 1000*workload``; FP32
Q, K, V, dO ~ N(0,1) drawn in that order with shape [B,H,N,d]; then one offset
direction per (b,h) (a single one for workload 1) ~ N(0,I_d), scaled to the
stated L2 norm, added in FP32; one rounding to BF16.  softmax_scale is the FP32
value of 1/sqrt(d).  The same arrays feed the oracle and the GPU.
"""
import math
from dataclasses import dataclass, replace

import numpy as np
import torch

BASE_SEED = 260934272


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    N: int
    d: int
    causal: bool
    k_offset: float = 0.0
    q_offset: float = 0.0
    shared_offset: bool = False   # one offset vector for every head (workload 1)
    seed: int = BASE_SEED
    Hkv: int = 0                  # key / value heads; 0 = same as H (no grouped queries)

    @property
    def kv_heads(self) -> int:
        return self.Hkv if self.Hkv else self.H

    @property
    def softmax_scale(self) -> float:
        return float(np.float32(1.0 / math.sqrt(self.d)))

    @property
    def elements(self) -> int:
        return self.B * self.H * self.N * self.d

    def gemm_unit_flops(self) -> float:
        """FLOPs of one N x N x d contraction over the whole problem (x0.5 if causal)."""
        return 2.0 * self.B * self.H * self.N * self.N * self.d * (0.5 if self.causal else 1.0)


WORKLOADS = {
    1: Workload("cfg1_tiny_causal_d64", 1, 2, 256, 64, True, k_offset=8.0, shared_offset=True, seed=BASE_SEED + 1000),
    2: Workload("cfg2_causal_h16_n4096_d64", 1, 16, 4096, 64, True, k_offset=16.0, seed=BASE_SEED + 2000),
    3: Workload("cfg3_causal_h8_n4096_d128", 1, 8, 4096, 128, True, k_offset=16.0, seed=BASE_SEED + 3000),
    4: Workload("cfg4_noncausal_b4_h32_n8192_d128", 4, 32, 8192, 128, False, k_offset=16.0, q_offset=16.0,
                seed=BASE_SEED + 4000),
    5: Workload("cfg5_causal_h8_n32768_d128", 1, 8, 32768, 128, True, k_offset=32.0, seed=BASE_SEED + 5000),
    # Not one of the five benchmark configurations: the paper's own layout (16 query / 4 KV heads, d = 64, 4096 tokens,
    # batch one; Appendix "Accuracy and Cost", "Captured inputs"), used by the grouped-query tests.
    6: Workload("gqa_causal_h16_kv4_n4096_d64", 1, 16, 4096, 64, True, k_offset=16.0, seed=BASE_SEED + 6000, Hkv=4),
}
CFG3_OFFSET_NORMS = (0.0, 4.0, 16.0, 64.0)


def workload(cfg: int, **overrides) -> Workload:
    w = WORKLOADS[cfg]
    return replace(w, **overrides) if overrides else w


def _offset(gen, B, H, d, norm, shared):
    n = 1 if shared else B * H
    c = torch.randn(n, d, generator=gen, dtype=torch.float32)
    c = c / c.norm(dim=1, keepdim=True) * norm
    if shared:
        c = c.expand(B * H, d)
    return c.reshape(B, H, 1, d)


def make_inputs(w: Workload):
    """Returns dict of CPU torch.bfloat16 tensors Q, dO [B,H,N,d] and K, V [B,Hkv,N,d] (Hkv = H unless grouped)."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(w.seed)
    shape = (w.B, w.H, w.N, w.d)
    kv_shape = (w.B, w.kv_heads, w.N, w.d)
    Q = torch.randn(shape, generator=gen, dtype=torch.float32)
    K = torch.randn(kv_shape, generator=gen, dtype=torch.float32)
    V = torch.randn(kv_shape, generator=gen, dtype=torch.float32)
    dO = torch.randn(shape, generator=gen, dtype=torch.float32)
    # Offset directions are always drawn (even for norm 0) so that variants share the base draw.
    ck = _offset(gen, w.B, w.kv_heads, w.d, w.k_offset, w.shared_offset)
    cq = _offset(gen, w.B, w.H, w.d, w.q_offset, w.shared_offset)
    K = K + ck
    Q = Q + cq
    return {name: t.to(torch.bfloat16).contiguous() for name, t in (("Q", Q), ("K", K), ("V", V), ("dO", dO))}


def bits(t: torch.Tensor) -> np.ndarray:
    """BF16 tensor (CPU) -> numpy uint16 bit patterns, same shape, no copy."""
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def from_bits(x: np.ndarray) -> torch.Tensor:
    """numpy uint16 bit patterns -> CPU torch.bfloat16 tensor."""
    return torch.from_numpy(np.ascontiguousarray(x).view(np.int16)).view(torch.bfloat16)


def sample_rows(w: Workload, count: int, salt: int = 0) -> np.ndarray:
    """Seeded query/key row sample that always contains the tile-boundary rows 0, 127, 128, N-1."""
    rng = np.random.default_rng(w.seed + 7919 * (salt + 1))
    fixed = [r for r in (0, 127, 128, w.N - 1) if r < w.N]
    rest = rng.choice(w.N, size=max(0, count - len(fixed)), replace=False).tolist()
    return np.array(sorted(set(fixed + rest)), dtype=np.int32)
