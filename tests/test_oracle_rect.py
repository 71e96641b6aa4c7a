"""Pins of the rectangular (N_q != N_k) FP64 oracle against things other than itself (CPU only)."""
import math

import numpy as np
import pytest
import torch

import oracle
from helpers import as_bits, randn_bf16


def _torch_reference(Q, K, V, dO, alpha, causal):
    """Library routine: torch float64 masked softmax and autograd; rows without support are set to zero output."""
    q, k, v = (t.to(torch.float64).clone().requires_grad_(True) for t in (Q, K, V))
    G = Q.shape[1] // K.shape[1]
    kk, vv = k.repeat_interleave(G, dim=1), v.repeat_interleave(G, dim=1)
    Nq, Nk = Q.shape[2], K.shape[2]
    s = alpha * q @ kk.transpose(-1, -2)
    keep = torch.ones(Nq, Nk, dtype=torch.bool)
    if causal:
        i = torch.arange(Nq)[:, None]; j = torch.arange(Nk)[None, :]
        keep = j <= i + (Nk - Nq)
    live = keep.any(dim=1)                                   # rows with a non-empty support
    s = s.masked_fill(~keep, float("-inf"))
    p = torch.zeros_like(s)
    p[..., live, :] = torch.softmax(s[..., live, :], dim=-1)
    o = p @ vv
    lse = torch.full(s.shape[:-1], float("inf"), dtype=torch.float64)
    lse[..., live] = torch.logsumexp(s[..., live, :], dim=-1).detach()
    (o * dO.to(torch.float64)).sum().backward()
    return o.detach().numpy(), lse.numpy(), q.grad.numpy(), k.grad.numpy(), v.grad.numpy(), live.numpy()


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("Nq,Nk", [(5, 9), (9, 5), (1, 7), (7, 1), (40, 130), (130, 40), (33, 33)])
def test_rect_matches_torch_float64_autograd(Nq, Nk, causal):
    # Appendix "Synthetic Numerical Suite" lists unequal lengths and empty causal rows; the definition is Eq. "row-attention"
    # / Eq. "row-gradients" with the support restricted as stated in the oracle's header.
    d, H, Hkv = 8, 4, 2
    Q, dO = randn_bf16((2, H, Nq, d), 11), randn_bf16((2, H, Nq, d), 12)
    K, V = randn_bf16((2, Hkv, Nk, d), 13), randn_bf16((2, Hkv, Nk, d), 14)
    alpha = float(np.float32(1 / math.sqrt(d)))
    got = oracle.attn_rect_f64(as_bits(Q), as_bits(K), as_bits(V), as_bits(dO), alpha, causal)
    o, lse, dq, dk, dv, live = _torch_reference(Q, K, V, dO, alpha, causal)
    for name, ref in (("O", o), ("dQ", dq), ("dK", dk), ("dV", dv)):
        err = np.abs(got[name] - ref).max()
        assert err <= 1e-12 * max(1.0, np.abs(ref).max()), (name, err)
    assert np.abs(got["LSE"][..., live] - lse[..., live]).max() <= 1e-12 * max(1.0, np.abs(lse[..., live]).max())
    assert np.all(np.isposinf(got["LSE"][..., ~live]))


def test_rect_with_equal_lengths_is_the_square_oracle():
    # N_q = N_k: the support is j <= i, the very loops of the square functions, so the results agree bit for bit
    Q, K, V, dO = (randn_bf16((1, 2, 45, 16), 20 + i) for i in range(4))
    for causal in (True, False):
        a = oracle.attn_rect_f64(as_bits(Q), as_bits(K), as_bits(V), as_bits(dO), 0.25, causal)
        b = oracle.attn_fwd_bwd_f64(as_bits(Q), as_bits(K), as_bits(V), as_bits(dO), 0.25, causal)
        for n in ("O", "LSE", "MUA", "dQ", "dK", "dV"):
            assert np.array_equal(a[n], b[n]), n


def test_empty_rows_and_single_key_rows_closed_form():
    # N_q = 6 queries, N_k = 2 keys, causal: rows 0..3 see nothing (O = 0, dQ = 0, LSE = +inf, no key / value gradient from
    # them), row 4 sees key 0 only (O = v_0, LSE = alpha q.k_0, dQ = 0), row 5 sees both keys.
    d = 4
    Q, dO = randn_bf16((1, 1, 6, d), 31), randn_bf16((1, 1, 6, d), 32)
    K, V = randn_bf16((1, 1, 2, d), 33), randn_bf16((1, 1, 2, d), 34)
    r = oracle.attn_rect_f64(as_bits(Q), as_bits(K), as_bits(V), as_bits(dO), 0.5, True)
    q, k, v, u = (t[0, 0].to(torch.float64).numpy() for t in (Q, K, V, dO))
    assert np.all(r["O"][0, 0, :4] == 0) and np.all(r["dQ"][0, 0, :4] == 0) and np.all(np.isposinf(r["LSE"][0, 0, :4]))
    assert np.allclose(r["O"][0, 0, 4], v[0], rtol=0, atol=1e-15) and np.all(r["dQ"][0, 0, 4] == 0)
    assert abs(r["LSE"][0, 0, 4] - 0.5 * q[4] @ k[0]) <= 1e-14
    # value gradient of key 1: only row 5 sees it, with its two-key softmax weight
    s5 = 0.5 * (k @ q[5]); p5 = np.exp(s5 - s5.max()); p5 /= p5.sum()
    assert np.allclose(r["dV"][0, 0, 1], p5[1] * u[5], rtol=1e-13, atol=1e-15)
    assert np.allclose(r["dV"][0, 0, 0], u[4] + p5[0] * u[5], rtol=1e-13, atol=1e-15)
