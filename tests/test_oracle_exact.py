"""Pins of the exact FP64 oracle against things other than itself (CPU only).

Each test names the passage that fixes the expected value.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from helpers import as_bits, grid_bf16, np64, randn_bf16


def _run(Q, K, V, dO, alpha, causal):
    return oracle.attn_fwd_bwd_f64(as_bits(Q), as_bits(K), as_bits(V), as_bits(dO), alpha, causal)


def _torch_reference(Q, K, V, dO, alpha, causal):
    """Library routine: torch float64 softmax / logsumexp / autograd."""
    q, k, v = (t.to(torch.float64).clone().requires_grad_(True) for t in (Q, K, V))
    s = alpha * q @ k.transpose(-1, -2)
    if causal:
        N = s.shape[-1]
        s = s.masked_fill(~torch.tril(torch.ones(N, N, dtype=torch.bool)), float("-inf"))
    o = torch.softmax(s, dim=-1) @ v
    lse = torch.logsumexp(s, dim=-1)
    (o * dO.to(torch.float64)).sum().backward()
    return o.detach().numpy(), lse.detach().numpy(), q.grad.numpy(), k.grad.numpy(), v.grad.numpy()


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("N,d", [(1, 4), (5, 3), (37, 16), (130, 8)])
def test_matches_torch_float64_autograd(N, d, causal):
    # Appendix "Synthetic Numerical Suite", "References": small cases agree with autograd to ~1e-15.
    shape = (2, 3, N, d)
    Q, K, V, dO = (randn_bf16(shape, 100 + i) for i in range(4))
    alpha = float(np.float32(1 / math.sqrt(d)))
    got = _run(Q, K, V, dO, alpha, causal)
    o, lse, dq, dk, dv = _torch_reference(Q, K, V, dO, alpha, causal)
    for name, ref in (("O", o), ("LSE", lse), ("dQ", dq), ("dK", dk), ("dV", dv)):
        err = np.abs(got[name] - ref).max()
        assert err <= 1e-12 * max(1.0, np.abs(ref).max()), (name, err)


@pytest.mark.parametrize("causal", [True, False])
def test_central_finite_differences(causal):
    # Eq. "row-gradients": dQ, dK, dV are the derivatives of L = sum(O * dO).
    # Inputs sit on a 1/8 grid below 2 so that +-2^-7 perturbations stay exactly BF16.
    N, d, h = 6, 3, 2.0 ** -7
    shape = (1, 1, N, d)
    Q, K, V, dO = (grid_bf16(shape, 7 + i, step=0.125, span=15) for i in range(4))
    alpha = 0.5
    base = _run(Q, K, V, dO, alpha, causal)
    U = np64(dO)

    def loss(Qx, Kx, Vx):
        return float((_run(Qx, Kx, Vx, dO, alpha, causal)["O"] * U).sum())

    for which, grad in (("Q", base["dQ"]), ("K", base["dK"]), ("V", base["dV"])):
        for i in range(N):
            for c in range(d):
                tens = {"Q": Q, "K": K, "V": V}
                plus = {k: v.clone() for k, v in tens.items()}
                minus = {k: v.clone() for k, v in tens.items()}
                plus[which][0, 0, i, c] += h
                minus[which][0, 0, i, c] -= h
                assert float(plus[which][0, 0, i, c]) - float(minus[which][0, 0, i, c]) == 2 * h
                fd = (loss(plus["Q"], plus["K"], plus["V"]) - loss(minus["Q"], minus["K"], minus["V"])) / (2 * h)
                assert abs(fd - grad[0, 0, i, c]) <= 2e-4 * max(1.0, np.abs(grad).max()), (which, i, c)


@pytest.mark.parametrize("causal", [True, False])
def test_second_formulation_covariance_and_jacobian(causal):
    # Proposition "Exact translation structure": G_Q = alpha sum_j p_j (k_j - mu_k)(a_j - mu_a);
    # explicit softmax Jacobian dS = (diag(p) - p p^T) a.  Two references agree within 1e-10 + 1e-9 ||G||
    # (Appendix "Synthetic Numerical Suite", "References").
    N, d = 48, 8
    shape = (1, 2, N, d)
    Q, K, V, dO = (randn_bf16(shape, 40 + i, offset=(3.0 if i == 1 else None)) for i in range(4))
    alpha = float(np.float32(1 / math.sqrt(d)))
    got = _run(Q, K, V, dO, alpha, causal)
    q, k, v, u = (np64(t) for t in (Q, K, V, dO))
    dQ = np.zeros_like(q); dK = np.zeros_like(k); dV = np.zeros_like(v)
    for h in range(2):
        for i in range(N):
            L = i + 1 if causal else N
            s = alpha * k[0, h, :L] @ q[0, h, i]
            p = np.exp(s - s.max()); p /= p.sum()
            a = v[0, h, :L] @ u[0, h, i]
            mu_k = p @ k[0, h, :L]; mu_a = p @ a
            dQ[0, h, i] = alpha * ((p * (a - mu_a)) @ (k[0, h, :L] - mu_k))
            dS = (np.diag(p) - np.outer(p, p)) @ a
            assert abs(dS.sum()) <= 1e-14 * max(1.0, np.abs(dS).sum())      # 1^T g = 0
            dK[0, h, :L] += alpha * np.outer(dS, q[0, h, i])
            dV[0, h, :L] += np.outer(p, u[0, h, i])
    for name, ref in (("dQ", dQ), ("dK", dK), ("dV", dV)):
        assert np.linalg.norm(got[name] - ref) <= 1e-10 + 1e-9 * np.linalg.norm(ref), name


def test_key_gradient_sums_to_zero_and_translation_invariance():
    # sum_j g_ij = 0  =>  sum_j dK_j = alpha sum_i (sum_j g_ij) q_i = 0.
    # Common key / value translations leave the VJP unchanged at fixed dO (Proposition "Exact translation structure").
    N, d = 40, 8
    shape = (1, 2, N, d)
    Q, K, V, dO = (grid_bf16(shape, 11 + i, step=0.125, span=15) for i in range(4))
    alpha = 0.25
    base = _run(Q, K, V, dO, alpha, True)
    assert np.abs(base["dK"].sum(axis=2)).max() <= 1e-12 * np.abs(base["dK"]).max()
    b = torch.tensor([4.0, -4.0, 2.0, 0.0, 8.0, -2.0, 4.0, 1.0]).to(torch.bfloat16)
    Kb = (K.float() + b.float()).to(torch.bfloat16)
    assert torch.equal(Kb.float(), K.float() + b.float())            # translation is exact in BF16
    moved = _run(Q, Kb, V, dO, alpha, True)
    for name in ("O", "dQ", "dK", "dV"):
        assert np.abs(moved[name] - base[name]).max() <= 1e-11, name
    shift = alpha * (np64(Q) @ np64(b))                                 # LSE moves by alpha q.b
    assert np.abs(moved["LSE"] - base["LSE"] - shift).max() <= 1e-11
    Vc = (V.float() + b.float()).to(torch.bfloat16)
    assert torch.equal(Vc.float(), V.float() + b.float())
    movedv = _run(Q, K, Vc, dO, alpha, True)
    for name in ("dQ", "dK", "dV", "LSE"):
        assert np.abs(movedv[name] - base[name]).max() <= 1e-11, name
    assert np.abs(movedv["O"] - base["O"] - np64(b)).max() <= 1e-12


def test_closed_forms():
    d = 4
    alpha = 0.5
    # (i) causal row 0 has one legal key: p_00 = 1, o_0 = v_0, LSE_0 = s_00, dq_0 = 0
    #     (Appendix "Channel One", fixed-forward paragraph on the first query row).
    Q, K, V, dO = (randn_bf16((1, 1, 9, d), 70 + i) for i in range(4))
    out = _run(Q, K, V, dO, alpha, True)
    assert np.array_equal(out["O"][0, 0, 0], np64(V)[0, 0, 0])
    assert out["LSE"][0, 0, 0] == alpha * float(np64(Q)[0, 0, 0] @ np64(K)[0, 0, 0])
    assert np.all(out["dQ"][0, 0, 0] == 0.0)
    # (ii) q = 0: uniform attention, LSE = ln n, o = mean(v) (setting of the four-key example).
    n = 8
    Q0 = torch.zeros((1, 1, n, d), dtype=torch.bfloat16)
    K, V, dO = (randn_bf16((1, 1, n, d), 80 + i) for i in range(3))
    out = _run(Q0, K, V, dO, alpha, False)
    assert np.allclose(out["LSE"], math.log(n), rtol=0, atol=1e-15)
    assert np.abs(out["O"][0, 0] - np64(V)[0, 0].mean(axis=0)).max() <= 1e-15
    # (iii) two keys: G_Q = alpha eps (1-eps) (a_1 - a_2)(k_1 - k_2)   (Eq. "two-key").
    q = torch.tensor([[1.0, -0.5, 2.0, 0.25]]); k = torch.tensor([[0.5, 1.0, -1.0, 2.0], [1.5, -1.0, 0.5, 0.0]])
    v = torch.tensor([[1.0, 2.0, -1.0, 0.5], [-2.0, 0.5, 1.0, 3.0]]); u = torch.tensor([[0.5, -1.0, 2.0, 1.0]])
    bf = lambda t: t.to(torch.bfloat16).reshape(1, 1, *t.shape)
    # non-causal with a single query needs N_q = N_k, so replicate the query row
    out = _run(bf(q.repeat(2, 1)), bf(k), bf(v), bf(u.repeat(2, 1)), alpha, False)
    s = alpha * (k.double() @ q.double()[0]); p = torch.softmax(s, 0)
    a = v.double() @ u.double()[0]
    expect = alpha * p[0] * p[1] * (a[0] - a[1]) * (k.double()[0] - k.double()[1])
    assert np.abs(out["dQ"][0, 0, 0] - expect.numpy()).max() <= 1e-15
    # (iv) constant values => dQ = dK = 0 exactly; dO = 0 => all gradients zero
    #      (Appendix "Synthetic Numerical Suite", "Exact zeros").
    Q, K, _, dO = (randn_bf16((1, 2, 17, d), 90 + i) for i in range(4))
    Vc = torch.full((1, 2, 17, d), 1.5, dtype=torch.bfloat16)
    out = _run(Q, K, Vc, dO, alpha, True)
    assert np.abs(out["dQ"]).max() <= 1e-14 and np.abs(out["dK"]).max() <= 1e-14
    out = _run(Q, K, randn_bf16((1, 2, 17, d), 99), torch.zeros_like(dO), alpha, True)
    assert all(np.all(out[n] == 0.0) for n in ("dQ", "dK", "dV"))


def test_row_and_key_subsets_match_full():
    N, d = 64, 8
    Q, K, V, dO = (randn_bf16((1, 1, N, d), 120 + i) for i in range(4))
    alpha = 0.3
    full = _run(Q, K, V, dO, alpha, True)
    rows = np.array([0, 5, 31, 63], dtype=np.int32)
    q, k, v, u = (as_bits(t)[0, 0] for t in (Q, K, V, dO))
    O, LSE, MUA, dQ = oracle.head_rows_f64(q, k, v, u, alpha, True, rows)
    assert np.array_equal(O, full["O"][0, 0, rows]) and np.array_equal(dQ, full["dQ"][0, 0, rows])
    assert np.array_equal(LSE, full["LSE"][0, 0, rows])
    dK, dV = oracle.head_keys_f64(q, k, v, u, alpha, True, full["LSE"][0, 0], full["MUA"][0, 0], rows)
    assert np.array_equal(dK, full["dK"][0, 0, rows]) and np.array_equal(dV, full["dV"][0, 0, rows])


def test_grouped_queries_match_torch_autograd():
    # Section 3.1: key and value contributions sum over the query heads that share a KV head.  Library reference:
    # torch float64 autograd with the K / V heads repeated for their groups.
    B, H, Hkv, N, d = 2, 6, 2, 33, 8
    Q, dO = (randn_bf16((B, H, N, d), 300 + i) for i in range(2))
    K, V = (randn_bf16((B, Hkv, N, d), 310 + i) for i in range(2))
    alpha = 0.3
    got = oracle.attn_fwd_bwd_f64(as_bits(Q), as_bits(K), as_bits(V), as_bits(dO), alpha, True)
    q = Q.double().requires_grad_(True); k = K.double().requires_grad_(True); v = V.double().requires_grad_(True)
    kk, vv = k.repeat_interleave(H // Hkv, dim=1), v.repeat_interleave(H // Hkv, dim=1)
    s = alpha * q @ kk.transpose(-1, -2)
    s = s.masked_fill(~torch.tril(torch.ones(N, N, dtype=torch.bool)), float("-inf"))
    o = torch.softmax(s, dim=-1) @ vv
    (o * dO.double()).sum().backward()
    assert got["dK"].shape == (B, Hkv, N, d)
    for name, ref in (("O", o.detach()), ("dQ", q.grad), ("dK", k.grad), ("dV", v.grad)):
        assert np.abs(got[name] - ref.numpy()).max() <= 1e-12 * max(1.0, ref.abs().max().item()), name


def test_rel_l2_metric():
    # 100 ||G^ - G|| / ||G||  (Appendix "Accuracy and Cost", "Reference and metric").
    g = np.array([3.0, 4.0]); gh = np.array([3.0, 4.5])
    assert oracle.rel_l2_percent(gh, g) == pytest.approx(10.0)
    assert oracle.rel_l2_percent(np.zeros(3), np.zeros(3)) == 0.0
