"""Pins of the Algorithm-1 rounding model (CPU only): the -24 witness, the projector
identities, the per-row bound of the projection, and agreement with the exact VJP."""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import emulation as em
from helpers import as_bits, load_values, randn_bf16, witness128_arrays

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "witness_minus24.txt")


def load_golden():
    vals = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if line:
                key, *rest = line.split()
                vals[key] = np.array([float(x) for x in rest])
    return vals


def witness_inputs(gold, d=2):
    pad = lambda rows: np.array([np.concatenate([r, np.zeros(d - r.size)]) for r in rows])
    K = pad([gold[f"k{j}"] for j in range(1, 5)])
    V = pad([gold[f"v{j}"] for j in range(1, 5)])
    Q = np.tile(pad([gold["q"]]), (4, 1))
    U = np.tile(pad([gold["u"]]), (4, 1))
    return tuple(em.f64_to_bf16_bits(x) for x in (Q, K, V, U))


def test_witness_inputs_are_exact_in_bf16():
    gold = load_golden()
    for key in ("k1", "k4", "v1", "v3", "u", "eta"):
        assert np.array_equal(em.bf16(gold[key]), gold[key]), key
    assert gold["eta"][0] == 3 / 1024


@pytest.mark.parametrize("d", [2, 64])
def test_minus24_witness(d):
    # Appendix A "An exact -24 witness": every printed intermediate, then -24 without and 0 with GProj.
    gold = load_golden()
    q, k, v, u = witness_inputs(gold, d)
    alpha = float(gold["alpha"][0])
    on = em.emulate_head(q, k, v, u, alpha, causal=False)
    off = em.emulate_head(q, k, v, u, alpha, causal=False, correct_q=False, correct_k=False)
    for row in range(4):                                   # every (identical) query row reproduces it
        assert np.array_equal(on["r"][row], gold["p"])
        assert np.array_equal(on["O"][row, :2], gold["o"])
        assert on["D"][row] == gold["uTo"][0]
        assert np.array_equal(on["t"][row], gold["t"])
        assert on["rho"][row] == gold["rho"][0]
        assert on["m"][row] == 1.0
        assert off["dQ"][row, 0] == gold["dq0_uncorrected"][0] == -24.0
        assert on["dQ"][row, 0] == gold["dq0_gproj"][0] == 0.0
    # the exact VJP agrees with the printed g and with dq[0] = 0
    ex = oracle.attn_fwd_bwd_f64(q[None, None], k[None, None], v[None, None], u[None, None], alpha, False)
    assert np.all(ex["dQ"][0, 0, :, 0] == gold["dq0_exact"][0])
    K = em.bf16_bits_to_f64(k)
    assert np.allclose(ex["dQ"][0, 0, 0], alpha * gold["g"] @ K, rtol=0, atol=1e-12)
    a = em.bf16_bits_to_f64(v) @ em.bf16_bits_to_f64(u)[0]
    assert np.array_equal(a, gold["a"])


def test_projector_identities():
    # Proposition "Projection with consistent operand mass" and Proposition "Exact leakage decomposition".
    rng = np.random.default_rng(3)
    n, d, alpha = 12, 5, 0.37
    r = em.bf16(rng.random(n)); t = em.bf16(rng.standard_normal(n)); K = rng.standard_normal((n, d))
    Pi = em.projector(r)
    assert np.allclose(Pi @ Pi, Pi, atol=1e-14)
    assert np.allclose(np.ones(n) @ Pi, 0, atol=1e-14)
    rho, m = t.sum(), r.sum()
    tp = Pi @ t
    assert np.allclose(tp, t - (rho / m) * r, atol=1e-15) and abs(tp.sum()) < 1e-14
    mu_r = (r @ K) / m
    assert np.allclose(alpha * (t @ K - (rho / m) * (r @ K)), alpha * t @ (K - mu_r), atol=1e-13)
    b = rng.standard_normal(d) * 1e3
    assert np.allclose(alpha * t @ (K + b) - alpha * t @ K, alpha * rho * b, rtol=1e-10)     # moves by alpha rho b
    assert np.allclose(alpha * tp @ (K + b), alpha * tp @ K, atol=1e-9)                    # invariant
    assert np.isclose((t - rho * r).sum(), rho * (1 - m), atol=1e-15)                      # lambda = rho leaves rho(1-m)
    # minimal r-weighted norm among zero-sum vectors
    for _ in range(20):
        z = rng.standard_normal(n); z -= z.mean()
        assert ((tp - t) ** 2 / r).sum() <= ((z - t) ** 2 / r).sum() + 1e-12


def test_projection_bound_is_offset_independent():
    # Theorem "Forward repair versus projection" (b): ||E_proj|| <= alpha u_b sigma_k sigma_a, at any key offset;
    # (a): the direct contraction's error grows with the offset.
    rng = np.random.default_rng(5)
    n, d, alpha, ub = 256, 16, 0.25, 2.0 ** -8
    direct_err = []
    for offset in (0.0, 1e2, 1e4):
        worst = 0.0
        for _ in range(20):
            z = rng.standard_normal((n, d)); b = rng.standard_normal(d); b *= offset / np.linalg.norm(b)
            keys = z + b
            s = 3.0 * rng.standard_normal(n); p = np.exp(s - s.max()); p /= p.sum()
            a = rng.standard_normal(n)
            got, exact = em.ideal_cast_row(p, a, keys, alpha, project=True)
            mu_k = p @ keys; mu_a = p @ a
            sig_k = math.sqrt((p * ((keys - mu_k) ** 2).sum(axis=1)).sum()); sig_a = math.sqrt((p * (a - mu_a) ** 2).sum())
            assert np.linalg.norm(got - exact) <= alpha * ub * sig_k * sig_a * (1 + 1e-9) + 1e-12 * (1 + offset)
            got_d, _ = em.ideal_cast_row(p, a, keys, alpha, project=False)
            worst = max(worst, np.linalg.norm(got_d - exact) / np.linalg.norm(exact))
        direct_err.append(worst)
    assert direct_err[2] > 50 * direct_err[0]


@pytest.mark.parametrize("causal", [True, False])
def test_emulation_tracks_exact_vjp_and_correction_helps(causal):
    N, d = 256, 64
    alpha = float(np.float32(1 / math.sqrt(d)))
    g = torch.Generator().manual_seed(1); c = torch.randn(d, generator=g); c = c / c.norm() * 256.0
    Q, K, V, dO = (randn_bf16((N, d), 200 + i, offset=(c if i == 1 else None)) for i in range(4))
    q, k, v, u = (as_bits(t) for t in (Q, K, V, dO))
    ex = oracle.attn_fwd_bwd_f64(q[None, None], k[None, None], v[None, None], u[None, None], alpha, causal)
    on = em.emulate_head(q, k, v, u, alpha, causal)
    off = em.emulate_head(q, k, v, u, alpha, causal, correct_q=False, correct_k=False)
    err = lambda r, n: oracle.rel_l2_percent(r[n], ex[n][0, 0])
    assert err(on, "O") < 0.3
    for name in ("dQ", "dK", "dV"):
        assert err(on, name) < 0.5, (name, err(on, name))              # BF16 floor (suite medians ~0.22 %)
    assert err(off, "dQ") > 5 * err(on, "dQ")                           # leak alpha rho mu_k with a 256-norm offset
    # each correction changes only the gradient it targets (Section "Translation invariance and robustness")
    only_q = em.emulate_head(q, k, v, u, alpha, causal, correct_k=False)
    assert np.array_equal(only_q["dQ"], on["dQ"]) and np.array_equal(only_q["dK"], off["dK"])
    assert np.array_equal(only_q["dV"], on["dV"]) and np.array_equal(off["dV"], on["dV"])
    # operand mass stays near one (Appendix "Synthetic Numerical Suite", "Operand masses")
    assert np.all(on["m"] > 0) and np.abs(on["m"] - 1).max() < 0.01


# ---------------------------------------------------------------------------------------------------------------
# Hand-derived pins of the key pass, of lambda with m != 1, of D from the saved output and of dV from r.
# The expected values live in tests/golden/*.txt with their derivations; none was produced by the model under test.

def test_key_pass_on_the_128_row_witness():
    # Algorithm 1 lines 15-18, Eq. "gproj-key-implemented": dK = BF16(alpha (t^T Q - r^T z)), z = BF16(lambda q).
    gold = load_golden()
    hand = load_values("witness128_key_pass.txt")
    q, k, v, u = (em.f64_to_bf16_bits(x) for x in witness128_arrays())
    alpha = float(gold["alpha"][0])
    on = em.emulate_head(q, k, v, u, alpha, causal=False)
    only_q = em.emulate_head(q, k, v, u, alpha, causal=False, correct_k=False)
    off = em.emulate_head(q, k, v, u, alpha, causal=False, correct_q=False, correct_k=False)
    assert np.all(on["m"] == 1.0) and np.all(on["rho"] == gold["rho"][0]) and np.all(on["lam"] == gold["rho"][0])
    assert np.array_equal(on["dK"][:4, 2], hand["dk2_gproj"])
    assert np.array_equal(only_q["dK"][:4, 2], hand["dk2_uncorrected"])
    assert np.array_equal(off["dK"][:4, 2], hand["dk2_uncorrected"])
    assert np.all(on["dK"][:4, 3] == hand["dk3_gproj"]) and np.array_equal(only_q["dK"][:4, 3], hand["dk3_uncorrected"])
    rest = on["dK"].copy(); rest[:4, 2:4] = 0
    assert not rest.any()
    assert np.all(on["dV"][:4, :2] == hand["dv01"]) and not on["dV"][4:].any() and not on["dV"][:, 2:].any()
    assert np.all(on["dQ"][:, 0] == 0.0) and np.all(off["dQ"][:, 0] == -24.0)
    ex = oracle.attn_fwd_bwd_f64(q[None, None], k[None, None], v[None, None], u[None, None], alpha, False)
    assert np.allclose(ex["dK"][0, 0, :4, 2], hand["dk2_exact"], rtol=0, atol=1e-9)
    assert np.allclose(ex["dK"][0, 0, :4, 3], hand["dk3_exact"], rtol=0, atol=1e-9)


def small_case_inputs(vals, n=3):
    rows = lambda stem: np.array([vals[f"{stem}{j}"] for j in range(1, n + 1)])
    Q = rows("q") if "q1" in vals else np.tile(vals["q"], (n, 1))
    return tuple(em.f64_to_bf16_bits(x) for x in (Q, rows("k"), rows("v"), rows("u")))


def test_lambda_divides_by_the_operand_mass():
    # Algorithm 1 line 14 / Eq. "gproj-row-mass": lambda = rho / m with m the sum of the ROUNDED probabilities
    # (three keys at BF16(1/3): m = 513/512); lambda = rho would leave the mass rho (1 - m) on the mean key.
    hand = load_values("three_key_mass.txt")
    q, k, v, u = small_case_inputs(hand)
    alpha = float(hand["alpha"][0])
    on = em.emulate_head(q, k, v, u, alpha, causal=False)
    only_q = em.emulate_head(q, k, v, u, alpha, causal=False, correct_k=False)
    assert np.all(on["r"] == hand["r"][0]) and np.all(on["m"] == hand["m"][0])
    assert np.array_equal(on["t"], np.tile(hand["t"], (3, 1))) and np.all(on["rho"] == hand["rho"][0])
    assert np.all(on["D"] == 0.0)
    assert np.all(on["lam"] == hand["lam"][0])
    assert np.all(on["dQ"][:, 0] == hand["dq0"][0])
    assert np.all(on["dQ"][:, 1] == hand["dq1"][0])
    assert np.array_equal(on["dK"][:, 2], hand["dk2_gproj"])
    assert np.array_equal(only_q["dK"][:, 2], hand["dk2_uncorrected"])
    assert np.all(on["dV"][:, 3] == hand["dv3"][0])
    assert np.all(on["dV"][:, :2] == hand["dv01"])


def test_row_term_comes_from_the_saved_bf16_output_and_operands_are_the_rounded_probabilities():
    # Algorithm 1 line 1 / Eq. "main-delta": D = rowsum(dO * BF16(o)); line 6: dV += r^T dO with r = BF16(P);
    # lines 16-17: the key correction contracts the rounded probabilities with z = BF16(lambda q).
    hand = load_values("three_key_saved_output.txt")
    q, k, v, u = small_case_inputs(hand)
    alpha = float(hand["alpha"][0])
    on = em.emulate_head(q, k, v, u, alpha, causal=False)
    only_q = em.emulate_head(q, k, v, u, alpha, causal=False, correct_k=False)
    assert np.all(on["O"][:, 0] == hand["o0"][0])
    assert np.all(on["D"] == hand["D"][0])
    assert np.array_equal(on["t"], np.tile(hand["t"], (3, 1))) and np.all(on["rho"] == hand["rho"][0])
    assert np.all(on["r"] == hand["r"][0]) and np.all(on["lam"] == hand["lam"][0])
    assert np.all(on["dQ"][:, 0] == hand["dq0"][0]) and np.all(on["dQ"][:, 1] == hand["dq1"][0])
    assert np.array_equal(on["dK"][:, 3], hand["dk3_gproj"])
    assert np.array_equal(only_q["dK"][:, 3], hand["dk3_uncorrected"])
    assert np.all(on["dV"][:, 3] == hand["dv3"][0]) and np.all(on["dV"][:, 0] == hand["dv0"][0])
    # the model's exact-D switch reproduces the alternative worked out beside the golden values
    ideal = em.emulate_head(q, k, v, u, alpha, causal=False, exact_D=True)
    assert np.all(ideal["rho"] == -0.22265625) and np.all(ideal["dQ"][:, 1] == -10.6875)
