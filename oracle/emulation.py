"""Rounding-model restatement of Algorithm 1 (test infrastructure only).

Untiled, one head at a time, in numpy.  Contractions and row sums are exact-ish
(FP64); BF16 / FP32 roundings sit where the paper puts them:

* saved output  O^ = BF16(o), saved LSE in FP32            (Appendix "Implemented Arithmetic", "Forward and saved state")
* D = rowsum(dO * O^)                                       (Algorithm 1, line 1)
* P = exp(S - LSE), r = BF16(P), t = BF16(fl32[P (dP - D)]) (lines 5-8, Eq. "gproj-row-mass")
* rho = rowsum(t), m = rowsum(r), lambda = rho/m, 0 if m=0  (lines 8, 14)
* dQ = BF16(fl32[alpha (tK - lambda rK)])                   (line 14, Eq. "gproj-query-implemented")
* z = BF16(lambda q), dK = BF16(fl32[alpha (t^T Q - r^T z)])(lines 17-18, Eq. "gproj-key-implemented")
* dV = BF16(r^T dO)                                         (lines 6, 12)

This is not a bitwise model of any kernel (accumulation order and the exponential
differ); it pins what the correction computes and what switching it off gives.
"""
import numpy as np


def bf16_bits_to_f64(x):
    x = np.ascontiguousarray(x, dtype=np.uint16)
    return (x.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def fl32(x):
    """Round to FP32 (nearest even), returned as FP64 for further exact arithmetic."""
    return np.asarray(x, dtype=np.float64).astype(np.float32).astype(np.float64)


def bf16(x):
    """cast_BF16 of an FP32 value: round-to-nearest-even to 8 significand bits (finite inputs)."""
    b = np.asarray(x, dtype=np.float64).astype(np.float32).view(np.uint32)
    b = b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))
    b = b & np.uint32(0xFFFF0000)
    return b.view(np.float32).astype(np.float64)


def f64_to_bf16_bits(x):
    """BF16 bit patterns of values that are (assumed) exactly representable or to be rounded RNE."""
    b = np.asarray(x, dtype=np.float64).astype(np.float32).view(np.uint32)
    b = b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))
    return (b >> np.uint32(16)).astype(np.uint16)


def projector(r):
    """Pi_r = I - r 1^T / m  (Proposition "Projection with consistent operand mass")."""
    r = np.asarray(r, dtype=np.float64)
    return np.eye(r.size) - np.outer(r, np.ones(r.size)) / r.sum()


def emulate_head(q, k, v, u, alpha, causal, correct_q=True, correct_k=True, exact_D=False):
    """Algorithm 1 on one head.  q,k,v,u: BF16 bits [N,d].  alpha: the FP32 scale value.

    Returns a dict with BF16-valued (as FP64) O, dQ, dK, dV and the intermediates
    LSE, D, t, r, rho, m, lam.
    """
    Q, K, V, U = (bf16_bits_to_f64(x) for x in (q, k, v, u))
    N = Q.shape[0]
    alpha = float(np.float32(alpha))
    S = alpha * (Q @ K.T)
    mask = np.tril(np.ones((N, N), dtype=bool)) if causal else np.ones((N, N), dtype=bool)
    Sm = np.where(mask, S, -np.inf)
    smax = Sm.max(axis=1, keepdims=True)
    w = np.exp(Sm - smax)
    Z = w.sum(axis=1, keepdims=True)
    lse = (smax + np.log(Z))[:, 0]
    o = (w / Z) @ V
    O_hat = bf16(fl32(o))
    LSE32 = fl32(lse)
    a = fl32(U @ V.T)                                         # dP, FP32 accumulator
    D = fl32((U * O_hat).sum(axis=1)) if not exact_D else ((w / Z) * (U @ V.T)).sum(axis=1)
    P_hat = np.where(mask, fl32(np.exp(fl32(S) - LSE32[:, None])), 0.0)
    r = bf16(P_hat)
    t = bf16(fl32(P_hat * fl32(a - D[:, None])))
    rho = t.sum(axis=1)
    m = r.sum(axis=1)
    with np.errstate(divide="ignore", invalid="ignore"):
        lam = np.where(m != 0.0, fl32(fl32(rho) / fl32(m)), 0.0)
    A = t @ K
    Bm = r @ K
    lam_q = lam if correct_q else np.zeros_like(lam)
    dQ = bf16(fl32(alpha * (A - lam_q[:, None] * Bm)))
    lam_k = lam if correct_k else np.zeros_like(lam)
    z = bf16(fl32(lam_k[:, None] * Q))
    dK = bf16(fl32(alpha * (t.T @ Q - r.T @ z)))
    dV = bf16(fl32(r.T @ U))
    return {"O": O_hat, "LSE": LSE32, "D": D, "t": t, "r": r, "rho": rho, "m": m, "lam": lam,
            "dQ": dQ, "dK": dK, "dV": dV, "A": A, "B": Bm}


def ideal_cast_row(p, a, keys, alpha, project):
    """Theorem "Forward repair versus projection" setting for one query row.

    Exact probabilities ``p``, exact centre mu_a, the only rounding is t = BF16(g);
    contraction in FP64.  ``project`` selects GProj with r = p (part b) or the direct
    contraction (part a).  Returns (dq_hat, dq_exact).
    """
    p = np.asarray(p, dtype=np.float64); a = np.asarray(a, dtype=np.float64); keys = np.asarray(keys, dtype=np.float64)
    g = p * (a - (p * a).sum())
    t = bf16(g)
    if project:
        t = t - (t.sum() / p.sum()) * p
    return alpha * (t @ keys), alpha * (g @ keys)
