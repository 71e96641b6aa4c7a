"""GPU parity with unequal query and key lengths (through the C ABI).

Appendix "Synthetic Numerical Suite" lists unequal lengths and empty causal rows among the shapes the correction must
survive.  The causal diagonal ends at the last query and the last key (support of query i: keys j <= i + (Nk - Nq)); with
more queries than keys the leading queries see nothing and must come back as O = 0, dQ = 0, LSE = +inf (no correction:
Algorithm 1, line 14).  Every case is compared with the FP64 oracle for this shape on the full tensors.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_34272_b200 as g

pytestmark = pytest.mark.gpu


def make(B, H, Hkv, Nq, Nk, d, seed, k_offset=0.5):
    gen = torch.Generator().manual_seed(seed)
    Q = torch.randn(B, H, Nq, d, generator=gen).to(torch.bfloat16)
    K = (torch.randn(B, Hkv, Nk, d, generator=gen) + k_offset).to(torch.bfloat16)   # shifted keys: the paper's biased regime
    V = torch.randn(B, Hkv, Nk, d, generator=gen).to(torch.bfloat16)
    dO = torch.randn(B, H, Nq, d, generator=gen).to(torch.bfloat16)
    return Q, K, V, dO


def tobits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def f64(t):
    return t.float().cpu().numpy().astype(np.float64)


def run(Q, K, V, dO, alpha, causal, flags=0):
    q, k, v, do = (x.cuda() for x in (Q, K, V, dO))
    # poisoned outputs: a row the kernels forget to write shows as NaN
    O = torch.full_like(q, float("nan")); LSE = torch.full(q.shape[:3], float("nan"), device="cuda")
    dQ = torch.full_like(q, float("nan")); dK = torch.full_like(k, float("nan")); dV = torch.full_like(v, float("nan"))
    g.gproj_attn_fwd_rect(q, k, v, alpha, causal, O=O, LSE=LSE)
    g.gproj_attn_bwd_rect(q, k, v, O, LSE, do, alpha, causal, flags=flags, dQ=dQ, dK=dK, dV=dV)
    rc, detail = g.gproj_last_device_status()
    assert rc == 0, (g.status_string(rc), hex(detail))
    return {"O": f64(O), "LSE": LSE.cpu().numpy().astype(np.float64), "dQ": f64(dQ), "dK": f64(dK), "dV": f64(dV)}


def check(got, ex, bar=1.0):
    empty = np.isinf(ex["LSE"])
    assert np.array_equal(np.isposinf(got["LSE"]), empty)
    assert np.all(np.abs(got["LSE"][~empty] - ex["LSE"][~empty]) <= 1e-4 + 1e-5 * np.abs(ex["LSE"][~empty]))
    assert np.all(got["O"][empty] == 0.0) and np.all(got["dQ"][empty] == 0.0)
    errs = {}
    for n in ("O", "dQ", "dK", "dV"):
        assert got[n].shape == ex[n].shape
        assert np.all(np.isfinite(got[n])), n
        scale = np.abs(ex[n]).max()
        if scale == 0.0:          # a gradient that vanishes exactly (one key): only rounding residue may remain
            assert np.abs(got[n]).max() <= 1e-3, n
            continue
        errs[n] = oracle.rel_l2_percent(got[n], ex[n])
        assert errs[n] <= bar, (n, errs)
        assert np.abs(got[n] - ex[n]).max() <= 0.03 * scale, (n, "element-wise")
    return errs


# (Nq, Nk): one side a single tile, ragged both ways, several tiles, a single query / key, more queries than keys
SHAPES = [(128, 256), (256, 128), (100, 333), (333, 100), (1, 200), (200, 1), (64, 640), (700, 190), (129, 130), (517, 1029)]


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("shape", SHAPES)
def test_unequal_lengths(shape, d, causal):
    Nq, Nk = shape
    Q, K, V, dO = make(1, 2, 1, Nq, Nk, d, seed=Nq * 7 + Nk * 3 + d)
    alpha = d ** -0.5
    ex = oracle.attn_rect_f64(tobits(Q), tobits(K), tobits(V), tobits(dO), alpha, causal)
    got = run(Q, K, V, dO, alpha, causal)
    if causal and Nq > Nk:
        assert int(np.isinf(ex["LSE"]).sum()) == 2 * (Nq - Nk)       # the leading queries of both heads see no key
    check(got, ex)


@pytest.mark.parametrize("case", [(2, 4, 2, 300, 555, 64, True), (2, 6, 2, 555, 300, 128, True), (2, 4, 4, 1000, 2048, 64, False),
                                  (1, 3, 3, 2048, 300, 128, False)])
def test_unequal_lengths_batched_grouped(case):
    B, H, Hkv, Nq, Nk, d, causal = case
    Q, K, V, dO = make(B, H, Hkv, Nq, Nk, d, seed=sum(case[:6]))
    alpha = d ** -0.5
    ex = oracle.attn_rect_f64(tobits(Q), tobits(K), tobits(V), tobits(dO), alpha, causal)
    check(run(Q, K, V, dO, alpha, causal), ex)


@pytest.mark.parametrize("d", [64, 128])
def test_equal_lengths_give_the_square_call_bit_for_bit(d):
    Q, K, V, dO = make(2, 4, 2, 333, 333, d, seed=11 + d)
    alpha = d ** -0.5
    got = run(Q, K, V, dO, alpha, True)
    q, k, v, do = (x.cuda() for x in (Q, K, V, dO))
    O, LSE = g.gproj_attn_fwd(q, k, v, alpha, True)
    dQ, dK, dV = g.gproj_attn_bwd(q, k, v, O, LSE, do, alpha, True)
    for n, t in (("O", O), ("dQ", dQ), ("dK", dK), ("dV", dV)):
        assert np.array_equal(got[n], f64(t)), n
    assert np.array_equal(got["LSE"], LSE.cpu().numpy().astype(np.float64))


def test_decode_like_block_of_new_queries():
    # a short block of new queries against a long key history, the causal diagonal at the end: each query's rows must
    # equal what the square causal call of the full length gives for the same rows
    d, Nk, Nq = 64, 1000, 72
    Qf, K, V, dOf = make(1, 2, 2, Nk, Nk, d, seed=4242)
    alpha = d ** -0.5
    Q, dO = Qf[:, :, Nk - Nq:].contiguous(), dOf[:, :, Nk - Nq:].contiguous()
    got = run(Q, K, V, dO, alpha, True)
    q, k, v = Qf.cuda(), K.cuda(), V.cuda()
    O, LSE = g.gproj_attn_fwd(q, k, v, alpha, True)
    assert np.array_equal(got["O"], f64(O[:, :, Nk - Nq:]))
    assert np.allclose(got["LSE"], LSE[:, :, Nk - Nq:].cpu().numpy().astype(np.float64), rtol=1e-6, atol=1e-6)


def test_uncorrected_backward_and_empty_rows():
    # the ablation flags take the same masked path; empty rows stay exactly zero
    Q, K, V, dO = make(1, 2, 2, 400, 150, 64, seed=9)
    alpha = 0.125
    ex = oracle.attn_rect_f64(tobits(Q), tobits(K), tobits(V), tobits(dO), alpha, True)
    check(run(Q, K, V, dO, alpha, True, flags=g.FLAG_NO_Q_CORRECTION | g.FLAG_NO_K_CORRECTION), ex, bar=5.0)


def test_shape_errors():
    q = torch.zeros(1, 2, 64, 64, dtype=torch.bfloat16, device="cuda")
    k = torch.zeros(1, 2, 32, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(ValueError):
        g.gproj_attn_fwd_rect(q, k, k, 0.125, True)
    k3 = torch.zeros(1, 3, 32, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(ValueError):
        g.gproj_attn_fwd_rect(q, k3, k3, 0.125, True)
