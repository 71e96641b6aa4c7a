"""Key smoothing (the comparison arm of Section 5.1) built from this library's calls, through the C ABI.

The arm: K~ = K - mean key (per sequence, per KV head), the fused-exponent forward on (Q, K~, V), the backward with both
corrections off, and dK = dK~ - mean_j dK~_j (the vector-Jacobian product of the subtraction).  The tests say what the
arm removes (a component common to all keys, which is what the leaked row mass multiplies) and what it does not (the
leak itself: when most rows select one key, the mean that matters is that key).
"""
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2609_34272_b200 as g
from paper_2609_34272_b200.workloads import Workload, bits, make_inputs

pytestmark = pytest.mark.gpu


def smooth_cpu(X, cu=None):
    """Mean in FP64 rounded to FP32, subtraction in FP32, one rounding to BF16 (per sequence if offsets are given)."""
    Xf = X.float()
    Y = torch.empty_like(Xf)
    rows = X.shape[-2]
    cu = [0, rows] if cu is None else cu
    for a, b in zip(cu[:-1], cu[1:]):
        if b > a:
            seg = Xf[..., a:b, :]
            Y[..., a:b, :] = seg - seg.double().mean(dim=-2, keepdim=True).float()
    return Y.to(torch.bfloat16)


def ulp_distance(a, b):
    """Distance in BF16 steps between two BF16 tensors of the same sign pattern (bit patterns are monotone per sign)."""
    ia = a.view(torch.int16).to(torch.int32); ib = b.view(torch.int16).to(torch.int32)
    return (ia - ib).abs()


@pytest.mark.parametrize("d", [64, 128])
def test_smoothing_kernel_against_a_cpu_restatement(d):
    gen = torch.Generator().manual_seed(3 + d)
    X = (torch.randn(2, 3, 1000, d, generator=gen) + 5.0 * torch.randn(2, 3, 1, d, generator=gen)).to(torch.bfloat16)
    want = smooth_cpu(X)
    got = g.gproj_key_smooth(X.cuda()).cpu()
    # the FP32 column sum is taken in another order than the CPU's FP64 one: a handful of entries may round the other way
    same_sign = (got.float() * want.float()) >= 0
    dist = ulp_distance(got, want)
    assert (dist[same_sign] <= 1).all() and (dist > 0).float().mean().item() < 2e-3
    assert (got.float() - want.float()).abs().max().item() <= 0.04
    assert got.float().mean(dim=2).abs().max().item() < 5e-3            # the mean row is gone (BF16 rounding noise remains)
    again = g.gproj_key_smooth(X.cuda()).cpu()
    assert torch.equal(got, again)                                      # fixed summation order: reproducible
    # packed layout with host offsets, in place; an empty sequence is skipped
    cu = [0, 130, 130, 700, 1000]
    P = X[0].contiguous()
    want_p = smooth_cpu(P, cu)
    buf = P.cuda()
    g.gproj_key_smooth(buf, Y=buf, cu_seqlens=cu)
    dist = ulp_distance(buf.cpu(), want_p)
    assert (dist <= 1).all() or ((buf.cpu().float() - want_p.float()).abs().max().item() <= 0.04)
    assert (dist > 0).float().mean().item() < 2e-3
    with pytest.raises(g.GprojError):
        g.gproj_key_smooth(buf, cu_seqlens=[0, 10, 5, 1000])


def smoothing_arm(Q, K, V, dO, alpha, causal):
    """The arm on CPU-smoothed keys (so that the oracle sees the very same BF16 inputs); returns GPU results and K~."""
    Ks = smooth_cpu(K)
    Qd, Kd, Vd, Ud = (t.cuda() for t in (Q, Ks, V, dO))
    O, LSE = g.gproj_attn_fwd(Qd, Kd, Vd, alpha, causal, fwd_flags=g.FWD_FLAG_FMA_SOFTMAX)
    dQ, dKs, dV = g.gproj_attn_bwd(Qd, Kd, Vd, O, LSE, Ud, alpha, causal, flags=g.FLAG_NO_Q_CORRECTION | g.FLAG_NO_K_CORRECTION)
    dK = g.gproj_key_smooth(dKs)
    rc, detail = g.gproj_last_device_status()
    assert rc == 0, hex(detail)
    return {"O": O, "dQ": dQ, "dK": dK, "dV": dV, "dK_before_fixup": dKs}, Ks


def errors(out, ex):
    return {n: oracle.rel_l2_percent(out[n].float().cpu().numpy(), ex[n]) for n in ("O", "dQ", "dK", "dV")}


def test_smoothing_removes_a_common_key_offset():
    # workload-3-like inputs with a key offset of norm 64: the plain uncorrected backward degrades (about 1.6 % on dQ),
    # the smoothing arm is back at the BF16 floor, like GProj on the raw keys.
    w = Workload("smooth", 1, 4, 1024, 128, True, k_offset=64.0, seed=31)
    inp = make_inputs(w)
    a = w.softmax_scale
    arm, Ks = smoothing_arm(inp["Q"], inp["K"], inp["V"], inp["dO"], a, True)
    ex_s = oracle.attn_fwd_bwd_f64(bits(inp["Q"]), bits(Ks), bits(inp["V"]), bits(inp["dO"]), a, True)
    e_arm = errors(arm, ex_s)
    dev = {k: v.cuda() for k, v in inp.items()}
    O, LSE = g.gproj_attn_fwd(dev["Q"], dev["K"], dev["V"], a, True)
    plain = g.gproj_attn_bwd(dev["Q"], dev["K"], dev["V"], O, LSE, dev["dO"], a, True, flags=3)
    ex = oracle.attn_fwd_bwd_f64(*(bits(inp[k]) for k in ("Q", "K", "V", "dO")), a, True)
    e_plain_dq = oracle.rel_l2_percent(plain[0].float().cpu().numpy(), ex["dQ"])
    print("smoothing arm:", {k: round(v, 3) for k, v in e_arm.items()}, " plain uncorrected dQ on the raw keys: %.3f %%" % e_plain_dq)
    assert all(v <= 1.0 for v in e_arm.values()), e_arm
    assert e_plain_dq >= 3 * e_arm["dQ"]
    # the fix-up of dK removes exactly the column sum (Proposition 3.1: the exact one is zero)
    col = arm["dK"].float().sum(dim=2).abs().max().item()
    col_before = arm["dK_before_fixup"].float().sum(dim=2).abs().max().item()
    assert col <= 0.05 * max(col_before, 1e-6) + 0.5, (col, col_before)


def test_smoothing_zeroes_a_gauge_coordinate():
    # key coordinate 0 holds one common value b: after the subtraction it is exactly zero, so nothing is left for a
    # leaked row mass to multiply in that coordinate (and q[:, 0] = 0 keeps the scores independent of b)
    w = Workload("smooth_gauge", 1, 2, 512, 64, True, seed=32)
    inp = make_inputs(w)
    inp["Q"][..., 0] = 0
    inp["K"][..., 0] = 4096.0
    arm, Ks = smoothing_arm(inp["Q"], inp["K"], inp["V"], inp["dO"], w.softmax_scale, True)
    assert not Ks[..., 0].any()
    assert not arm["dQ"][..., 0].any()


@pytest.mark.parametrize("d,common_query,sink_norm", [(64, 8.0, 16.0), (128, 12.0, 16.0)])
def test_smoothing_does_not_help_when_rows_select_one_key(d, common_query, sink_norm):
    # attention sink: most rows put nearly all probability on key 0.  The leaked row mass then multiplies that key
    # (the row's own mean key), which the subtraction of the average key barely moves: the arm stays as wrong as the
    # plain backward, while the projection on the raw keys is at the floor.
    N = 512
    gen = torch.Generator().manual_seed(4242 + d)
    Q, K, V, U = (torch.randn(N, d, generator=gen) for _ in range(4))
    c = torch.randn(d, generator=gen); c = c / c.norm()
    Q = Q + common_query * c
    K[0] = 0.1 * K[0] + sink_norm * c
    Q, K, V, U = (x.to(torch.bfloat16).reshape(1, 1, N, d) for x in (Q, K, V, U))
    alpha = float(np.float32(1 / math.sqrt(d)))
    arm, Ks = smoothing_arm(Q, K, V, U, alpha, True)
    ex_s = oracle.attn_fwd_bwd_f64(bits(Q), bits(Ks), bits(V), bits(U), alpha, True)
    e_arm = errors(arm, ex_s)
    O, LSE = g.gproj_attn_fwd(Q.cuda(), K.cuda(), V.cuda(), alpha, True)
    dQ, dK, dV = g.gproj_attn_bwd(Q.cuda(), K.cuda(), V.cuda(), O, LSE, U.cuda(), alpha, True)
    ex = oracle.attn_fwd_bwd_f64(bits(Q), bits(K), bits(V), bits(U), alpha, True)
    e_gproj = errors({"O": O, "dQ": dQ, "dK": dK, "dV": dV}, ex)
    print("sink regime d=%d: smoothing arm %s, GProj %s" % (d, {k: round(v, 2) for k, v in e_arm.items()}, {k: round(v, 3) for k, v in e_gproj.items()}))
    assert all(v <= 1.0 for v in e_gproj.values()), e_gproj
    assert e_arm["dQ"] >= 20 * e_gproj["dQ"] and e_arm["dK"] >= 20 * e_gproj["dK"]
