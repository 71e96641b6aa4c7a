"""GPU checks of exact identities and designed cases (through the C ABI)."""
import math
import os

import numpy as np
import pytest
import torch

import oracle
import paper_2609_34272_b200 as g
from oracle import emulation as em
from helpers import load_values, witness128_arrays
from paper_2609_34272_b200.workloads import Workload, bits, from_bits, make_inputs

pytestmark = pytest.mark.gpu


def fwd_bwd(Q, K, V, dO, alpha, causal, flags=0):
    Q, K, V, dO = (t.cuda() for t in (Q, K, V, dO))
    O, LSE = g.gproj_attn_fwd(Q, K, V, alpha, causal)
    dQ, dK, dV = g.gproj_attn_bwd(Q, K, V, O, LSE, dO, alpha, causal, flags=flags)
    rc, detail = g.gproj_last_device_status()
    assert rc == 0, hex(detail)
    return O, LSE, dQ, dK, dV


def witness_problem():
    """The four-key -24 witness embedded in a 128 x 128, d = 64 non-causal problem.

    Every query is (0, 0, 256, c, 0, ...); keys 0..3 are the witness keys (third and fourth coordinate 0); the
    other 124 keys are (0, 0, -256, 0, ...), whose logits -8192 give probability exactly 0 in FP32 and FP64.
    Every row therefore reproduces the witness (Appendix A, "An exact -24 witness"), and the third and fourth
    query coordinates make the key-side correction visible in dK (tests/golden/witness128_key_pass.txt).
    """
    vals = load_values("witness_minus24.txt")
    N, d = 128, 64
    tens = [from_bits(em.f64_to_bf16_bits(x)).reshape(1, 1, N, d) for x in witness128_arrays()]
    return tens, vals


def test_minus24_witness_on_gpu():
    (Q, K, V, U), vals = witness_problem()
    hand = load_values("witness128_key_pass.txt")
    alpha = float(vals["alpha"][0])
    O, LSE, dQ, dK, dV = fwd_bwd(Q, K, V, U, alpha, False)
    assert torch.all(O[0, 0, :, 0].float() == vals["o"][0]) and torch.all(O[0, 0, :, 1].float() == vals["o"][1])
    assert torch.all(dQ[0, 0, :, 0].float() == vals["dq0_gproj"][0])                    # exactly zero with GProj
    _, _, dQ_off, dK_noq, _ = fwd_bwd(Q, K, V, U, alpha, False, flags=g.FLAG_NO_Q_CORRECTION)
    assert torch.all(dQ_off[0, 0, :, 0].float() == vals["dq0_uncorrected"][0])          # -24 without it
    # the remaining coordinates agree with the rounding model of Algorithm 1
    q, k, v, u = (bits(t)[0, 0] for t in (Q, K, V, U))
    model = em.emulate_head(q, k, v, u, alpha, causal=False)
    assert np.array_equal(dQ[0, 0].float().cpu().numpy(), model["dQ"])
    assert np.array_equal(dV[0, 0].float().cpu().numpy(), model["dV"])
    # key pass (Algorithm 1 lines 15-18): the hand-derived values, with and without the correction
    dK_np = dK[0, 0].float().cpu().numpy()
    assert np.array_equal(dK_np, model["dK"])
    assert np.array_equal(dK_np[:4, 2], hand["dk2_gproj"]) and np.array_equal(dK_np[:4, 3], hand["dk3_gproj"])
    assert torch.equal(dK_noq, dK)
    _, _, dQ_nok, dK_nok, dV_nok = fwd_bwd(Q, K, V, U, alpha, False, flags=g.FLAG_NO_K_CORRECTION)
    dK_nok = dK_nok[0, 0].float().cpu().numpy()
    assert np.array_equal(dK_nok[:4, 2], hand["dk2_uncorrected"]) and np.array_equal(dK_nok[:4, 3], hand["dk3_uncorrected"])
    assert torch.equal(dQ_nok, dQ) and torch.equal(dV_nok, dV)
    rest = dK_np.copy(); rest[:4, 2:4] = 0
    assert not rest.any()
    assert np.all(dV[0, 0, :4, :2].float().cpu().numpy() == hand["dv01"])


def three_key_problem(name):
    """A hand-worked three-key case of tests/golden, zero-padded from d = 4 to d = 64 (N = 3: one ragged tile)."""
    hand = load_values(name)
    rows = lambda stem: np.array([hand[f"{stem}{j}"] for j in (1, 2, 3)])
    Qs = rows("q") if "q1" in hand else np.tile(hand["q"], (3, 1))
    pad = lambda x: np.concatenate([x, np.zeros((3, 60))], axis=1)
    tens = [from_bits(em.f64_to_bf16_bits(pad(x))).reshape(1, 1, 3, 64) for x in (Qs, rows("k"), rows("v"), rows("u"))]
    return tens, hand


def test_three_key_operand_mass_on_gpu():
    # lambda = rho / m with m = 513/512 (Algorithm 1 line 14): hand values of tests/golden/three_key_mass.txt
    (Q, K, V, U), hand = three_key_problem("three_key_mass.txt")
    alpha = float(hand["alpha"][0])
    O, LSE, dQ, dK, dV = fwd_bwd(Q, K, V, U, alpha, False)
    dQ, dK, dV = (x[0, 0].float().cpu().numpy() for x in (dQ, dK, dV))
    assert np.all(np.abs(dQ[:, 0]) <= 1e-6)               # one FP32 rounding of lambda away from 0 (0.046875 with lambda = rho)
    assert np.all(dQ[:, 1] == hand["dq1"][0])
    assert np.array_equal(dK[:, 2], hand["dk2_gproj"])
    assert np.all(dV[:, 3] == hand["dv3"][0]) and np.all(dV[:, :2] == hand["dv01"])
    _, _, _, dK_nok, _ = fwd_bwd(Q, K, V, U, alpha, False, flags=g.FLAG_NO_K_CORRECTION)
    assert np.array_equal(dK_nok[0, 0, :, 2].float().cpu().numpy(), hand["dk2_uncorrected"])


def test_three_key_saved_output_on_gpu():
    # D from the saved BF16 output, dV and the key correction from the rounded probabilities
    # (Algorithm 1 lines 1, 6, 16-17): hand values of tests/golden/three_key_saved_output.txt
    (Q, K, V, U), hand = three_key_problem("three_key_saved_output.txt")
    alpha = float(hand["alpha"][0])
    O, LSE, dQ, dK, dV = fwd_bwd(Q, K, V, U, alpha, False)
    assert torch.all(O[0, 0, :, 0].float() == hand["o0"][0])
    dQ, dK, dV = (x[0, 0].float().cpu().numpy() for x in (dQ, dK, dV))
    assert np.all(np.abs(dQ[:, 0]) <= 1e-6) and np.all(dQ[:, 1] == hand["dq1"][0])
    assert np.array_equal(dK[:, 3], hand["dk3_gproj"])
    assert np.all(dV[:, 3] == hand["dv3"][0]) and np.all(dV[:, 0] == hand["dv0"][0])
    _, _, _, dK_nok, _ = fwd_bwd(Q, K, V, U, alpha, False, flags=g.FLAG_NO_K_CORRECTION)
    assert np.array_equal(dK_nok[0, 0, :, 3].float().cpu().numpy(), hand["dk3_uncorrected"])


def sink_problem(N, d, seed, common_query, sink_norm):
    """Late-training-like inputs: every query carries a large common component and key 0 is aligned with it, so
    most rows put nearly all their probability on key 0 (an attention sink).  Input construction only."""
    gen = torch.Generator().manual_seed(seed)
    Q, K, V, U = (torch.randn(N, d, generator=gen) for _ in range(4))
    c = torch.randn(d, generator=gen); c = c / c.norm()
    Q = Q + common_query * c
    K[0] = 0.1 * K[0] + sink_norm * c
    return [x.to(torch.bfloat16).reshape(1, 1, N, d) for x in (Q, K, V, U)]


@pytest.mark.parametrize("d,common_query,sink_norm", [(64, 8.0, 16.0), (64, 32.0, 4.0), (128, 12.0, 16.0)])
def test_key_pass_is_material_with_an_attention_sink(d, common_query, sink_norm):
    # The regime in which the paper's per-capture table shows the key pass mattering (dK error falling by more
    # than an order of magnitude): the leaked row mass of every row lands on the one key all rows select, times the
    # common query component.  Against the exact FP64 VJP: GProj dK at the BF16 floor, without the key pass >= 10x worse.
    N = 512
    Q, K, V, U = sink_problem(N, d, 4242 + d, common_query, sink_norm)
    alpha = float(np.float32(1 / math.sqrt(d)))
    ex = oracle.attn_fwd_bwd_f64(bits(Q), bits(K), bits(V), bits(U), alpha, True)
    on = fwd_bwd(Q, K, V, U, alpha, True)
    no_k = fwd_bwd(Q, K, V, U, alpha, True, flags=g.FLAG_NO_K_CORRECTION)
    err = lambda t, n: oracle.rel_l2_percent(t.float().cpu().numpy(), ex[n])
    e_on = {n: err(t, n) for n, t in zip(("O", "dQ", "dK", "dV"), (on[0], on[2], on[3], on[4]))}
    e_nok = err(no_k[3], "dK")
    print("sink regime d=%d: GProj %s, dK without the key pass %.2f %%" % (d, {k: round(v, 3) for k, v in e_on.items()}, e_nok))
    assert all(v <= 1.0 for v in e_on.values()), e_on
    assert e_nok >= 10 * e_on["dK"], (e_nok, e_on)


@pytest.mark.parametrize("d", [64, 128])
def test_gauge_coordinate(d):
    # Query coordinate 0 is zero and key coordinate 0 is a common value b: scores, O and LSE do not depend on b
    # and the exact dQ[:, 0] is zero (Appendix "Saved-state crosses and the remaining gauge defect").
    N = 256
    w = Workload("gauge", 1, 2, N, d, True, seed=991 + d)
    inp = make_inputs(w)
    inp["Q"][..., 0] = 0
    ref = None
    leak = {}
    for b in (0.0, 256.0, 65536.0):
        inp["K"][..., 0] = b
        O, LSE, dQ, dK, dV = fwd_bwd(inp["Q"], inp["K"], inp["V"], inp["dO"], w.softmax_scale, True)
        _, _, dQ_off, _, _ = fwd_bwd(inp["Q"], inp["K"], inp["V"], inp["dO"], w.softmax_scale, True, flags=3)
        if ref is None:
            ref = (O.clone(), LSE.clone())
        assert torch.equal(O, ref[0]) and torch.equal(LSE, ref[1])                       # bitwise unchanged
        leak[b] = (dQ[..., 0].float().abs().max().item(), dQ_off[..., 0].float().abs().max().item())
    print("gauge leak (corrected, uncorrected):", leak)
    assert leak[0.0] == (0.0, 0.0)
    assert leak[65536.0][0] <= 0.05                                                      # paper: <= 0.0117 on its case
    assert leak[65536.0][1] >= 20 * max(leak[65536.0][0], 1e-3)                          # uncorrected: grows with b
    assert leak[65536.0][1] == pytest.approx(256.0 * leak[256.0][1], rel=1e-2)           # and linearly in b


@pytest.mark.parametrize("d", [64, 128])
def test_first_causal_row_and_zero_targets(d):
    N = 384
    w = Workload("ident", 1, 2, N, d, True, k_offset=16.0, seed=77 + d)
    inp = make_inputs(w)
    O, LSE, dQ, dK, dV = fwd_bwd(inp["Q"], inp["K"], inp["V"], inp["dO"], w.softmax_scale, True)
    # one legal key: o_0 = v_0 bitwise and dq_0 = 0 exactly (subtract-before-scale restores the identity)
    assert torch.equal(O[:, :, 0].cpu(), inp["V"][:, :, 0])
    assert torch.all(dQ[:, :, 0] == 0)
    # zero upstream gradient: every gradient is exactly zero
    z = torch.zeros_like(inp["dO"])
    _, _, dQ0, dK0, dV0 = fwd_bwd(inp["Q"], inp["K"], inp["V"], z, w.softmax_scale, True)
    assert not dQ0.any() and not dK0.any() and not dV0.any()
    # constant values: exact dQ = dK = 0; the kernel's residual is rounding-level
    Vc = torch.full_like(inp["V"], 1.5)
    _, _, dQc, dKc, _ = fwd_bwd(inp["Q"], inp["K"], Vc, inp["dO"], w.softmax_scale, True)
    assert dQc.float().abs().max().item() <= 1e-3 and dKc.float().abs().max().item() <= 1e-3


def test_flags_change_only_their_gradient_and_runs_are_reproducible():
    w = Workload("flags", 1, 2, 512, 64, True, k_offset=64.0, seed=5)
    inp = make_inputs(w)
    base = fwd_bwd(inp["Q"], inp["K"], inp["V"], inp["dO"], w.softmax_scale, True)
    again = fwd_bwd(inp["Q"], inp["K"], inp["V"], inp["dO"], w.softmax_scale, True)
    for a, b in zip(base, again):
        assert torch.equal(a, b)                                                          # bitwise reproducible
    no_q = fwd_bwd(inp["Q"], inp["K"], inp["V"], inp["dO"], w.softmax_scale, True, flags=g.FLAG_NO_Q_CORRECTION)
    no_k = fwd_bwd(inp["Q"], inp["K"], inp["V"], inp["dO"], w.softmax_scale, True, flags=g.FLAG_NO_K_CORRECTION)
    O, LSE, dQ, dK, dV = base
    assert torch.equal(no_q[0], O) and torch.equal(no_q[3], dK) and torch.equal(no_q[4], dV) and not torch.equal(no_q[2], dQ)
    assert torch.equal(no_k[0], O) and torch.equal(no_k[2], dQ) and torch.equal(no_k[4], dV) and not torch.equal(no_k[3], dK)


def test_error_codes_on_device():
    x = torch.zeros(1, 1, 128, 64, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(1, 1, 128, dtype=torch.float32, device="cuda")
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(g.GprojError) as e:
        g.gproj_attn_bwd(x, x, x, x, lse, x, 0.125, True, workspace=small)
    assert e.value.status == -4
    with pytest.raises(g.GprojError) as e:
        g.gproj_attn_fwd(x, x, x, float("inf"), True)
    assert e.value.status == -5


def test_bounded_wait_reports_timeout_and_context_survives():
    # Failure detection without a GPU fault: a wait that can never be satisfied runs out of its budget, the kernel
    # returns, the host reads the code; the next real call works again.
    g.gproj_selftest_wait_timeout()
    rc, detail = g.gproj_last_device_status()
    assert rc == -8 and detail == 0x7e01, (rc, hex(detail))
    assert g.status_string(rc).startswith("a bounded in-kernel wait gave up")
    rc, detail = g.gproj_last_device_status()
    assert (rc, detail) == (0, 0)                                  # cleared by the read
    w = Workload("after_timeout", 1, 2, 256, 64, True, seed=3)
    inp = make_inputs(w)
    O, LSE, dQ, dK, dV = fwd_bwd(inp["Q"], inp["K"], inp["V"], inp["dO"], w.softmax_scale, True)
    assert torch.equal(O[:, :, 0].cpu(), inp["V"][:, :, 0])


def test_sharp_attention_far_keys_stress():
    # The regime the paper calls late training (sharp attention, keys far from the origin; Section 5.3): here the
    # uncorrected BF16 backward loses dQ entirely while the projected one stays at the BF16 floor.
    N, d, H = 1024, 64, 4
    gen = torch.Generator().manual_seed(77)
    z = torch.randn(1, H, N, d, generator=gen)
    b = torch.randn(1, H, 1, d, generator=gen); b = b / b.norm(dim=-1, keepdim=True) * 2048.0
    K = (z + b).to(torch.bfloat16)
    Q = (6.0 * torch.randn(1, H, N, d, generator=gen)).to(torch.bfloat16)      # logit spread ~6: nearly one-hot rows
    V = torch.randn(1, H, N, d, generator=gen).to(torch.bfloat16)
    dO = torch.randn(1, H, N, d, generator=gen).to(torch.bfloat16)
    alpha = 0.125
    ex = oracle.attn_fwd_bwd_f64(bits(Q), bits(K), bits(V), bits(dO), alpha, True)
    on = fwd_bwd(Q, K, V, dO, alpha, True)
    off = fwd_bwd(Q, K, V, dO, alpha, True, flags=3)
    err = lambda t, n: oracle.rel_l2_percent(t.float().cpu().numpy(), ex[n])
    e_on = {n: err(t, n) for n, t in zip(("O", "dQ", "dK", "dV"), (on[0], on[2], on[3], on[4]))}
    e_off = {n: err(t, n) for n, t in zip(("dQ", "dK"), (off[2], off[3]))}
    print("stress: corrected", e_on, "uncorrected", e_off)
    assert all(v <= 1.0 for v in e_on.values()), e_on
    assert e_off["dQ"] > 20.0 and e_off["dQ"] > 50 * e_on["dQ"]


def test_fma_softmax_breaks_the_one_key_identity_and_sbs_restores_it():
    # Appendix "The source of the saved-output error" / "Prescribed FMA cases": all 64 query coordinates equal c 2^k, all
    # key coordinates equal one, so every dot product is known exactly; the first causal row has a single key.  With the
    # fused exponent r = fma(x, a, -fl32(x a)) the row's own score does not map to zero, z = 2^r != 1, and the output is
    # v_0 BF16(z) / z instead of v_0.  Subtract-before-scale restores o_0 = v_0 in every case; GProj keeps dq_0 = 0.
    N, d, alpha = 128, 64, 0.125
    a32 = np.float32(np.float64(np.float32(alpha)) * 1.4426950408889634)
    gen = torch.Generator().manual_seed(9)
    V = torch.randn(1, 1, N, d, generator=gen).to(torch.bfloat16)
    dO = torch.randn(1, 1, N, d, generator=gen).to(torch.bfloat16)
    K = torch.ones(1, 1, N, d, dtype=torch.bfloat16)
    violations = 0
    for c in (3, 5, 7):
        for k in range(16):
            Q = torch.full((1, 1, N, d), float(c * 2 ** k), dtype=torch.bfloat16)
            x = np.float64(64.0 * c * 2 ** k)                                   # exact logit of every (row, key) pair
            r = np.float32(np.float64(x) * np.float64(a32) - np.float64(np.float32(np.float32(x) * a32)))   # fma residue
            z = 2.0 ** np.float64(r)
            Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
            O_sbs, LSE = g.gproj_attn_fwd(Qd, Kd, Vd, alpha, True)
            O_fma, LSE_f = g.gproj_attn_fwd(Qd, Kd, Vd, alpha, True, fwd_flags=g.FWD_FLAG_FMA_SOFTMAX)
            assert torch.equal(O_sbs[0, 0, 0].cpu(), V[0, 0, 0]), (c, k)       # identity holds with subtract-before-scale
            v0 = V[0, 0, 0].double().numpy()
            zb = float(torch.tensor(z, dtype=torch.float32).to(torch.bfloat16))
            model = v0 * zb / z                                                # scalar model of the fused form
            got = O_fma[0, 0, 0].double().cpu().numpy()
            assert np.all(np.abs(got - model) <= 2.0 ** -7 * np.abs(model) + 1e-30), (c, k, r)
            if r == 0.0:
                assert torch.equal(O_fma[0, 0, 0].cpu(), V[0, 0, 0]), (c, k)
            elif not torch.equal(O_fma[0, 0, 0].cpu(), V[0, 0, 0]):
                violations += 1
                # the backward on this saved state: exact dq_0 is zero; GProj returns exactly zero, the plain backward not
                dQ, _, _ = g.gproj_attn_bwd(Qd, Kd, Vd, O_fma, LSE_f, dO.cuda(), alpha, True)
                assert torch.all(dQ[0, 0, 0] == 0), (c, k)
    rc, detail = g.gproj_last_device_status()
    assert rc == 0, hex(detail)
    print("one-key violations with the fused exponent:", violations, "of 48")
    assert violations >= 3


def test_host_buffer_entry_point_matches_device_calls():
    # forward + backward from pinned host tensors: same kernels, so bit for bit the results of the device-pointer calls
    w = Workload("host", 2, 4, 320, 64, True, k_offset=4.0, seed=31, Hkv=2)
    inp = make_inputs(w)
    O, LSE, dQ, dK, dV = fwd_bwd(inp["Q"], inp["K"], inp["V"], inp["dO"], w.softmax_scale, True)
    host = {k: v.pin_memory() for k, v in inp.items()}
    hO = torch.empty_like(host["Q"]).pin_memory(); hL = torch.empty(w.B, w.H, w.N, dtype=torch.float32).pin_memory()
    hdQ = torch.empty_like(host["Q"]).pin_memory(); hdK = torch.empty_like(host["K"]).pin_memory(); hdV = torch.empty_like(host["K"]).pin_memory()
    staging = torch.empty(g.gproj_attn_host_staging_bytes(w.B, w.H, w.kv_heads, w.N, w.d), dtype=torch.uint8, device="cuda")
    g.gproj_attn_fwd_bwd_host(host["Q"], host["K"], host["V"], host["dO"], hdQ, hdK, hdV, w.softmax_scale, True, staging, O=hO, LSE=hL)
    rc, detail = g.gproj_last_device_status()      # synchronises the stream
    assert rc == 0, hex(detail)
    assert torch.equal(hO, O.cpu()) and torch.equal(hL, LSE.cpu())
    assert torch.equal(hdQ, dQ.cpu()) and torch.equal(hdK, dK.cpu()) and torch.equal(hdV, dV.cpu())
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(g.GprojError) as e:
        g.gproj_attn_fwd_bwd_host(host["Q"], host["K"], host["V"], host["dO"], hdQ, hdK, hdV, w.softmax_scale, True, small)
    assert e.value.status == -4


@pytest.mark.parametrize("shape", [(2, 8, 8, 2048, 64), (1, 10, 5, 8192, 64), (3, 2, 1, 16384, 128)])
def test_host_buffer_entry_point_pipelined_slabs(shape):
    # Problems above a few MiB are cut into slabs of KV heads whose copies overlap the kernels on internal streams
    # (2 even slabs; 2 slabs over 5 KV heads; 3 slabs of one KV head with two query heads each).  A slab may run the forward in
    # another tile mode than the whole problem, so the comparison with the device-pointer calls is to rounding, not bits;
    # a slab offset or ordering mistake is a gross error.  Two calls back to back on one stream reuse the staging buffer.
    B, H, Hkv, N, d = shape
    staging = torch.empty(g.gproj_attn_host_staging_bytes(B, H, Hkv, N, d), dtype=torch.uint8, device="cuda")
    pending = []
    for rep in range(2):
        w = Workload("host_slabs", B, H, N, d, True, k_offset=4.0, seed=57 + rep, Hkv=Hkv)
        inp = make_inputs(w)
        host = {k: v.pin_memory() for k, v in inp.items()}
        out = {"O": torch.empty_like(host["Q"]).pin_memory(), "LSE": torch.empty(B, H, N, dtype=torch.float32).pin_memory(),
               "dQ": torch.empty_like(host["Q"]).pin_memory(), "dK": torch.empty_like(host["K"]).pin_memory(),
               "dV": torch.empty_like(host["K"]).pin_memory()}
        for t in out.values():
            t.fill_(float("nan"))
        g.gproj_attn_fwd_bwd_host(host["Q"], host["K"], host["V"], host["dO"], out["dQ"], out["dK"], out["dV"], w.softmax_scale, True,
                                  staging, O=out["O"], LSE=out["LSE"])
        assert g.gproj_last_launch_count() >= 6          # at least two slabs of three kernels
        pending.append((w, inp, host, out))
    rc, detail = g.gproj_last_device_status()          # synchronises the stream, which waits for the last copy-out
    assert rc == 0, hex(detail)
    for w, inp, host, out in pending:
        O, LSE, dQ, dK, dV = fwd_bwd(inp["Q"], inp["K"], inp["V"], inp["dO"], w.softmax_scale, True)
        assert torch.allclose(out["LSE"], LSE.cpu(), rtol=1e-5, atol=1e-5)
        for name, ref in (("O", O), ("dQ", dQ), ("dK", dK), ("dV", dV)):
            got, ref = out[name].double(), ref.cpu().double()
            assert torch.isfinite(got).all(), name
            assert float((got - ref).norm() / ref.norm()) <= 2e-3, name


def test_cuda_graph_capture_and_replay():
    # The entry points only enqueue work on the given stream (no allocation, no synchronisation once the per-device
    # set-up of the first call is done), so forward + backward can be captured into a CUDA graph and replayed.
    w = Workload("graph", 1, 4, 512, 64, True, k_offset=4.0, seed=17)
    inp = {k: v.cuda() for k, v in make_inputs(w).items()}
    O = torch.empty_like(inp["Q"]); LSE = torch.empty(w.B, w.H, w.N, dtype=torch.float32, device="cuda")
    dQ, dK, dV = (torch.empty_like(inp["Q"]) for _ in range(3))
    ws = torch.empty(g.gproj_attn_bwd_workspace_bytes(w.B, w.H, w.N, w.d), dtype=torch.uint8, device="cuda")

    def step():
        g.gproj_attn_fwd(inp["Q"], inp["K"], inp["V"], w.softmax_scale, True, O=O, LSE=LSE)
        g.gproj_attn_bwd(inp["Q"], inp["K"], inp["V"], O, LSE, inp["dO"], w.softmax_scale, True, workspace=ws, dQ=dQ, dK=dK, dV=dV)

    step()                                               # eager: also performs the one-time set-up
    torch.cuda.synchronize()
    ref = [t.clone() for t in (O, LSE, dQ, dK, dV)]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()                                           # warm-up on the capture stream
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for t in (O, LSE, dQ, dK, dV):
        t.zero_()
    graph.replay()
    torch.cuda.synchronize()
    rc, detail = g.gproj_last_device_status()
    assert rc == 0, hex(detail)
    for a, b in zip(ref, (O, LSE, dQ, dK, dV)):
        assert torch.equal(a, b)


def test_two_streams_run_concurrently_without_interference():
    # Calls on different streams share nothing but the read-only per-device state (each launch carries its own tensor maps,
    # each call its own workspace): results equal those of the same calls run one after the other.
    ws = [Workload("s0", 1, 8, 1024, 64, True, k_offset=4.0, seed=41), Workload("s1", 2, 4, 640, 128, False, k_offset=8.0, seed=42)]
    inps = [{k: v.cuda() for k, v in make_inputs(w).items()} for w in ws]
    ref = [fwd_bwd(i["Q"], i["K"], i["V"], i["dO"], w.softmax_scale, w.causal) for w, i in zip(ws, inps)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    torch.cuda.synchronize()
    out = [None, None]
    for rep in range(3):
        for k, (w, i) in enumerate(zip(ws, inps)):
            with torch.cuda.stream(streams[k]):
                O, LSE = g.gproj_attn_fwd(i["Q"], i["K"], i["V"], w.softmax_scale, w.causal)
                out[k] = (O, LSE) + tuple(g.gproj_attn_bwd(i["Q"], i["K"], i["V"], O, LSE, i["dO"], w.softmax_scale, w.causal))
    torch.cuda.synchronize()
    rc, detail = g.gproj_last_device_status()
    assert rc == 0, hex(detail)
    for r, o in zip(ref, out):
        for a, b in zip(r, o):
            assert torch.equal(a, b)


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("causal", [False, True])
def test_row_maximum_that_creeps_up_across_key_tiles(d, causal):
    # The forward subtracts a lazily raised running maximum (raised only when a key tile exceeds it by more than 8 in
    # the base-two exponent domain).  Here every row's maximum grows a little with every key tile: by less than the
    # threshold from one tile to the next (so the stale reference is kept for several tiles and z exceeds one), but by
    # far more than it over the row.  O and LSE must stay inside the bars either way, and so must the fused variant,
    # which always takes the true running maximum.
    N, H = 2048, 2
    gen = torch.Generator().manual_seed(515 + d)
    Q, K, V, dO = (torch.randn(1, H, N, d, generator=gen) for _ in range(4))
    c = torch.randn(d, generator=gen); c = c / c.norm()
    alpha = float(np.float32(1 / math.sqrt(d)))
    ramp = torch.arange(N, dtype=torch.float32) / N                  # key j carries ramp_j * 40 / (alpha * 4) along c
    Q = Q * 0.5 + 4.0 * c
    K = K * 0.5 + (ramp[:, None] * (40.0 / (alpha * 4.0))) * c        # score grows by about 40 nats over the row, 2.5 per tile
    Q, K, V, dO = (t.to(torch.bfloat16) for t in (Q, K, V, dO))
    ex = oracle.attn_fwd_bwd_f64(bits(Q), bits(K), bits(V), bits(dO), alpha, causal)
    for fwd_flags in (0, g.FWD_FLAG_FMA_SOFTMAX):
        O, LSE = g.gproj_attn_fwd(Q.cuda(), K.cuda(), V.cuda(), alpha, causal, fwd_flags=fwd_flags)
        rc, detail = g.gproj_last_device_status()
        assert rc == 0, hex(detail)
        eO = oracle.rel_l2_percent(O.float().cpu().numpy(), ex["O"])
        dL = np.abs(LSE.cpu().numpy().astype(np.float64) - ex["LSE"])
        assert eO <= 1.0, (fwd_flags, eO)
        assert np.all(dL <= 1e-4 + 1e-5 * np.abs(ex["LSE"])), (fwd_flags, dL.max())
        if fwd_flags == 0:
            dQ, dK, dV = g.gproj_attn_bwd(Q.cuda(), K.cuda(), V.cuda(), O, LSE, dO.cuda(), alpha, causal)
            for n, t in (("dQ", dQ), ("dK", dK), ("dV", dV)):
                assert oracle.rel_l2_percent(t.float().cpu().numpy(), ex[n]) <= 1.0, n
    span = (ex["LSE"][0, 0, -1] - ex["LSE"][0, 0, 0]) if causal else None
    if causal:
        assert span > 20.0                                            # the construction does what it says
