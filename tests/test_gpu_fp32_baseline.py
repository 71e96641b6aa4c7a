"""The fused FP32 comparison arm (plain FP32 arithmetic on the CUDA cores) against the FP64 oracle, through the C ABI.

Appendix "Accuracy and Cost", paragraph "Fused FP32 baseline": BF16 inputs decoded, FP32 arithmetic, BF16 outputs and
gradients, FP32 saved output and row statistics.  Its error is the final BF16 cast and little else: the paper's table
has 0.385 / 0.371 / 0.165 % (dQ / dK / dV) on its captures; on the synthetic workloads every tensor sits at the BF16
rounding floor of about 0.17 %, below the tensor-core path's 0.23 %, whose operands r, t are rounded as well.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_34272_b200 as g
from paper_2609_34272_b200.workloads import Workload, bits, make_inputs

pytestmark = pytest.mark.gpu


def run(w):
    inp = make_inputs(w)
    dev = {k: v.cuda() for k, v in inp.items()}
    O, saved = g.gproj_fp32_attn_fwd(dev["Q"], dev["K"], dev["V"], w.softmax_scale, w.causal)
    dQ, dK, dV = g.gproj_fp32_attn_bwd(dev["Q"], dev["K"], dev["V"], dev["dO"], saved, w.softmax_scale, w.causal)
    torch.cuda.synchronize()
    ex = oracle.attn_fwd_bwd_f64(*(bits(inp[k]) for k in ("Q", "K", "V", "dO")), w.softmax_scale, w.causal)
    rows = w.B * w.H * w.N
    stats = saved.view(torch.float32)[rows * w.d: rows * w.d + 3 * rows].reshape(w.B * w.H, 3, w.N)
    errs = {n: oracle.rel_l2_percent(t.float().cpu().numpy(), ex[n]) for n, t in (("O", O), ("dQ", dQ), ("dK", dK), ("dV", dV))}
    o32 = saved.view(torch.float32)[: rows * w.d].reshape(w.B, w.H, w.N, w.d).cpu().numpy()
    return errs, ex, stats.cpu().numpy(), o32, (inp, dev)


@pytest.mark.parametrize("B,H,N,d,causal,koff", [(1, 2, 256, 64, True, 8.0), (2, 2, 384, 128, False, 16.0), (1, 3, 200, 64, True, 32.0),
                                                  (1, 2, 129, 128, True, 0.0), (1, 1, 1, 64, True, 0.0), (1, 2, 1024, 64, True, 64.0)])
def test_fp32_arm_matches_the_oracle(B, H, N, d, causal, koff):
    w = Workload("fp32", B, H, N, d, causal, k_offset=koff, seed=808 + N + d)
    errs, ex, stats, o32, _ = run(w)
    print("fused FP32 arm:", {k: round(v, 4) for k, v in errs.items()})
    assert all(v <= 0.3 for v in errs.values()), errs                       # the BF16 cast of the results and nothing more
    # the saved FP32 state itself is far tighter than anything BF16 can hold
    lse = stats[:, 0].reshape(B, H, N)
    assert np.all(np.abs(lse - ex["LSE"]) <= 2e-5 + 2e-6 * np.abs(ex["LSE"]))
    assert oracle.rel_l2_percent(o32, ex["O"]) <= 2e-3
    assert np.allclose(stats[:, 0], stats[:, 1] - np.log(stats[:, 2]), rtol=0, atol=1e-4)      # lse = max + ln l, 1 / l saved


def test_fp32_arm_needs_no_correction_where_the_bf16_backward_breaks():
    # the attention-sink regime of the key-pass test: the uncorrected BF16 backward loses dQ and dK, the FP32 arm does not
    N, d = 512, 64
    gen = torch.Generator().manual_seed(4242 + d)
    Q, K, V, U = (torch.randn(N, d, generator=gen) for _ in range(4))
    c = torch.randn(d, generator=gen); c = c / c.norm()
    Q = Q + 8.0 * c
    K[0] = 0.1 * K[0] + 16.0 * c
    Q, K, V, U = (x.to(torch.bfloat16).reshape(1, 1, N, d) for x in (Q, K, V, U))
    ex = oracle.attn_fwd_bwd_f64(bits(Q), bits(K), bits(V), bits(U), 0.125, True)
    O, saved = g.gproj_fp32_attn_fwd(Q.cuda(), K.cuda(), V.cuda(), 0.125, True)
    dQ, dK, dV = g.gproj_fp32_attn_bwd(Q.cuda(), K.cuda(), V.cuda(), U.cuda(), saved, 0.125, True)
    e32 = {n: oracle.rel_l2_percent(t.float().cpu().numpy(), ex[n]) for n, t in (("dQ", dQ), ("dK", dK), ("dV", dV))}
    O2, LSE = g.gproj_attn_fwd(Q.cuda(), K.cuda(), V.cuda(), 0.125, True)
    off = g.gproj_attn_bwd(Q.cuda(), K.cuda(), V.cuda(), O2, LSE, U.cuda(), 0.125, True, flags=3)
    e_off = oracle.rel_l2_percent(off[0].float().cpu().numpy(), ex["dQ"])
    print("sink regime: fused FP32", {k: round(v, 3) for k, v in e32.items()}, "uncorrected BF16 dQ %.1f %%" % e_off)
    assert all(v <= 0.3 for v in e32.values()) and e_off > 20.0


def test_fp32_arm_argument_errors():
    x = torch.zeros(1, 1, 128, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(g.GprojError) as e:
        g.gproj_fp32_attn_fwd(x, x, x, 0.125, True, saved=torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == -4
    with pytest.raises(g.GprojError) as e:
        g.gproj_fp32_attn_fwd(x, x, x, float("nan"), True)
    assert e.value.status == -5
