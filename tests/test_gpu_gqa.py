"""Grouped-query attention on the GPU (through the C ABI) against the FP64 oracle.

The paper's own layout is 16 query / 4 KV heads with d = 64; key and value gradients sum over the query heads of a
group (Section 3.1).  Same bar as the other parity tests: full-tensor relative L2 <= 1 %.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_34272_b200 as g
from paper_2609_34272_b200.workloads import Workload, bits, make_inputs, workload

pytestmark = pytest.mark.gpu


def run(w, flags=0):
    inp = make_inputs(w)
    ex = oracle.attn_fwd_bwd_f64(*(bits(inp[k]) for k in ("Q", "K", "V", "dO")), w.softmax_scale, w.causal)
    dev = {k: v.cuda() for k, v in inp.items()}
    O, LSE = g.gproj_attn_fwd(dev["Q"], dev["K"], dev["V"], w.softmax_scale, w.causal)
    dQ, dK, dV = g.gproj_attn_bwd(dev["Q"], dev["K"], dev["V"], O, LSE, dev["dO"], w.softmax_scale, w.causal, flags=flags)
    rc, detail = g.gproj_last_device_status()
    assert rc == 0, hex(detail)
    assert dK.shape == dev["K"].shape and dV.shape == dev["V"].shape
    got = {"O": O, "dQ": dQ, "dK": dK, "dV": dV}
    errs = {n: oracle.rel_l2_percent(t.float().cpu().numpy(), ex[n]) for n, t in got.items()}
    assert np.all(np.abs(LSE.cpu().numpy() - ex["LSE"]) <= 1e-4 + 1e-5 * np.abs(ex["LSE"]))
    return errs, got


@pytest.mark.parametrize("B,H,Hkv,N,d,causal", [(2, 4, 2, 256, 64, True), (1, 8, 2, 384, 128, False), (1, 4, 1, 512, 64, True),
                                                 (1, 6, 3, 256, 128, True)])
def test_small_grouped_shapes(B, H, Hkv, N, d, causal):
    w = Workload("gqa_small", B, H, N, d, causal, k_offset=16.0, seed=900 + H * 7 + N, Hkv=Hkv)
    errs, _ = run(w)
    assert all(v <= 1.0 for v in errs.values()), errs


def test_paper_layout_16q_4kv():
    w = workload(6)
    errs, got = run(w)
    print("16q/4kv:", errs)
    assert all(v <= 1.0 for v in errs.values()), errs
    # each correction still changes only the gradient it targets
    _, off = run(w, flags=g.FLAG_NO_K_CORRECTION)
    assert torch.equal(off["dQ"], got["dQ"]) and torch.equal(off["dV"], got["dV"]) and not torch.equal(off["dK"], got["dK"])
