"""The backward's scratch memory may hold anything on entry (through the C ABI).

The dQ-side kernel writes the row statistics and the scaled-query operand that the dK/dV-side kernel reads.  At
d = 64 the second kernel fetches two 64-row statistic blocks per step, so for lengths with N mod 128 in 1..64 it also
reads a block the first kernel never wrote for that step (the spare block, or the next head's); those words belong to
masked columns.  A workspace full of 0xFF bytes (NaN patterns: ordinary arithmetic, nothing faults) must therefore
give the same bits as a zeroed one.
"""
import numpy as np
import pytest
import torch

import paper_2609_34272_b200 as g
from paper_2609_34272_b200 import binding
from paper_2609_34272_b200.workloads import Workload, make_inputs

pytestmark = pytest.mark.gpu


def _dense(N, d, causal, fill, H=3):
    w = Workload("ws", 1, H, N, d, causal, k_offset=8.0, seed=900 + N + d)
    inp = {k: v.cuda() for k, v in make_inputs(w).items()}
    O, LSE = g.gproj_attn_fwd(inp["Q"], inp["K"], inp["V"], w.softmax_scale, causal)
    ws = torch.full((g.gproj_attn_bwd_workspace_bytes(1, H, N, d) + 4096,), fill, dtype=torch.uint8, device="cuda")
    out = g.gproj_attn_bwd(inp["Q"], inp["K"], inp["V"], O, LSE, inp["dO"], w.softmax_scale, causal, workspace=ws)
    rc, detail = g.gproj_last_device_status()
    assert rc == 0, hex(detail)
    return out


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("N", [192, 320, 64, 129])
@pytest.mark.parametrize("causal", [True, False])
def test_dense_backward_ignores_what_the_workspace_held(N, d, causal):
    zero = _dense(N, d, causal, 0)
    poison = _dense(N, d, causal, 0xFF)
    for name, a, b in zip(("dQ", "dK", "dV"), zero, poison):
        assert torch.equal(a, b), name
        assert torch.isfinite(b.float()).all(), name


@pytest.mark.parametrize("d", [64, 128])
def test_packed_backward_ignores_what_the_workspace_held(d):
    lens = [192, 320, 1, 65, 200]
    H, Hkv = 4, 2
    gen = torch.Generator().manual_seed(77 + d)
    T = sum(lens)
    Q, dO = (torch.randn(H, T, d, generator=gen).to(torch.bfloat16).cuda() for _ in range(2))
    K, V = (torch.randn(Hkv, T, d, generator=gen).to(torch.bfloat16).cuda() for _ in range(2))
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    for causal in (True, False):
        plan = g.VarlenPlan(cu, causal)
        O, LSE = g.gproj_attn_fwd_varlen(Q, K, V, plan, 0.125)
        outs = []
        for fill in (0, 0xFF):
            need = int(binding.load().gproj_attn_bwd_varlen_workspace_bytes(plan.cu, plan.num_seqs, H, d))
            ws = torch.full((need + 4096,), fill, dtype=torch.uint8, device="cuda")
            outs.append(g.gproj_attn_bwd_varlen(Q, K, V, O, LSE, dO, plan, 0.125, workspace=ws))
        rc, detail = g.gproj_last_device_status()
        assert rc == 0, hex(detail)
        for name, a, b in zip(("dQ", "dK", "dV"), *outs):
            assert torch.equal(a, b), (name, causal)
            assert torch.isfinite(b.float()).all(), (name, causal)
