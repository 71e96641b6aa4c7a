"""The synthetic offset sweep of Fig. 1, panel 2, on the GPU kernels (through the C ABI).

Appendix "Gauge Projection: Proofs", paragraph "Synthetic offset sweep": 256 query rows, L = 1024 keys k_j = z_j + b in
d = 64 dimensions, z_j ~ N(0, I), a common translation b with norm from 1 to 1e4, logits with standard deviation 3,
standard-normal values and upstream derivative; the translation leaves p, g and the exact dQ unchanged, the projected
contraction stays at a floor of 0.12-0.17 % and the direct one grows linearly with the offset.

Reading taken here: the paper's sweep is an FP64 emulation whose only rounding is t = BF16(g); the kernels take BF16
inputs, and BF16(z + b) would lose z altogether for a large b along a random direction.  So b lies along one coordinate
axis (that coordinate of z is lost, the other 63 are kept), and the reference is the exact FP64 VJP at those BF16 inputs.
"""
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2609_34272_b200 as g
from paper_2609_34272_b200.workloads import bits

pytestmark = pytest.mark.gpu

OFFSETS = (1.0, 10.0, 1e2, 1e3, 1e4)


def sweep_inputs(offset, seed=2609):
    Nq, L, d = 256, 1024, 64
    gen = torch.Generator().manual_seed(seed)
    z = torch.randn(1, 1, L, d, generator=gen)
    Q = 3.0 * torch.randn(1, 1, Nq, d, generator=gen)          # alpha q . z has standard deviation alpha * 3 * sqrt(64) = 3
    V = torch.randn(1, 1, L, d, generator=gen)
    dO = torch.randn(1, 1, Nq, d, generator=gen)
    K = z.clone()
    K[..., 0] += offset
    return [t.to(torch.bfloat16) for t in (Q, K, V, dO)]


def test_offset_sweep_projected_curve_is_flat_and_direct_curve_grows_linearly():
    alpha = 0.125
    rows = []
    for b in OFFSETS:
        Q, K, V, dO = sweep_inputs(b)
        ex = oracle.attn_rect_f64(bits(Q), bits(K), bits(V), bits(dO), alpha, False)
        Qd, Kd, Vd, Ud = (t.cuda() for t in (Q, K, V, dO))
        O, LSE = g.gproj_attn_fwd_rect(Qd, Kd, Vd, alpha, False)
        on = g.gproj_attn_bwd_rect(Qd, Kd, Vd, O, LSE, Ud, alpha, False)
        off = g.gproj_attn_bwd_rect(Qd, Kd, Vd, O, LSE, Ud, alpha, False, flags=3)
        rc, detail = g.gproj_last_device_status()
        assert rc == 0, hex(detail)
        err = lambda t, n: oracle.rel_l2_percent(t.float().cpu().numpy(), ex[n])
        rows.append({"offset": b, "dQ_gproj": err(on[0], "dQ"), "dQ_direct": err(off[0], "dQ"), "dK_gproj": err(on[1], "dK"),
                     "dK_direct": err(off[1], "dK"), "dV": err(on[2], "dV"), "O": err(O, "O")})
        print({k: (round(v, 4) if k != "offset" else v) for k, v in rows[-1].items()})
    proj = np.array([r["dQ_gproj"] for r in rows]); direct = np.array([r["dQ_direct"] for r in rows])
    assert np.all(proj <= 1.0) and all(r["dK_gproj"] <= 1.0 and r["dV"] <= 1.0 and r["O"] <= 1.0 for r in rows)
    assert proj.max() <= 2.5 * proj.min()                               # flat (paper: a floor of 0.12-0.17 %)
    # linear growth of the direct contraction once the leak dominates: a decade in the offset is a decade in the error
    assert direct[2] > 3 * proj[2]
    assert direct[3] / direct[2] == pytest.approx(10.0, rel=0.25) and direct[4] / direct[3] == pytest.approx(10.0, rel=0.25)
    assert direct[4] > 100 * proj[4]
