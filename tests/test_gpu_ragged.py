"""GPU parity on sequence lengths that are not a multiple of the 128-row tile (through the C ABI).

The kernels round tiles and 64-row steps up; rows past N are zero-filled by the tensor-map loads and clipped by the
tensor-map stores, and key columns past N are masked where they would enter a row statistic.  Every case is compared
with the FP64 oracle on the full tensors (same bar as the tile-aligned parity tests), with more than one head so that
a tile reaching into the next head's rows would show.
"""
import os

import numpy as np
import pytest
import torch

import oracle
import paper_2609_34272_b200 as g
from oracle import emulation as em
from paper_2609_34272_b200.workloads import Workload, bits, from_bits, make_inputs

pytestmark = pytest.mark.gpu

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "witness_minus24.txt")


def to_np(t):
    return t.float().cpu().numpy().astype(np.float64)


def run_gpu(inp, alpha, causal, flags=0):
    dev = {k: v.cuda() for k, v in inp.items()}
    O, LSE = g.gproj_attn_fwd(dev["Q"], dev["K"], dev["V"], alpha, causal)
    dQ, dK, dV = g.gproj_attn_bwd(dev["Q"], dev["K"], dev["V"], O, LSE, dev["dO"], alpha, causal, flags=flags)
    rc, detail = g.gproj_last_device_status()
    assert rc == 0, (g.status_string(rc), hex(detail))
    return {"O": to_np(O), "LSE": LSE.cpu().numpy().astype(np.float64), "dQ": to_np(dQ), "dK": to_np(dK), "dV": to_np(dV)}


def check(got, ex, bar=1.0):
    errs = {}
    for n in ("O", "dQ", "dK", "dV"):
        assert got[n].shape == ex[n].shape
        assert np.all(np.isfinite(got[n])), n
        errs[n] = oracle.rel_l2_percent(got[n], ex[n])
        assert errs[n] <= bar, (n, errs)
        assert np.abs(got[n] - ex[n]).max() <= 0.03 * np.abs(ex[n]).max(), (n, "element-wise")
    assert np.all(np.abs(got["LSE"] - ex["LSE"]) <= 1e-4 + 1e-5 * np.abs(ex["LSE"]))
    return errs


# N: below one 64-row step, on and around step and tile boundaries, several tiles with a ragged tail
LENGTHS = [4, 63, 64, 65, 127, 129, 200, 320, 1000]


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("N", LENGTHS)
def test_ragged_lengths(N, d, causal):
    w = Workload("ragged", 2, 3, N, d, causal, k_offset=8.0, seed=5150 + 31 * N + d + (7 if causal else 0))
    inp = make_inputs(w)
    ex = oracle.attn_fwd_bwd_f64(*(bits(inp[k]) for k in ("Q", "K", "V", "dO")), w.softmax_scale, causal)
    check(run_gpu(inp, w.softmax_scale, causal), ex)


@pytest.mark.parametrize("causal", [True, False])
def test_ragged_grouped_queries(causal):
    w = Workload("ragged_gqa", 2, 4, 200, 64, causal, k_offset=8.0, seed=6160, Hkv=2)
    inp = make_inputs(w)
    ex = oracle.attn_fwd_bwd_f64(*(bits(inp[k]) for k in ("Q", "K", "V", "dO")), w.softmax_scale, causal)
    check(run_gpu(inp, w.softmax_scale, causal), ex)


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("d", [64, 128])
def test_single_token(d, causal):
    # N = 1: the row has one key, so O = v, LSE = alpha q.k, dV = dO, and the exact dQ and dK vanish.  With the
    # projection dQ is exactly zero (t k - (t / 1) (1 k)); dK keeps only the rounding of BF16(lambda q).
    w = Workload("one", 2, 2, 1, d, causal, k_offset=4.0, seed=77 + d)
    inp = make_inputs(w)
    got = run_gpu(inp, w.softmax_scale, causal)
    assert np.array_equal(got["O"], to_np(inp["V"]))
    assert np.array_equal(got["dV"], to_np(inp["dO"]))
    assert np.all(got["dQ"] == 0.0)
    assert np.abs(got["dK"]).max() <= 1e-4
    lse = w.softmax_scale * (to_np(inp["Q"]) * to_np(inp["K"])).sum(-1)
    assert np.all(np.abs(got["LSE"] - lse) <= 1e-4 + 1e-5 * np.abs(lse))


def test_uncorrected_backward_on_ragged_length():
    # the ablation flags take the same masked path
    w = Workload("ragged_off", 1, 2, 333, 64, True, k_offset=4.0, seed=99)
    inp = make_inputs(w)
    ex = oracle.attn_fwd_bwd_f64(*(bits(inp[k]) for k in ("Q", "K", "V", "dO")), w.softmax_scale, True)
    check(run_gpu(inp, w.softmax_scale, True, flags=3), ex, bar=5.0)


def test_minus24_witness_at_its_own_size():
    # The four-key witness of Appendix A ("An exact -24 witness") as an N = 4 problem, columns zero-padded to d = 64:
    # nothing but the four printed keys is in the row's support.
    vals = {}
    for line in open(GOLDEN):
        line = line.split("#", 1)[0].strip()
        if line:
            key, *rest = line.split()
            vals[key] = [float(x) for x in rest]
    N, d = 4, 64
    Q = np.zeros((N, d)); K = np.zeros((N, d)); V = np.zeros((N, d)); U = np.zeros((N, d))
    for j in range(4):
        K[j, :2] = vals[f"k{j + 1}"]
        V[j, :2] = vals[f"v{j + 1}"]
    U[:, :2] = vals["u"]
    inp = {n: from_bits(em.f64_to_bf16_bits(x)).reshape(1, 1, N, d) for n, x in (("Q", Q), ("K", K), ("V", V), ("dO", U))}
    alpha = vals["alpha"][0]
    on = run_gpu(inp, alpha, False)
    off = run_gpu(inp, alpha, False, flags=g.FLAG_NO_Q_CORRECTION)
    assert np.all(on["O"][0, 0, :, 0] == vals["o"][0]) and np.all(on["O"][0, 0, :, 1] == vals["o"][1])
    assert np.all(on["dQ"][0, 0, :, 0] == vals["dq0_gproj"][0])
    assert np.all(off["dQ"][0, 0, :, 0] == vals["dq0_uncorrected"][0])


def test_many_heads_short_sequences():
    # more (batch, head) problems than SMs, one tile each: exercises the tile -> (head, tile) decode of the persistent
    # schedule far from the benchmark shapes
    w = Workload("many_heads", 8, 40, 96, 64, True, k_offset=4.0, seed=4711)
    inp = make_inputs(w)
    ex = oracle.attn_fwd_bwd_f64(*(bits(inp[k]) for k in ("Q", "K", "V", "dO")), w.softmax_scale, True)
    check(run_gpu(inp, w.softmax_scale, True), ex)


@pytest.mark.parametrize("seed", range(6))
def test_random_shapes(seed):
    # seeded random shapes: lengths off every grid, head counts with and without grouping, both head dimensions
    rng = np.random.default_rng(1234 + seed)
    d = int(rng.choice([64, 128]))
    Hkv = int(rng.integers(1, 4))
    G = int(rng.choice([1, 1, 2, 3]))
    B = int(rng.integers(1, 3))
    N = int(rng.integers(2, 700))
    causal = bool(rng.integers(0, 2))
    w = Workload("rand", B, Hkv * G, N, d, causal, k_offset=float(rng.choice([0.0, 4.0, 16.0])), seed=900 + seed, Hkv=Hkv)
    inp = make_inputs(w)
    ex = oracle.attn_fwd_bwd_f64(*(bits(inp[k]) for k in ("Q", "K", "V", "dO")), w.softmax_scale, causal)
    print("shape", B, Hkv * G, Hkv, N, d, causal, check(run_gpu(inp, w.softmax_scale, causal), ex))


@pytest.mark.parametrize("d", [64, 128])
def test_many_heads_long_causal_matches_chunks_of_heads(d):
    # 40 heads x 8192 rows stream more than 64 MB of K / V: the kernels then deal groups of adjacent tiles per head (so
    # that concurrent CTAs share a head's rows in L2) instead of every head's longest tile first.  Scheduling must not
    # change a single bit of the backward: the same heads run in chunks of 8 (plain longest-first order) give identical
    # gradients from the same saved O and LSE; the forward, whose tile pairing may differ, agrees to rounding.
    B, H, N = 1, 40, 8192
    gen = torch.Generator().manual_seed(4040 + d)
    Q, K, V, dO = (torch.randn(B, H, N, d, generator=gen).to(torch.bfloat16).cuda() for _ in range(4))
    alpha = d ** -0.5
    O, LSE = g.gproj_attn_fwd(Q, K, V, alpha, True)
    dQ, dK, dV = g.gproj_attn_bwd(Q, K, V, O, LSE, dO, alpha, True)
    for h0 in range(0, H, 8):
        sl = slice(h0, h0 + 8)
        q, k, v, do, o, lse = (t[:, sl].contiguous() for t in (Q, K, V, dO, O, LSE))
        o2, lse2 = g.gproj_attn_fwd(q, k, v, alpha, True)
        assert torch.allclose(lse2, lse, rtol=1e-5, atol=1e-5)
        assert float((o2.float() - o.float()).abs().max()) <= 0.02 * float(o.float().abs().max())
        dq2, dk2, dv2 = g.gproj_attn_bwd(q, k, v, o, lse, do, alpha, True)
        assert torch.equal(dq2, dQ[:, sl]) and torch.equal(dk2, dK[:, sl]) and torch.equal(dv2, dV[:, sl]), h0
    rc, detail = g.gproj_last_device_status()
    assert rc == 0, hex(detail)


@pytest.mark.parametrize("d,causal", [(64, True), (128, False)])
def test_head_shards_give_the_bits_of_the_whole_call(d, causal):
    # The multi-GPU launch cuts the flat (batch, head) axis into contiguous shares (one per rank, no exchange).  Run the
    # shares one after the other on this GPU: laid side by side they must be the whole call's outputs bit for bit.
    from paper_2609_34272_b200.sharding import shard_heads
    B, H, N = 2, 5, 640
    gen = torch.Generator().manual_seed(606 + d)
    Q, K, V, dO = (torch.randn(B, H, N, d, generator=gen).to(torch.bfloat16).cuda() for _ in range(4))
    alpha = d ** -0.5
    O, LSE = g.gproj_attn_fwd(Q, K, V, alpha, causal)
    dQ, dK, dV = g.gproj_attn_bwd(Q, K, V, O, LSE, dO, alpha, causal)
    fl = lambda t: t.reshape((1, B * H) + t.shape[2:])
    for world in (2, 3, 4):
        for r in range(world):
            mine = shard_heads(B * H, world, r)
            q, k, v, u = (fl(t)[:, mine.start:mine.stop].contiguous() for t in (Q, K, V, dO))
            o, lse = g.gproj_attn_fwd(q, k, v, alpha, causal)
            dq, dk, dv = g.gproj_attn_bwd(q, k, v, o, lse, u, alpha, causal)
            sl = slice(mine.start, mine.stop)
            assert torch.equal(lse, fl(LSE)[:, sl]) or torch.allclose(lse, fl(LSE)[:, sl], rtol=1e-5, atol=1e-5)
            dq2, dk2, dv2 = g.gproj_attn_bwd(q, k, v, fl(O)[:, sl].contiguous(), fl(LSE)[:, sl].contiguous(), u, alpha, causal)
            assert torch.equal(dq2, fl(dQ)[:, sl]) and torch.equal(dk2, fl(dK)[:, sl]) and torch.equal(dv2, fl(dV)[:, sl]), (world, r)
    rc, detail = g.gproj_last_device_status()
    assert rc == 0, hex(detail)


@pytest.mark.parametrize("B,H,N,d,causal", [(2, 24, 1000, 64, True), (1, 160, 300, 64, False), (2, 80, 257, 128, True), (1, 300, 65, 64, True)])
def test_ragged_lengths_with_several_tiles_per_cta(B, H, N, d, causal):
    # More tiles than twice the SM count, with a ragged last tile in every head: a CTA walks three or more tiles, so the
    # per-tile hand-overs that only start at a CTA's second and third tile (row constants prepared one tile ahead in the
    # other stationary buffer, buffers reused across tiles) are exercised on ragged data.  The oracle runs on eight heads.
    w = Workload("ragged_many", B, H, N, d, causal, k_offset=8.0, seed=900 + N + H)
    inp = make_inputs(w)
    dev = {k: v.cuda() for k, v in inp.items()}
    O, LSE = g.gproj_attn_fwd(dev["Q"], dev["K"], dev["V"], w.softmax_scale, causal)
    dQ, dK, dV = g.gproj_attn_bwd(dev["Q"], dev["K"], dev["V"], O, LSE, dev["dO"], w.softmax_scale, causal)
    rc, detail = g.gproj_last_device_status()
    assert rc == 0, (g.status_string(rc), hex(detail))
    rng = np.random.default_rng(N + H)
    for hh in sorted(set(rng.integers(0, B * H, size=6).tolist()) | {0, B * H - 1}):
        b, h = divmod(hh, H)
        one = lambda t: t[b:b + 1, h:h + 1]
        ex = oracle.attn_fwd_bwd_f64(*(bits(one(inp[k])) for k in ("Q", "K", "V", "dO")), w.softmax_scale, causal)
        got = {"O": to_np(one(O)), "LSE": LSE[b:b + 1, h:h + 1].cpu().numpy().astype(np.float64),
               "dQ": to_np(one(dQ)), "dK": to_np(one(dK)), "dV": to_np(one(dV))}
        check(got, ex)
