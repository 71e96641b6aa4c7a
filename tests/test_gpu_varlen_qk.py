"""GPU parity on packed sequences whose query and key lengths differ, through the C ABI.

Appendix "Synthetic Numerical Suite" lists packed segments, unequal lengths and empty causal rows.  Sequence s owns
query rows cu_q[s] .. cu_q[s+1]-1 of [H, Tq, d] and key rows cu_k[s] .. cu_k[s+1]-1 of [Hkv, Tk, d]; causal means query
i sees the keys j <= i + (Lk - Lq) of its own sequence.  The oracle (the unequal-length one, which knows nothing of
packing) is run sequence by sequence and the results laid side by side; a sequence without queries must get zero key
and value gradients, one without keys zero outputs and LSE = +inf.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_34272_b200 as g

pytestmark = pytest.mark.gpu


def f64(t):
    return t.float().cpu().numpy().astype(np.float64)


def tobits(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def make(H, Hkv, lq, lk, d, seed):
    gen = torch.Generator().manual_seed(seed)
    Tq, Tk = sum(lq), sum(lk)
    Q = torch.randn(H, Tq, d, generator=gen)
    K = torch.randn(Hkv, Tk, d, generator=gen) + 0.5
    V = torch.randn(Hkv, Tk, d, generator=gen)
    dO = torch.randn(H, Tq, d, generator=gen)
    return {n: t.to(torch.bfloat16).contiguous() for n, t in (("Q", Q), ("K", K), ("V", V), ("dO", dO))}


def oracle_packed(inp, lq, lk, alpha, causal):
    H, Tq, d = inp["Q"].shape
    Hkv, Tk = inp["K"].shape[:2]
    out = {"O": np.zeros((H, Tq, d)), "LSE": np.full((H, Tq), np.inf), "dQ": np.zeros((H, Tq, d)),
           "dK": np.zeros((Hkv, Tk, d)), "dV": np.zeros((Hkv, Tk, d))}
    q0 = k0 = 0
    for nq, nk in zip(lq, lk):
        if nq > 0 and nk > 0:
            sq, sk = slice(q0, q0 + nq), slice(k0, k0 + nk)
            ex = oracle.attn_rect_f64(tobits(inp["Q"][:, sq].unsqueeze(0)), tobits(inp["K"][:, sk].unsqueeze(0)),
                                      tobits(inp["V"][:, sk].unsqueeze(0)), tobits(inp["dO"][:, sq].unsqueeze(0)), alpha, causal)
            for n in ("O", "LSE", "dQ"):
                out[n][:, sq] = ex[n][0]
            for n in ("dK", "dV"):
                out[n][:, sk] = ex[n][0]
        q0 += nq; k0 += nk
    return out


def run_gpu(inp, lq, lk, alpha, causal, flags=0):
    cu_q = np.concatenate([[0], np.cumsum(lq)]); cu_k = np.concatenate([[0], np.cumsum(lk)])
    plan = g.VarlenPlan(cu_q, causal, cu_seqlens_k=cu_k)
    dev = {k: v.cuda() for k, v in inp.items()}
    O, LSE = g.gproj_attn_fwd_varlen_qk(dev["Q"], dev["K"], dev["V"], plan, alpha)
    dQ, dK, dV = g.gproj_attn_bwd_varlen_qk(dev["Q"], dev["K"], dev["V"], O, LSE, dev["dO"], plan, alpha, flags=flags)
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
        assert np.all(np.isfinite(got[n])), n
        errs[n] = oracle.rel_l2_percent(got[n], ex[n])
        assert errs[n] <= bar, (n, errs)
        assert np.abs(got[n] - ex[n]).max() <= 0.03 * np.abs(ex[n]).max(), (n, "element-wise")
    return errs


CASES = [  # (query lengths, key lengths)
    ([100, 300, 30, 257], [300, 130, 64, 257]),          # fewer / more queries than keys, ragged everywhere
    ([128, 1, 200], [256, 500, 1]),                      # aligned; one query against many keys; many queries, one key
    ([70, 0, 200, 40], [200, 50, 90, 0]),                # a sequence without queries, one without keys
    ([0, 333], [128, 100]),                              # the first sequence has keys only
    ([64, 64, 64, 64, 64], [640, 64, 1, 130, 300]),      # five short query blocks behind key histories
]


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("case", range(len(CASES)))
def test_packed_unequal_lengths(case, d, causal):
    lq, lk = CASES[case]
    inp = make(2, 2, lq, lk, d, seed=100 * case + d)
    ex = oracle_packed(inp, lq, lk, d ** -0.5, causal)
    got = run_gpu(inp, lq, lk, d ** -0.5, causal)
    check(got, ex)
    q0 = k0 = 0
    for nq, nk in zip(lq, lk):
        if nq == 0:        # keys nobody asks for: exact zeros, not rounding residue
            assert np.all(got["dK"][:, k0:k0 + nk] == 0.0) and np.all(got["dV"][:, k0:k0 + nk] == 0.0)
        q0 += nq; k0 += nk


@pytest.mark.parametrize("causal", [True, False])
def test_packed_unequal_lengths_grouped_queries(causal):
    lq, lk = [300, 77, 512], [512, 300, 100]
    inp = make(6, 2, lq, lk, 64, seed=7)
    ex = oracle_packed(inp, lq, lk, 0.125, causal)
    check(run_gpu(inp, lq, lk, 0.125, causal), ex)


@pytest.mark.parametrize("d", [64, 128])
def test_one_sequence_equals_the_dense_unequal_call_bit_for_bit(d):
    lq, lk = [333], [500]
    inp = make(3, 3, lq, lk, d, seed=21 + d)
    got = run_gpu(inp, lq, lk, d ** -0.5, True)
    q, k, v, do = (inp[n].cuda().unsqueeze(0) for n in ("Q", "K", "V", "dO"))
    O, LSE = g.gproj_attn_fwd_rect(q, k, v, d ** -0.5, True)
    dQ, dK, dV = g.gproj_attn_bwd_rect(q, k, v, O, LSE, do, d ** -0.5, True)
    # the dense call pairs query tiles in the forward when there are enough of them; three heads of three tiles are not
    for n, t in (("dQ", dQ), ("dK", dK), ("dV", dV), ("O", O)):
        assert np.array_equal(got[n], f64(t[0])), n


def test_equal_offsets_equal_the_packed_call_bit_for_bit():
    lens = [100, 300, 257]
    inp = make(2, 2, lens, lens, 64, seed=5)
    got = run_gpu(inp, lens, lens, 0.125, True)
    cu = np.concatenate([[0], np.cumsum(lens)])
    plan = g.VarlenPlan(cu, True)
    dev = {k: v.cuda() for k, v in inp.items()}
    O, LSE = g.gproj_attn_fwd_varlen(dev["Q"], dev["K"], dev["V"], plan, 0.125)
    dQ, dK, dV = g.gproj_attn_bwd_varlen(dev["Q"], dev["K"], dev["V"], O, LSE, dev["dO"], plan, 0.125)
    for n, t in (("O", O), ("dQ", dQ), ("dK", dK), ("dV", dV)):
        assert np.array_equal(got[n], f64(t)), n


@pytest.mark.parametrize("seed", range(4))
def test_random_packings(seed):
    rng = np.random.default_rng(77 + seed)
    S = int(rng.integers(2, 7))
    lq = [int(x) for x in rng.integers(0, 400, S)]
    lk = [int(x) for x in rng.integers(0, 400, S)]
    lq[0] = max(lq[0], 1); lk[-1] = max(lk[-1], 1)
    d = int(rng.choice([64, 128])); Hkv = int(rng.integers(1, 3)); G = int(rng.choice([1, 2]))
    causal = bool(rng.integers(0, 2))
    inp = make(Hkv * G, Hkv, lq, lk, d, seed=seed)
    ex = oracle_packed(inp, lq, lk, d ** -0.5, causal)
    print("packing", lq, lk, d, Hkv * G, Hkv, causal, check(run_gpu(inp, lq, lk, d ** -0.5, causal), ex))
