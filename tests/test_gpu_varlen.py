"""GPU parity on packed (variable-length) sequences, through the C ABI.

Several sequences share the row axis of [H, T, d] tensors; a query attends only inside its own sequence.  The oracle is
run sequence by sequence on the slices (it knows nothing of packing) and the results are laid side by side.  Lengths are
chosen off the 64 / 128 grid so that tiles reach into the next sequence's rows: those rows must be masked as keys and as
queries and must not be written.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_34272_b200 as g
from paper_2609_34272_b200.workloads import bits

pytestmark = pytest.mark.gpu


def to_np(t):
    return t.float().cpu().numpy().astype(np.float64)


def make_packed(H, Hkv, lens, d, seed, koff=8.0):
    gen = torch.Generator().manual_seed(seed)
    T = sum(lens)
    Q = torch.randn(H, T, d, generator=gen)
    K = torch.randn(Hkv, T, d, generator=gen)
    V = torch.randn(Hkv, T, d, generator=gen)
    dO = torch.randn(H, T, d, generator=gen)
    c = torch.randn(Hkv, 1, d, generator=gen)
    K = K + c / c.norm(dim=-1, keepdim=True) * koff          # a common key offset per head, as in the dense workloads
    return {n: t.to(torch.bfloat16).contiguous() for n, t in (("Q", Q), ("K", K), ("V", V), ("dO", dO))}


def oracle_packed(inp, lens, alpha, causal):
    H, T, d = inp["Q"].shape
    Hkv = inp["K"].shape[0]
    out = {"O": np.zeros((H, T, d)), "LSE": np.zeros((H, T)), "dQ": np.zeros((H, T, d)),
           "dK": np.zeros((Hkv, T, d)), "dV": np.zeros((Hkv, T, d))}
    r0 = 0
    for n in lens:
        if n > 0:
            sl = slice(r0, r0 + n)
            ex = oracle.attn_fwd_bwd_f64(*(bits(inp[k][:, sl].contiguous().unsqueeze(0)) for k in ("Q", "K", "V", "dO")), alpha, causal)
            for k in out:
                out[k][:, sl] = ex[k][0]
        r0 += n
    return out


def run_gpu(inp, lens, alpha, causal, flags=0):
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    plan = g.VarlenPlan(cu, causal)
    dev = {k: v.cuda() for k, v in inp.items()}
    O, LSE = g.gproj_attn_fwd_varlen(dev["Q"], dev["K"], dev["V"], plan, alpha)
    dQ, dK, dV = g.gproj_attn_bwd_varlen(dev["Q"], dev["K"], dev["V"], O, LSE, dev["dO"], plan, alpha, flags=flags)
    rc, detail = g.gproj_last_device_status()
    assert rc == 0, (g.status_string(rc), hex(detail))
    return {"O": to_np(O), "LSE": LSE.cpu().numpy().astype(np.float64), "dQ": to_np(dQ), "dK": to_np(dK), "dV": to_np(dV)}


def check(got, ex, bar=1.0):
    errs = {}
    for n in ("O", "dQ", "dK", "dV"):
        assert np.all(np.isfinite(got[n])), n
        errs[n] = oracle.rel_l2_percent(got[n], ex[n])
        assert errs[n] <= bar, (n, errs)
        assert np.abs(got[n] - ex[n]).max() <= 0.03 * np.abs(ex[n]).max(), (n, "element-wise")
    assert np.all(np.abs(got["LSE"] - ex["LSE"]) <= 1e-4 + 1e-5 * np.abs(ex["LSE"]))
    return errs


CASES = [  # lengths: singleton, below a step, across steps and tiles, an empty sequence, tile-aligned, long
    [1, 5, 64, 100, 128, 129, 300, 0, 257],
    [200, 200, 200],
    [128, 256, 384],
    [700],
    [3, 1000, 17],
]


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("lens", CASES)
def test_packed_sequences(lens, d, causal):
    inp = make_packed(3, 3, lens, d, seed=8800 + sum(lens) + d + (1 if causal else 0))
    alpha = float(np.float32(d ** -0.5))
    check(run_gpu(inp, lens, alpha, causal), oracle_packed(inp, lens, alpha, causal))


@pytest.mark.parametrize("causal", [True, False])
def test_packed_grouped_queries(causal):
    lens = [70, 333, 129]
    inp = make_packed(4, 2, lens, 64, seed=9901)
    check(run_gpu(inp, lens, 0.125, causal), oracle_packed(inp, lens, 0.125, causal))


def test_packed_equals_dense_for_one_sequence():
    # one sequence filling the whole row axis is the dense problem with B = 1: same kernels, same arithmetic, same bits
    lens = [384]
    inp = make_packed(2, 2, lens, 64, seed=5)
    got = run_gpu(inp, lens, 0.125, True)
    dev = {k: v.cuda().unsqueeze(0) for k, v in inp.items()}
    O, LSE = g.gproj_attn_fwd(dev["Q"], dev["K"], dev["V"], 0.125, True)
    dQ, dK, dV = g.gproj_attn_bwd(dev["Q"], dev["K"], dev["V"], O, LSE, dev["dO"], 0.125, True)
    for name, t in (("O", O), ("dQ", dQ), ("dK", dK), ("dV", dV)):
        assert np.array_equal(got[name], to_np(t[0])), name


def test_sequences_do_not_leak_into_each_other():
    # changing one sequence's data must leave every other sequence's results bit for bit unchanged
    lens = [100, 150, 90]
    inp = make_packed(2, 2, lens, 64, seed=77)
    base = run_gpu(inp, lens, 0.125, True)
    inp2 = {k: v.clone() for k, v in inp.items()}
    for k in inp2:
        inp2[k][:, 100:250] = (inp2[k][:, 100:250].float() * 1.5 + 0.25).to(torch.bfloat16)
    other = run_gpu(inp2, lens, 0.125, True)
    keep = np.r_[0:100, 250:340]
    for name in ("O", "dQ", "dK", "dV"):
        assert np.array_equal(base[name][:, keep], other[name][:, keep]), name
        assert not np.array_equal(base[name][:, 100:250], other[name][:, 100:250]), name


def test_malformed_cu_seqlens_is_rejected():
    for bad in ([1, 5], [0, 5, 3], [0, 0]):
        with pytest.raises(g.GprojError):
            g.VarlenPlan(bad, True)


@pytest.mark.parametrize("seed", range(10))
def test_random_packings(seed):
    rng = np.random.default_rng(4321 + seed)
    d = int(rng.choice([64, 128]))
    Hkv = int(rng.integers(1, 3))
    G = int(rng.choice([1, 2]))
    lens = [int(x) for x in rng.integers(0, 400, size=int(rng.integers(2, 7)))]
    lens = [0 if n == 1 else n for n in lens]      # one-token sequences (exact zero dQ, dK) have their own dense test
    if sum(lens) == 0:
        lens[0] = 17
    causal = bool(rng.integers(0, 2))
    inp = make_packed(Hkv * G, Hkv, lens, d, seed=7000 + seed)
    alpha = float(np.float32(d ** -0.5))
    print("packing", lens, Hkv * G, Hkv, d, causal, check(run_gpu(inp, lens, alpha, causal), oracle_packed(inp, lens, alpha, causal)))


@pytest.mark.parametrize("d", [64, 128])
def test_many_short_sequences_repeat_bitwise(d):
    # Hundreds of one- and two-step tiles per CTA: tile boundaries dominate, where the kernels hand buffers over between
    # tiles (stationary tiles, the saved-output rows copied ahead for the next tile, statistics, accumulators).  A wrong
    # hand-over shows as a result that depends on timing: forty repetitions must give the same bits, and those bits must
    # pass the oracle.
    rng = np.random.default_rng(2718 + d)
    lens = [int(x) for x in rng.integers(1, 200, 260)]
    inp = make_packed(8, 4, lens, d, seed=99 + d, koff=4.0)
    alpha = d ** -0.5
    first = run_gpu(inp, lens, alpha, True)
    check(first, oracle_packed(inp, lens, alpha, True))
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    plan = g.VarlenPlan(cu, True)
    dev = {k: v.cuda() for k, v in inp.items()}
    ws = torch.empty(int(g.binding.load().gproj_attn_bwd_varlen_workspace_bytes(plan.cu, plan.num_seqs, 8, d)), dtype=torch.uint8, device="cuda")
    for _ in range(40):
        O, LSE = g.gproj_attn_fwd_varlen(dev["Q"], dev["K"], dev["V"], plan, alpha)
        dQ, dK, dV = g.gproj_attn_bwd_varlen(dev["Q"], dev["K"], dev["V"], O, LSE, dev["dO"], plan, alpha, workspace=ws)
        for n, t in (("O", O), ("dQ", dQ), ("dK", dK), ("dV", dV)):
            assert np.array_equal(to_np(t), first[n]), n
    rc, detail = g.gproj_last_device_status()
    assert rc == 0, hex(detail)
