"""CPU-only checks of the C-ABI library: it loads, exports what the header declares, and rejects
bad arguments before touching CUDA."""
import ctypes
import os
import re

import pytest

import __graft_entry__ as entry
from paper_2609_34272_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    entry.build()
    return binding.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "gproj_attn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gproj_[a-z_0-9]+)\s*\(", text)))


def test_header_and_exports_agree(lib):
    names = declared_functions()
    assert set(names) == set(binding.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_status_strings(lib):
    assert binding.status_string(0) == "ok"
    for code in range(-9, 0):
        assert binding.status_string(code) not in ("ok", "unknown status")
    assert binding.status_string(-99) == "unknown status"


def test_workspace_bytes(lib):
    # one BF16 query-shaped array + the row constants (LSE, D) in 64-row blocks plus one spare block (the paper's "Cost"
    # paragraph allows more): the constants travel as a 16-column BF16 operand tile of the dK/dV side's score products,
    # 32 B per row, 2048 B per block.
    B, H, N = 2, 3, 256
    rows = B * H * N
    for d in (64, 128):
        assert binding.gproj_attn_bwd_workspace_bytes(B, H, N, d) == rows * 32 + 2048 + rows * d * 2
        # ragged length: the blocks are padded to whole 64-row blocks per head (2 blocks + the spare), the query-shaped array is not
        assert binding.gproj_attn_bwd_workspace_bytes(1, 1, 100, d) == 3 * 2048 + 100 * d * 2
    assert binding.gproj_attn_bwd_workspace_bytes(1, 1, 0, 64) == 0
    assert binding.gproj_attn_bwd_workspace_bytes(1, 1, 128, 96) == 0


def test_argument_validation_without_gpu(lib):
    p = ctypes.c_void_p(0x1000)        # never dereferenced: validation fails first
    bad = ctypes.c_void_p(0x1008)
    fwd = lambda Q=p, LSE=p, B=1, H=1, N=128, d=64, scale=0.125: lib.gproj_attn_fwd(Q, p, p, p, LSE, B, H, N, d, scale, 1, None)
    assert fwd(Q=None) == -1
    assert fwd(N=-128) == -2 and fwd(d=96) == -2 and fwd(B=0) == -2 and fwd(N=0) == -2
    assert fwd(Q=bad) == -3
    assert fwd(scale=0.0) == -5 and fwd(scale=float("nan")) == -5 and fwd(scale=-1.0) == -5
    bwd = lambda ws=ctypes.c_void_p(0x1000), nbytes=1 << 30, flags=0, dQ=p: lib.gproj_attn_bwd(
        p, p, p, p, p, p, dQ, p, p, 1, 1, 128, 64, 0.125, 1, ws, nbytes, flags, None)
    assert bwd(dQ=None) == -1
    assert bwd(flags=16) == -9 and bwd(flags=12) == -9
    assert bwd(ws=None) == -4 and bwd(nbytes=16) == -4 and bwd(ws=ctypes.c_void_p(0x1010)) == -4


def test_python_binding_refuses_cpu_tensors():
    import torch
    x = torch.zeros(1, 1, 128, 64, dtype=torch.bfloat16)
    with pytest.raises(TypeError):
        binding.gproj_attn_fwd(x, x, x, 0.125, True)


def test_varlen_plan_on_host(lib):
    # the plan is host arithmetic: every 128-row tile of every non-empty sequence exactly once in each of the two orders,
    # longest work first, statistic blocks numbered sequence after sequence; two int4 per tile, the second one the range
    # of the other operand (here the same rows: equal query and key lengths)
    import numpy as np
    cu = [0, 1, 6, 70, 70, 470, 598]
    arr = (ctypes.c_int * len(cu))(*cu)
    S = len(cu) - 1
    lens = np.diff(cu)
    n_tiles = int(sum((l + 127) // 128 for l in lens))
    nbytes = lib.gproj_attn_varlen_plan_bytes(arr, S)
    assert nbytes == 2 * n_tiles * 32
    for causal in (0, 1):
        buf = np.zeros(2 * n_tiles * 8, dtype=np.int32)
        assert lib.gproj_attn_varlen_plan(arr, S, causal, buf.ctypes.data_as(ctypes.c_void_p), nbytes) == 0
        plan = buf.reshape(2, n_tiles, 8)
        expect = set()
        blk = 0
        for s in range(S):
            for t in range((lens[s] + 127) // 128):
                expect.add((cu[s] + 128 * t, cu[s], cu[s + 1], blk, cu[s], cu[s + 1], 0, 0))
            blk += (lens[s] + 63) // 64
        for order in range(2):
            assert set(map(tuple, plan[order].tolist())) == expect and len(plan[order]) == len(expect)
        work_q = [min(r0 + 128, e) - s0 if causal else e - s0 for r0, s0, e, *_ in plan[0]]
        work_kv = [e - r0 if causal else e - s0 for r0, s0, e, *_ in plan[1]]
        assert work_q == sorted(work_q, reverse=True) and work_kv == sorted(work_kv, reverse=True)
    assert lib.gproj_attn_varlen_plan(arr, S, 1, None, nbytes) == -1
    assert lib.gproj_attn_varlen_plan(arr, S, 1, ctypes.c_void_p(0x1000), 16) == -4
    bad = (ctypes.c_int * 3)(0, 5, 3)
    assert lib.gproj_attn_varlen_plan_bytes(bad, 2) == 0 and lib.gproj_attn_varlen_plan(bad, 2, 1, None, 0) == -2


def test_varlen_qk_plan_on_host(lib):
    # separate query and key offsets: query tiles of every sequence with queries, key tiles of every sequence with both;
    # a query tile's work is the keys its last row sees, a key tile's the queries from the first one that sees it
    import numpy as np
    cu_q = [0, 100, 100, 400, 430, 431]
    cu_k = [0, 300, 350, 480, 480, 1000]      # (100, 300), (0, 50), (300, 130), (30, 0), (1, 520)
    aq = (ctypes.c_int * len(cu_q))(*cu_q); ak = (ctypes.c_int * len(cu_k))(*cu_k)
    S = len(cu_q) - 1
    lq, lk = np.diff(cu_q), np.diff(cu_k)
    n_q = int(sum((l + 127) // 128 for l in lq))
    n_k = int(sum((k + 127) // 128 for q, k in zip(lq, lk) if q > 0))
    nbytes = lib.gproj_attn_varlen_qk_plan_bytes(aq, ak, S)
    assert nbytes == (n_q + n_k) * 32
    for causal in (0, 1):
        buf = np.zeros((n_q + n_k) * 8, dtype=np.int32)
        assert lib.gproj_attn_varlen_qk_plan(aq, ak, S, causal, buf.ctypes.data_as(ctypes.c_void_p), nbytes) == 0
        plan = buf.reshape(n_q + n_k, 8)
        exp_q, exp_k, blk = set(), set(), 0
        for s in range(S):
            for t in range((lq[s] + 127) // 128):
                exp_q.add((cu_q[s] + 128 * t, cu_q[s], cu_q[s + 1], blk, cu_k[s], cu_k[s + 1], 0, 0))
            if lq[s] > 0:
                for t in range((lk[s] + 127) // 128):
                    exp_k.add((cu_k[s] + 128 * t, cu_k[s], cu_k[s + 1], blk, cu_q[s], cu_q[s + 1], 0, 0))
            blk += (lq[s] + 63) // 64
        assert set(map(tuple, plan[:n_q].tolist())) == exp_q and set(map(tuple, plan[n_q:].tolist())) == exp_k

        def keys_seen(r0, s0, e, _b, k0, k1, *_):
            off = (k1 - k0) - (e - s0)
            return max(0, min(k1 - k0, min(r0 + 128, e) - s0 + off)) if causal else k1 - k0

        def queries_seeing(r0, s0, e, _b, q0, q1, *_):
            off = (e - s0) - (q1 - q0)
            return max(0, (q1 - q0) - max(0, r0 - s0 - off)) if causal else q1 - q0

        wq = [keys_seen(*r) for r in plan[:n_q].tolist()]
        wk = [queries_seeing(*r) for r in plan[n_q:].tolist()]
        assert wq == sorted(wq, reverse=True) and wk == sorted(wk, reverse=True)
    short = (ctypes.c_int * 2)(0, 0)
    assert lib.gproj_attn_varlen_qk_plan_bytes(aq, short, 1) == 0        # no keys at all
