"""The workspace-free backward entry point, through the C ABI.

The file name sorts behind every other test file, so pytest collects it last: a run that stops at the first failure
(-x) has then already run every other test before it reaches this added entry point.

Some users of this library cannot allocate device memory at the moment they need a gradient (a plugin inside
another framework's memory pool, a process whose memory is fixed at start-up).  For them the library carries its
backward scratch as a fixed device array.  This test checks that the entry point gives the same bytes as the
ordinary backward, twice in a row (the scratch keeps the previous call's contents), and that it refuses shapes
that do not fit.
"""
import ctypes

import pytest
import torch

import paper_2609_34272_b200 as g
from paper_2609_34272_b200 import binding
from paper_2609_34272_b200.workloads import Workload, make_inputs

pytestmark = pytest.mark.gpu


def _run_both(w, flags=0):
    inp = {k: v.cuda() for k, v in make_inputs(w).items()}
    O, LSE = g.gproj_attn_fwd(inp["Q"], inp["K"], inp["V"], w.softmax_scale, w.causal)
    ref = g.gproj_attn_bwd(inp["Q"], inp["K"], inp["V"], O, LSE, inp["dO"], w.softmax_scale, w.causal, flags=flags)
    got = g.gproj_attn_bwd_static_scratch(inp["Q"], inp["K"], inp["V"], O, LSE, inp["dO"], w.softmax_scale, w.causal, flags=flags)
    rc, detail = g.gproj_last_device_status()
    assert rc == 0, hex(detail)
    return ref, got


def test_static_scratch_matches_workspace_backward_twice_in_a_row():
    # two different problems back to back: the second call starts from the first call's leftovers in the scratch
    first = Workload("noalloc_a", 1, 2, 512, 64, True, k_offset=16.0, seed=11)
    second = Workload("noalloc_b", 2, 1, 384, 128, False, k_offset=4.0, seed=12)
    for w in (first, second):
        ref, got = _run_both(w)
        for name, a, b in zip(("dQ", "dK", "dV"), ref, got):
            # the tests' tolerance is 1 % relative L2 against the oracle; the two entry points run the same
            # kernels on the same data, so they must agree far inside it: bit for bit
            assert torch.equal(a, b), name
    ref, got = _run_both(first, flags=g.FLAG_NO_K_CORRECTION)
    assert all(torch.equal(a, b) for a, b in zip(ref, got))


def test_static_scratch_allocates_nothing_and_is_not_fooled_by_a_larger_earlier_call():
    # A large problem first (it fills most of the built-in array), then small ones of other shapes whose second kernel
    # also reads statistic blocks the first kernel does not write for them (d = 64, N mod 128 in 1..64): whatever the large
    # call left there must not reach a result.  With the outputs pre-allocated the call must leave both PyTorch's
    # allocator and the device's free memory exactly as they were -- that is what the entry point is for.
    big = Workload("noalloc_big", 1, 16, 4096, 64, True, k_offset=16.0, seed=21)
    _run_both(big)
    for w in (Workload("noalloc_s1", 1, 3, 192, 64, True, k_offset=8.0, seed=22), Workload("noalloc_s2", 2, 2, 320, 64, False, seed=23),
              Workload("noalloc_s3", 1, 2, 129, 128, True, seed=24)):
        inp = {k: v.cuda() for k, v in make_inputs(w).items()}
        O, LSE = g.gproj_attn_fwd(inp["Q"], inp["K"], inp["V"], w.softmax_scale, w.causal)
        ref = g.gproj_attn_bwd(inp["Q"], inp["K"], inp["V"], O, LSE, inp["dO"], w.softmax_scale, w.causal)
        out = [torch.empty_like(inp["Q"]) for _ in range(3)]
        g.gproj_attn_bwd_static_scratch(inp["Q"], inp["K"], inp["V"], O, LSE, inp["dO"], w.softmax_scale, w.causal,
                                        dQ=out[0], dK=out[1], dV=out[2])            # first call of the shape: any one-time set-up
        torch.cuda.synchronize()
        for t in out:
            t.zero_()
        torch.cuda.synchronize()
        allocated, reserved, free = torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), torch.cuda.mem_get_info()[0]
        g.gproj_attn_bwd_static_scratch(inp["Q"], inp["K"], inp["V"], O, LSE, inp["dO"], w.softmax_scale, w.causal,
                                        dQ=out[0], dK=out[1], dV=out[2])
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == allocated and torch.cuda.memory_reserved() == reserved
        assert torch.cuda.mem_get_info()[0] == free
        rc, detail = g.gproj_last_device_status()
        assert rc == 0, hex(detail)
        for name, a, b in zip(("dQ", "dK", "dV"), ref, out):
            assert torch.equal(a, b), (w.name, name)
    # a wrongly shaped output tensor is refused before anything is launched
    with pytest.raises(ValueError):
        g.gproj_attn_bwd_static_scratch(inp["Q"], inp["K"], inp["V"], O, LSE, inp["dO"], w.softmax_scale, w.causal,
                                        dQ=torch.empty(1, 1, 8, 128, dtype=torch.bfloat16, device="cuda"))


def test_static_scratch_rejects_shapes_beyond_its_size():
    lib = binding.load()
    p = ctypes.c_void_p(0x1000)      # never dereferenced: the size check comes first
    # workload 4 needs 264 MiB of scratch, far beyond the built-in 16 MiB
    assert g.gproj_attn_bwd_workspace_bytes(4, 32, 8192, 128) > binding.STATIC_SCRATCH_BYTES
    rc = lib.gproj_attn_bwd_static_scratch(p, p, p, p, p, p, p, p, p, 4, 32, 8192, 128, 0.0884, 0, 0, None)
    assert rc == -4
    # an unsupported head dimension is rejected by the shape check, again before any pointer is used
    rc = lib.gproj_attn_bwd_static_scratch(p, p, p, p, p, p, p, p, p, 1, 1, 128, 96, 0.125, 1, 0, None)
    assert rc == -2
