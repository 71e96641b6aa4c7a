#!/usr/bin/env python
"""Benchmark of the fused attention forward + backward (GProj) path on B200.

One step = one forward and one backward over one batch of the synthetic workload.
  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 2] [--impl reference]
For N > 1 launch with torch.distributed.run (one rank per GPU); every rank runs the same
independent problem on its own GPU (the path shards over (batch, head) with no exchange), the
timed region is bracketed by a barrier and a device synchronize on both sides, and the reported
time is the maximum over ranks.

Headline `value`: backward TFLOP/s, counting the 7 contractions Algorithm 1 needs per tile pair
(S, dP, dV, tK, rK, t^T Q, r^T Z; causal x 0.5), divided by the CUDA-event time of the backward call
(both kernels).  The 5-contraction FlashAttention convention is printed next to it.
"""
import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "fused attn bwd TFLOP/s & % BF16 tensor peak; dQ/dK/dV rel-L2 vs FP64"
UNIT = "TFLOP/s"
# dram__bytes_read.sum + dram__bytes_write.sum of one launch, from the ncu capture summarised under profiles/
NCU_DRAM_BYTES_PER_LAUNCH = {("bwd_dkv_kernel", 2): 42.519e6 + 0.696e6, ("bwd_dkv_kernel", 3): 42.252e6 + 0.861e6,
                             ("bwd_dkv_kernel", 4): 1351.866e6 + 516.820e6}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons through NVML (read only) while the timed region runs."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index, period=0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        while not self._stop_evt.is_set():
            try:
                self.samples.append(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
                mask = self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=2)
        return {"sm_mhz": (statistics.median(self.samples) if self.samples else None),
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def flops(w):
    unit = w.gemm_unit_flops()
    return {"fwd": 2 * unit, "bwd7": 7 * unit, "bwd5": 5 * unit, "dkv_kernel": 5 * unit, "dq_kernel": 4 * unit}


# --------------------------------------------------------------------------------------------
# reference arm: the FP64 oracle as it stands, on the host cores
# --------------------------------------------------------------------------------------------
def oracle_sample(w, inp_bits, heads):
    import oracle
    t0 = time.perf_counter()
    oracle.attn_fwd_bwd_f64(inp_bits["Q"], inp_bits["K"], inp_bits["V"], inp_bits["dO"], w.softmax_scale, w.causal, heads=heads)
    return time.perf_counter() - t0


def run_reference(args):
    import oracle
    from paper_2609_34272_b200.workloads import bits, make_inputs, workload
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = workload(args.workload)
    inp = make_inputs(w)
    b = {k: bits(v) for k, v in inp.items()}
    per_head = flops(w)["bwd7"] / (w.B * w.H)
    heads = [0]
    for _ in range(args.warmup):
        oracle_sample(w, b, heads)
    times = [oracle_sample(w, b, heads) for _ in range(args.steps)]
    total = sum(times)
    value = per_head * len(heads) * args.steps / total / 1e12
    sample = (f"{len(heads)} of {w.B * w.H} (batch, head) problems of {w.name} per step, FP64 forward + backward; "
              f"FLOPs counted as the 7-contraction backward of the sample")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "B": w.B, "H": w.H, "N": w.N, "d": w.d, "causal": w.causal, "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# --------------------------------------------------------------------------------------------
# the CUDA path
# --------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", type=int, default=2, help="1..5 (default 2: B=1 H=16 N=4096 d=64 causal)")
    ap.add_argument("--impl", default="gproj", choices=["gproj", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    args.warmup = max(args.warmup, 3)

    import torch
    import paper_2609_34272_b200 as g
    from paper_2609_34272_b200.sharding import max_over_ranks, init_process_group_from_env
    from paper_2609_34272_b200.workloads import bits, make_inputs, workload

    world, rank, local_rank = init_process_group_from_env(args.gpus)
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    peaks, peak_kind = load_peaks()

    w = workload(args.workload)
    fl = flops(w)
    host = {k: v.pin_memory() for k, v in make_inputs(w).items()}
    d_in = {k: v.to(dev) for k, v in host.items()}
    O = torch.empty_like(d_in["Q"]); LSE = torch.empty((w.B, w.H, w.N), dtype=torch.float32, device=dev)
    dQ, dK, dV = (torch.empty_like(d_in["Q"]) for _ in range(3))
    ws = torch.empty(max(256, g.gproj_attn_bwd_workspace_bytes(w.B, w.H, w.N, w.d)), dtype=torch.uint8, device=dev)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)      # > 126 MB L2
    a, c = w.softmax_scale, w.causal

    def fwd():
        g.gproj_attn_fwd(d_in["Q"], d_in["K"], d_in["V"], a, c, O=O, LSE=LSE)

    def bwd(flags=0):
        g.gproj_attn_bwd(d_in["Q"], d_in["K"], d_in["V"], O, LSE, d_in["dO"], a, c, flags=flags, workspace=ws, dQ=dQ, dK=dK, dV=dV)

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    stream = torch.cuda.current_stream()

    def timed_steps(nsteps, body):
        """body(i, ev) records CUDA events on the launching stream; returns list of per-step event tuples."""
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(nsteps)]
        barrier()
        t0 = time.perf_counter()
        for i in range(nsteps):
            flush.zero_()                         # L2 flush between timed iterations (inputs fit in L2)
            body(evs[i])
        barrier()
        return evs, (time.perf_counter() - t0)

    def step_body(ev):
        ev[0].record(stream); fwd(); ev[1].record(stream)
        ev[2].record(stream); bwd(); ev[3].record(stream)

    for _ in range(args.warmup):
        flush.zero_(); fwd(); bwd()
    rc, detail = g.gproj_last_device_status()
    if rc != 0:
        raise RuntimeError(f"device status {g.status_string(rc)} {hex(detail)}")

    sampler = ClockSampler(local_rank)
    sampler.start()
    evs, wall = timed_steps(args.steps, step_body)
    clocks = sampler.stop()
    fwd_ms = sum(e[0].elapsed_time(e[1]) for e in evs)
    bwd_ms = sum(e[2].elapsed_time(e[3]) for e in evs)
    fwd_ms, bwd_ms = max_over_ranks(fwd_ms, world), max_over_ranks(bwd_ms, world)
    rc, detail = g.gproj_last_device_status()
    if rc != 0:
        raise RuntimeError(f"device status {g.status_string(rc)} {hex(detail)}")

    # dominant kernel alone (dK/dV side; 5 of the 9 executed contractions), CUDA events around single launches
    def dkv_body(ev):
        ev[0].record(stream); bwd(g.FLAG_ONLY_DKV_PASS); ev[1].record(stream)

    def dq_body(ev):
        ev[0].record(stream); bwd(g.FLAG_ONLY_DQ_PASS); ev[1].record(stream)

    n_k = max(10, min(args.steps, 50))
    evk, _ = timed_steps(n_k, dq_body)
    dq_ms = max_over_ranks(sum(e[0].elapsed_time(e[1]) for e in evk), world) / n_k
    evk, _ = timed_steps(n_k, dkv_body)
    dkv_ms = max_over_ranks(sum(e[0].elapsed_time(e[1]) for e in evk), world) / n_k

    # end to end through the C ABI with host buffers (gproj_attn_fwd_bwd_host): H2D of Q, K, V, dO, forward, backward,
    # D2H of dQ, dK, dV, all inside the timed region
    h_out = [torch.empty_like(host[k]).pin_memory() for k in ("Q", "K", "V")]
    staging = torch.empty(g.gproj_attn_host_staging_bytes(w.B, w.H, w.kv_heads, w.N, w.d), dtype=torch.uint8, device=dev)
    n_e2e = max(5, min(args.steps, 30))

    def e2e_body(ev):
        ev[0].record(stream)
        g.gproj_attn_fwd_bwd_host(host["Q"], host["K"], host["V"], host["dO"], h_out[0], h_out[1], h_out[2], a, c, staging)
        ev[1].record(stream)

    for _ in range(3):
        e2e_body([torch.cuda.Event(enable_timing=True) for _ in range(2)])
    eve, _ = timed_steps(n_e2e, e2e_body)
    e2e_ms = max_over_ranks(sum(e[0].elapsed_time(e[1]) for e in eve), world) / n_e2e
    tensor_bytes = w.elements * 2

    steps = args.steps
    bwd_t = bwd_ms / steps / 1e3
    fwd_t = fwd_ms / steps / 1e3
    value = world * fl["bwd7"] / bwd_t / 1e12
    # Denominator: the burst GEMM figure for kernels timed alone (workloads 1-3: 0.1 ms launches between L2 flushes); the
    # sustained figure when the run itself sat under the power cap (workloads 4, 5: tens of ms per step, clocks sampled).
    capped = "sw_power_cap" in (clocks.get("reasons") or [])
    peak_key = "bf16_tflops_sustained" if capped else "bf16_tflops"
    peak = peaks.get(peak_key, FALLBACK_PEAKS[peak_key])
    dkv_achieved = fl["dkv_kernel"] / (dkv_ms / 1e3) / 1e12

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": args.warmup,
        "ms_per_step": (fwd_ms + bwd_ms) / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "H": w.H, "N": w.N, "d": w.d, "causal": w.causal,
                   "key_offset_norm": w.k_offset, "query_offset_norm": w.q_offset, "per_gpu": "one full workload per GPU",
                   "l2": "512 MiB buffer rewritten before every timed step",
                   "flop_convention": "7 contractions x 2 B H N^2 d x 0.5 (causal) for the backward"},
        "bwd_ms": bwd_ms / steps, "fwd_ms": fwd_ms / steps,
        "bwd_tflops_7unit": value, "bwd_tflops_5unit_fa_convention": world * fl["bwd5"] / bwd_t / 1e12,
        "fwd_tflops": world * fl["fwd"] / fwd_t / 1e12,
        "bwd_frac_of_bf16_peak": value / world / peak, "peak_source": peak_kind,
        "wall_ms_per_step_incl_l2_flush": 1e3 * wall / steps,
        "kernels_ms": {"bwd_dq_kernel": dq_ms, ("bwd_dkv_w128_kernel" if w.d == 64 else "bwd_dkv_kernel"): dkv_ms},
        "roofline": {"bound": "tensor", "kernel": "bwd_dkv_w128_kernel" if w.d == 64 else "bwd_dkv_kernel", "achieved": dkv_achieved, "peak": peak, "unit": "TFLOP/s",
                     "frac": dkv_achieved / peak, "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get(("bwd_dkv_kernel", args.workload)),
                     "peak_source": peak_kind + (" (sustained bf16 GEMM, run was power-capped)" if capped else " (burst bf16 GEMM)"),
                     "algorithmic_flops_per_launch": fl["dkv_kernel"]},
        "e2e": {"value": world * fl["bwd7"] / (e2e_ms / 1e3) / 1e12, "unit": UNIT, "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": 4 * tensor_bytes, "d2h_bytes_per_step": 3 * tensor_bytes,
                "what": "gproj_attn_fwd_bwd_host: pinned host Q,K,V,dO -> device, forward, backward, dQ,dK,dV -> pinned host (slabs of heads pipelined on internal copy streams); same FLOP count"},
        "gpu_launches": 3 * steps,
        "clocks": clocks,
    }

    if rank == 0 and not args.no_extras and args.workload == 2:
        # the other 4096-token workload (d = 128), few iterations, for context
        w3 = workload(3)
        i3 = {k: v.to(dev) for k, v in make_inputs(w3).items()}
        O3 = torch.empty_like(i3["Q"]); L3 = torch.empty((w3.B, w3.H, w3.N), dtype=torch.float32, device=dev)
        g3 = [torch.empty_like(i3["Q"]) for _ in range(3)]
        ws3 = torch.empty(g.gproj_attn_bwd_workspace_bytes(w3.B, w3.H, w3.N, w3.d), dtype=torch.uint8, device=dev)

        def body3(ev):
            ev[0].record(stream); g.gproj_attn_fwd(i3["Q"], i3["K"], i3["V"], w3.softmax_scale, True, O=O3, LSE=L3); ev[1].record(stream)
            ev[2].record(stream)
            g.gproj_attn_bwd(i3["Q"], i3["K"], i3["V"], O3, L3, i3["dO"], w3.softmax_scale, True, workspace=ws3, dQ=g3[0], dK=g3[1], dV=g3[2])
            ev[3].record(stream)

        for _ in range(3):
            body3([torch.cuda.Event(enable_timing=True) for _ in range(4)])
        e3, _ = timed_steps(30, body3)
        f3 = sum(e[0].elapsed_time(e[1]) for e in e3) / 30 / 1e3
        b3 = sum(e[2].elapsed_time(e[3]) for e in e3) / 30 / 1e3
        fl3 = flops(w3)
        line["also"] = {w3.name: {"bwd_ms": b3 * 1e3, "fwd_ms": f3 * 1e3, "bwd_tflops_7unit": fl3["bwd7"] / b3 / 1e12,
                                  "bwd_frac_of_bf16_peak": fl3["bwd7"] / b3 / 1e12 / peak, "fwd_tflops": fl3["fwd"] / f3 / 1e12}}

        # the paper's own layout for context: four packed 4096-token causal sequences, 16 query / 4 KV heads, d = 64
        lens, Hq, Hkv, dd = [4096] * 4, 16, 4, 64
        T = sum(lens)
        gen = torch.Generator().manual_seed(260934272 + 9000)
        pk = {n: torch.randn((Hq if n in ("Q", "dO") else Hkv, T, dd), generator=gen).to(torch.bfloat16).to(dev) for n in ("Q", "K", "V", "dO")}
        cu = [0]
        for n in lens:
            cu.append(cu[-1] + n)
        plan = g.VarlenPlan(cu, True, device=dev)

        def bodyp(ev):
            ev[0].record(stream); Op, Lp = g.gproj_attn_fwd_varlen(pk["Q"], pk["K"], pk["V"], plan, 0.125); ev[1].record(stream)
            ev[2].record(stream); g.gproj_attn_bwd_varlen(pk["Q"], pk["K"], pk["V"], Op, Lp, pk["dO"], plan, 0.125); ev[3].record(stream)

        for _ in range(3):
            bodyp([torch.cuda.Event(enable_timing=True) for _ in range(4)])
        ep, _ = timed_steps(20, bodyp)
        fp = sum(e[0].elapsed_time(e[1]) for e in ep) / 20 / 1e3
        bp = sum(e[2].elapsed_time(e[3]) for e in ep) / 20 / 1e3
        unit_p = sum(2.0 * Hq * n * n * dd * 0.5 for n in lens)
        line["also"]["packed_4x4096_causal_h16_kv4_d64"] = {
            "bwd_ms": bp * 1e3, "fwd_ms": fp * 1e3, "bwd_tflops_7unit": 7 * unit_p / bp / 1e12,
            "bwd_frac_of_bf16_peak": 7 * unit_p / bp / 1e12 / peak, "fwd_tflops": 2 * unit_p / fp / 1e12,
            "note": "timed with output allocation inside the call (binding allocates O, LSE, dQ, dK, dV, workspace)"}

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        b = {k: bits(v) for k, v in host.items()}
        heads = list(range(min(4, w.B * w.H)))
        secs = oracle_sample(w, b, heads)
        line["cpu_baseline"] = {"value": fl["bwd7"] / (w.B * w.H) * len(heads) / secs / 1e12, "unit": UNIT,
                                "cores": oracle.num_threads(), "kind": "oracle", "seconds": secs,
                                "sample": f"{len(heads)} of {w.B * w.H} (batch, head) problems of {w.name}, FP64 forward + backward, "
                                          f"FLOPs counted as the 7-contraction backward of the sample"}

    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
