#!/usr/bin/env python
"""Benchmark of the fused attention forward + backward (GProj) path on B200.

One step = one forward and one backward over one batch of the synthetic workload.
  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 2] [--shard replicas|heads] [--impl reference]
For N > 1 launch with torch.distributed.run (one rank per GPU).  The path shards over (batch, head) with no
exchange: with `--shard replicas` (default) every rank runs the whole workload on its own GPU (weak scaling),
with `--shard heads` rank r runs the (batch, head) pairs shard_heads(B H, N, r) of ONE workload (strong
scaling).  The timed region is bracketed by a barrier and a device synchronize on both sides, and the reported
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
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of each kernel on the whole workload, keyed by
# (kernel, workload), from the ncu captures summarised under profiles/ (file named beside each entry)
NCU_DRAM_BYTES_PER_LAUNCH = {
    ("bwd_dkv_w128_kernel", 2): (44.1e6 + 1.1e6, "profiles/bwd_fwd_kernels_cfg2_ncu.md"),
    ("bwd_dq_kernel", 2): (42.3e6 + 0.7e6, "profiles/bwd_fwd_kernels_cfg2_ncu.md"),
    ("attn_fwd_kernel", 2): (25.2e6 + 0.0e6, "profiles/bwd_fwd_kernels_cfg2_ncu.md"),
    ("bwd_dkv_kernel", 4): (1351.9e6 + 516.8e6, "profiles/bwd_fwd_kernels_cfg4_dram_ncu.md"),
    ("bwd_dq_kernel", 4): (1347.8e6 + 521.5e6, "profiles/bwd_fwd_kernels_cfg4_dram_ncu.md"),
    ("attn_fwd_kernel", 4): (805.6e6 + 253.8e6, "profiles/bwd_fwd_kernels_cfg4_dram_ncu.md"),
    ("bwd_dkv_kernel", 5): (1552.6e6 + 110.8e6, "profiles/bwd_fwd_kernels_cfg4_dram_ncu.md"),
    ("bwd_dq_kernel", 5): (1057.8e6 + 114.4e6, "profiles/bwd_fwd_kernels_cfg4_dram_ncu.md"),
    ("attn_fwd_kernel", 5): (557.8e6 + 61.1e6, "profiles/bwd_fwd_kernels_cfg4_dram_ncu.md"),
}
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

    def __init__(self, index, period=0.002):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz, self.power_w = [], set(), None, []
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
                self.power_w.append(self.nv.nvmlDeviceGetPowerUsage(self.h) / 1e3)
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
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples),
                "power_w_median": (statistics.median(self.power_w) if self.power_w else None),
                "power_w_max": (max(self.power_w) if self.power_w else None)}


def flops(w):
    unit = w.gemm_unit_flops()
    return {"unit": unit, "fwd": 2 * unit, "bwd7": 7 * unit, "bwd5": 5 * unit, "bwd9": 9 * unit}


# Contractions per tile pair of each kernel: executed, and the share of the 7 the method itself needs (Algorithm 1: S, dP,
# dV, tK, rK, t^T Q, r^T Z).  The dQ side computes S, dP, tK, rK (all four are the method's); the dK/dV side computes S^T,
# dP^T again (recomputation of the two-kernel design) and dV, t^T Q, r^T Z (the method's).
KERNEL_UNITS = {"bwd_dq_kernel": (4, 4), "bwd_dkv_w128_kernel": (5, 3), "bwd_dkv_kernel": (5, 3), "attn_fwd_kernel": (2, 2)}


def stats_ms(xs):
    return {"mean": sum(xs) / len(xs), "median": statistics.median(xs), "min": min(xs)}


# --------------------------------------------------------------------------------------------
# reference arm: the FP64 oracle as it stands, on the host cores
# --------------------------------------------------------------------------------------------
def config_of(w, shard):
    """The `config` object of the JSON line; both arms print the same one."""
    return {"workload": w.name, "B": w.B, "H": w.H, "N": w.N, "d": w.d, "causal": w.causal,
            "key_offset_norm": w.k_offset, "query_offset_norm": w.q_offset,
            "per_gpu": ("one full workload per GPU" if shard == "replicas" else "a contiguous share of the (batch, head) pairs of one workload"),
            "l2": "512 MiB buffer rewritten before every timed step",
            "flop_convention": "7 contractions x 2 B H N^2 d x 0.5 (causal) for the backward"}


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
            "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps, "higher_is_better": True,
            "scaling": "weak" if args.shard == "replicas" else "strong",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config_of(w, args.shard),
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
    ap.add_argument("--shard", default="replicas", choices=["replicas", "heads"],
                    help="N > 1: every rank runs the whole workload (weak scaling) or its share of the (batch, head) pairs (strong)")
    ap.add_argument("--impl", default="gproj", choices=["gproj", "reference"])
    ap.add_argument("--sustained-seconds", type=float, default=2.0, help="length of the back-to-back region (0 = skip)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    args.warmup = max(args.warmup, 3)

    import torch
    import paper_2609_34272_b200 as g
    from paper_2609_34272_b200.sharding import max_over_ranks, init_process_group_from_env, shard_heads
    from paper_2609_34272_b200.workloads import bits, make_inputs, workload

    world, rank, local_rank = init_process_group_from_env(args.gpus)
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    peaks, peak_kind = load_peaks()

    w = workload(args.workload)
    fl = flops(w)
    host = {k: v.pin_memory() for k, v in make_inputs(w).items()}
    total_heads = w.B * w.H
    if args.shard == "heads" and world > 1:
        # strong scaling: this rank's contiguous share of the flat (batch, head) index; every pair is an independent
        # problem, so a share is itself a dense call with B = 1 and H = (pairs in the share)
        mine = shard_heads(total_heads, world, rank)
        host = {k: v.reshape(1, total_heads, w.N, w.d)[:, mine.start:mine.stop].contiguous().pin_memory() for k, v in host.items()}
        Bl, Hl = 1, len(mine)
        job_flops_scale = 1.0                    # the job is ONE workload
    else:
        Bl, Hl = w.B, w.H
        job_flops_scale = float(world)           # one workload per rank
    my_share = (Bl * Hl) / total_heads
    d_in = {k: v.to(dev) for k, v in host.items()}
    O = torch.empty_like(d_in["Q"]); LSE = torch.empty((Bl, Hl, w.N), dtype=torch.float32, device=dev)
    dQ, dK, dV = (torch.empty_like(d_in["Q"]) for _ in range(3))
    ws = torch.empty(max(256, g.gproj_attn_bwd_workspace_bytes(Bl, Hl, w.N, w.d)), dtype=torch.uint8, device=dev)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)      # > 126 MB L2
    a, c = w.softmax_scale, w.causal
    have_work = Hl > 0

    def fwd():
        if have_work:
            g.gproj_attn_fwd(d_in["Q"], d_in["K"], d_in["V"], a, c, O=O, LSE=LSE)

    def bwd(flags=0):
        if have_work:
            g.gproj_attn_bwd(d_in["Q"], d_in["K"], d_in["V"], O, LSE, d_in["dO"], a, c, flags=flags, workspace=ws, dQ=dQ, dK=dK, dV=dV)

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    stream = torch.cuda.current_stream()
    launches = [0]

    def timed_steps(nsteps, body, do_flush=True):
        """body(ev) records CUDA events on the launching stream; returns the per-step event tuples and the wall time."""
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(nsteps)]
        barrier()
        t0 = time.perf_counter()
        for i in range(nsteps):
            if do_flush:
                flush.zero_()                     # L2 flush between timed iterations (inputs fit in L2)
            body(evs[i])
        barrier()
        return evs, (time.perf_counter() - t0)

    def step_body(ev):
        ev[0].record(stream); fwd(); launches[0] += g.gproj_last_launch_count() if have_work else 0; ev[1].record(stream)
        ev[2].record(stream); bwd(); launches[0] += g.gproj_last_launch_count() if have_work else 0; ev[3].record(stream)

    for _ in range(args.warmup):
        flush.zero_(); fwd(); bwd()
    rc, detail = g.gproj_last_device_status()
    if rc != 0:
        raise RuntimeError(f"device status {g.status_string(rc)} {hex(detail)}")

    launches[0] = 0
    sampler = ClockSampler(local_rank)
    sampler.start()
    evs, wall = timed_steps(args.steps, step_body)
    clocks = sampler.stop()
    gpu_launches = launches[0]
    fwd_each = [e[0].elapsed_time(e[1]) for e in evs]
    bwd_each = [e[2].elapsed_time(e[3]) for e in evs]
    fwd_ms, bwd_ms = max_over_ranks(sum(fwd_each), world), max_over_ranks(sum(bwd_each), world)
    rc, detail = g.gproj_last_device_status()
    if rc != 0:
        raise RuntimeError(f"device status {g.status_string(rc)} {hex(detail)}")

    # each kernel alone, CUDA events around single launches (L2 flushed before each)
    dkv_name = "bwd_dkv_w128_kernel" if w.d == 64 else "bwd_dkv_kernel"
    n_k = max(10, min(args.steps, 50))

    def alone(fn):
        def body(ev):
            ev[0].record(stream); fn(); ev[1].record(stream)
        evk, _ = timed_steps(n_k, body)
        return max_over_ranks(sum(e[0].elapsed_time(e[1]) for e in evk), world) / n_k

    kernels_ms = {"bwd_dq_kernel": alone(lambda: bwd(g.FLAG_ONLY_DQ_PASS)), dkv_name: alone(lambda: bwd(g.FLAG_ONLY_DKV_PASS)),
                  "attn_fwd_kernel": alone(fwd)}

    # a second, long region: backward calls back to back (no L2 flush, no gaps) for a few seconds, with the SM clock
    # sampled throughout -- the rate the part sustains under its power limit, next to the burst number above
    sustained = None
    if args.sustained_seconds > 0 and have_work:
        per_call = max(1e-5, bwd_ms / args.steps / 1e3)
        chunk = max(10, int(0.02 / per_call))
        n_chunks = max(3, int(args.sustained_seconds / (chunk * per_call)) + 1)
        sampler2 = ClockSampler(local_rank, period=0.01)
        barrier()
        sampler2.start()
        marks = [torch.cuda.Event(enable_timing=True) for _ in range(n_chunks + 1)]
        marks[0].record(stream)
        for i in range(n_chunks):
            for _ in range(chunk):
                bwd()
            marks[i + 1].record(stream)
        barrier()
        clk2 = sampler2.stop()
        total_ms = max_over_ranks(marks[0].elapsed_time(marks[-1]), world)
        ms_call = total_ms / (n_chunks * chunk)
        tf = job_flops_scale * fl["bwd7"] / (ms_call / 1e3) / 1e12      # whole job; the slowest rank's time bounds every call
        sus_peak = peaks.get("bf16_tflops_sustained", FALLBACK_PEAKS["bf16_tflops_sustained"])
        sustained = {"what": "backward calls back to back, no L2 flush", "seconds": total_ms / 1e3, "calls": n_chunks * chunk,
                     "bwd_ms": ms_call, "bwd_tflops_7unit": tf, "bwd_tflops_9unit_executed": tf * 9 / 7,
                     "frac_of_bf16_sustained_peak": tf / world / sus_peak,
                     "frac_of_bf16_burst_peak": tf / world / peaks.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"]),
                     "clocks": clk2,
                     "mclk_per_call": (ms_call * 1e-3 * clk2["sm_mhz"]) if clk2.get("sm_mhz") else None}

    # end to end through the C ABI with host buffers (gproj_attn_fwd_bwd_host): H2D of Q, K, V, dO, forward, backward,
    # D2H of dQ, dK, dV, all inside the timed region
    e2e_ms = None
    tensor_bytes = Bl * Hl * w.N * w.d * 2
    if have_work:
        h_out = [torch.empty_like(host[k]).pin_memory() for k in ("Q", "K", "V")]
        staging = torch.empty(g.gproj_attn_host_staging_bytes(Bl, Hl, Hl, w.N, w.d), dtype=torch.uint8, device=dev)
        n_e2e = max(5, min(args.steps, 30))

        def e2e_body(ev):
            ev[0].record(stream)
            g.gproj_attn_fwd_bwd_host(host["Q"], host["K"], host["V"], host["dO"], h_out[0], h_out[1], h_out[2], a, c, staging)
            ev[1].record(stream)

        for _ in range(3):
            e2e_body([torch.cuda.Event(enable_timing=True) for _ in range(2)])
        eve, _ = timed_steps(n_e2e, e2e_body)
        e2e_ms = sum(e[0].elapsed_time(e[1]) for e in eve) / n_e2e
    e2e_ms = max_over_ranks(e2e_ms or 0.0, world)

    steps = args.steps
    bwd_t = bwd_ms / steps / 1e3
    fwd_t = fwd_ms / steps / 1e3
    job_bwd7 = job_flops_scale * fl["bwd7"]
    value = job_bwd7 / bwd_t / 1e12
    # Fractions are always quoted against the BURST bf16 GEMM figure (a kernel timed alone between L2 flushes); the
    # sustained figure is printed beside it and is the denominator of the `sustained` block only.
    burst = peaks.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"])
    sus = peaks.get("bf16_tflops_sustained", FALLBACK_PEAKS["bf16_tflops_sustained"])
    hbm_peak = peaks.get("hbm_gbs", FALLBACK_PEAKS["hbm_gbs"])
    per_gpu_tf = value / world

    # roofline of the dominant kernel = the longest of the three, chosen from this run's own times
    dom = max(kernels_ms, key=kernels_ms.get)
    u_exec, u_alg = KERNEL_UNITS[dom]
    share_unit = fl["unit"] * my_share
    dom_t = kernels_ms[dom] / 1e3
    traffic = NCU_DRAM_BYTES_PER_LAUNCH.get((dom, args.workload)) if my_share == 1.0 else None
    roofline = {"bound": "tensor", "kernel": dom, "unit": "TFLOP/s", "peak": burst,
                "peak_source": peak_kind + " (burst bf16 GEMM)",
                "algorithmic_flops_per_launch": u_alg * share_unit, "executed_flops_per_launch": u_exec * share_unit,
                "achieved": u_alg * share_unit / dom_t / 1e12, "frac": u_alg * share_unit / dom_t / 1e12 / burst,
                "achieved_executed": u_exec * share_unit / dom_t / 1e12, "frac_executed": u_exec * share_unit / dom_t / 1e12 / burst,
                "contractions": {"executed": u_exec, "algorithmic": u_alg,
                                 "note": "the dK/dV side recomputes S and dP (2 of its 5); the dQ side and the forward execute only the method's own"},
                "ms": kernels_ms[dom],
                "traffic": traffic[0] if traffic else None, "traffic_source": traffic[1] if traffic else None}
    # bytes the backward has to move: read Q, K, V, O, dO and LSE, write dQ, dK, dV
    alg_bytes = 16.0 * tensor_bytes / 2 + 4.0 * Bl * Hl * w.N
    ncu_bytes = [NCU_DRAM_BYTES_PER_LAUNCH.get((k, args.workload)) for k in ("bwd_dq_kernel", dkv_name)]
    hbm = {"bwd_algorithmic_bytes": alg_bytes, "bwd_gbs_algorithmic": alg_bytes / bwd_t / 1e9, "peak_gbs": hbm_peak,
           "frac_of_hbm_peak": alg_bytes / bwd_t / 1e9 / hbm_peak,
           "bwd_gbs_ncu": (sum(b[0] for b in ncu_bytes) / bwd_t / 1e9) if all(ncu_bytes) and my_share == 1.0 else None}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": args.warmup,
        "ms_per_step": (fwd_ms + bwd_ms) / steps, "higher_is_better": True,
        "scaling": "weak" if args.shard == "replicas" else "strong", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic", "config": config_of(w, args.shard),
        "bwd_ms": bwd_ms / steps, "fwd_ms": fwd_ms / steps,
        "bwd_ms_stats_this_rank": stats_ms(bwd_each), "fwd_ms_stats_this_rank": stats_ms(fwd_each),
        "bwd_tflops_7unit": value, "bwd_tflops_5unit_fa_convention": value * 5 / 7, "bwd_tflops_9unit_executed": value * 9 / 7,
        "fwd_tflops": job_flops_scale * fl["fwd"] / fwd_t / 1e12,
        "bwd_frac_of_bf16_peak": per_gpu_tf / burst, "bwd_frac_of_bf16_sustained_peak": per_gpu_tf / sus,
        "bwd_frac_of_bf16_peak_executed": per_gpu_tf * 9 / 7 / burst,
        "target": {"what": "backward >= 50 % of the measured burst bf16 peak (7-contraction count)", "met": bool(per_gpu_tf / burst >= 0.5)},
        "peaks": {"bf16_tflops_burst": burst, "bf16_tflops_sustained": sus, "hbm_gbs": hbm_peak, "source": peak_kind},
        "wall_ms_per_step_incl_l2_flush": 1e3 * wall / steps,
        "kernels_ms": kernels_ms, "roofline": roofline, "hbm": hbm, "sustained": sustained,
        "e2e": {"value": job_bwd7 / (e2e_ms / 1e3) / 1e12 if e2e_ms else None, "unit": UNIT, "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": 4 * tensor_bytes, "d2h_bytes_per_step": 3 * tensor_bytes,
                "what": "gproj_attn_fwd_bwd_host: pinned host Q,K,V,dO -> device, forward, backward, dQ,dK,dV -> pinned host (slabs of heads pipelined on internal copy streams); same FLOP count"},
        "gpu_launches": gpu_launches,
        "clocks": clocks,
    }

    if rank == 0 and not args.no_extras and args.workload == 2 and args.shard == "replicas":
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
                                  "bwd_frac_of_bf16_peak": fl3["bwd7"] / b3 / 1e12 / burst, "fwd_tflops": fl3["fwd"] / f3 / 1e12}}

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
            "bwd_frac_of_bf16_peak": 7 * unit_p / bp / 1e12 / burst, "fwd_tflops": 2 * unit_p / fp / 1e12,
            "note": "timed with output allocation inside the call (binding allocates O, LSE, dQ, dK, dV, workspace)"}

    if rank == 0 and not args.no_extras and args.workload == 2 and args.shard == "replicas":
        # the paper's fused FP32 comparison arm on the same workload (plain FP32 arithmetic on the CUDA cores), for context
        saved = torch.empty(g.binding.load().gproj_fp32_attn_saved_bytes(w.B, w.H, w.N, w.d), dtype=torch.uint8, device=dev)

        def body32(ev):
            ev[0].record(stream); g.gproj_fp32_attn_fwd(d_in["Q"], d_in["K"], d_in["V"], a, c, saved=saved); ev[1].record(stream)
            ev[2].record(stream); g.gproj_fp32_attn_bwd(d_in["Q"], d_in["K"], d_in["V"], d_in["dO"], saved, a, c); ev[3].record(stream)

        for _ in range(2):
            body32([torch.cuda.Event(enable_timing=True) for _ in range(4)])
        e32, _ = timed_steps(5, body32)
        f32 = sum(e[0].elapsed_time(e[1]) for e in e32) / 5
        b32 = sum(e[2].elapsed_time(e[3]) for e in e32) / 5
        line["also"]["fused_fp32_arm_" + w.name] = {
            "fwd_ms": f32, "bwd_ms": b32, "bwd_tflops_5unit": fl["bwd5"] / (b32 / 1e3) / 1e12, "fwd_tflops": fl["fwd"] / (f32 / 1e3) / 1e12,
            "step_ms_ratio_to_tensor_core_path": (f32 + b32) / ((fwd_ms + bwd_ms) / steps),
            "note": "comparison arm: FP32 FMAs on the CUDA cores, FP32 saved output; the paper's fused FP32 attention cost its training step +33 %"}

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
