#!/usr/bin/env python
"""Benchmark of the MoE layer forward under an expert placement (route -> dispatch -> grouped SwiGLU
expert FFN -> combine -> placement cost) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config c2_mixtral] [--impl ours|reference]

One "step" is one pass of the whole layer over one batch of seeded synthetic input.  The default
workload is the Mixtral-8x7B-shaped layer (4096 tokens, hidden 4096, 8 experts top-2, FFN 14336, 8
logical ranks, the two hottest experts replicated).  Prints ONE JSON line (rank 0).

With N > 1 (launched under torch.distributed.run) every rank runs an independent replica of the layer on
its own GPU - the path has no inter-GPU exchange - and the value is the aggregate over ranks divided by
the slowest rank's time ("weak" scaling).

--impl reference times the CPU oracle (the plain fp64 restatement of the method) on the host cores, on a
bounded sample of the same workload per step.
"""
from __future__ import annotations

import argparse
import json
import os
import signal
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "moe_layer_tokens_per_s"
UNIT = "tokens/s"

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of the dominant kernel, from the
# committed ncu summary of that kernel on that workload (None until a capture for the workload exists).
NCU_TRAFFIC_BYTES = {
    # gate||up GEMM, full-size workload: 1 955 644 416 B read + 229 357 568 B written
    "c2_mixtral": 2185001984,
}


# ------------------------------------------------------------------------------------------------
# clock sampling (child process; NVML, read only)
# ------------------------------------------------------------------------------------------------

REASON_BITS = {
    0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
    0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
    0x100: "display_clock_setting",
}


def _sample_clocks_main(uuid: str, out_path: str, period_s: float = 0.001):
    """Child process: polls SM clock, power and clock-event reasons of one GPU until SIGTERM."""
    import pynvml
    pynvml.nvmlInit()
    h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if isinstance(uuid, str) else uuid)
    stop = {"now": False}
    signal.signal(signal.SIGTERM, lambda *_: stop.__setitem__("now", True))
    max_sm = pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM)
    with open(out_path, "w") as f:
        f.write(f"max {max_sm}\n")
        while not stop["now"]:
            sm = pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)
            try:
                reasons = pynvml.nvmlDeviceGetCurrentClocksEventReasons(h)
            except Exception:
                reasons = pynvml.nvmlDeviceGetCurrentClocksThrottleReasons(h)
            try:
                power = pynvml.nvmlDeviceGetPowerUsage(h) / 1000.0
            except Exception:
                power = -1.0
            f.write(f"{time.time():.4f} {sm} {reasons} {power:.1f}\n")
            time.sleep(period_s)


class ClockSampler:
    def __init__(self, uuid: str):
        self.path = tempfile.mktemp(prefix="director_clocks_", suffix=".txt")
        self.proc = subprocess.Popen([sys.executable, os.path.abspath(__file__), "--sample-clocks", uuid, self.path],
                                     stdout=subprocess.DEVNULL, stderr=subprocess.DEVNULL)
        for _ in range(200):                      # wait until the child has written its header
            if os.path.exists(self.path) and os.path.getsize(self.path) > 0:
                break
            time.sleep(0.02)

    def stop(self) -> None:
        """Ends the child and reads its samples; window() then summarises any time interval."""
        self.proc.send_signal(signal.SIGTERM)
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.max_mhz, self.samples = None, []
        try:
            lines = open(self.path).read().split("\n")
            os.unlink(self.path)
        except OSError:
            return
        for ln in lines:
            p = ln.split()
            if len(p) == 2 and p[0] == "max":
                self.max_mhz = int(p[1])
            elif len(p) == 4:
                self.samples.append((float(p[0]), int(p[1]), int(p[2]), float(p[3])))

    def window(self, t0: float, t1: float) -> dict:
        """Median SM clock, clock-event reasons and peak power of the samples taken in [t0, t1] (wall clock)."""
        out = {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        sel = [smp for smp in self.samples if t0 <= smp[0] <= t1]
        if sel:
            bits = 0
            for smp in sel:
                bits |= smp[2]
            out["sm_mhz"] = statistics.median(smp[1] for smp in sel)
            out["sm_mhz_min"] = min(smp[1] for smp in sel)
            out["samples"] = len(sel)
            out["power_w_max"] = max(smp[3] for smp in sel)
            out["reasons"] = [name for bit, name in REASON_BITS.items() if bits & bit and name != "gpu_idle"]
        return out


# ------------------------------------------------------------------------------------------------
# workload
# ------------------------------------------------------------------------------------------------

WORKLOAD_TEXT = {
    "c1_tiny": "tiny MoE layer: 64 tokens, hidden 256, 8 experts top-2, FFN 512, 4 ranks x 2 slots, seeded random placement",
    "c2_mixtral": "Mixtral-8x7B-shaped layer: 4096 tokens, hidden 4096, 8 experts top-2, SwiGLU FFN 14336, "
                  "8 logical ranks, 2 hottest experts replicated",
    "c3_dsv2lite": "DeepSeek-V2-Lite-shaped layer: 8192 tokens, hidden 2048, 64 experts top-6 + 2 shared, FFN 1408, "
                   "8 ranks x 9 slots, spare slots filled by greedy replication",
    "c4_qwen15": "Qwen1.5-MoE-A2.7B-shaped layer: 16384 tokens, hidden 2048, 60 experts top-4 + 4 shared, FFN 1408, "
                 "8 ranks x 8 slots, popularity shifting every 512 tokens",
    "c5_qwen3": "Qwen3-30B-A3B-shaped layer: hidden 2048, 128 experts top-8, FFN 768, 16 ranks x 9 slots, "
                "greedy load-balanced placement",
}


def algorithmic_work(s, T):
    """Bytes / FLOP the method itself must move or compute for one batch (per-token figures times T)."""
    A = T * s.K
    return {
        "route_bytes": T * (4 * s.E + 8 * s.K),
        "dispatch_bytes": T * (2 * s.H + 2 * s.H * s.K + 16 * s.K),
        "combine_bytes": T * (2 * s.H * s.K + 8 * s.K + 2 * s.H + (2 * s.H if s.S > 0 else 0)),
        "cost_bytes": T * 8 * s.K,
        "gemm1_flop": 4 * s.H * s.F * A,            # gate and up projections
        "gemm2_flop": 2 * s.H * s.F * A,            # down projection
        "shared_flop": 6 * s.H * s.F * s.S * T,
        "ffn_flop": 6 * s.H * s.F * (A + T * s.S),
    }


def build_layer(args, device):
    """Generates the workload on the host, uploads it, derives the placement through the product path
    (route -> placement-cost histogram -> greedy helper) and returns everything the timed loops need."""
    import numpy as np
    import torch
    from paper_2607_08782_b200 import placement, synth
    from paper_2607_08782_b200.layer import MoELayer, bf16_bits_to_tensor

    wl = synth.make_workload(args.config, args.tokens, E=args.experts)
    s, w = wl.shape, wl.weights
    wg, wu, wd = (bf16_bits_to_tensor(a, device) for a in (w.w_gate, w.w_up, w.w_down))
    sg = su = sd = None
    if s.S > 0:
        sg = bf16_bits_to_tensor(w.ws_gate.reshape(s.S * s.F, s.H), device)
        su = bf16_bits_to_tensor(w.ws_up.reshape(s.S * s.F, s.H), device)
        sd = bf16_bits_to_tensor(synth.concat_shared_down(w.ws_down), device)
    layer = MoELayer(s.T, s.H, s.F, s.E, s.K, s.S, s.R, s.C_max, wg, wu, wd, sg, su, sd, device)
    logits = torch.from_numpy(wl.logits).to(device)
    x = bf16_bits_to_tensor(wl.x, device)

    # placement from the layer's own histograms of this batch (ground-truth routing)
    layer.set_placement(wl.X_primary)
    layer.route(s.T, logits)
    layer.placement_cost(s.T)
    torch.cuda.synchronize()
    N = placement.expert_counts(layer.workload.cpu().numpy())
    if args.placement == "primary" or s.name == "c1_tiny":
        X, pname = wl.X_primary, "primary"
    elif s.name == "c2_mixtral":
        X, pname = placement.replicate_hottest(N, wl.X_primary, 2), "2 hottest experts replicated"
    elif s.name == "c5_qwen3":
        X, pname = placement.greedy_balanced(N, s.R, s.C_max), "greedy load-balanced"
    else:
        X, pname = placement.greedy_balanced(N, s.R, s.C_max, synth.primary_ranks(s)), "primaries + greedy replicas"
    layer.set_placement(X)
    if args.ffn_variant is not None:
        layer.set_ffn_variant(args.ffn_variant)
    if args.replica_policy == "local_first":
        layer.set_replica_policy(1)
    return wl, layer, logits, x, X, pname


# ------------------------------------------------------------------------------------------------
# CPU oracle legs (cpu_baseline and --impl reference)
# ------------------------------------------------------------------------------------------------

def oracle_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return 1


def oracle_weights(wl):
    """The oracle's parameters decoded once into its compute precision (fp64), the counterpart of the
    GPU path's weights being resident in HBM before the timed region."""
    from oracle import director_oracle as orc
    from paper_2607_08782_b200.synth import Weights
    w = wl.weights
    dec = lambda a: None if a is None else orc.bf16_to_f64(a)
    return Weights(dec(w.w_gate), dec(w.w_up), dec(w.w_down), dec(w.ws_gate), dec(w.ws_up), dec(w.ws_down))


def oracle_step(wl, w, X, n_tokens):
    """The oracle, as it stands, on the first n_tokens tokens of the batch as a batch of their own."""
    from oracle import director_oracle as orc
    s = wl.shape
    logits, x = wl.logits[:n_tokens], wl.x[:n_tokens]
    idx, _, w64 = orc.route(logits, s.K)
    d = orc.dispatch(idx, X, s.C_max, x)
    yp = orc.expert_ffn(d["xp"], d["seg_offsets"], d["slot_expert"], w.w_gate, w.w_up, w.w_down)
    ysh = orc.shared_ffn(x, w.ws_gate, w.ws_up, w.ws_down) if s.S > 0 else None
    y = orc.combine(yp, d["inv_row"], w64, ysh)
    orc.placement_cost(idx, X, s.C_max, s.H)
    return y


def oracle_sample_tokens(s, target_flop):
    """Sub-batch size whose fp64 FFN work is about target_flop (a few seconds on a many-core host)."""
    per_token = 6.0 * s.H * s.F * (s.K + s.S)
    n = int(max(1, min(s.T, target_flop // per_token)))
    return n


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    from paper_2607_08782_b200 import synth
    from oracle import director_oracle as orc
    wl = synth.make_workload(args.config, args.tokens)
    s = wl.shape
    idx, _, _ = orc.route(wl.logits, s.K)
    N = np.bincount(idx.ravel(), minlength=s.E)
    if s.name == "c2_mixtral":
        X = orc.replicate_hottest(N, wl.X_primary, 2)
    elif s.name == "c5_qwen3":
        X = orc.balanced_placement(N, s.R, s.C_max)
    elif s.name == "c1_tiny":
        X = wl.X_primary
    else:
        X = orc.balanced_placement(N, s.R, s.C_max, synth.primary_ranks(s))
    n = oracle_sample_tokens(s, 2.0e11)
    w64 = oracle_weights(wl)
    for _ in range(args.warmup):
        oracle_step(wl, w64, X, n)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(wl, w64, X, n)
    dt = time.perf_counter() - t0
    value = n * args.steps / dt
    cores = oracle_threads()
    sample = f"each step = the oracle on the first {n} of {s.T} tokens as a batch of their own (all stages, fp64)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD_TEXT[args.config], "tokens": s.T, "sample_tokens_per_step": n},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------------------------------------
# main (CUDA arm)
# ------------------------------------------------------------------------------------------------

DOMINANT_KERNEL = "grouped_gemm_swiglu_kernel"      # the gate||up grouped GEMM: ~63 % of a step

STAGE_KERNELS = {
    "route": ["route_topk_kernel", "front_small_kernel"],   # the fused front end (T <= 256) is booked under route
    "dispatch": ["dispatch_plan_kernel", "dispatch_count_scan_kernel", "dispatch_index_kernel", "dispatch_scatter_rows_kernel",
                 "dispatch_travel_count_scan_kernel", "dispatch_slot_count_scan_kernel", "dispatch_local_index_kernel"],
    "expert_ffn": ["grouped_gemm_swiglu_kernel", "grouped_gemm_down_kernel", "one_segment_kernel",
                   "small_ffn_swiglu_kernel", "small_ffn_down_kernel", "grouped_gemm_down_fused_kernel",
                   "fused_combine_prepare_kernel"],
    "combine": ["combine_kernel", "fused_combine_finish_kernel"],
    "placement_cost": ["cost_workload_hist_kernel", "cost_from_workload_kernel", "cost_count_scan_kernel", "cost_kernel",
                       "cost_travel_count_scan_kernel", "cost_local_kernel"],
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        under_load = p.get("clocks_under_load", {})
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                "sm_max_mhz": p.get("sm_max_mhz", 1965.0),
                "sustained_sm_mhz": under_load.get("sm_mhz_median", 1342.0), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "sm_max_mhz": 1965.0,
            "sustained_sm_mhz": 1300.0, "source": "fallback"}


def tensor_peak_for_clock(peaks, sm_mhz):
    """The cuBLAS bf16 ceiling that belongs to the clock regime a kernel was timed in.

    The two measured ceilings were taken at two clocks: the burst figure at the maximum SM clock (a kernel timed
    alone, before the power cap bites) and the sustained figure at the clock the GPU settles to under the 1 kW cap.
    A timed region whose median SM clock is within 5 % of the maximum is compared with the burst ceiling, one at or
    below the sustained clock with the sustained ceiling, and one in between with the straight line between the two
    points.  Without clock samples the burst ceiling (the stricter one) is used.
    Returns (peak TFLOP/s, regime name)."""
    burst, sust = peaks["bf16_tflops"], peaks["bf16_tflops_sustained"]
    f_max, f_sust = float(peaks["sm_max_mhz"]), float(peaks["sustained_sm_mhz"])
    if sm_mhz is None:
        return burst, "burst (no clock samples)"
    if sm_mhz >= 0.95 * f_max:
        return burst, "burst"
    if sm_mhz <= f_sust or f_max <= f_sust:
        return sust, "sustained"
    return sust + (burst - sust) * (sm_mhz - f_sust) / (f_max - f_sust), "between"


def run_placement_search(args, device):
    """Extra measurement (not the headline): candidates per second of director_placement_cost_batch, the scoring
    loop of the placement search (Section VI-C), and one full search on the workload."""
    import numpy as np
    import torch
    from paper_2607_08782_b200 import optimizer as opt
    from paper_2607_08782_b200 import synth
    from paper_2607_08782_b200.binding import Director
    shape = synth.shape_for(args.config, args.tokens)
    s = shape
    logits = torch.from_numpy(synth.make_logits(s)).to(device)
    d = Director(s.T, s.H, s.F, s.E, s.K, s.S, s.R, s.C_max)
    X0 = synth.placement_from_ranks(synth.primary_ranks(s), s.R)
    d.set_placement(X0)
    idx = torch.empty((s.T, s.K), dtype=torch.int32, device=device)
    w = torch.empty((s.T, s.K), dtype=torch.float32, device=device)
    W = torch.empty((s.R, s.E), dtype=torch.int64, device=device)
    load = torch.empty((s.R,), dtype=torch.int64, device=device)
    dt = torch.empty((s.R, s.R), dtype=torch.int64, device=device)
    db = torch.empty((s.R, s.R), dtype=torch.int64, device=device)
    d.route(s.T, logits, idx, w)
    d.placement_cost(s.T, idx, None, W, load, dt, db)
    torch.cuda.synchronize()
    n = 4096
    rng = np.random.default_rng(0)
    Xb = np.zeros((n, s.E, s.R), dtype=np.uint8)
    for c in range(n):
        ranks_c = np.repeat(np.arange(s.R), s.C_max)[rng.permutation(s.R * s.C_max)[:s.E]]
        Xb[c, np.arange(s.E), ranks_c] = 1
    Xd = torch.from_numpy(Xb).to(device)
    o_load = torch.empty((n, s.R), dtype=torch.int64, device=device)
    o_disp = torch.empty((n, s.R, s.R), dtype=torch.int64, device=device)
    o_sum = torch.empty((n, 4), dtype=torch.int64, device=device)
    for _ in range(3):
        d.placement_cost_batch(W, n, Xd, o_load, o_disp, o_sum)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        d.placement_cost_batch(W, n, Xd, o_load, o_disp, o_sum)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    model = opt.LatencyModel(1.0, 0.0, 0.2 / (2 * s.H), 2 * s.H)
    ev = opt.GpuPlacementEvaluator(d, W)
    base = ev(X0[None])[0]
    t0 = time.perf_counter()
    res = opt.optimize_placement(W.cpu().numpy(), s.C_max, model, ev, allow_replicas=True)
    search_s = time.perf_counter() - t0
    print(json.dumps({
        "metric": "placement_candidates_per_s", "value": n / (ms * 1e-3), "unit": "candidates/s", "n_gpus": 1,
        "steps": args.steps, "ms_per_step": ms, "higher_is_better": True, "data": "synthetic",
        "config": {"workload": WORKLOAD_TEXT[args.config], "candidates_per_call": n, "E": s.E, "R": s.R},
        "search": {"seconds": search_s, "candidates_scored": ev.evaluated, "rounds": res["rounds"],
                   "latency_before": float(model.latency(base[0], base[1])), "latency_after": res["latency"],
                   "lp_bound": res["lp_bound"]}}))


def run_index_kernels(args, device):
    """Extra measurement (not the headline): the routing and index kernels far above their launch latency.  At the
    paper-shaped batch sizes these kernels move ~1-20 MB and finish in microseconds, so their bandwidth there says
    little; here the same routing shape (E, K, R, C_max of --config) runs on 2^20 tokens (hidden size cut to 256:
    neither kernel touches hidden states), logits tiled from the seeded generator."""
    import numpy as np
    import torch
    from paper_2607_08782_b200 import placement, synth
    from paper_2607_08782_b200.binding import Director
    base = synth.shape_for(args.config, None)
    T = args.tokens or (1 << 20)
    s = base
    block = torch.from_numpy(synth.make_logits(base)).to(device)
    logits = block.repeat((T + base.T - 1) // base.T, 1)[:T].contiguous()
    d = Director(T, 256, 128, s.E, s.K, 0, s.R, s.C_max)
    d.set_placement(synth.placement_from_ranks(synth.primary_ranks(s), s.R))
    A = T * s.K
    i32 = dict(dtype=torch.int32, device=device)
    idx, w = torch.empty((T, s.K), **i32), torch.empty((T, s.K), dtype=torch.float32, device=device)
    row_token, inv_row, dest = torch.empty(A, **i32), torch.empty((T, s.K), **i32), torch.empty((T, s.K), **i32)
    seg = torch.empty(s.R * s.C_max + 1, **i32)
    peaks = measured_peaks()

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / args.steps

    out = {}
    ms = timed(lambda: d.route(T, logits, idx, w))
    by = T * (4 * s.E + 8 * s.K)
    out["route"] = {"ms": ms, "GB/s": by / ms / 1e6, "frac_of_peak": by / ms / 1e6 / peaks["hbm_gbs"]}
    for policy, name in ((0, "dispatch_index_round_robin"), (1, "dispatch_index_local_first")):
        d.set_replica_policy(policy)
        ms = timed(lambda: d.dispatch(T, None, idx, None, row_token, inv_row, dest, seg))
        by = T * 16 * s.K                                     # topk_idx read, inv_row / dest_rank / row_token written
        out[name] = {"ms": ms, "GB/s": by / ms / 1e6, "frac_of_peak": by / ms / 1e6 / peaks["hbm_gbs"]}
    d.set_replica_policy(0)
    d.check_device_status()
    print(json.dumps({"metric": "index_kernel_bandwidth", "unit": "GB/s", "n_gpus": 1, "steps": args.steps,
                      "data": "synthetic", "peak": {"hbm_gbs": peaks["hbm_gbs"], "source": peaks["source"]},
                      "config": {"workload": WORKLOAD_TEXT[args.config], "tokens": T, "E": s.E, "K": s.K, "R": s.R},
                      "kernels": out}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="c2_mixtral", choices=sorted(WORKLOAD_TEXT))
    ap.add_argument("--tokens", type=int, default=None, help="batch size override (c5_qwen3 sweep: 1, 64, 1024, 32768)")
    ap.add_argument("--experts", type=int, default=None,
                    help="cut the workload down to this many routed experts (same tile shapes, smaller device footprint: "
                         "for profiler captures; not the headline workload)")
    ap.add_argument("--placement", default="auto", choices=["auto", "primary"])
    ap.add_argument("--ffn-variant", type=int, default=None, choices=[0, 1, 2, 6],
                    help="expert-FFN tile scheme: 0 = one CTA per 128x256 tile, 1 = CTA pairs (256x256), 2 = weight-stationary CTA pairs "
                         "(the library's default), 6 = scheme 2 with the tensor-core kernels also for batches of at most 4 tokens")
    ap.add_argument("--replica-policy", default="round_robin", choices=["round_robin", "local_first"],
                    help="which replica of a replicated expert an assignment uses (the default is the headline setting)")
    ap.add_argument("--fused", action="store_true",
                    help="index-only dispatch + director_expert_ffn_gather (the GEMM gathers rows from x) instead of the "
                         "materialised permutation")
    ap.add_argument("--fused-combine", action="store_true",
                    help="director_expert_ffn_combine: the down projection combines in its epilogue (fp32 atomic adds; "
                         "opt-in, not bit-reproducible) instead of writing Yp for a separate combine kernel")
    ap.add_argument("--graph", action="store_true",
                    help="replay the device-resident step from a CUDA graph (decode-sized batches); no per-kernel timings")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--stage", default="layer", choices=["layer", "placement_search", "index_kernels"],
                    help="layer (default): the MoE layer step; placement_search: batched scoring of candidate placements; "
                         "index_kernels: routing and dispatch-index kernels on 2^20 tokens")
    ap.add_argument("--sample-clocks", nargs=2, metavar=("UUID", "PATH"), help=argparse.SUPPRESS)
    args = ap.parse_args()
    if args.sample_clocks:
        _sample_clocks_main(*args.sample_clocks)
        return
    if args.impl == "reference":
        run_reference(args)
        return

    import numpy as np
    import torch
    from paper_2607_08782_b200.multirank import Ranks

    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the layer has no CPU implementation")
    torch.cuda.set_device(local_rank)
    device = f"cuda:{local_rank}"
    ranks = Ranks("nccl", device)
    rank, world = ranks.rank, ranks.world
    barrier = ranks.barrier

    if args.stage == "placement_search":
        run_placement_search(args, device)
        ranks.close()
        return
    if args.stage == "index_kernels":
        run_index_kernels(args, device)
        ranks.close()
        return
    wl, layer, logits, x, X, pname = build_layer(args, device)
    s = wl.shape
    T = s.T
    peaks = measured_peaks()

    # ---- device-resident throughput ----
    for _ in range(max(args.warmup, 3)):
        layer.forward(T, logits, x, fused=args.fused, fused_combine=args.fused_combine)
    torch.cuda.synchronize()
    layer.d.check_device_status()

    sampler = None
    if rank == 0:
        try:
            uuid = str(torch.cuda.get_device_properties(local_rank).uuid)
            sampler = ClockSampler(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
        except Exception:
            sampler = None
    # keep the GPU busy while the sampler starts so that the first samples see load clocks
    for _ in range(3):
        layer.forward(T, logits, x, fused=args.fused, fused_combine=args.fused_combine)
    barrier()
    torch.cuda.synchronize()
    graph, launches_per_pass = None, 0
    if args.graph:
        n_c = layer.d.launch_count()
        graph = layer.capture(T, logits, x, fused=args.fused, fused_combine=args.fused_combine)
        launches_per_pass = (layer.d.launch_count() - n_c) // 2      # capture() runs the pass twice (warm-up + record)
    else:
        # inside the timed region only the dominant kernel is bracketed by events (its live duration is what the
        # roofline object needs); the other kernels are timed in a pass of their own afterwards
        layer.d.set_profiling(True, only=DOMINANT_KERNEL)
    n0 = layer.d.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    wall0 = time.time()
    ev0.record()
    for _ in range(args.steps):
        if graph is None:
            layer.forward(T, logits, x, fused=args.fused, fused_combine=args.fused_combine)
        else:
            graph.replay()
    ev1.record()
    torch.cuda.synchronize()
    wall1 = time.time()
    barrier()
    launches = layer.d.launch_count() - n0
    if graph is not None:                                  # replays launch the kernels recorded in the graph
        launches = args.steps * launches_per_pass
    ms_total = ev0.elapsed_time(ev1)
    # the SM clock during the last gate||up / down launch of the timed region, measured by the kernels themselves
    kernel_clock = None
    try:
        (mhz1, us1), (mhz2, us2) = layer.d.gemm_sm_mhz(0), layer.d.gemm_sm_mhz(1)
        kernel_clock = {"gate_up_sm_mhz": round(mhz1, 1), "gate_up_us": round(us1, 1), "down_sm_mhz": round(mhz2, 1),
                        "down_us": round(us2, 1),
                        "how": "cycle counter / global timer inside the last launch of the timed region (tile scheme 2)",
                        "gate_up": {k: round(v, 4) for k, v in layer.d.gemm_counters(0).items()},
                        "down": {k: round(v, 4) for k, v in layer.d.gemm_counters(1).items()}}
    except Exception:
        kernel_clock = None
    kernel_ms = {}
    stage_ms_measured = {}
    wallx0 = wallx1 = None
    if graph is None:
        ms, n = layer.d.kernel_time(DOMINANT_KERNEL)
        dominant = (ms / n, n // args.steps) if n else None
        # every kernel, in an extra pass outside the timed region (same steps, events around every launch)
        extra = min(args.steps, 100)
        layer.d.set_profiling(True)
        wallx0 = time.time()
        for _ in range(extra):
            layer.forward(T, logits, x, fused=args.fused, fused_combine=args.fused_combine)
        torch.cuda.synchronize()
        wallx1 = time.time()
        for names in STAGE_KERNELS.values():
            for k in names:
                ms, n = layer.d.kernel_time(k)
                if n:
                    kernel_ms[k] = (ms / n, n // extra)
        if dominant:
            kernel_ms[DOMINANT_KERNEL] = dominant        # the figure from the timed region itself
        # every stage, in a third pass: ONE pair of events around all launches of a stage, so a stage of several small
        # kernels pays the bracket once (a pair of events around a microsecond kernel costs as much as the kernel)
        layer.d.set_profiling(2)
        for _ in range(extra):
            layer.forward(T, logits, x, fused=args.fused, fused_combine=args.fused_combine)
        torch.cuda.synchronize()
        wallx1 = time.time()
        for stage in STAGE_KERNELS:
            ms, n = layer.d.kernel_time("stage_" + stage)
            if n:
                stage_ms_measured[stage] = ms / extra
        ms, n = layer.d.kernel_time("stage_front_small")
        if n:
            stage_ms_measured["front_small"] = ms / extra
    layer.d.set_profiling(False)
    layer.d.check_device_status()
    no_clocks = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
    clocks, clocks_extra = dict(no_clocks), dict(no_clocks)
    if sampler:
        sampler.stop()
        clocks = sampler.window(wall0, wall1)
        if wallx0 is not None:
            clocks_extra = sampler.window(wallx0, wallx1)
    ms_total = ranks.max_over_ranks(ms_total)
    ms_per_step = ms_total / args.steps
    value = world * T * args.steps / (ms_total * 1e-3)

    # ---- end to end through the host-buffer entry points (pipelined submit / wait) ----
    h_logits = torch.from_numpy(wl.logits).pin_memory()
    h_x = torch.from_numpy(wl.x.view(np.int16)).pin_memory()
    h_y = [torch.empty((T, s.H), dtype=torch.int16).pin_memory() for _ in range(2)]
    h_load = [torch.empty((s.R,), dtype=torch.int64).pin_memory() for _ in range(2)]
    h_bytes = [torch.empty((s.R, s.R), dtype=torch.int64).pin_memory() for _ in range(2)]

    def e2e_run(n):
        """n batches through director_layer_submit_host / director_layer_wait_host, two in flight: every batch
        pays its own host->device and device->host copies, which overlap the kernels of its neighbours."""
        prev = None
        for i in range(n):
            b = i & 1
            tk = layer.d.layer_submit_host(T, h_logits, h_x, *layer.w, *layer.ws, h_y[b], h_load[b], h_bytes[b])
            if prev is not None:
                layer.d.layer_wait_host(prev)
            prev = tk
        layer.d.layer_wait_host(prev)

    e2e_run(3)
    barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    e2e_run(args.steps)
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t0) * 1e3
    barrier()
    # one unpipelined call for the latency of a single batch
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    layer.d.layer_forward_host(T, h_logits, h_x, *layer.w, *layer.ws, h_y[0], h_load[0], h_bytes[0])
    single_ms = (time.perf_counter() - t0) * 1e3
    e2e_ms = ranks.max_over_ranks(e2e_ms)
    layer.d.check_device_status()
    # the host-path result must be the same bits as the device-path result
    same = bool(torch.equal(h_y[0].cuda().view(torch.bfloat16), layer.y[:T])) and \
        bool(torch.equal(h_y[1].cuda().view(torch.bfloat16), layer.y[:T])) and \
        bool(torch.equal(h_load[0].cuda(), layer.rank_load))
    e2e = {"value": world * T * args.steps / (e2e_ms * 1e-3), "unit": UNIT,
           "h2d_bytes_per_step": int(h_logits.numel() * 4 + h_x.numel() * 2),
           "d2h_bytes_per_step": int(h_y[0].numel() * 2 + h_load[0].numel() * 8 + h_bytes[0].numel() * 8),
           "ms_per_step": e2e_ms / args.steps, "single_batch_latency_ms": single_ms, "matches_device_path": same,
           "api": "director_layer_submit_host / director_layer_wait_host: pinned host logits and x in, y and "
                  "histograms out, two batches in flight; wall clock around the loop, synchronised on both sides"}

    if rank != 0:
        ranks.close()
        return

    # ---- roofline of the dominant kernel and per-stage figures ----
    work = algorithmic_work(s, T)
    dom = DOMINANT_KERNEL
    dom_ms, dom_per_step = kernel_ms.get(dom, (None, 0))
    shared_frac = work["shared_flop"] / work["ffn_flop"] if work["ffn_flop"] else 0.0
    # with shared experts the kernel is launched twice per step (routed + shared); flops per launch averaged
    gemm1_flop_per_launch = (work["gemm1_flop"] + work["shared_flop"] * 2 / 3) / max(dom_per_step, 1)
    achieved = gemm1_flop_per_launch / (dom_ms * 1e-3) / 1e12 if dom_ms else None
    # the denominator follows the clock regime of the timed region itself (median SM clock sampled inside it; the
    # dominant kernel is ~63 % of that region, so the region's median is the clock it ran at)
    # The regime is read from the NVML-sampled clock, the instrument the two measured ceilings were recorded with.  The
    # clock the kernel measures itself at (cycle counter against the global timer) is lower - the GPU is power-limited
    # inside a dense GEMM long before the sampled clock shows it - and is reported beside it: cycles per launch =
    # duration x that clock is the figure that compares runs at different clocks.
    dom_mhz = kernel_clock["gate_up_sm_mhz"] if kernel_clock and kernel_clock["gate_up_sm_mhz"] > 0 else None
    peak, regime = tensor_peak_for_clock(peaks, clocks.get("sm_mhz"))
    roofline = {"kernel": dom, "bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": (achieved / peak) if achieved else None,
                "traffic": NCU_TRAFFIC_BYTES.get(args.config),
                "regime": regime, "sm_mhz_kernel": dom_mhz, "sm_mhz_median": clocks.get("sm_mhz"),
                "clock_samples": clocks.get("samples", 0),
                "peak_source": f"{peaks['source']} cuBLAS bf16: burst {peaks['bf16_tflops']} at {peaks['sm_max_mhz']:.0f} MHz, "
                               f"sustained {peaks['bf16_tflops_sustained']} at {peaks['sustained_sm_mhz']:.0f} MHz; "
                               "chosen by the median NVML-sampled SM clock of the timed region",
                "flop_per_launch": gemm1_flop_per_launch, "ms_per_launch": dom_ms,
                "mcycles_per_launch": (dom_ms * dom_mhz * 1e-3) if dom_ms and dom_mhz else None,
                "frac_of_pipe_at_kernel_clock": (achieved * 1e12 / (148 * 8192 * dom_mhz * 1e6)) if achieved and dom_mhz else None,
                "frac_of_burst_peak": (achieved / peaks["bf16_tflops"]) if achieved else None,
                "frac_of_sustained_peak": (achieved / peaks["bf16_tflops_sustained"]) if achieved else None,
                "frac_of_nominal_2250": (achieved / 2250.0) if achieved else None}

    def stage_ms(stage):
        """Time of a stage per step: its own bracket (one pair of events around all its launches) when that pass ran,
        else the sum of its individually bracketed kernels."""
        if stage in stage_ms_measured and stage != "expert_ffn":   # the GEMMs are long: their kernel brackets are exact
            return stage_ms_measured[stage]
        return sum(kernel_ms[k][0] * kernel_ms[k][1] for k in STAGE_KERNELS[stage] if k in kernel_ms)

    stages = {}
    for stage, key, unit in (("route", "route_bytes", "GB/s"), ("dispatch", "dispatch_bytes", "GB/s"),
                             ("combine", "combine_bytes", "GB/s"), ("placement_cost", "cost_bytes", "GB/s"),
                             ("expert_ffn", "ffn_flop", "TFLOP/s")):
        ms = stage_ms(stage)
        if ms <= 0:
            continue
        rate = work[key] / (ms * 1e-3) / (1e9 if unit == "GB/s" else 1e12)
        # stage times come from the extra pass (events around every launch): its own clock window picks the ceiling
        pk = peaks["hbm_gbs"] if unit == "GB/s" else tensor_peak_for_clock(peaks, clocks_extra.get("sm_mhz"))[0]
        stages[stage] = {"ms": round(ms, 4), "rate": round(rate, 2), "unit": unit, "frac_of_measured_peak": round(rate / pk, 4),
                         "timing": "one event pair around the stage" if stage in stage_ms_measured and stage != "expert_ffn" else "sum of per-kernel event pairs",
                         "ms_sum_of_kernel_brackets": round(sum(kernel_ms[k][0] * kernel_ms[k][1] for k in STAGE_KERNELS[stage]
                                                                 if k in kernel_ms), 4)}
    if "front_small" in stage_ms_measured:
        stages["front_small"] = {"ms": round(stage_ms_measured["front_small"], 4), "unit": "ms",
                                 "what": "gate + dispatch indices + placement cost of a decode batch in one launch"}
    kernels = {k: {"ms_per_launch": round(v[0], 4), "launches_per_step": v[1]} for k, v in kernel_ms.items()}

    # ---- CPU baseline: the oracle on a bounded sample, on this machine's host cores ----
    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        n = oracle_sample_tokens(s, 1.5e13)
        w64 = oracle_weights(wl)
        t0 = time.perf_counter()
        oracle_step(wl, w64, X, n)
        dt = time.perf_counter() - t0
        cpu_baseline = {"value": n / dt, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                        "sample": f"the oracle (all stages, fp64, weights pre-decoded to fp64) on the first {n} of {T} "
                                  f"tokens as a batch of their own, one run, {dt:.1f} s", "host_cpus": os.cpu_count()}

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": WORKLOAD_TEXT[args.config] + (f" [cut down to {s.E} experts]" if args.experts else ""),
                   "tokens": T, "placement": pname,
                   "replica_policy": args.replica_policy,
                   "l2": "inputs larger than L2: every step streams the expert weights "
                         f"({3 * s.E * s.F * s.H * 2 / 1e9:.2f} GB) and activations through HBM",
                   "parallelism": "single GPU, logical ranks" if world == 1 else f"{world} independent replicas"},
        "clocks": clocks, "clocks_stage_pass": clocks_extra, "kernel_clock": kernel_clock, "e2e": e2e, "gpu_launches": int(launches), "cuda_graph": bool(args.graph), "roofline": roofline,
        "cpu_baseline": cpu_baseline, "stages": stages, "kernels": kernels,
        "ffn_tflops": round(work["ffn_flop"] / (stage_ms("expert_ffn") * 1e-3) / 1e12, 1) if stage_ms("expert_ffn") else None,
    }
    print(json.dumps(out))
    ranks.close()


if __name__ == "__main__":
    main()
