#!/usr/bin/env python
"""Benchmark of the Monarch multiply hot path on B200.

One step = one pass of the hot path over one batch of synthetic tokens.  The headline is the largest
forward + backward configuration, workload 4 (n = 16384, m = 128, 4096 tokens per GPU, bf16):
    monarch_fwd (y), then monarch_bwd (dx, dL, dR in one call, reusing the intermediate the forward call left
    in its workspace).
The same JSON line carries, under "workloads", every other workload of the contract (1: fp32 forward, 2: m = 32
forward, 3: m = 64 forward + backward, 5: feed-forward block) timed the same way with fewer steps.
Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
`--workload N` picks another headline; `--calls fwd,bwd_dx,bwd_dw` times the three separately exported calls;
`--workload 5 --calls mlp_fwd,mlp_bwd` adds the backward of the feed-forward block; workloads 6-8 are the
general (rectangular) class, the projection and the complex multiply.

`python bench.py --gpus N` starts N ranks itself (torch.distributed.run, one per GPU, NCCL); under an external
launcher (WORLD_SIZE set) it is one of the ranks.  Tokens are sharded over ranks (fixed tokens per GPU: weak
scaling); the only exchange is one all-reduce of the packed (dL, dR) gradients per step.
"""
from __future__ import annotations

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

FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None,
                    help="timed steps (default: 1000, so that the timed region spans several clock samples; "
                         "100 for workload 7; 30 for --impl reference)")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=4, choices=[1, 2, 3, 4, 5, 6, 7, 8, 9],
                    help="1-5: the square workloads; 6: the general (rectangular) class, forward only; "
                         "7: projection of a dense matrix onto the Monarch class + dense materialisation; "
                         "8: complex multiply (planar), y = M x then z = M^H y; 9: the rectangular class with "
                         "wrapped-diagonal blocks (b2 != b3)")
    ap.add_argument("--kernels", default="auto", choices=["auto", "staged", "fused"])
    ap.add_argument("--calls", default="", help="comma-separated subset of the workload's calls "
                    "(profiling aid; the default step runs them all)")
    ap.add_argument("--no-side-workloads", dest="side_workloads", action="store_false",
                    help="time only the headline workload (default: the other workloads of the contract are "
                         "timed too, with fewer steps, and reported under \"workloads\")")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    if args.steps is None:
        args.steps = 30 if args.impl == "reference" else (100 if args.workload == 7 else 1000)
    return args


# ----------------------------------------------------------------------------- accounting

def esize(dtype):
    return 4 if dtype == "f32" else 2


def call_flops(call, n, m, T):
    """Algorithmic FLOPs: 4 n m per token per pass (two block-diagonal stages of 2 n m each)."""
    return {"fwd": 4, "bwd_dx": 4, "bwd_dw": 4, "bwd": 8, "mlp_fwd": 8, "mlp_bwd": 16}[call] * n * m * T


def call_bytes(call, n, m, T, dtype):
    """Algorithmic bytes: the token tensors read and written once, plus the weights once."""
    s = esize(dtype)
    w = 2 * n * m * s
    if call in ("fwd", "bwd_dx"):
        return 2 * T * n * s + w
    if call == "bwd_dw":
        return 2 * T * n * s + w + 2 * n * m * 4
    if call == "bwd":          # read x, dy; write dx, dL, dR
        return 3 * T * n * s + w + 2 * n * m * 4
    if call == "mlp_fwd":
        return 2 * T * n * s + 2 * w + 2 * n * s
    if call == "mlp_bwd":      # read x, dy; write dx and the six parameter gradients
        return 3 * T * n * s + 2 * w + n * s + 4 * n * m * 4 + 2 * n * 4
    raise ValueError(call)


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "source": "measured"}
    except Exception:
        return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": FALLBACK_BF16_TFLOPS,
                "source": "fallback"}


# ----------------------------------------------------------------------------- clocks

class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
            "hw_power_brake": getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(0.02)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        return {
            "sm_mhz": statistics.median(self.samples) if self.samples else None,
            "sm_max_mhz": self.max_mhz,
            "reasons": sorted(self.reasons),
            "samples": len(self.samples),
        }


# ----------------------------------------------------------------------------- CPU oracle timing

def time_oracle(cfg, d, target_s=12.0, calls=None, tokens=None):
    """Time the oracle (as it stands) on a bounded token sample of the workload: `tokens` of them, or (None) as many
    as a short calibration says take about target_s seconds."""
    from oracle import monarch_oracle as O
    c = cfg
    calls = list(c.ops) if calls is None else [k for k in calls if k != "bwd"] + (
        ["bwd_dx", "bwd_dw"] if "bwd" in calls else [])

    def run(T):
        t0 = time.perf_counter()
        if "fwd" in calls:
            O.fwd(d["x"][:T], d["L"], d["R"])
        if "bwd_dx" in calls or "bwd_dw" in calls:
            want = tuple(k for k, op in (("dx", "bwd_dx"), ("dL", "bwd_dw"), ("dR", "bwd_dw"))
                         if op in calls)
            O.bwd(d["x"][:T], d["dy"][:T], d["L"], d["R"], want=want)
        if "mlp_fwd" in calls:
            O.mlp_fwd(d["x"][:T], d["L"], d["R"], d["b1"], d["L2"], d["R2"], d["b2"])
        if "mlp_bwd" in calls:
            O.mlp_bwd(d["x"][:T], d["dy"][:T], d["L"], d["R"], d["b1"], d["L2"], d["R2"])
        return time.perf_counter() - t0

    if tokens is not None:
        T = int(min(c.tokens, max(1, tokens)))
        dt = run(T)
    else:
        T = min(32, c.tokens)
        dt = run(T)
        while dt < min(0.5, target_s) and T < c.tokens:
            T = min(T * 4, c.tokens)
            dt = run(T)
        Ts = int(min(c.tokens, max(8, T * target_s / max(dt, 1e-9))))
        if Ts != T:
            dt = run(Ts)
            T = Ts
    flops = sum(call_flops(k, c.n, c.m, T) for k in calls)
    return {"tflops": flops / dt / 1e12, "tokens": T, "seconds": dt, "cores": O.num_threads(),
            "tokens_per_s": T / dt}


# ----------------------------------------------------------------------------- main

# Kernels behind each timed call, and the DRAM traffic one call generated under ncu (dram__bytes_read.sum +
# dram__bytes_write.sum of the call's kernels; the note names the capture under profiles/ and says when the
# value was scaled from a smaller token count).
KERNELS_OF = {
    (16, "f32", "fwd"): "fused_fwd_m16_kernel (1 launch)",
    (32, "bf16", "fwd"): "fused_fwd_m32_kernel (1 launch)",
    (64, "bf16", "fwd"): "fused_fwd_m64_team_kernel (1 launch)",
    (64, "bf16", "bwd"): "fused_bwd_all_m64_kernel (1 launch, 2 memset nodes)",
    (64, "bf16", "bwd_dx"): "fused_bwd_dx_m64_kernel (1 launch)",
    (64, "bf16", "bwd_dw"): "fused_fwd_m64_kernel (stage 1 only) + fused_bwd_all_m64_kernel without dx "
                            "(2 launches, 2 memset nodes)",
    (64, "bf16", "mlp_fwd"): "fused_fwd_m64_team_kernel (2 launches)",
    (64, "bf16", "mlp_bwd"): "fused_fwd_m64_team_kernel + mlp_act_kernel + fused_fwd_m64_kernel (stage 1 only) + "
                             "2 x fused_bwd_all_m64_kernel + mlp_dact_kernel + merge_status_kernel (7 launches)",
    (128, "bf16", "fwd"): "chain_fused_fwd_kernel (1 persistent launch; chain_gemm_kernel x 2 + plane_transpose_kernel "
                          "beyond 8192 tiles)",
    (128, "bf16", "bwd"): "plane_transpose_kernel + chain_gemm_kernel x 2 with the token reductions (3 launches)",
    (128, "bf16", "bwd_dx"): "plane_transpose_kernel + chain_gemm_kernel x 2 (3 launches)",
    (128, "bf16", "bwd_dw"): "chain_gemm_kernel (stage 1) + plane_transpose_kernel + chain_gemm_kernel x 2 (4 launches)",
}
_W3 = "profiles/fused_m64_workload3_ncu.md, full size"
_W4 = "profiles/chain_m128_workload4_ncu.md, full size, cold L2 per launch (upper bound)"
NCU_TRAFFIC_MB = {
    (1, "fwd"): (0.1, "profiles/fused_fwd_m16_workload1_ncu.md, full size; the 65 KB output is still in L2 at kernel end"),
    (2, "fwd"): (33.9, "profiles/fused_fwd_m32_workload2_ncu.md, full size; the 33.6 MB output is still in L2 at kernel end"),
    (3, "fwd"): (146.9, _W3),
    (3, "bwd"): (364.0, _W3),
    (3, "bwd_dx"): (139.8, _W3),
    (3, "bwd_dw"): (408.3, _W3),
    (4, "fwd"): (460.8, _W4),
    (4, "bwd"): (924.8, _W4),
    (4, "bwd_dx"): (637.8, _W4),
    (4, "bwd_dw"): (1055.3, _W4),
    (5, "mlp_fwd"): (1511.0, "profiles/mlp_fwd_workload5_ncu.md, full size, both passes"),
}


def main_rect(args):
    """Workload 6: forward of the general Monarch class (appendix), q = 4 blocks of 1024 x 1024, one GPU or
    token-sharded replicas; bound by the tensor pipe (stage 1 holds nearly all the FLOPs)."""
    from paper_2204_00595_b200.inputs import RECT_WORKLOAD, RECTW_WORKLOAD, make_rect_inputs, make_rectw_inputs
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    wrapped = args.workload == 9                          # wrapped-diagonal blocks: b is R's block height b2, b3 that of L's blocks
    c = RECTW_WORKLOAD if wrapped else RECT_WORKLOAD
    q, b1, b, r, T = c["q"], c["b1"], c["b2" if wrapped else "b"], c["r"], c["tokens"]
    b3 = c["b3"] if wrapped else b
    nL = r * q * max(b, b3)                               # stored entries of L
    with_bwd = "rect_bwd" in args.calls.split(",")
    fwd_flops = 2 * T * (q * b * b1 + nL)
    flops = fwd_flops * (3 if with_bwd else 1)           # backward: dx and the two weight gradients, 2x the forward
    nbytes = T * (q * b1 + r * b3) * 2 + (q * b * b1 + nL) * 2
    workload = (f"workload {args.workload}: rect_fwd{'+rect_bwd' if with_bwd else ''} bf16 q={q} b1={b1} "
                + (f"b2={b} b3={b3}" if wrapped else f"b={b}") + f" r={r} tokens/GPU={T}")
    metric, unit = "monarch_rect_fwd_tflops", "TFLOP/s"
    make_inputs_ = make_rectw_inputs if wrapped else make_rect_inputs

    def time_oracle_rect(d, target_s):
        from oracle import monarch_oracle as O
        Ts, dt = 8, 0.0
        while True:
            t0 = time.perf_counter()
            if wrapped:
                O.rectw_fwd(d["x"][:Ts], d["L"], d["R"], b3)
            else:
                O.rect_fwd(d["x"][:Ts], d["L"], d["R"])
            dt = time.perf_counter() - t0
            if dt >= target_s / 4 or Ts >= T:
                break
            Ts = min(T, Ts * 4)
        return {"tflops": flops * Ts / T / dt / 1e12, "tokens": Ts, "seconds": dt, "cores": O.num_threads()}

    if args.impl == "reference":
        if rank != 0:
            return 0
        from oracle import monarch_oracle as O
        O.build()
        d = make_inputs_()
        rs = [time_oracle_rect(d, 8.0) for _ in range(args.warmup + args.steps)][args.warmup:]
        tfl = statistics.mean(x["tflops"] for x in rs)
        print(json.dumps({
            "impl": "reference", "metric": metric, "value": tfl, "unit": unit, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": statistics.mean(x["seconds"] for x in rs) * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload, "sample_tokens_per_step": rs[-1]["tokens"]},
            "cpu_baseline": {"value": tfl, "unit": unit, "cores": rs[-1]["cores"], "kind": "oracle",
                             "sample": f"{rs[-1]['tokens']} tokens of the workload per step"},
            "e2e": {"value": tfl, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))
        return 0

    import torch
    import __graft_entry__ as entry
    entry.build()
    import paper_2204_00595_b200 as P
    from paper_2204_00595_b200.inputs import to_device
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    P.monarch_set_impl({"auto": P.IMPL_AUTO, "staged": P.IMPL_STAGED, "fused": P.IMPL_AUTO}[args.kernels])
    d = make_inputs_()
    R, L = to_device(d["R"], "bf16"), to_device(d["L"], "bf16")
    sets = []
    for s in range(2):                          # two rotating sets, each larger than L2 with its output
        x = torch.roll(to_device(d["x"], "bf16"), shifts=17 * s + 5 * rank, dims=0).contiguous()
        sets.append((x, torch.empty(T, r * b3, dtype=torch.bfloat16, device="cuda")))
    if wrapped:
        ws = P.Workspace(P.monarch_rectw_workspace_bytes(T, q, b1, b, b3, r, P.BF16))
        ws_b = P.Workspace(P.monarch_rectw_bwd_workspace_bytes(T, q, b1, b, b3, r, P.BF16))
    else:
        ws = P.Workspace(P.monarch_rect_workspace_bytes(T, q, b1, b, r, P.BF16))
        ws_b = P.Workspace(P.monarch_rect_bwd_workspace_bytes(T, q, b1, b, r, P.BF16))
    stream = torch.cuda.current_stream()
    if with_bwd:
        dy = torch.randn(T, r * b3, device="cuda", generator=torch.Generator("cuda").manual_seed(595006)).bfloat16()
        dxs = [torch.empty_like(sets[0][0]) for _ in range(2)]
        gL = torch.zeros(L.shape, dtype=torch.float32, device="cuda")
        gR = torch.zeros(q, b, b1, dtype=torch.float32, device="cuda")
    mid = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    nmid = [0]

    def step(i, timed=False):
        x, y = sets[i % 2]
        if wrapped:
            P.monarch_rectw_fwd(x, L, R, y, T, q, b1, b, b3, r, ws)
        else:
            P.monarch_rect_fwd(x, L, R, y, T, q, b1, b, r, ws)
        if timed and with_bwd:                   # boundary between the two calls of a step
            mid[nmid[0]].record(stream)
            nmid[0] += 1
        if with_bwd and wrapped:
            P.monarch_rectw_bwd(x, dy, L, R, dxs[i % 2], gL, gR, 0, T, q, b1, b, b3, r, ws_b)
        elif with_bwd:
            P.monarch_rect_bwd(x, dy, L, R, dxs[i % 2], gL, gR, 0, T, q, b1, b, r, ws_b, fwd_workspace=ws)
            if dist is not None:
                dist.all_reduce(gL)
                dist.all_reduce(gR)

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    launches0 = P.monarch_launch_count()
    t_start, t_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t_start.record(stream)
    for i in range(args.steps):
        if with_bwd:
            starts[i].record(stream)
        step(args.warmup + i, True)
    t_stop.record(stream)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    total_ms = t_start.elapsed_time(t_stop)
    clocks = sampler.stop()
    launches = P.monarch_launch_count() - launches0
    # a wait that ran out in any kernel of the timed region shows in the status word of the workspace it used
    status = P.monarch_last_device_status(ws) | (P.monarch_last_device_status(ws_b) if with_bwd else 0)
    if dist is not None:
        tmax = torch.tensor([total_ms], device="cuda")
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        total_ms = float(tmax.item())
    ms = total_ms / args.steps
    fwd_ms = statistics.mean(starts[i].elapsed_time(mid[i]) for i in range(args.steps)) if with_bwd else ms
    peaks = load_peaks()
    tfl = flops / (ms * 1e-3) / 1e12
    line = {
        "metric": metric, "value": tfl * world, "unit": unit, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "tokens_per_s": T * world / (ms * 1e-3),
        "config": {"workload": workload, "l2": "inputs larger than L2; 2 rotating buffer sets",
                   "kernels": args.kernels, "device_status": status},
        "clocks": clocks, "gpu_launches": int(launches),
        "calls": {"rect_fwd": {"ms": fwd_ms, "tflops": fwd_flops / fwd_ms / 1e9},
                  **({"rect_bwd": {"ms": ms - fwd_ms, "tflops": 2 * fwd_flops / (ms - fwd_ms) / 1e9}} if with_bwd else {})},
        "roofline": {"bound": "tensor", "kernel": "rect_fwd: rect_stage1_kernel<256> (tcgen05) + "
                                                  + ("relabel_kernel + " if wrapped else "") +
                                                  "rect_stage2_stream_kernel (%d launches)" % (3 if wrapped else 2)
                                                  + ("; rect_bwd: stage 1, adjoint stage 2, adjoint stage 1 (tcgen05), "
                                                     "rect_wgrad_kernel (tcgen05), dl_small4_kernel" if with_bwd else ""),
                     "achieved": tfl, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                     "frac": tfl / peaks["bf16_tflops"], "peak_source": peaks["source"], "traffic": None,
                     "algorithmic_mb": nbytes / 1e6,
                     "hbm_time_ms": nbytes / (peaks["hbm_gbs"] * 1e9) * 1e3},
        "e2e": None,
    }
    if status != 0:
        line["invalid"] = "a device-side wait ran out inside the timed region"
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        rr = time_oracle_rect(d, 12.0)
        line["cpu_baseline"] = {"value": rr["tflops"], "unit": unit, "cores": rr["cores"], "kind": "oracle",
                                "sample": f"first {rr['tokens']} tokens of the workload, {rr['seconds']:.1f} s"}
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


def main_project(args):
    """Workload 7: Algorithm 1 (projection, one rank-1 SVD per m x m slice) followed by Eq. (2) (dense
    materialisation) for n = 4096, m = 64, fp32.  The projection is bound by instruction issue on the CUDA
    cores; its FLOPs are counted from the plane rotations the kernel reports (12 m per rotation: three dot
    products and two column updates of length m)."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    m, n = 64, 4096
    workload = f"workload 7: project+dense f32 n={n} m={m} ({m * m} slices of {m} x {m})"
    metric, unit = "monarch_project_matrices_per_s", "matrices/s"
    import numpy as np
    rng = np.random.default_rng(595007)

    if args.impl == "reference":
        if rank != 0:
            return 0
        from oracle import monarch_oracle as O
        sub = 16                                  # the oracle (numpy SVD per slice) on a 16 x 16-block instance
        A = rng.standard_normal((sub * sub, sub * sub))
        ts = []
        for i in range(args.warmup + args.steps):
            t0 = time.perf_counter()
            L, R = O.project(A, sub)
            O.dense(L, R)
            ts.append(time.perf_counter() - t0)
        dt = statistics.mean(ts[args.warmup:])
        # scale by slice count and the cubic cost of an SVD to the workload's 64 x 64 slices
        est = dt * (m * m) / (sub * sub) * (m / sub) ** 3
        print(json.dumps({
            "impl": "reference", "metric": metric, "value": 1.0 / est, "unit": unit, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": est * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload, "sample": f"m={sub} instance timed ({dt * 1e3:.1f} ms), scaled by "
                                                       "slice count and m^3"},
            "cpu_baseline": {"value": 1.0 / est, "unit": unit, "cores": 1, "kind": "oracle",
                             "sample": f"m={sub} instance, scaled"},
            "e2e": {"value": 1.0 / est, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))
        return 0

    import torch
    import __graft_entry__ as entry
    entry.build()
    import paper_2204_00595_b200 as P
    torch.cuda.set_device(local_rank)
    A = torch.from_numpy(rng.standard_normal((n, n), dtype=np.float32)).cuda()
    L = torch.empty(m, m, m, device="cuda")
    R = torch.empty_like(L)
    M = torch.empty_like(A)
    rot = torch.zeros(1, dtype=torch.int64, device="cuda")
    stream = torch.cuda.current_stream()
    for _ in range(args.warmup):
        P.monarch_project(A, L, R, n, m)
        P.monarch_dense(L, R, M, n, m)
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    sampler.start()
    launches0 = P.monarch_launch_count()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * args.steps + 1)]
    ev[0].record(stream)
    for i in range(args.steps):
        P.monarch_project(A, L, R, n, m, rotation_count=rot)
        ev[2 * i + 1].record(stream)
        P.monarch_dense(L, R, M, n, m)
        ev[2 * i + 2].record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    launches = P.monarch_launch_count() - launches0
    t_proj = statistics.mean(ev[2 * i].elapsed_time(ev[2 * i + 1]) for i in range(args.steps))
    t_dense = statistics.mean(ev[2 * i + 1].elapsed_time(ev[2 * i + 2]) for i in range(args.steps))
    ms = ev[0].elapsed_time(ev[-1]) / args.steps
    flops = int(rot.item()) / args.steps * 12 * m
    sm_mhz = clocks.get("sm_max_mhz") or 1965
    alu_peak = 148 * 128 * 2 * sm_mhz * 1e6 / 1e12          # fp32 FMA lanes x 2 FLOP x clock
    line = {
        "metric": metric, "value": world / (ms * 1e-3), "unit": unit, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload, "l2": "A (67 MB) + M (67 MB) exceed L2"},
        "clocks": clocks, "gpu_launches": int(launches),
        "calls": {"project": {"ms": t_proj, "rotations": int(rot.item()) // args.steps,
                              "tflops": flops / t_proj / 1e9},
                  "dense": {"ms": t_dense, "gbs": n * n * 4 / t_dense / 1e6}},
        "roofline": {"bound": "alu", "kernel": "project_kernel<float, 64>", "achieved": flops / t_proj / 1e9,
                     "peak": alu_peak, "unit": "TFLOP/s", "frac": flops / t_proj / 1e9 / alu_peak,
                     "peak_source": "148 SMs x 128 fp32 FMA lanes x 2 FLOP x max SM clock", "traffic": None},
        "e2e": None,
    }
    if rank == 0:
        print(json.dumps(line))
    return 0


def main_cplx(args):
    """Workload 8: complex Monarch multiply on planar bf16 tensors, n = 4096, m = 64, 8192 tokens: y = M x followed by
    z = M^H y (the two halves of an MM* product).  Algorithmic work per call: 16 n m FLOP per token (a complex
    multiply-add is four real ones) and 2 x 2 n s bytes (two planes in, two out)."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    import numpy as np
    m, n, T = 64, 4096, 8192
    flops = 2 * 16 * n * m * T
    nbytes = 2 * (4 * T * n * 2 + 4 * n * m * 2)
    workload = f"workload 8: cplx_fwd + adjoint bf16 (planar) n={n} m={m} tokens/GPU={T}"
    metric, unit = "monarch_cplx_tflops", "TFLOP/s"
    rng = np.random.default_rng(595008)

    def draw(shape, std):
        from paper_2204_00595_b200.inputs import round_to_storage
        return round_to_storage(rng.standard_normal(shape, dtype=np.float32) * np.float32(std), "bf16")

    x = draw((2, T, n), 1.0)
    L, R = draw((2, m, m, m), 1.0 / np.sqrt(2 * m)), draw((2, m, m, m), 1.0 / np.sqrt(2 * m))

    def time_oracle_cplx(target_s):
        from oracle import monarch_oracle as O
        Lc, Rc = L[0] + 1j * L[1], R[0] + 1j * R[1]
        Ts = 8
        while True:
            xc = x[0, :Ts] + 1j * x[1, :Ts]
            t0 = time.perf_counter()
            O.cplx_fwd(O.cplx_fwd(xc, Lc, Rc), Lc, Rc, adjoint=True)
            dt = time.perf_counter() - t0
            if dt >= target_s / 4 or Ts >= T:
                break
            Ts = min(T, Ts * 4)
        return {"tflops": flops * Ts / T / dt / 1e12, "tokens": Ts, "seconds": dt, "cores": os.cpu_count()}

    if args.impl == "reference":
        if rank != 0:
            return 0
        rs = [time_oracle_cplx(8.0) for _ in range(args.warmup + args.steps)][args.warmup:]
        tfl = statistics.mean(r["tflops"] for r in rs)
        print(json.dumps({
            "impl": "reference", "metric": metric, "value": tfl, "unit": unit, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": statistics.mean(r["seconds"] for r in rs) * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "c128", "data": "synthetic",
            "config": {"workload": workload, "sample_tokens_per_step": rs[-1]["tokens"]},
            "cpu_baseline": {"value": tfl, "unit": unit, "cores": rs[-1]["cores"], "kind": "oracle",
                             "sample": f"{rs[-1]['tokens']} tokens of the workload per step (numpy einsum)"},
            "e2e": {"value": tfl, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))
        return 0

    import torch
    import __graft_entry__ as entry
    entry.build()
    import paper_2204_00595_b200 as P
    from paper_2204_00595_b200.inputs import to_device
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dx, dL, dR = to_device(x, "bf16"), to_device(L, "bf16"), to_device(R, "bf16")
    y, z = torch.empty_like(dx), torch.empty_like(dx)
    ws = P.Workspace(P.monarch_workspace_bytes(P.OP_CPLX, T, n, m, P.BF16))
    stream = torch.cuda.current_stream()

    def step():
        P.monarch_cplx_fwd(dx, dL, dR, y, 0, T, n, m, ws)
        P.monarch_cplx_fwd(y, dL, dR, z, 1, T, n, m, ws)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    launches0 = P.monarch_launch_count()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0.record(stream)
    for _ in range(args.steps):
        step()
    t1.record(stream)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    total_ms = t0.elapsed_time(t1)
    clocks = sampler.stop()
    launches = P.monarch_launch_count() - launches0
    status = P.monarch_last_device_status(ws)
    if dist is not None:
        tmax = torch.tensor([total_ms], device="cuda")
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        total_ms = float(tmax.item())
    ms = total_ms / args.steps
    peaks = load_peaks()
    line = {
        "metric": metric, "value": flops * world / (ms * 1e-3) / 1e12, "unit": unit, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "tokens_per_s": T * world / (ms * 1e-3),
        "config": {"workload": workload, "l2": "each call streams > 1 GB of planes and partial results",
                   "device_status": status},
        "clocks": clocks, "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": "per call: 4 x fused_fwd_m64_team_kernel (or fused_bwd_dx_m64_kernel) "
                                               "on 2 x tokens rows + cplx_combine_kernel",
                     "achieved": nbytes / ms / 1e6, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": nbytes / ms / 1e6 / peaks["hbm_gbs"], "peak_source": peaks["source"], "traffic": None,
                     "algorithmic_mb": nbytes / 1e6},
        "e2e": None,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        rr = time_oracle_cplx(12.0)
        line["cpu_baseline"] = {"value": rr["tflops"], "unit": unit, "cores": rr["cores"], "kind": "oracle",
                                "sample": f"first {rr['tokens']} tokens of the workload, {rr['seconds']:.1f} s"}
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


def launch_ranks(args):
    """`python bench.py --gpus N` outside a launcher: start N ranks of this script under torch.distributed.run
    (one per GPU, NCCL rendezvous on 127.0.0.1) and pass rank 0's JSON line through."""
    import socket
    import subprocess
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def default_calls(cfg, requested):
    calls = list(cfg.ops)
    if requested:
        # the backward of the feed-forward block is an optional extra call of the workload that has the block
        extra = ["mlp_bwd"] if "mlp_fwd" in calls else []
        return [k for k in calls + extra if k in requested.split(",")]
    if calls == ["fwd", "bwd_dx", "bwd_dw"]:
        # default: the backward pass as one call (dx, dL, dR) that reuses the intermediate the forward
        # call left in its workspace; --calls fwd,bwd_dx,bwd_dw times the three separate entry points
        return ["fwd", "bwd"]
    return calls


def measure(P, torch, dist, cfg, calls, steps, warmup, rank, local_rank, sample_clocks):
    """Time `steps` steps of `calls` on workload `cfg` (device-resident inputs, CUDA events on the launching
    stream, rotating buffer sets).  Returns the step time, per-call figures and what the run needs to report."""
    from paper_2204_00595_b200.inputs import make_inputs, to_device
    n, m, T = cfg.n, cfg.m, cfg.tokens
    code = P.F32 if cfg.dtype == "f32" else P.BF16
    d = make_inputs(cfg.index, with_dy="mlp_bwd" in calls)   # every rank draws the same recipe, then offsets it
    # Rotating sets of token tensors so that no launch finds its operands in L2 from the previous step: enough
    # sets that together they hold at least 512 MB (each set of workloads 3-5 alone exceeds the 126 MB L2).
    per_set = T * n * esize(cfg.dtype) * (4 if "dy" in d else 2)
    SETS = max(2, min(8, -(-(512 << 20) // per_set))) if per_set < (1 << 30) else 1
    sets = []
    for s in range(SETS):
        x = to_device(d["x"], cfg.dtype)
        if s or rank:
            x = torch.roll(x, shifts=17 * s + 5 * rank, dims=0).contiguous()
        e = {"x": x, "y": torch.empty_like(x)}
        if "dy" in d:
            e["dy"] = torch.roll(to_device(d["dy"], cfg.dtype), shifts=3 * s + rank, dims=0).contiguous()
            e["dx"] = torch.empty_like(x)
        sets.append(e)
    W = {k: to_device(d[k], cfg.dtype) for k in ("L", "R", "L2", "R2", "b1", "b2") if k in d}
    grads = torch.zeros(2, m, m, m, dtype=torch.float32, device="cuda")   # packed (dL, dR)
    mlp_grads = ([torch.zeros(m, m, m, dtype=torch.float32, device="cuda") for _ in range(4)] +
                 [torch.zeros(n, dtype=torch.float32, device="cuda") for _ in range(2)]) if "mlp_bwd" in calls else []
    op_of = {"fwd": P.OP_FWD, "bwd_dx": P.OP_BWD_DX, "bwd_dw": P.OP_BWD_DW, "mlp_fwd": P.OP_MLP_FWD,
             "bwd": P.OP_BWD, "mlp_bwd": P.OP_MLP_BWD}
    ws = P.Workspace(max([P.monarch_workspace_bytes(op_of[k], T, n, m, code) for k in calls if k != "bwd"]
                         + [256]))
    ws_b = P.Workspace(P.monarch_workspace_bytes(P.OP_BWD, T, n, m, code)) if "bwd" in calls else None
    stream = torch.cuda.current_stream()

    # One boundary event between consecutive calls (pre-created: nothing but the records sits between two
    # launches): call k of a timed step runs between marks[j] and marks[j+1].
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(steps * len(calls) + 1)]
    nmark = [0]

    def step(i, timed):
        e = sets[i % SETS]
        for k in calls:
            if k == "fwd":
                P.monarch_fwd(e["x"], W["L"], W["R"], e["y"], T, n, m, ws)
            elif k == "bwd_dx":
                P.monarch_bwd_dx(e["dy"], W["L"], W["R"], e["dx"], T, n, m, ws)
            elif k == "bwd_dw":
                P.monarch_bwd_dw(e["x"], e["dy"], W["L"], W["R"], grads[0], grads[1], 0, T, n, m, ws)
                if dist is not None:
                    dist.all_reduce(grads)
            elif k == "bwd":
                P.monarch_bwd(e["x"], e["dy"], W["L"], W["R"], e["dx"], grads[0], grads[1], 0, T, n, m,
                              ws_b, fwd_workspace=ws)
                if dist is not None:
                    dist.all_reduce(grads)
            elif k == "mlp_fwd":
                P.monarch_mlp_fwd(e["x"], W["L"], W["R"], W["b1"], W["L2"], W["R2"], W["b2"],
                                  e["y"], T, n, m, ws)
            elif k == "mlp_bwd":
                g = mlp_grads
                P.monarch_mlp_bwd(e["x"], e["dy"], W["L"], W["R"], W["b1"], W["L2"], W["R2"], e["dx"],
                                  g[0], g[1], g[4], g[2], g[3], g[5], 0, T, n, m, ws)
                if dist is not None:
                    for t in g:
                        dist.all_reduce(t)
            if timed:
                nmark[0] += 1
                marks[nmark[0]].record(stream)

    for i in range(warmup):
        step(i, False)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    sampler = ClockSampler(local_rank) if sample_clocks else None
    if sampler:
        sampler.start()
    launches0 = P.monarch_launch_count()
    torch.cuda.synchronize()
    t_start = torch.cuda.Event(enable_timing=True)
    t_stop = torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    marks[0].record(stream)
    for i in range(steps):
        step(warmup + i, True)
    t_stop.record(stream)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    total_ms = t_start.elapsed_time(t_stop)
    clocks = sampler.stop() if sampler else None
    launches = P.monarch_launch_count() - launches0
    # a wait that ran out in any kernel of the timed region shows in the status word of the workspace it used
    status = P.monarch_last_device_status(ws) | (P.monarch_last_device_status(ws_b) if ws_b is not None else 0)
    if dist is not None:
        tmax = torch.tensor([total_ms], device="cuda")
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        total_ms = float(tmax.item())
    ms_per_step = total_ms / steps

    peaks = load_peaks()
    per_call = {}
    for ci, k in enumerate(calls):
        ts = [marks[st * len(calls) + ci].elapsed_time(marks[st * len(calls) + ci + 1]) for st in range(steps)]
        ms = statistics.mean(ts)
        by = call_bytes(k, n, m, T, cfg.dtype)
        fl = call_flops(k, n, m, T)
        roof_ms = max(by / (peaks["hbm_gbs"] * 1e9), fl / (peaks["bf16_tflops"] * 1e12)) * 1e3
        tr = NCU_TRAFFIC_MB.get((cfg.index, k))
        per_call[k] = {"ms": ms, "ms_min": min(ts), "gbs": by / ms / 1e6, "tflops": fl / ms / 1e9,
                       "roofline_ms": roof_ms, "roofline_frac": roof_ms / ms,
                       "impl": P.monarch_impl_name(op_of[k], m, code),
                       "kernels": KERNELS_OF.get((m, cfg.dtype, k)),
                       "algorithmic_mb": by / 1e6,
                       "traffic_mb": tr[0] if tr else None, "traffic_note": tr[1] if tr else None}
    return {"ms_per_step": ms_per_step, "calls": per_call, "clocks": clocks, "launches": int(launches),
            "status": int(status), "sets": SETS, "inputs": d, "weights": W, "grads": grads}


def main():
    args = parse_args()
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return launch_ranks(args)
    if args.workload == 8:
        return main_cplx(args)
    if args.workload in (6, 9):
        return main_rect(args)
    if args.workload == 7:
        return main_project(args)
    from paper_2204_00595_b200.inputs import CONFIGS, make_inputs
    cfg = CONFIGS[args.workload]
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    calls = default_calls(cfg, args.calls)
    n, m, T = cfg.n, cfg.m, cfg.tokens
    workload = (f"workload {cfg.index}: {'+'.join(calls)} {cfg.dtype} n={n} m={m} "
                f"tokens/GPU={T}")
    metric, unit = "monarch_fwd_bwd_tflops", "TFLOP/s"
    step_flops = sum(call_flops(k, n, m, T) for k in calls)

    if args.impl == "reference":
        if rank != 0:
            return 0
        import __graft_entry__ as entry
        from oracle import monarch_oracle as O
        O.build()
        d = make_inputs(cfg.index, with_dy="mlp_bwd" in calls)
        # every step runs the oracle on the same bounded sample: sized once (first step) so that warm-up plus timed
        # steps take about two minutes, whatever --steps is
        times, sample = [], None
        per_step = max(0.05, min(8.0, 120.0 / (args.warmup + args.steps)))
        for i in range(args.warmup + args.steps):
            r = time_oracle(cfg, d, target_s=per_step, calls=calls, tokens=sample["tokens"] if sample else None)
            sample = r
            if i >= args.warmup:
                times.append(r)
        tfl = statistics.mean(r["tflops"] for r in times)
        tps = statistics.mean(r["tokens_per_s"] for r in times)
        ms = statistics.mean(r["seconds"] for r in times) * 1e3
        line = {
            "impl": "reference", "metric": metric, "value": tfl, "unit": unit, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "tokens_per_s": tps,
            "config": {"workload": workload, "sample_tokens_per_step": sample["tokens"]},
            "cpu_baseline": {"value": tfl, "unit": unit, "cores": sample["cores"], "kind": "oracle",
                             "sample": f"{sample['tokens']} tokens of the workload per step"},
            "e2e": {"value": tfl, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        }
        print(json.dumps(line))
        return 0

    import torch
    import __graft_entry__ as entry
    entry.build()
    import paper_2204_00595_b200 as P
    from paper_2204_00595_b200.inputs import to_device

    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    P.monarch_set_impl({"auto": P.IMPL_AUTO, "staged": P.IMPL_STAGED, "fused": P.IMPL_FUSED}[args.kernels])
    code = P.F32 if cfg.dtype == "f32" else P.BF16

    res = measure(P, torch, dist, cfg, calls, args.steps, args.warmup, rank, local_rank, True)
    d, W, grads = res.pop("inputs"), res.pop("weights"), res.pop("grads")
    ms_per_step, per_call = res["ms_per_step"], res["calls"]
    value = step_flops * world / (ms_per_step * 1e-3) / 1e12
    tokens_per_s = T * world / (ms_per_step * 1e-3)

    peaks = load_peaks()
    dom = max(calls, key=lambda k: per_call[k]["ms"])
    roofline = {
        "bound": "hbm", "kernel": f"{dom}: {per_call[dom]['kernels'] or per_call[dom]['impl']}",
        "achieved": per_call[dom]["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
        "frac": per_call[dom]["gbs"] / peaks["hbm_gbs"], "peak_source": peaks["source"],
        "traffic": per_call[dom]["traffic_mb"],
        "traffic_unit": "MB per call (dram__bytes_read.sum + dram__bytes_write.sum, summed over the "
                        "call's kernels, from the ncu capture named in the call's traffic_note)",
        "algorithmic_mb": per_call[dom]["algorithmic_mb"],
    }

    line = {
        "metric": metric, "value": value, "unit": unit, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
        "tokens_per_s": tokens_per_s,
        "config": {"workload": workload, "l2": f"inputs larger than L2; {res['sets']} rotating buffer sets",
                   "kernels": args.kernels, "device_status": res["status"]},
        "clocks": res["clocks"], "gpu_launches": res["launches"], "roofline": roofline, "calls": per_call,
    }

    # The other workloads of the contract, timed the same way with fewer steps (per call: time, fraction of the
    # roofline, kernels, algorithmic and measured DRAM megabytes).  The headline above is the largest
    # forward + backward configuration; these entries carry the rest.
    if args.side_workloads and not args.calls:
        side = {str(cfg.index): {"calls": per_call, "ms_per_step": ms_per_step, "steps": args.steps}}
        for idx in (1, 2, 3, 4, 5):
            if idx == cfg.index:
                continue
            c2 = CONFIGS[idx]
            k2 = default_calls(c2, "")
            torch.cuda.empty_cache()
            steps2 = max(20, min(args.steps, 200))
            r2 = measure(P, torch, dist, c2, k2, steps2, max(args.warmup, 3), rank, local_rank, False)
            for key in ("inputs", "weights", "grads"):
                r2.pop(key)
            side[str(idx)] = {"calls": r2["calls"], "ms_per_step": r2["ms_per_step"], "steps": steps2,
                              "device_status": r2["status"], "gpu_launches": r2["launches"],
                              "workload": f"{'+'.join(k2)} {c2.dtype} n={c2.n} m={c2.m} tokens/GPU={c2.tokens}"}
            line["config"]["device_status"] |= r2["status"]
        line["workloads"] = dict(sorted(side.items()))
    if line["config"]["device_status"] != 0:
        line["invalid"] = "a device-side wait ran out inside the timed region"

    if not args.no_e2e:
        e2e = None
        if "fwd" in calls and ("bwd" in calls or "bwd_dw" in calls):
            # the same step through the host-buffer entry point: pinned host tensors in, host tensors
            # out, uploads and downloads inside the timed region (wall clock around blocking calls)
            torch.cuda.empty_cache()
            hx = torch.roll(to_device(d["x"], cfg.dtype), 5 * rank, 0).cpu().pin_memory()
            hdy = torch.roll(to_device(d["dy"], cfg.dtype), rank, 0).cpu().pin_memory()
            hL, hR = W["L"].cpu().pin_memory(), W["R"].cpu().pin_memory()
            hy, hdx = torch.empty_like(hx).pin_memory(), torch.empty_like(hx).pin_memory()
            hg = torch.empty(2, m, m, m, dtype=torch.float32).pin_memory()
            ctx = P.HostContext(T, n, m, code)

            def host_step():
                ctx.fwd_bwd(hx, hdy, hL, hR, hy, hdx, hg[0], hg[1], T)
                if dist is not None:
                    grads.copy_(hg, non_blocking=True)
                    dist.all_reduce(grads)
                    hg.copy_(grads, non_blocking=True)
                    torch.cuda.synchronize()

            for _ in range(3):
                host_step()
            torch.cuda.synchronize()
            if dist is not None:
                dist.barrier()
            k_e2e = max(1, min(args.steps, 10))
            t0 = time.perf_counter()
            for _ in range(k_e2e):
                host_step()
            torch.cuda.synchronize()
            dt = (time.perf_counter() - t0) / k_e2e
            if dist is not None:
                tmax = torch.tensor([dt], device="cuda")
                dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
                dt = float(tmax.item())
            act = T * n * esize(cfg.dtype)
            wbytes = n * m * esize(cfg.dtype)
            e2e = {"value": step_flops * world / dt / 1e12, "unit": unit, "ms_per_step": dt * 1e3,
                   "h2d_bytes_per_step": 2 * act + 2 * wbytes, "d2h_bytes_per_step": 2 * act + 2 * n * m * 4,
                   "steps": k_e2e, "api": "monarch_host_fwd_bwd (pinned host tensors, chunked 3-stream staging)",
                   "timer": "host wall clock around blocking calls"}
            ctx.close()
        line["e2e"] = e2e
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        r = time_oracle(cfg, d, calls=calls)
        line["cpu_baseline"] = {"value": r["tflops"], "unit": unit, "cores": r["cores"],
                                "kind": "oracle", "tokens_per_s": r["tokens_per_s"],
                                "sample": f"first {r['tokens']} tokens of the workload, "
                                          f"{r['seconds']:.1f} s"}
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
