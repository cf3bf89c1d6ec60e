#!/usr/bin/env python
"""Benchmark of the W4A4 linear hot path (transform + quant + MXFP4 GEMM).

One "step" is one pass of the whole path over one batch: for each projection of
the workload, the fused activation transform/clip/quantiser kernel followed by
the block-scaled tensor-core GEMM, on seeded synthetic inputs.  Prints ONE JSON
line (rank 0).  `--impl reference` times the CPU oracle instead, on a bounded
sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2603_16590_b200 import synth  # noqa: E402

METRIC = "w4a4_linear_tflops"
UNIT = "TFLOP/s"
WORKLOADS = {
    # name: (tokens, projections, vision-row fraction, outlier-channel fraction)
    "cfg1_llama8b_prefill": (2048, synth.LLAMA8B_PREFILL, 0.0, 0.01),
    "cfg3_qwen2vl7b_prefill": (8192, synth.QWEN2VL7B_PREFILL, 0.75, 0.005),
    "cfg0_single_layer": (128, [("lin", 1024, 1024)], 0.0, 0.01),
    # single-kernel cases for profiler captures (m = 0: quantiser only, input larger than L2)
    "profile_gemm_gate_up": (2048, [("gate_up", 4096, 28672)], 0.0, 0.01),
    "profile_gemm_down": (2048, [("down", 14336, 4096)], 0.0, 0.01),
    "profile_quant_32768x4096": (32768, [("quant", 4096, 0)], 0.0, 0.01),
}
FP4_OVER_BF16 = 4.0  # nominal dense peak ratio 9 / 2.25 PFLOP/s


def workload_flops(S, projs):
    return sum(2.0 * S * n * m for _, n, m in projs)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p["bf16_tflops_sustained"], "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def make_inputs(workload, seed):
    S, projs, vis_frac, och = WORKLOADS[workload]
    layers = []
    for i, (name, n, m) in enumerate(projs):
        xb = synth.make_activations(S, n, seed + 16 * i, outlier_channel_frac=och, vision_rows=int(S * vis_frac))
        t = synth.make_transform(n, seed + 16 * i + 1, "baseline")
        layers.append({"name": name, "n": n, "m": m, "x_bits": xb, "t": t, "w_seed": seed + 16 * i + 2})
    return S, layers


# ------------------------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU during the timed region (read-only NVML
    queries from a thread, every ~2 ms; falls back to one nvidia-smi query if NVML is missing)."""
    REASONS = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}

    def __init__(self, index):
        self.index, self.sm, self.reasons, self.power = index, [], set(), []
        self._stop = threading.Event()
        self._thread = None
        self.max_mhz = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = int(vis.split(",")[index]) if vis and vis.split(",")[index].isdigit() else index
            self.h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                for name, bit in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
                self.power.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvml unavailable"], "samples": 0}
        self._stop.set()
        self._thread.join()
        return {"sm_mhz": float(np.median(self.sm)) if self.sm else None, "sm_min_mhz": min(self.sm) if self.sm else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.sm),
                "power_w_max": max(self.power) if self.power else None}


# ------------------------------------------------------------------------------------ oracle arm
def oracle_sample(workload, seed, rows, feats):
    """A bounded sample of the workload for the CPU oracle: the first projection,
    `rows` token rows and `feats` output features (weights prepared offline)."""
    from oracle import batq_oracle as O
    S, projs, vis_frac, och = WORKLOADS[workload]
    name, n, m = projs[0]
    rows, feats = min(rows, S), min(feats, m)
    xb = synth.make_activations(rows, n, seed, outlier_channel_frac=och, vision_rows=int(rows * vis_frac))
    t = synth.make_transform(n, seed + 1, "baseline")
    wb = synth.make_weight(feats, n, seed + 2)
    qw = O.prepare_weight(wb, t.left, t.right)

    def step():
        qx = O.quantize_act(xb, t.left, t.right, t.clip_lo, t.clip_hi)
        return O.gemm_mxfp4(qx[0], qx[1], qw[0], qw[1])[0]

    flops = 2.0 * rows * n * feats
    desc = f"{name} projection, {rows} of {S} token rows x {n} -> {feats} of {m} features (weights prepared offline)"
    return step, flops, desc


def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


def time_oracle(workload, seed, rows, feats, steps, warmup):
    step, flops, desc = oracle_sample(workload, seed, rows, feats)
    for _ in range(warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    dt = (time.perf_counter() - t0) / max(steps, 1)
    return flops / dt / 1e12, dt, desc


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    S, projs, _, _ = WORKLOADS[args.workload]
    val, dt, desc = time_oracle(args.workload, synth.BASE_SEED, 256, 1024, args.steps, args.warmup)
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "tokens": S, "projections": [list(p) for p in projs]},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle", "sample": desc},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------ CUDA arm
def run_ours(args):
    import torch
    from paper_2603_16590_b200 import binding as B

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    B.load()
    B.batq_debug_force_tile_width(args.tile_width)
    B.batq_debug_set_gemm_flags(args.gemm_debug_flags)
    B.batq_debug_force_quantizer(args.quantizer)
    peaks = load_peaks()

    # weak scaling: every rank runs the same workload on its own seeded batch, no exchange step
    S, layers = make_inputs(args.workload, synth.BASE_SEED + 1000 * rank)
    projs = WORKLOADS[args.workload][1]
    for L in layers:
        L["tr"] = B.batq_transform_create(L["n"], L["t"].left, L["t"].right, L["t"].clip_lo, L["t"].clip_hi)
        L["x"] = B.bits_to_cuda_bf16(L["x_bits"])
        L["codes"] = torch.empty((S, L["n"] // 2), dtype=torch.uint8, device="cuda")
        L["sf"] = torch.empty(B.batq_sf_bytes(S, L["n"], B.SF_MMA), dtype=torch.uint8, device="cuda")
        if L["m"] == 0:
            continue
        wdev = B.bits_to_cuda_bf16(synth.make_weight(L["m"], L["n"], L["w_seed"]))
        L["w"] = B.batq_prepare_weight(L["tr"], wdev)
        del wdev
        L["y"] = torch.empty((S, L["m"]), dtype=torch.bfloat16, device="cuda")
        L["ws"] = B.aligned_workspace(B.batq_linear_workspace_bytes(L["w"], S))
        L["x_host"] = torch.from_numpy(L["x_bits"].view(np.int16)).pin_memory()
        L["y_host"] = torch.empty((S, L["m"]), dtype=torch.bfloat16).pin_memory()
    torch.cuda.synchronize()
    flops_step = workload_flops(S, projs)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms):
        if world == 1:
            return ms
        t = torch.tensor([ms], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    # ---- device-resident arm: quantise + GEMM per projection, events around every launch
    ev = lambda: torch.cuda.Event(enable_timing=True)
    marks = [[(ev(), ev(), ev()) for _ in layers] for _ in range(args.steps)]

    def step(m=None):
        for i, L in enumerate(layers):
            if m is not None:
                m[i][0].record()
            B.batq_quantize_act(L["tr"], L["x"], L["codes"], L["sf"], B.SF_MMA)
            if m is not None:
                m[i][1].record()
            if L["m"]:
                B.batq_gemm_mxfp4(L["codes"], L["sf"], L["w"], S, L["y"])
            if m is not None:
                m[i][2].record()

    for _ in range(args.warmup):
        step()
    sampler = ClockSampler(local)
    barrier()
    if rank == 0:
        sampler.start()
    e0, e1 = ev(), ev()
    e0.record()
    for k in range(args.steps):
        step(marks[k])
    e1.record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    ms = max_over_ranks(e0.elapsed_time(e1))
    status = B.batq_last_device_status()
    if status != 0:
        raise SystemExit(f"device status {status} after the timed region")
    q_ms = np.array([[m[i][0].elapsed_time(m[i][1]) for i in range(len(layers))] for m in marks]).mean(axis=0)
    g_ms = np.array([[m[i][1].elapsed_time(m[i][2]) for i in range(len(layers))] for m in marks]).mean(axis=0)

    # ---- end-to-end arm: host buffers in, host buffers out, through the C-ABI host entry point
    def step_host():
        for L in layers:
            if L["m"] == 0:
                continue
            B.batq_linear_w4a4_host(L["tr"], L["w"], L["x_host"], L["y_host"], L["x"], L["y"], L["ws"])

    e2e_steps = max(1, min(args.steps, 5))
    for _ in range(2):
        step_host()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        step_host()
    torch.cuda.synchronize()
    e2e_ms = max_over_ranks((time.perf_counter() - t0) * 1e3)
    h2d = sum(S * L["n"] * 2 for L in layers)
    d2h = sum(S * L["m"] * 2 for L in layers)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    value = flops_step * args.steps * world / (ms * 1e-3) / 1e12
    fp4_peak = peaks["bf16_tflops_sustained"] * FP4_OVER_BF16
    gemm_flops = [2.0 * S * L["n"] * L["m"] for L in layers]
    gemm_achieved = sum(gemm_flops) / (max(g_ms.sum(), 1e-9) * 1e-3) / 1e12
    q_bytes = [S * L["n"] * 2.53125 for L in layers]
    quant_gbs = sum(q_bytes) / (q_ms.sum() * 1e-3) / 1e9
    cpu_val, cpu_dt, cpu_desc = time_oracle(args.workload, synth.BASE_SEED, 256, 1024, 3, 1)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "mxfp4", "data": "synthetic",
        "config": {"workload": args.workload, "tokens": S, "projections": [list(p) for p in projs],
                   "transform": "shared 4x4 (x) private 8x8 per 32-group, clip U[0.8,1]", "output": "bf16",
                   "l2": "inputs larger than L2: one step touches %.0f MB" % (
                       (h2d + d2h + sum(L["n"] * L["m"] * 0.53125 for L in layers)) / 1e6)},
        "roofline": {"bound": "tensor", "kernel": "gemm_mxfp4_kernel", "achieved": gemm_achieved, "peak": fp4_peak,
                     "unit": "TFLOP/s", "frac": gemm_achieved / fp4_peak, "traffic": None,
                     "peak_source": "%s bf16 sustained x %.0f (nominal fp4:bf16)" % (peaks["source"], FP4_OVER_BF16)},
        "act_quant": {"bound": "hbm", "kernel": "quantize_act_kernel", "achieved": quant_gbs, "peak": peaks["hbm_gbs"],
                      "unit": "GB/s", "frac": quant_gbs / peaks["hbm_gbs"], "peak_source": peaks["source"]},
        "kernels": [{"name": L["name"], "n": L["n"], "m": L["m"], "quant_us": float(q_ms[i] * 1e3),
                     "quant_gbs": q_bytes[i] / (q_ms[i] * 1e-3) / 1e9, "gemm_us": float(g_ms[i] * 1e3),
                     "gemm_tflops": gemm_flops[i] / (max(g_ms[i], 1e-9) * 1e-3) / 1e12} for i, L in enumerate(layers)],
        "cpu_baseline": {"value": cpu_val, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                         "sample": cpu_desc},
        "e2e": {"value": flops_step * e2e_steps * world / (e2e_ms * 1e-3) / 1e12, "unit": UNIT,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "gpu_launches": 2 * len(layers) * args.steps,
        "clocks": clocks,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg1_llama8b_prefill", choices=sorted(WORKLOADS))
    ap.add_argument("--gemm-debug-flags", type=int, default=0, help="timing experiments only; results invalid")
    ap.add_argument("--quantizer", type=int, default=0, help="0 auto, 1 ALU kernel, 2 tensor-core kernel (tuning)")
    ap.add_argument("--tile-width", type=int, default=0, help="force the GEMM tile width (tuning); 0 = automatic")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
