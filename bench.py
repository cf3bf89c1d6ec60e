#!/usr/bin/env python
"""Benchmark of the W4A4 linear hot path (transform + clip + MXFP4 quantise + MXFP4 GEMM).

One "step" is one pass of the whole path over one batch of seeded synthetic input: for each
projection of the workload, the activation transform/clip/quantiser kernel followed by the
block-scaled tensor-core GEMM (prefill workloads), the whole-layer call (decode workload), or
the quantiser alone (quantiser sweep).  Prints ONE JSON line (rank 0).  `--impl reference`
times the CPU oracle instead, on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2603_16590_b200 import synth  # noqa: E402

METRIC = "w4a4_linear_tflops"
UNIT = "TFLOP/s"
FP4_OVER_BF16 = 4.0       # nominal dense peak ratio 9 / 2.25 PFLOP/s
QUANT_BYTES_PER_ELEM = 2.53125   # 2 (bf16 in) + 0.5 (codes) + 1/32 (scale byte)
WEIGHT_BYTES_PER_ELEM = 0.53125  # 0.5 (codes) + 1/32 (scale byte)
EVENT_EVERY = 8                  # prefill: every 8th timed step carries per-launch events
MIN_BRACKETED = 50               # prefill: at least this many bracketed steps (extra ones follow the timed region)
NOMINAL_FP4_TFLOPS = 9000.0      # vendor figure for dense FP4 at the maximum SM clock (context, not the denominator)
# The CPU oracle is timed on this fixed sample of the workload's first projection (rows, output features)
ORACLE_SAMPLE = {"prefill": (512, 4096), "decode": (16, 4096), "quant": (2048, 0)}

# kind, tokens, projections (name, n in, m out), vision-row fraction, outlier-channel fraction
WORKLOADS = {
    "cfg0_single_layer": ("prefill", [128], [("lin", 1024, 1024)], 0.0, 0.01),
    "cfg1_llama8b_prefill": ("prefill", [2048], synth.LLAMA8B_PREFILL, 0.0, 0.01),
    "cfg2_llama8b_decode": ("decode", [1, 4, 16], synth.LLAMA8B_PREFILL, 0.0, 0.01),
    "cfg3_qwen2vl7b_prefill": ("prefill", [8192], synth.QWEN2VL7B_PREFILL, 0.75, 0.005),
    "cfg4_quantizer_sweep": ("quant", [1024, 8192, 32768], [("h2048", 2048, 0), ("h4096", 4096, 0), ("h8192", 8192, 0)],
                             0.0, 0.01),
    # the W4A8 settings (MXFP8 activations x MXFP4 weights) on the config-1 shapes
    "cfg1_llama8b_prefill_w4a8": ("prefill", [2048], synth.LLAMA8B_PREFILL, 0.0, 0.01),
    # single-kernel cases for profiler captures (inputs larger than L2, a few hundred MB on the device)
    "profile_gemm_gate_up": ("prefill", [2048], [("gate_up", 4096, 28672)], 0.0, 0.01),
    "profile_gemm_down": ("prefill", [2048], [("down", 14336, 4096)], 0.0, 0.01),
    "profile_quant_32768x4096": ("quant", [32768], [("h4096", 4096, 0)], 0.0, 0.01),
    "profile_decode_gate_up": ("decode", [16], [("gate_up", 4096, 28672)] * 4, 0.0, 0.01),
}

A8_WORKLOADS = {"cfg1_llama8b_prefill_w4a8"}   # activations quantised to MXFP8 (E4M3), GEMM on kind::mxf8f6f4
FP8_OVER_BF16 = 2.0       # nominal dense peak ratio 4.5 / 2.25 PFLOP/s

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum, MB per step = the four GEMM launches of
# cfg1_llama8b_prefill) from the ncu capture summarised under profiles/, valid for the kernel source
# with this hash only.
GEMM_TRAFFIC = {"workload": "cfg1_llama8b_prefill", "mb_per_step": 214.5, "source_sha256": "86454977d11cfd34"}


def kernel_source_hash():
    h = hashlib.sha256()
    for f in ("gemm_mxfp4.cuh", "gemm_mxfp4_pair.cuh", "gemm_mxfp4_wide.cuh", "ptx.cuh"):
        with open(os.path.join(ROOT, "paper_2603_16590_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p["bf16_tflops_sustained"], "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def workload_config(workload):
    """The `config` object of the JSON line: a function of the workload name alone, so that both
    arms (--impl ours / reference) print the same object."""
    kind, tokens, projs, vis_frac, och = WORKLOADS[workload]
    cfg = {"workload": workload, "tokens": tokens[0] if kind == "prefill" else tokens,
           "projections": [list(p) for p in projs],
           "transform": "shared 4x4 (x) private 8x8 per 32-group, clip U[0.8,1]"}
    if workload in A8_WORKLOADS:
        cfg["activations"] = "MXFP8 (E4M3), weights MXFP4"
    if kind == "prefill":
        S = tokens[0]
        touched = sum(S * n * 2 + S * m * 2 + n * m * WEIGHT_BYTES_PER_ELEM for _, n, m in projs)
        cfg.update({"output": "bf16", "l2": "inputs larger than L2: one step touches %.0f MB" % (touched / 1e6)})
    elif kind == "decode":
        copies = 4
        cfg.update({"output": "bf16",
                    "launch": "per token count one CUDA graph of %d layers x %d projections in model order" % (
                        copies, len(projs)),
                    "l2": "%d copies of each prepared weight used in turn: %.0f MB cycle through L2 between reuses" % (
                        copies, copies * sum(n * m * WEIGHT_BYTES_PER_ELEM for _, n, m in projs) / 1e6)})
    else:
        cfg.update({"hidden": [p[1] for p in projs], "ablation": "T = I (plain MXFP4); 8-bit elements (MXFP8)",
                    "l2": "a 256 MB buffer is read between launches (outside the per-launch events)",
                    "value_note": "transform flops (24 per element) over quantiser time; the GB/s figures are the point"})
    return cfg


def make_layer_inputs(workload, S, seed):
    _, _, projs, vis_frac, och = WORKLOADS[workload]
    layers = []
    for i, (name, n, m) in enumerate(projs):
        xb = synth.make_activations(S, n, seed + 16 * i, outlier_channel_frac=och, vision_rows=int(S * vis_frac))
        t = synth.make_transform(n, seed + 16 * i + 1, "baseline")
        layers.append({"name": name, "n": n, "m": m, "x_bits": xb, "t": t, "w_seed": seed + 16 * i + 2})
    return layers


# ------------------------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock, power and throttle reasons of one GPU during the timed region (read-only
    NVML queries from a thread, every ~2 ms)."""
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
    kind, tokens, projs, vis_frac, och = WORKLOADS[workload]
    S = tokens[-1]
    name, n, m = projs[0]
    rows, feats = max(1, min(rows, S)), max(1, min(feats, m if m else 1))
    xb = synth.make_activations(rows, n, seed, outlier_channel_frac=och, vision_rows=int(rows * vis_frac))
    t = synth.make_transform(n, seed + 1, "baseline")
    if kind == "quant":
        def step():
            return O.quantize_act(xb, t.left, t.right, t.clip_lo, t.clip_hi)
        return step, 24.0 * rows * n, f"quantiser only, {rows} of {S} token rows x {n} channels"
    wb = synth.make_weight(feats, n, seed + 2)
    qw = O.prepare_weight(wb, t.left, t.right)

    def step():
        if workload in A8_WORKLOADS:
            qx = O.quantize_act_mxfp8(xb, t.left, t.right, t.clip_lo, t.clip_hi)
            return O.gemm_mxfp8_mxfp4(qx[0], qx[1], qw[0], qw[1])[0]
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


def time_oracle(workload, seed, steps, warmup, threads=None):
    """Times the oracle as it stands on the workload's fixed sample (ORACLE_SAMPLE); `threads`
    limits the BLAS / OpenMP pools it runs on (None = as the libraries choose: all cores).
    Returns (TFLOP/s, seconds per step, sample description, threads used)."""
    kind = WORKLOADS[workload][0]
    rows, feats = ORACLE_SAMPLE[kind]
    step, flops, desc = oracle_sample(workload, seed, rows, feats)

    def run():
        for _ in range(warmup):
            step()
        t0 = time.perf_counter()
        for _ in range(steps):
            step()
        return (time.perf_counter() - t0) / max(steps, 1)

    if threads is None:
        dt, used = run(), oracle_threads()
    else:
        from threadpoolctl import threadpool_limits
        with threadpool_limits(limits=threads):
            dt, used = run(), threads
    return flops / dt / 1e12, dt, desc, used


def cpu_baseline(workload, seed):
    """The oracle on all host cores (3 steps) and on one core (1 step), same fixed sample."""
    val, dt, desc, cores = time_oracle(workload, seed, 3, 1)
    val1, dt1, _, _ = time_oracle(workload, seed, 1, 0, threads=1)
    return {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc, "seconds_per_sample": dt,
            "one_core": {"value": val1, "cores": 1, "seconds_per_sample": dt1}}


def run_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    if args.workload not in WORKLOADS:
        print(json.dumps({"impl": "reference", "unavailable": "the MMA-only measurement has no CPU counterpart"}))
        return
    steps = args.steps if args.steps is not None else 5
    val, dt, desc, cores = time_oracle(args.workload, synth.BASE_SEED, steps, args.warmup)
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(args.workload),
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------ CUDA arm
class Harness:
    """Process-group plumbing shared by the workload kinds: one process per GPU, no data-path
    collective (token rows are independent, so ranks are replicas on their own batches).  The
    benchmark always uses NCCL on CUDA devices; the "gloo" backend exists so that this plumbing
    (rank seeds, barrier, max-over-ranks, whole-job aggregation) can be tested on CPU ranks."""

    def __init__(self, backend="nccl"):
        import torch
        self.torch = torch
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        self.cuda = backend == "nccl"
        if self.cuda:
            if not torch.cuda.is_available():
                raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
            torch.cuda.set_device(self.local)
        self.device = torch.device("cuda", self.local) if self.cuda else torch.device("cpu")
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            if self.cuda:
                dist.init_process_group("nccl", device_id=self.device)
            else:
                dist.init_process_group("gloo")
            self.dist = dist

    def rank_seed(self, base):
        """Weak scaling: every rank draws its own batch."""
        return base + 1000 * self.rank

    def barrier(self):
        if self.cuda:
            self.torch.cuda.synchronize()
        if self.dist is not None:
            self.dist.barrier()
        if self.cuda:
            self.torch.cuda.synchronize()

    def max_over_ranks(self, ms):
        if self.dist is None:
            return ms
        t = self.torch.tensor([ms], dtype=self.torch.float64, device=self.device)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def whole_job_rate(self, units_per_rank_step, steps, ms):
        """Units all ranks processed per second: every rank did `steps` steps of
        `units_per_rank_step`, in the max-over-ranks time `ms`."""
        return units_per_rank_step * steps * self.world / (ms * 1e-3)

    def close(self):
        if self.dist is not None:
            self.dist.destroy_process_group()


def timed_region(h, step, steps, warmup):
    """W warm-up steps, then K steps bracketed by barrier + synchronize, CUDA events on the
    launching stream, clocks sampled meanwhile; returns (ms max over ranks, clocks)."""
    torch = h.torch
    for _ in range(warmup):
        step(None)
    sampler = ClockSampler(h.local)
    h.barrier()
    if h.rank == 0:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for k in range(steps):
        step(k)
    e1.record()
    h.barrier()
    clocks = sampler.stop() if h.rank == 0 else None
    return h.max_over_ranks(e0.elapsed_time(e1)), clocks


def measure_mma_peak(B, torch, iters, a8=False):
    """The block-scaled tensor-core rate with operands resident in shared memory (MMA-only loop, every
    SM busy, nothing loaded or stored): CTA pairs on 256 x 256 tiles and single CTAs on 128 x 256
    tiles, one timed launch each after a short warm-up launch.  a8: kind::mxf8f6f4 (the W4A8 GEMM's
    instruction) instead of kind::mxf4.  For kind::mxf4 also: the CTA-pair GEMM's own issue loop on
    the same resident operands, and the wide-tile GEMM's issue pattern (a second MMA of width 192
    into a second accumulator after every MMA)."""
    def timed(pair, sfc):
        B.batq_debug_mma_peak(pair, 256, max(64, iters // 50), sfc)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        flops = B.batq_debug_mma_peak(pair, 256, iters, sfc)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        return {"tflops": flops / (ms * 1e-3) / 1e12, "ms": ms}
    out = {}
    B.batq_debug_mma_peak_kind(a8)
    try:
        for name, pair, sfc in (("pair_256x256", True, False), ("cta_128x256", False, False),
                                ("pair_256x256_with_scale_copies", True, True), ("cta_128x256_with_scale_copies", False, True)):
            out[name] = timed(pair, sfc)
        if not a8:
            B.batq_debug_mma_peak_gemm_loop(True)
            out["pair_256x256_issued_by_the_gemm_loop"] = timed(True, True)
            B.batq_debug_mma_peak_gemm_loop(False)
            B.batq_debug_mma_peak_second_width(192)
            out["pair_256x448_two_accumulators"] = timed(True, True)
    finally:
        B.batq_debug_mma_peak_kind(False)
        B.batq_debug_mma_peak_gemm_loop(False)
        B.batq_debug_mma_peak_second_width(0)
    if B.batq_last_device_status() != 0:
        raise SystemExit("device status after the MMA-only loop")
    best = max((k for k in ("pair_256x256", "cta_128x256")), key=lambda k: out[k]["tflops"])
    return {"tflops": out[best]["tflops"], "shape": best, "variants": out,
            "how": "tcgen05.mma kind::%s.block_scale only, %d K-steps per CTA (pair), CUDA events"
                   % ("mxf8f6f4" if a8 else "mxf4", iters)}


def measure_mma_with_loads(B, torch, w, iters=8192):
    """A probe of how the tensor cores and the path from L2 into shared memory get along: the MMA-only
    loop with, beside it in every CTA, a TMA load stream of a 256 x 256 pair tile's volume (32 KiB
    of a prepared weight, L2-resident, per K-step) into a ring nobody reads.  No barrier couples
    the two.  Also the two alone, and the MMAs with fewer loads.  Context for the GEMM's fraction,
    not a ceiling: the GEMM's own access pattern takes in more bytes per second than this stream."""
    def timed(it, lit):
        B.batq_debug_mma_peak_with_loads(w, True, 256, min(it, 256), min(lit, 256))
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        flops, nbytes = B.batq_debug_mma_peak_with_loads(w, True, 256, it, lit)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        return {"tflops": flops / (ms * 1e-3) / 1e12, "load_gbs": nbytes / (ms * 1e-3) / 1e9, "ms": ms}
    out = {"mma_and_loads": timed(iters, iters), "loads_only": timed(0, iters), "mma_only": timed(iters, 0),
           "mma_and_three_quarters_of_the_loads": timed(iters, iters * 3 // 4),
           "mma_and_half_the_loads": timed(iters, iters // 2)}
    if B.batq_last_device_status() != 0:
        raise SystemExit("device status after the MMA + loads loop")
    return {"tflops": out["mma_and_loads"]["tflops"], "variants": out,
            "how": "CTA pairs, tcgen05.mma kind::mxf4.block_scale on resident operands (scale copies every K-step) "
                   "and an unsynchronised TMA stream of 32 KiB per K-step and CTA from an L2-resident weight, "
                   "%d K-steps, CUDA events" % iters}


def measure_big_quantizer(B, torch, seed):
    """The quantiser at the largest size of the sweep, 32768 x 8192 (537 MB in, 143 MB out: far larger
    than L2), where it is meant to run at the HBM roofline.  The batch is a 4096-row draw repeated
    eight times (the kernel's time does not depend on the values)."""
    S, N, rep = 32768, 8192, 8
    t = synth.make_transform(N, seed + 901, "baseline")
    tr = B.batq_transform_create(N, t.left, t.right, t.clip_lo, t.clip_hi)
    x = B.bits_to_cuda_bf16(synth.make_activations(S // rep, N, seed + 900)).repeat(rep, 1)
    codes = torch.empty((S, N // 2), dtype=torch.uint8, device="cuda")
    sf = torch.empty(B.batq_sf_bytes(S, N, B.SF_MMA), dtype=torch.uint8, device="cuda")
    marks = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(10)]
    # as in the sweep: a 256 MB buffer is read before each launch (outside the events), so that the
    # timed launch does not also carry the write-back of its predecessor's dirty output lines
    flush = torch.zeros(256 << 18, dtype=torch.int32, device="cuda")
    for k in range(-3, len(marks)):
        flush.sum()
        if k >= 0:
            marks[k][0].record()
        B.batq_quantize_act(tr, x, codes, sf, B.SF_MMA)
        if k >= 0:
            marks[k][1].record()
    torch.cuda.synchronize()
    us = float(np.median([a.elapsed_time(b) for a, b in marks]) * 1e3)
    gbs = S * N * QUANT_BYTES_PER_ELEM / (us * 1e-6) / 1e9
    peaks = load_peaks()
    del x, codes, sf, flush
    return {"tokens": S, "hidden": N, "us": us, "achieved": gbs, "unit": "GB/s", "peak": peaks["hbm_gbs"],
            "frac": gbs / peaks["hbm_gbs"],
            "events": "around each of 10 launches, median; a 256 MB buffer is read between launches"}


def sweep_parity_counts(B, torch, cases, rows_per_case=256):
    """Part of the CPU-oracle leg of the quantiser sweep: for every case, the first and the last
    `rows_per_case` token rows quantised by the library and by the oracle (fp64 transform), codes and
    scale bytes compared.  Plain MXFP4 (T = I) must agree bit for bit; with the transform, the fp32
    arithmetic may move an element next to a rounding boundary to the neighbouring code."""
    from oracle import batq_oracle as O
    out = []
    for L in cases:
        S, n, k = L["S"], L["n"], L["n"] // 32
        rows = np.unique(np.concatenate([np.arange(min(rows_per_case, S)), np.arange(max(0, S - rows_per_case), S)]))
        idx = torch.from_numpy(rows).cuda()
        xb = L["x_bits"][rows]
        t = L["t"]
        rec = {"tokens": S, "hidden": n, "rows_checked": int(len(rows)), "elements_checked": int(len(rows)) * n}
        for name, tr, want in (("gpk", L["tr"], O.quantize_act(xb, t.left, t.right, t.clip_lo, t.clip_hi)),
                               ("identity", None, O.quantize_act(xb, None, None))):
            scales = torch.empty((S, k), dtype=torch.uint8, device="cuda")
            B.batq_quantize_act(tr, L["x"], L["codes"], scales, B.SF_ROWMAJOR)
            gc = O.unpack_codes(L["codes"][idx].cpu().numpy())
            gs = scales[idx].cpu().numpy()
            rec[name + "_code_mismatch"] = int((gc != want[0]).sum())
            rec[name + "_scale_mismatch"] = int((gs != want[1]).sum())
        out.append(rec)
    return out


def run_peak(args, h, B, peaks):
    """--workload peak_mxf4: the MMA-only rate as a burst (one launch of a few ms) and sustained
    (launches back to back for about a second, under the power cap), with the clocks sampled."""
    import torch
    burst = measure_mma_peak(B, torch, 20000)
    burst_a8 = measure_mma_peak(B, torch, 10000, a8=True)
    pair = burst["shape"].startswith("pair")
    wq = B.batq_prepare_weight(None, B.bits_to_cuda_bf16(synth.make_weight(8192, 4096, synth.BASE_SEED + 77)))
    with_loads = measure_mma_with_loads(B, torch, wq)
    sampler = ClockSampler(h.local)
    h.barrier()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n = args.steps if args.steps is not None else 150
    e0.record()
    flops = 0.0
    for _ in range(n):
        flops += B.batq_debug_mma_peak(pair, 256, 20000, False)
    e1.record()
    h.barrier()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1)
    if B.batq_last_device_status() != 0:
        raise SystemExit("device status after the MMA-only loop")
    sustained = flops / (ms * 1e-3) / 1e12
    if h.rank == 0:
        print(json.dumps({
            "metric": "mxf4_mma_only_tflops", "unit": UNIT, "value": sustained, "n_gpus": h.world, "steps": n,
            "warmup": 1, "ms_per_step": ms / n, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "mxfp4", "data": "synthetic",
            "config": {"workload": "peak_mxf4", "shape": burst["shape"], "k_steps_per_launch": 20000},
            "burst": burst, "burst_mxf8f6f4": burst_a8, "sustained": {"tflops": sustained, "ms": ms},
            "with_loads": with_loads,
            "context": {"cublas_bf16_x4_burst": peaks["bf16_tflops"] * FP4_OVER_BF16,
                        "cublas_bf16_x4_sustained": peaks["bf16_tflops_sustained"] * FP4_OVER_BF16,
                        "nominal": NOMINAL_FP4_TFLOPS, "source": peaks["source"]},
            "gpu_launches": n + 4 + 10, "clocks": clocks}))
    h.close()


def run_ours(args):
    import torch
    from paper_2603_16590_b200 import binding as B

    h = Harness()
    B.load()
    # tuning switches: touched only when a flag asks for something other than the automatic choice
    for value, hook in ((args.tile_width, B.batq_debug_force_tile_width), (args.quantizer, B.batq_debug_force_quantizer),
                        (args.gemm_kernel, B.batq_debug_force_gemm_kernel), (args.splits, B.batq_debug_force_small_s_splits),
                        (args.small_path, B.batq_debug_force_small_s_path),
                        (args.prefill_path, B.batq_debug_force_prefill_path),
                        (args.small_reduce, B.batq_debug_force_small_s_reduce)):
        if value != 0:
            hook(value)
    peaks = load_peaks()
    if args.workload == "peak_mxf4":
        return run_peak(args, h, B, peaks)
    kind, tokens, projs, _, _ = WORKLOADS[args.workload]
    # prefill: long enough (> 1 s) for the power cap to settle, so that the sustained peak is the fair denominator
    steps = args.steps if args.steps is not None else {"prefill": 5000, "decode": 300, "quant": 100}[kind]
    if args.workload == "cfg3_qwen2vl7b_prefill" and args.steps is None:
        steps = 1200
    seed = h.rank_seed(synth.BASE_SEED)
    ev = lambda: torch.cuda.Event(enable_timing=True)
    line = {"metric": METRIC, "unit": UNIT, "n_gpus": h.world, "steps": steps, "warmup": args.warmup,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "mxfp4", "data": "synthetic"}

    def mk_transform(L):
        return B.batq_transform_create(L["n"], L["t"].left, L["t"].right, L["t"].clip_lo, L["t"].clip_hi)

    if kind == "prefill":
        S = tokens[0]
        a8 = args.workload in A8_WORKLOADS
        # the three calls of the path, in the 4-bit or the 8-bit activation format
        f_linear = B.batq_linear_w4a8 if a8 else B.batq_linear_w4a4
        f_quant = B.batq_quantize_act_mxfp8 if a8 else B.batq_quantize_act
        f_gemm = B.batq_gemm_mxfp8_mxfp4 if a8 else B.batq_gemm_mxfp4
        f_ws = B.batq_linear_w4a8_workspace_bytes if a8 else B.batq_linear_workspace_bytes
        if a8:
            line["metric"], line["dtype"] = "w4a8_linear_tflops", "mxfp8 x mxfp4"
        layers = make_layer_inputs(args.workload, S, seed)
        for L in layers:
            L["tr"] = mk_transform(L)
            L["x"] = B.bits_to_cuda_bf16(L["x_bits"])
            L["codes"] = torch.empty((S, L["n"] if a8 else L["n"] // 2), dtype=torch.uint8, device="cuda")
            L["sf"] = torch.empty(B.batq_sf_bytes(S, L["n"], B.SF_MMA), dtype=torch.uint8, device="cuda")
            wdev = B.bits_to_cuda_bf16(synth.make_weight(L["m"], L["n"], L["w_seed"]))
            L["w"] = B.batq_prepare_weight(L["tr"], wdev)
            del wdev
            L["y"] = torch.empty((S, L["m"]), dtype=torch.bfloat16, device="cuda")
            L["ws"] = B.aligned_workspace(f_ws(L["w"], S))
            L["x_host"] = torch.from_numpy(L["x_bits"].view(np.int16)).pin_memory()
            L["y_host"] = torch.empty((S, L["m"]), dtype=torch.bfloat16).pin_memory()
        torch.cuda.synchronize()
        flops_step = sum(2.0 * S * L["n"] * L["m"] for L in layers)
        # Events around every launch cost about 8 % of a step (they close the gap-free hand-over between
        # consecutive kernels), so only every EVENT_EVERY-th step of the timed region carries them.
        sampled = [k for k in range(steps) if k % EVENT_EVERY == 0]
        marks = {k: [(ev(), ev(), ev()) for _ in layers] for k in sampled}

        # The other steps call the whole-layer entry point (the same two kernels, the GEMM launched as
        # a programmatic dependent of the quantiser); the bracketed steps call the two stages one by one.
        def step(k):
            m = marks.get(k)
            for i, L in enumerate(layers):
                if m is None:
                    f_linear(L["tr"], L["w"], L["x"], L["y"], L["ws"])
                    continue
                m[i][0].record()
                f_quant(L["tr"], L["x"], L["codes"], L["sf"], B.SF_MMA)
                m[i][1].record()
                f_gemm(L["codes"], L["sf"], L["w"], S, L["y"])
                m[i][2].record()

        ms, clocks = timed_region(h, step, steps, args.warmup)
        # A short run brackets only a few steps: add bracketed steps right after the timed region (same
        # calls, same buffers, device still warm) until MIN_BRACKETED have been taken.
        extra = max(0, MIN_BRACKETED - len(sampled))
        for k in range(steps, steps + extra):
            marks[k] = [(ev(), ev(), ev()) for _ in layers]
            step(k)
        torch.cuda.synchronize()
        q_all = np.array([[m[i][0].elapsed_time(m[i][1]) for i in range(len(layers))] for m in marks.values()])
        g_all = np.array([[m[i][1].elapsed_time(m[i][2]) for i in range(len(layers))] for m in marks.values()])
        q_ms, g_ms = q_all.mean(axis=0), g_all.mean(axis=0)

        # The same launches back to back (one CUDA graph of 8 steps' GEMMs, then one of 8 steps' quantisers):
        # no event between launches, so each kernel's prologue hides behind the one before it as it does in
        # the timed steps.  Reported next to the bracketed durations, not instead of them.
        def graph_of(fn, reps=8):
            side = torch.cuda.Stream()
            with torch.cuda.stream(side):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    for _ in range(reps):
                        fn()
            return g, reps

        def time_graph(g, reps, n=5):
            g.replay()
            torch.cuda.synchronize()
            a, b = ev(), ev()
            a.record()
            for _ in range(n):
                g.replay()
            b.record()
            torch.cuda.synchronize()
            return a.elapsed_time(b) / (n * reps)

        b2b = []
        for L in layers:
            gg, r = graph_of(lambda L=L: f_gemm(L["codes"], L["sf"], L["w"], S, L["y"]))
            gq, _ = graph_of(lambda L=L: f_quant(L["tr"], L["x"], L["codes"], L["sf"], B.SF_MMA))
            b2b.append((time_graph(gq, r), time_graph(gg, r)))
        mma_only = measure_mma_peak(B, torch, 20000, a8) if S > 128 else None
        big_w = max(layers, key=lambda L: L["m"] * L["n"])["w"]
        mma_loads = measure_mma_with_loads(B, torch, big_w) if (S > 128 and not a8) else None
        big_quant = measure_big_quantizer(B, torch, seed) if (S > 128 and h.rank == 0 and not a8) else None

        # end to end: host buffers in and out through the C-ABI host entry point
        def step_host():
            for L in layers:
                # every layer has staging buffers and a workspace of its own: enqueue all, wait once
                (B.batq_linear_w4a8_host_async if a8 else B.batq_linear_w4a4_host_async)(
                    L["tr"], L["w"], L["x_host"], L["y_host"], L["x"], L["y"], L["ws"])
            B.batq_host_drain()

        e2e_steps = max(1, min(steps, 5))
        for _ in range(2):
            step_host()
        h.barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            step_host()
        torch.cuda.synchronize()
        e2e_ms = h.max_over_ranks((time.perf_counter() - t0) * 1e3)
        h2d = sum(S * L["n"] * 2 for L in layers)
        d2h = sum(S * L["m"] * 2 for L in layers)

        gemm_flops = [2.0 * S * L["n"] * L["m"] for L in layers]
        gemm_achieved = sum(gemm_flops) / (g_ms.sum() * 1e-3) / 1e12
        q_bytes = [S * L["n"] * (3.03125 if a8 else QUANT_BYTES_PER_ELEM) for L in layers]
        quant_gbs = sum(q_bytes) / (q_ms.sum() * 1e-3) / 1e9
        sustained = ms >= 500.0   # a timed region this long runs under the power cap
        bf16_peak = peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]
        fp4_peak = bf16_peak * (FP8_OVER_BF16 if a8 else FP4_OVER_BF16)   # the 8-bit-container MMA runs at the FP8 rate
        traffic = None
        if GEMM_TRAFFIC["workload"] == args.workload and GEMM_TRAFFIC["source_sha256"] == kernel_source_hash():
            traffic = GEMM_TRAFFIC["mb_per_step"]
        b2b_gemm = sum(gemm_flops) / (sum(t[1] for t in b2b) * 1e-3) / 1e12
        b2b_quant = sum(q_bytes) / (sum(t[0] for t in b2b) * 1e-3) / 1e9
        # context: the vendor's dense-FP4 figure scaled to the SM clock sampled during the timed region
        mhz = (clocks or {}).get("sm_mhz") or 0.0
        mhz_max = (clocks or {}).get("sm_max_mhz") or 0.0
        nominal_at_clock = (NOMINAL_FP4_TFLOPS / 2 if a8 else NOMINAL_FP4_TFLOPS) * mhz / mhz_max if mhz and mhz_max else None
        nominal_peak = NOMINAL_FP4_TFLOPS / 2 if a8 else NOMINAL_FP4_TFLOPS
        b2b_peak = peaks["bf16_tflops"] * (FP8_OVER_BF16 if a8 else FP4_OVER_BF16)
        roof = {"bound": "tensor", "kernel": "gemm_w4a8_wide_kernel / gemm_w4a8_pair_kernel (per layer)" if a8 else ("gemm_mxfp4_wide_kernel / gemm_mxfp4_pair_kernel (per layer, by the "
                                                                "library's cost model)" if S > 128 else "gemm_mxfp4_kernel"),
                "achieved": gemm_achieved, "peak": fp4_peak,
                "events": "around every launch in every %dth step of the timed region (%d steps) and in %d more steps "
                          "right after it" % (EVENT_EVERY, len(sampled), extra),
                "unit": "TFLOP/s", "frac": gemm_achieved / fp4_peak, "traffic": traffic,
                "traffic_unit": "MB per step (4 launches)" if traffic else None,
                "peak_source": "%s cuBLAS bf16 %s x %.0f (nominal %s:bf16 ratio): a proxy that inherits cuBLAS's own "
                               "efficiency" % (peaks["source"], "sustained" if sustained else "burst",
                                               FP8_OVER_BF16 if a8 else FP4_OVER_BF16, "fp8" if a8 else "fp4"),
                "back_to_back": {"achieved": b2b_gemm, "peak": b2b_peak, "frac": b2b_gemm / b2b_peak,
                                 "how": "the same launches in a CUDA graph of 8 steps, no events between them; a few "
                                        "ms after the timed region, so against the burst peak"},
                "nominal": {"peak": nominal_peak, "frac": gemm_achieved / nominal_peak,
                            "peak_at_sampled_clock": nominal_at_clock,
                            "frac_at_sampled_clock": gemm_achieved / nominal_at_clock if nominal_at_clock else None,
                            "note": "vendor dense-FP4 figure (context, not the denominator of `frac` above); 70 % of "
                                    "the dense FP4 peak means frac >= 0.70 here"}}
        if mma_only is not None:
            roof["mma_only"] = dict(mma_only, frac=gemm_achieved / mma_only["tflops"],
                                    frac_back_to_back=b2b_gemm / mma_only["tflops"])
        if mma_loads is not None:
            roof["mma_with_loads"] = dict(mma_loads, frac=gemm_achieved / mma_loads["tflops"],
                                          frac_back_to_back=b2b_gemm / mma_loads["tflops"])
        line.update({
            "value": h.whole_job_rate(flops_step, steps, ms) / 1e12, "ms_per_step": ms / steps,
            "config": workload_config(args.workload),
            "roofline": roof,
            "act_quant": {"bound": "hbm", "kernel": "quantize_act_tc_kernel", "achieved": quant_gbs,
                          "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": quant_gbs / peaks["hbm_gbs"],
                          "peak_source": peaks["source"],
                          "note": "between events: the kernel plus the launch gaps on both sides, at 17-59 MB per launch",
                          "back_to_back": {"achieved": b2b_quant, "frac": b2b_quant / peaks["hbm_gbs"]},
                          "largest_sweep_case": big_quant},
            "kernels": [{"name": L["name"], "n": L["n"], "m": L["m"], "quant_us": float(q_ms[i] * 1e3),
                         "quant_gbs": q_bytes[i] / (q_ms[i] * 1e-3) / 1e9, "gemm_us": float(g_ms[i] * 1e3),
                         "gemm_tflops": gemm_flops[i] / (g_ms[i] * 1e-3) / 1e12,
                         "quant_us_back_to_back": float(b2b[i][0] * 1e3), "gemm_us_back_to_back": float(b2b[i][1] * 1e3),
                         "gemm_tflops_back_to_back": gemm_flops[i] / (b2b[i][1] * 1e-3) / 1e12}
                        for i, L in enumerate(layers)],
            "e2e": {"value": flops_step * e2e_steps * h.world / (e2e_ms * 1e-3) / 1e12, "unit": UNIT,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps},
            "gpu_launches": 2 * len(layers) * steps,
        })

    elif kind == "decode":
        # Per call: quantiser + small-s GEMM, or the fused kernel (one batq_linear_w4a4).  A decode loop
        # is launch-bound from Python, so for every token count the projections of `copies` layers, in
        # model order (qkv, o, gate/up, down; layer after layer, each layer with its own copy of the
        # prepared weights), are captured once as ONE CUDA graph.  The copies cycle through more than
        # 3 x L2 between reuses, so no call finds its weights in L2.  A step replays the graph of every
        # token count; events bracket each replay.
        copies = 4
        base = make_layer_inputs(args.workload, max(tokens), seed)
        cases = []
        for i, L in enumerate(base):
            L["tr"] = mk_transform(L)
            wdev = B.bits_to_cuda_bf16(synth.make_weight(L["m"], L["n"], L["w_seed"]))
            L["ws_list"] = [B.batq_prepare_weight(L["tr"], wdev) for _ in range(copies)]
            del wdev
            xfull = B.bits_to_cuda_bf16(L["x_bits"])
            for S in tokens:
                c = {"L": L, "S": S, "x": xfull[:S].contiguous(),
                     "y": torch.empty((S, L["m"]), dtype=torch.bfloat16, device="cuda"),
                     "ws": B.aligned_workspace(B.batq_linear_workspace_bytes(L["ws_list"][0], S)),
                     "x_host": torch.from_numpy(L["x_bits"][:S].copy().view(np.int16)).pin_memory(),
                     "y_host": torch.empty((S, L["m"]), dtype=torch.bfloat16).pin_memory(),
                     "launches": B.batq_linear_kernel_launches(L["tr"], L["ws_list"][0], S)}
                cases.append(c)
        order = [c for S in tokens for c in cases if c["S"] == S]   # all projections at S=1, then S=4, ...

        def call(c, layer):
            B.batq_linear_w4a4(c["L"]["tr"], c["L"]["ws_list"][layer], c["x"], c["y"], c["ws"])

        side = torch.cuda.Stream()
        layer_graphs = {}
        with torch.cuda.stream(side):
            for c in order:
                for layer in range(copies):   # first calls outside capture: per-device set-up
                    call(c, layer)
            torch.cuda.synchronize()
            for S in tokens:
                layer_graphs[S] = torch.cuda.CUDAGraph()
                with torch.cuda.graph(layer_graphs[S], stream=side):
                    for layer in range(copies):
                        for c in order:
                            if c["S"] == S:
                                call(c, layer)
            for c in order:                   # per-projection detail: each case alone, `copies` calls
                c["graph"] = torch.cuda.CUDAGraph()
                with torch.cuda.graph(c["graph"], stream=side):
                    for layer in range(copies):
                        call(c, layer)
        torch.cuda.synchronize()
        flops_step = copies * sum(2.0 * c["S"] * c["L"]["n"] * c["L"]["m"] for c in order)
        marks = [[(ev(), ev()) for _ in tokens] for _ in range(steps)]

        def step(k):
            for i, S in enumerate(tokens):
                if k is not None:
                    marks[k][i][0].record()
                layer_graphs[S].replay()
                if k is not None:
                    marks[k][i][1].record()

        ms, clocks = timed_region(h, step, steps, args.warmup)
        l_ms = np.array([[m[i][0].elapsed_time(m[i][1]) for i in range(len(tokens))] for m in marks]) / copies
        layer_bytes = sum(L["n"] * L["m"] * WEIGHT_BYTES_PER_ELEM for L in base)
        gbs = layer_bytes * len(tokens) / (l_ms.mean(axis=0).sum() * 1e-3) / 1e9

        # Per-projection detail, outside the timed region: every case in a graph of its own.
        d_steps = max(3, min(steps, 50))
        d_marks = [[(ev(), ev()) for _ in order] for _ in range(d_steps)]
        for k in range(-3, d_steps):
            for i, c in enumerate(order):
                if k >= 0:
                    d_marks[k][i][0].record()
                c["graph"].replay()
                if k >= 0:
                    d_marks[k][i][1].record()
        torch.cuda.synchronize()
        c_ms = np.array([[m[i][0].elapsed_time(m[i][1]) for i in range(len(order))] for m in d_marks]) / copies
        c_med = np.median(c_ms, axis=0)
        w_bytes = [c["L"]["n"] * c["L"]["m"] * WEIGHT_BYTES_PER_ELEM for c in order]

        def step_host():
            for c in order:   # every call has staging buffers and a workspace of its own: enqueue all, wait once
                B.batq_linear_w4a4_host_async(c["L"]["tr"], c["L"]["ws_list"][0], c["x_host"], c["y_host"], c["x"], c["y"],
                                              c["ws"])
            B.batq_host_drain()

        e2e_steps = max(1, min(steps, 20))
        for _ in range(2):
            step_host()
        h.barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            step_host()
        torch.cuda.synchronize()
        e2e_ms = h.max_over_ranks((time.perf_counter() - t0) * 1e3)
        h2d = sum(c["S"] * c["L"]["n"] * 2 for c in order)
        d2h = sum(c["S"] * c["L"]["m"] * 2 for c in order)
        line.update({
            "value": h.whole_job_rate(flops_step, steps, ms) / 1e12, "ms_per_step": ms / steps,
            "config": workload_config(args.workload),
            "roofline": {"bound": "hbm", "kernel": "gemm_small_s_kernel", "achieved": gbs, "peak": peaks["hbm_gbs"],
                         "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"], "traffic": None,
                         "peak_source": "%s copy bandwidth; achieved = weight bytes / time of the layer graphs "
                                        "(quantisers + GEMMs)" % peaks["source"]},
            "layers": [{"tokens": S, "layer_us": float(l_ms[:, i].mean() * 1e3),
                        "layer_us_median": float(np.median(l_ms[:, i]) * 1e3),
                        "weight_gbs": layer_bytes / (l_ms[:, i].mean() * 1e-3) / 1e9} for i, S in enumerate(tokens)],
            "kernels": [{"name": c["L"]["name"], "tokens": c["S"], "n": c["L"]["n"], "m": c["L"]["m"],
                         "launches_per_call": c["launches"],
                         "call_us": float(c_ms[:, i].mean() * 1e3), "call_us_median": float(c_med[i] * 1e3),
                         "weight_gbs": w_bytes[i] / (c_ms[:, i].mean() * 1e-3) / 1e9} for i, c in enumerate(order)],
            "kernels_note": "per projection, outside the timed region: each case alone in a graph of %d calls "
                            "(includes that short graph's launch and ramp)" % copies,
            "e2e": {"value": flops_step / copies * e2e_steps * h.world / (e2e_ms * 1e-3) / 1e12, "unit": UNIT,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                    "note": "one eager host-buffer call per case and step (no graph)"},
            "gpu_launches": copies * sum(c["launches"] for c in order) * steps,
        })

    else:  # quantiser sweep
        cases = []
        for S in tokens:
            for L in make_layer_inputs(args.workload, S, seed):
                L["S"] = S
                L["tr"] = mk_transform(L)
                L["x"] = B.bits_to_cuda_bf16(L["x_bits"])
                L["codes"] = torch.empty((S, L["n"] // 2), dtype=torch.uint8, device="cuda")
                L["sf"] = torch.empty(B.batq_sf_bytes(S, L["n"], B.SF_MMA), dtype=torch.uint8, device="cuda")
                L["x_host"] = torch.from_numpy(L["x_bits"].view(np.int16)).pin_memory()
                L["codes_host"] = torch.empty((S, L["n"] // 2), dtype=torch.uint8).pin_memory()
                cases.append(L)
        # > L2, read between cases: evicts the previous case without leaving dirty lines behind (a
        # written flush buffer would be drained to HBM during the timed launch)
        flush = torch.zeros(256 << 18, dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()
        # T_j = G (x) P_j with clip to MXFP4, plain MXFP4 (T = I), and the transform with 8-bit (E4M3) elements
        variants = [("gpk", True), ("identity", False), ("gpk_mxfp8", True)]
        for L in cases:
            L["codes8"] = torch.empty((L["S"], L["n"]), dtype=torch.uint8, device="cuda")
        marks = [[[(ev(), ev()) for _ in variants] for _ in cases] for _ in range(steps)]

        def step(k):
            for i, L in enumerate(cases):
                for v, (_, xf) in enumerate(variants):
                    flush.sum()
                    if k is not None:
                        marks[k][i][v][0].record()
                    if v == 2:
                        B.batq_quantize_act_mxfp8(L["tr"], L["x"], L["codes8"], L["sf"], B.SF_MMA)
                    else:
                        B.batq_quantize_act(L["tr"] if xf else None, L["x"], L["codes"], L["sf"], B.SF_MMA)
                    if k is not None:
                        marks[k][i][v][1].record()

        ms, clocks = timed_region(h, step, steps, args.warmup)
        t_ms = np.array([[[m[i][v][0].elapsed_time(m[i][v][1]) for v in range(3)] for i in range(len(cases))]
                         for m in marks]).mean(axis=0)
        bytes_case = np.array([L["S"] * L["n"] * QUANT_BYTES_PER_ELEM for L in cases])
        gbs = bytes_case.sum() / (t_ms[:, 0].sum() * 1e-3) / 1e9
        big = int(np.argmax(bytes_case))

        def step_host():
            for L in cases:
                L["x"].copy_(L["x_host"].view(torch.bfloat16), non_blocking=True)
                B.batq_quantize_act(L["tr"], L["x"], L["codes"], L["sf"], B.SF_MMA)
                L["codes_host"].copy_(L["codes"], non_blocking=True)
            torch.cuda.synchronize()

        step_host()
        h.barrier()
        t0 = time.perf_counter()
        step_host()
        e2e_ms = h.max_over_ranks((time.perf_counter() - t0) * 1e3)
        elems = float(sum(L["S"] * L["n"] for L in cases))
        # quantiser-only workloads have no GEMM flops: the metric's numerator is the transform's
        # 24 flop per element (Kronecker form), reported for completeness
        line.update({
            "value": 24.0 * elems * steps * h.world / (t_ms[:, 0].sum() * steps * 1e-3) / 1e12,
            "ms_per_step": float(t_ms[:, 0].sum()),
            "config": workload_config(args.workload),
            "roofline": {"bound": "hbm", "kernel": "quantize_act_tc_kernel", "achieved": gbs, "peak": peaks["hbm_gbs"],
                         "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"], "traffic": None,
                         "largest_case_gbs": float(bytes_case[big] / (t_ms[big, 0] * 1e-3) / 1e9),
                         "peak_source": "%s copy bandwidth" % peaks["source"]},
            "kernels": [{"tokens": L["S"], "hidden": L["n"], "gpk_us": float(t_ms[i, 0] * 1e3),
                         "gpk_gbs": float(bytes_case[i] / (t_ms[i, 0] * 1e-3) / 1e9),
                         "gpk_frac": float(bytes_case[i] / (t_ms[i, 0] * 1e-3) / 1e9 / peaks["hbm_gbs"]),
                         "identity_us": float(t_ms[i, 1] * 1e3),
                         "identity_gbs": float(bytes_case[i] / (t_ms[i, 1] * 1e-3) / 1e9),
                         "mxfp8_us": float(t_ms[i, 2] * 1e3),   # 2 + 1 + 1/32 bytes per element
                         "mxfp8_gbs": float(L["S"] * L["n"] * 3.03125 / (t_ms[i, 2] * 1e-3) / 1e9)}
                        for i, L in enumerate(cases)],
            "e2e": {"value": 24.0 * elems * h.world / (e2e_ms * 1e-3) / 1e12, "unit": UNIT,
                    "h2d_bytes_per_step": int(elems * 2), "d2h_bytes_per_step": int(elems // 2), "steps": 1},
            "gpu_launches": 3 * len(cases) * steps,
        })

    status = B.batq_last_device_status()
    if status != 0:
        raise SystemExit(f"device status {status} after the timed region")
    if h.rank == 0:
        line["cpu_baseline"] = cpu_baseline(args.workload, synth.BASE_SEED)
        if kind == "quant":
            line["cpu_baseline"]["parity_check"] = sweep_parity_counts(B, torch, cases)
        line["clocks"] = clocks
        print(json.dumps(line))
    h.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None, help="timed steps (default: per workload, about 0.3-1 s of GPU time)")
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg1_llama8b_prefill", choices=sorted(WORKLOADS) + ["peak_mxf4"])
    ap.add_argument("--quantizer", type=int, default=0, help="0 auto, 1 ALU kernel, 2 tensor-core kernel (tuning)")
    ap.add_argument("--gemm-kernel", type=int, default=0, help="0 auto, 1 one CTA per tile, 2 CTA pairs (tuning)")
    ap.add_argument("--tile-width", type=int, default=0, help="force the GEMM tile width (tuning); 0 = automatic")
    ap.add_argument("--small-path", type=int, default=0, help="0 auto, 1 two kernels, 2 fused kernel (tuning)")
    ap.add_argument("--prefill-path", type=int, default=0, help="0 auto, 1 quantiser + GEMM kernels, 2 one kernel (tuning)")
    ap.add_argument("--small-reduce", type=int, default=0, help="0 auto, 1 tickets, 2 cluster (split-K reduction, tuning)")
    ap.add_argument("--splits", type=int, default=0, help="force the small-s GEMM's K splits (tuning); 0 = automatic")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        args.warmup = max(args.warmup, 3)
        run_ours(args)


if __name__ == "__main__":
    main()
