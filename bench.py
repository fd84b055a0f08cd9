#!/usr/bin/env python
"""Benchmark of the hot path: bit-exact emulated MACs/s of one MMA model at 4096^3 on a B200.

One "step" is one evaluation D = Phi(A, B, C) of the workload named in ``config.workload`` (default: the FP8 E4M3
4096 x 4096 x 4096 GEMM under the paper's Hopper FP8 -> FP32 model, L = 32, F = 13, RZ-E8M13) with the inputs
resident in HBM.  The line also carries the issue-rate roofline of the dominant kernel (its multiply-add pipe, with
the paper-level integer operation count beside it), the end-to-end number
through the host-buffer entry point and the CPU oracle timed on a bounded sample.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfg3|cfg2|...]
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "emulated_macs_per_s"
UNIT = "MAC/s"

WORKLOADS = {
    # name: (registry key, (M, N, K), description)
    "cfg3": (("hopper", "e4m3", "fp32"), (4096, 4096, 4096),
             "FP8 E4M3 4096x4096x4096, A,B ~ N(0,1) scaled per row to the E4M3 range, C = +0; Hopper FP8->FP32 model (L=32, F=13, RZ-E8M13)"),
    "cfg3_chunk128": (("hopper", "e4m3", "fp32"), (4096, 4096, 4096),
                      "as cfg3 with FP32 promotion of partial sums every 128 elements of K and the row/column dequantisation epilogue"),
    "cfg3_2k": (("hopper", "e4m3", "fp32"), (2048, 2048, 2048),
                "FP8 E4M3 2048^3 (reduced case for profiler captures), inputs as cfg3; Hopper FP8->FP32 model"),
    "cfg2": (("ampere", "bf16", "fp32"), (2048, 2048, 2048),
             "BF16 2048^3, exponents uniform over +-20 binades, C ~ N(0,1); Ampere BF16->FP32 model (L=8, F=24, RZ-FP32)"),
    "hopper_fp16": (("hopper", "fp16", "fp32"), (4096, 4096, 4096),
                    "FP16 4096^3 N(0,1) inputs; Hopper FP16->FP32 model (L=16, F=25, RZ-FP32)"),
    "hopper_fp16_2k": (("hopper", "fp16", "fp32"), (2048, 2048, 2048),
                       "FP16 2048^3 N(0,1) inputs (reduced case for profiler captures); Hopper FP16->FP32 model"),
    "volta_fp16": (("volta", "fp16", "fp32"), (4096, 4096, 4096),
                   "FP16 4096^3 N(0,1) inputs; Volta FP16->FP32 model (L=4, F=23, RZ-FP32)"),
    "ampere_bf16": (("ampere", "bf16", "fp32"), (4096, 4096, 4096),
                    "BF16 4096^3 N(0,1) inputs; Ampere BF16->FP32 model (L=8, F=24, RZ-FP32)"),
    "cfg4_dot_hopper_fp16": (("hopper", "fp16", "fp32"), (1 << 20, 1, 32),
                             "probe-style batch: 2^20 independent dot products of length 32, FP16, eight seeded input classes (subnormals, cancellation, outliers, inf/NaN, bit streams); Hopper FP16->FP32 model via mmasim_dot_batch"),
    "cfg4_dot_cdna2_fp16": (("cdna2", "fp16", "fp32"), (1 << 20, 1, 32),
                            "probe-style batch: 2^20 independent dot products of length 32, FP16, eight seeded input classes; CDNA2 FP16 model (FTZ-AddMul, P=4) via mmasim_dot_batch"),
    "cdna3_bf16_2k": (("cdna3", "bf16", "fp32"), (2048, 2048, 2048),
                      "BF16 2048^3 N(0,1) inputs (reduced case for profiler captures); CDNA3 BF16 model (TR-FDPA, L=8, F=24, F2=31)"),
    "cdna1_fp16_2k": (("cdna1", "fp16", "fp32"), (2048, 2048, 2048),
                      "FP16 2048^3 N(0,1) inputs (reduced case for profiler captures); CDNA1 FP16 model (E-FDPA, L=4)"),
    "cdna3_tf32_2k": (("cdna3", "tf32", "fp32"), (2048, 2048, 2048),
                      "TF32 2048^3 N(0,1) inputs (reduced case for profiler captures); CDNA3 TF32 model (TR-FDPA, L=4)"),
    "cdna3_e4m3_2k": (("cdna3", "e4m3", "fp32"), (2048, 2048, 2048),
                      "FP8 E4M3 2048^3 N(0,1) inputs (reduced case for profiler captures); CDNA3 FP8 model (GTR-FDPA, L=16)"),
    "volta_fp16_2k": (("volta", "fp16", "fp32"), (2048, 2048, 2048),
                      "FP16 2048^3 N(0,1) inputs (reduced case for profiler captures); Volta FP16->FP32 model (L=4, F=23)"),
    "blackwell_mxf4_2k": (("blackwell", "mxf4", "fp32"), (2048, 2048, 2048),
                          "MXFP4 2048^3 N(0,1) inputs with E8M0 block scales (reduced case for profiler captures); Blackwell MXFP4 model (GST-FDPA, L=64, G=16, F=35)"),
    "cdna1_fp32_2k": (("cdna1", "fp32", "fp32"), (2048, 2048, 2048),
                      "FP32 2048^3 N(0,1) inputs (reduced case for profiler captures); CDNA1 FP32 model (FMA chain)"),
    "ampere_fp64_2k": (("ampere", "fp64", "fp64"), (2048, 2048, 2048),
                       "FP64 2048^3 N(0,1) inputs (reduced case for profiler captures); FP64 FMA chain on the FP64 matrix instruction"),
    "blackwell_e4m3": (("blackwell", "e4m3", "fp32"), (4096, 4096, 4096),
                       "FP8 E4M3 4096^3 N(0,1) inputs; Blackwell FP8->FP32 model (L=32, F=25, RZ-FP32)"),
}


def compute_dtype(kernel: str, model) -> str:
    """The arithmetic type the timed kernel computes in (the results are exact integers / model words either way)."""
    if kernel == "tfdpa_lut8" and model.F <= 13:
        return "f32"
    return {"tfdpa_lut8": "f64", "tfdpa_f16": "f64", "tfdpa_bf16": "f64", "tfdpa_tf32": "f64", "trfdpa": "f64", "gtrfdpa": "f64",
            "efdpa": "f64", "dot_tfdpa": "f64", "dot_ftz": "f32", "ftz_addmul": "f32", "fma_f32": "f32", "fma_f64": "f64", "gstfdpa": "int32"}.get(kernel, "int64")


# DRAM bytes per step (the main kernel and the two decode launches before it): dram__bytes_read.sum +
# dram__bytes_write.sum of a one-pass ncu capture of the same workload at its full size, a STORED CONSTANT, not a figure
# of this run.  Algorithmic bytes are 168 MB at 4096^3 (operands once, C and D); the rest is the decoded operand blocks
# (226 MB, larger than the L2) written once and re-read by the tiles of later waves.  The kernels are bound by arithmetic:
# 1.18 GB in 4.2 ms is 4 % of what the memory could move in that time.
NCU_DRAM_BYTES = {"cfg3": (980664832 + 65643264) + (16788480 + 52632832) + (16789248 + 49752576),
                  "cfg3_2k": (74762496 + 1387776) + 4204288 + 4204800}
NCU_ALGORITHMIC_BYTES = {"cfg3": 2 * 4096 * 4096 + 2 * 4 * 4096 * 4096, "cfg3_2k": 2 * 2048 * 2048 + 2 * 4 * 2048 * 2048}

# kernels one library call launches: the tuned fused-summation kernels decode A and B into scratch blocks first
KERNELS_PER_CALL = {"tfdpa_lut8": 3, "tfdpa_f16": 3, "tfdpa_bf16": 3, "tfdpa_tf32": 3, "trfdpa": 3, "gtrfdpa": 3, "efdpa": 3}

SMS = 148
# The pipe that bounds each kernel: (name, instruction kinds of the issue-rate micro-benchmark that witness its rate,
# nominal results per SM and clock, pipe instructions per emulated MAC).
#   f32 fused summation (F = 13): one FP32 fused multiply-add per term; f64 fused summation (F >= 23, TR, GTR, E): one
#   FP64 fused multiply-add per term; Phi_FMA: the multiply-add itself; Phi_FTZ-AddMul: one multiply and one add per
#   term (two FP32-pipe instructions); GST-FDPA: one 4-way byte dot product per four terms.
FP32_KINDS = ("ffma.rm", "ffma2.rm", "ffma.rn.x16", "ffma.rn.x32", "ffma.rm.x16", "ffma2.rm.x16")
FP64_KINDS = ("dfma", "dfma.rn.x16", "dfma.rn.x32", "dfma.rm.x16", "dmma.rm.k4")
PIPES = {
    "fp32_fma": ("FP32 fused multiply-add issue", FP32_KINDS, 128.0),
    "fp64_fma": ("FP64 fused multiply-add issue", FP64_KINDS, 64.0),
    "int_dp4a": ("4-way byte dot-product issue", ("dp4a",), 64.0),
    "int_alu": ("3-input integer add issue", ("iadd3",), 64.0),
}


def pipe_of(kernel: str, model):
    """(pipe key, pipe instructions per emulated MAC) of the kernel a model dispatches to."""
    if kernel == "tfdpa_lut8" and model.F <= 13:
        return "fp32_fma", 1.0
    if kernel in ("tfdpa_lut8", "tfdpa_f16", "tfdpa_bf16", "tfdpa_tf32", "trfdpa", "gtrfdpa", "efdpa", "fma_f64"):
        return "fp64_fma", 1.0
    if kernel == "fma_f32":
        return "fp32_fma", 1.0
    if kernel == "ftz_addmul":
        return "fp32_fma", 2.0
    if kernel == "gstfdpa":
        return "int_dp4a", 0.25
    return "int_alu", algorithmic_ops_per_mac(model)


def measure_pipe_peaks(mmasim, torch, dev, pipes):
    """Issue rates of the given pipes, measured live: every witness kind at 2, 4 and 8 CTAs of 256 threads per SM, best
    of three launches each; returns {pipe: {"peak": ops/s, "witness": kind, "ctas_per_sm": n, "all": {kind: ops/s}}}."""
    sink = torch.zeros(4, dtype=torch.int32, device=dev)
    out = {}
    for pipe in pipes:
        _, kinds, _ = PIPES[pipe]
        best, who, occ, every = 0.0, None, 0, {}
        for kind in kinds:
            kbest = 0.0
            for ctas in (2, 4, 8):
                mmasim.int_peak(kind, SMS * ctas, 256, sink)
                for _ in range(3):
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    ops = mmasim.int_peak(kind, SMS * ctas, 8192 // ctas, sink)
                    e1.record()
                    torch.cuda.synchronize()
                    rate = ops / (e0.elapsed_time(e1) * 1e-3)
                    kbest = max(kbest, rate)
                    if rate > best:
                        best, who, occ = rate, kind, ctas
            every[kind] = kbest
        out[pipe] = {"peak": best, "witness": who, "ctas_per_sm": occ, "all": every}
    return out


# One model per kernel template (and per block length where the per-block work matters): the per-model leg of the line.
PER_MODEL = [("hopper", "e4m3", "fp32"), ("hopper", "e4m3", "fp16"), ("ada", "e5m2", "fp32"),
             ("volta", "fp16", "fp32"), ("ampere", "fp16", "fp32"), ("hopper", "fp16", "fp32"), ("hopper", "fp16", "fp16"),
             ("ampere", "bf16", "fp32"), ("hopper", "bf16", "fp32"), ("ampere", "tf32", "fp32"), ("hopper", "tf32", "fp32"),
             ("blackwell", "e4m3", "fp32"), ("blackwell", "e2m1", "fp32"), ("blackwell", "mxe4m3", "fp32"),
             ("blackwell", "mxf4", "fp32"), ("blackwell", "nvf4", "fp32"),
             ("cdna3", "bf16", "fp32"), ("cdna3", "tf32", "fp32"), ("cdna3", "e4m3", "fp32"),
             ("cdna1", "fp16", "fp32"), ("cdna1", "bf16", "fp32"), ("cdna2", "fp16", "fp32"), ("cdna2", "bf16", "fp32"),
             ("cdna1", "fp32", "fp32"), ("hopper", "fp64", "fp64")]


def algorithmic_ops_per_mac(model) -> float:
    """Integer operations per emulated MAC of the T-FDPA family: multiply, exponent add, maximum, distance,
    shift, accumulate (6 per term) plus about 25 per block for the accumulator term, normalisation and rho."""
    L = max(model.l_max, 1)
    return 6.0 + 25.0 / L


def make_inputs(name):
    from paper_2511_10909_b200 import workloads as wl
    key, (M, N, K), _ = WORKLOADS[name]
    if name.startswith("cfg3"):
        A, B, C, sa, sb = wl.cfg3(M)
        inp = {"A": A, "B": B, "C": C}
        if name == "cfg3_chunk128":
            inp.update(k_chunk=128, row_scale=sa, col_scale=sb)
        return inp
    if name == "cfg2":
        A, B, C = wl.cfg2(M)
        return {"A": A, "B": B, "C": C}
    if name.startswith("cfg4_dot"):
        A, B, C = wl.cfg4(key[1], K, n=M)
        return {"A": A, "B": B, "C": C, "dot": True}
    d = wl.normal_inputs(key[1], key[2], M, N, K, seed=5)
    return {k: d[k] for k in ("A", "B", "C", "sfa", "sfb") if k in d}


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """The slowest rank's time: every rank contributes its own device-timed milliseconds."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(macs_per_rank_step: float, steps: int, world: int, slowest_ms: float) -> float:
    """Aggregate MAC/s of `world` replicas that each evaluate their own batch (weak scaling, no exchange)."""
    return macs_per_rank_step * world * steps / (slowest_ms * 1e-3)


class ClockSampler:
    """Samples SM clocks and throttle reasons while the timed region runs: through NVML every few milliseconds where
    the Python binding is there (read-only queries), else with nvidia-smi every 100 ms."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.lines, self.proc = index, [], None
        self.nvml, self.handle, self.samples, self.stop_flag, self.thread = None, None, [], False, None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            idx = self.index
            vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
            if vis and all(v.strip().isdigit() for v in vis.split(",")):
                idx = int(vis.split(",")[self.index])
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self.nvml = pynvml
            self.thread = threading.Thread(target=self._poll, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.nvml = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _poll(self):
        n = self.nvml
        reasons_of = getattr(n, "nvmlDeviceGetCurrentClocksEventReasons", None) or n.nvmlDeviceGetCurrentClocksThrottleReasons
        try:
            mx = n.nvmlDeviceGetMaxClockInfo(self.handle, n.NVML_CLOCK_SM)
        except Exception:
            mx = 0
        while not self.stop_flag:
            try:
                self.samples.append((n.nvmlDeviceGetClockInfo(self.handle, n.NVML_CLOCK_SM), mx, int(reasons_of(self.handle))))
            except Exception:
                pass
            time.sleep(0.001)

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.nvml is not None:
            self.stop_flag = True
            self.thread.join(timeout=1.0)
            n = self.nvml
            names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40}
            sm = [x[0] for x in self.samples]
            loaded = [x for x in sm if x > 0.5 * max(sm)] if sm else []
            reasons = sorted(k for k, bit in names.items() if any(x[2] & bit for x in self.samples))
            return {"sm_mhz": float(np.median(loaded)) if loaded else None,
                    "sm_max_mhz": float(max(x[1] for x in self.samples)) if self.samples else None,
                    "reasons": reasons, "samples": len(sm), "source": "nvml"}
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        loaded = [x for x in sm if x > 0.5 * max(sm)] if sm else []
        return {"sm_mhz": float(np.median(loaded)) if loaded else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons), "samples": len(sm), "source": "nvidia-smi"}


def oracle_sample_rate(name, inp, seconds_target=15.0, processes=None):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload's outputs; returns (MAC/s, info)."""
    import oracle
    from paper_2511_10909_b200 import workloads as wl
    key, (M, N, K), _ = WORKLOADS[name]
    m = oracle.lookup(*key)
    cores = processes or os.cpu_count() or 1
    kw = {}
    if "k_chunk" in inp:
        kw.update(k_chunk=inp["k_chunk"], row_scale=inp["row_scale"].view(np.uint32), col_scale=inp["col_scale"].view(np.uint32))
    if "sfa" in inp:
        kw.update(SFA=inp["sfa"], SFB=inp["sfb"])
    probe = wl.sample_pairs(M, N, 64 * cores, seed=77)
    t0 = time.perf_counter()
    oracle.phi_gemm_sampled(m, inp["A"], inp["B"], inp["C"], probe, processes=cores, **kw)
    dt = time.perf_counter() - t0
    n = int(max(64 * cores, min(200000, len(probe) * seconds_target / max(dt, 1e-3))))
    pairs = wl.sample_pairs(M, N, n, seed=78)
    t0 = time.perf_counter()
    oracle.phi_gemm_sampled(m, inp["A"], inp["B"], inp["C"], pairs, processes=cores, **kw)
    dt = time.perf_counter() - t0
    return n * K / dt, {"cores": cores, "sample": f"{n} seeded output elements x K={K} of {name} ({n * K:.3g} MACs in {dt:.1f} s)"}


def run_reference(args):
    """The reference arm: the CPU oracle on this machine's host cores, each step a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2511_10909_b200 import workloads as wl
    name = args.workload
    key, (M, N, K), desc = WORKLOADS[name]
    inp = make_inputs(name)
    m = oracle.lookup(*key)
    cores = os.cpu_count() or 1
    kw = {}
    if "k_chunk" in inp:
        kw.update(k_chunk=inp["k_chunk"], row_scale=inp["row_scale"].view(np.uint32), col_scale=inp["col_scale"].view(np.uint32))
    if "sfa" in inp:
        kw.update(SFA=inp["sfa"], SFB=inp["sfb"])
    n = 512 * cores
    times = []
    for step in range(args.warmup + args.steps):
        pairs = wl.sample_pairs(M, N, n, seed=100 + step)
        t0 = time.perf_counter()
        oracle.phi_gemm_sampled(m, inp["A"], inp["B"], inp["C"], pairs, processes=cores, **kw)
        if step >= args.warmup:
            times.append(time.perf_counter() - t0)
    total = sum(times)
    value = n * K * args.steps / total
    sample = f"{n} seeded output elements x K={K} per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int64", "data": "synthetic",
        "config": {"workload": f"{name}: {desc}", "model": "-".join(key), "M": M, "N": N, "K": K, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_ours(args):
    import torch
    from paper_2511_10909_b200.build import build
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if rank == 0:
        build()
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    from paper_2511_10909_b200 import mmasim
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    name = args.workload
    key, (M, N, K), desc = WORKLOADS[name]
    inp = make_inputs(name)          # every rank evaluates its own full batch of the workload (weak scaling, no exchange)
    model = mmasim.Model(*key)

    def to_dev(x):
        x = np.ascontiguousarray(x)
        view = {1: np.uint8, 2: np.int16, 4: np.int32, 8: np.int64}[x.dtype.itemsize]
        return torch.from_numpy(x.view(view) if x.dtype.kind != "f" else x).to(dev)

    dA, dB, dC = to_dev(inp["A"]), to_dev(inp["B"]), to_dev(inp["C"])
    kw = {}
    if "k_chunk" in inp:
        kw = dict(k_chunk=inp["k_chunk"], row_scale=to_dev(inp["row_scale"]), col_scale=to_dev(inp["col_scale"]))
    if "sfa" in inp:
        kw.update(sfa=to_dev(inp["sfa"]), sfb=to_dev(inp["sfb"]))
    dD = torch.empty((M, N), dtype={2: torch.int16, 4: torch.int32, 8: torch.int64}[model.acc_bytes], device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)      # larger than the 126 MB L2

    is_dot = bool(inp.get("dot"))
    if is_dot:
        dD = torch.empty((M,), dtype=torch.int32, device=dev)

    def step():
        if is_dot:
            mmasim.dot_batch(model, dA, dB, dC, out=dD)
        else:
            mmasim.gemm(model, dA, dB, dC, out=dD, **kw)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    kernel_name = mmasim.last_kernel()

    # issue-rate peaks, measured live (independent chains of one instruction kind on every SM, several witnesses and
    # occupancies per pipe, the best counts): the pipe the timed kernel is bound by, and the 3-input integer add that is
    # the unit of the paper-level operation count
    pipe_key, pipe_ops_per_mac = pipe_of(kernel_name, model)
    peaks = measure_pipe_peaks(mmasim, torch, dev, sorted({pipe_key, "int_alu"})) if not is_dot else {}

    # ---- timed region: K steps, device timers, L2 flushed between steps ----
    sampler = ClockSampler(local_rank)
    events = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    for e0, e1 in events:
        flush.zero_()
        e0.record()
        step()
        e1.record()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    clocks = sampler.stop()
    total_ms = max_over_ranks(sum(e0.elapsed_time(e1) for e0, e1 in events), dist, dev)
    macs_per_step = float(M) * N * K * world
    value = whole_job_value(float(M) * N * K, args.steps, world, total_ms)

    # ---- end to end through the host-buffer entry point (pinned host memory, copies inside the timed region) ----
    e2e = None
    if not args.skip_extras and not is_dot and (rank == 0 or world > 1):
        def pinned(x):
            x = np.ascontiguousarray(x)
            t = torch.from_numpy(x.view({1: np.uint8, 2: np.int16, 4: np.int32, 8: np.int64}[x.dtype.itemsize]) if x.dtype.kind != "f" else x)
            return t.pin_memory()
        hA, hB, hC = pinned(inp["A"]), pinned(inp["B"]), pinned(inp["C"])
        hD = torch.empty((M, N), dtype=dD.dtype).pin_memory()
        hkw = {}
        if "k_chunk" in inp:
            hkw = dict(k_chunk=inp["k_chunk"], row_scale=pinned(inp["row_scale"]), col_scale=pinned(inp["col_scale"]))
        if "sfa" in inp:
            hkw.update(sfa=pinned(inp["sfa"]), sfb=pinned(inp["sfb"]))
        n_e2e = max(1, min(args.steps, 3))
        mmasim.gemm_host(model, hA, hB, hC, out=hD.numpy(), **hkw)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            mmasim.gemm_host(model, hA, hB, hC, out=hD.numpy(), **hkw)
        torch.cuda.synchronize()
        e2e_s = (time.perf_counter() - t0) / n_e2e
        e2e_s = max_over_ranks(e2e_s, dist, dev)
        h2d = hA.numel() * hA.element_size() + hB.numel() * hB.element_size() + hC.numel() * hC.element_size()
        e2e = {"value": macs_per_step / e2e_s, "unit": UNIT, "h2d_bytes_per_step": int(h2d),
               "d2h_bytes_per_step": int(hD.numel() * hD.element_size()), "ms_per_step": 1e3 * e2e_s,
               "api": "mmasim_gemm_host (stream-ordered allocation, then row panels: H2D, kernel and D2H of different panels overlap; free; per call)"}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    per_gpu_macs_s = value / world
    sm_mhz = clocks.get("sm_mhz") or 1965.0
    hbm_peak, hbm_src = 6650.0, "fallback 6.65 TB/s (MEASURED_PEAKS.json absent)"
    try:
        hbm_peak = float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["hbm_gbs"])
        hbm_src = "MEASURED_PEAKS.json hbm_gbs (STREAM-style copy)"
    except (OSError, KeyError, ValueError):
        pass

    def pipe_view(pipe, ops_per_mac, macs_s):
        """Fractions of one pipe: against the best live witness and against the nominal rate at the sampled clock."""
        label, _, per_clk = PIPES[pipe]
        nominal = SMS * per_clk * sm_mhz * 1e6
        measured = peaks[pipe]["peak"]
        achieved = macs_s * ops_per_mac
        return {"pipe": label, "pipe_ops_per_mac": ops_per_mac, "achieved": achieved / 1e12, "peak": measured / 1e12,
                "unit": "Tops/s", "frac": achieved / measured, "peak_nominal": nominal / 1e12, "frac_nominal": achieved / nominal,
                "peak_source": f"measured live, best witness {peaks[pipe]['witness']} at {peaks[pipe]['ctas_per_sm']} CTAs/SM "
                               f"(= {measured / (SMS * sm_mhz * 1e6):.1f} per SM and clock at the sampled {sm_mhz:.0f} MHz); "
                               f"nominal {per_clk:.0f} per SM and clock",
                "witnesses": {k: v / 1e12 for k, v in peaks[pipe]["all"].items()}}

    if is_dot:
        esz = inp["A"].dtype.itemsize
        bytes_per_dot = 2 * K * esz + 8
        gbs = per_gpu_macs_s / K * bytes_per_dot / 1e9
        roofline = {"bound": "hbm", "achieved": gbs, "peak": hbm_peak, "unit": "GB/s", "frac": gbs / hbm_peak, "traffic": None,
                    "kernel": kernel_name, "algorithmic_bytes_per_dot": bytes_per_dot, "peak_source": hbm_src}
    else:
        ops_per_mac = algorithmic_ops_per_mac(model)
        int_view = pipe_view("int_alu", ops_per_mac, per_gpu_macs_s)
        int_view["note"] = ("the count of 6 integer operations per term + 25 per block is not a floor for this formulation: the "
                            "kernel replaces multiply / distance / shift / add by one fused multiply-add and the maximum by a "
                            "tensor-core product of powers, so this fraction may exceed 1 and bounds nothing")
        roofline = {"bound": "alu", **pipe_view(pipe_key, pipe_ops_per_mac, per_gpu_macs_s), "kernel": kernel_name,
                    "traffic": NCU_DRAM_BYTES.get(name),
                    "traffic_source": "stored constant from a one-pass ncu capture of this workload at full size, main kernel + both decode launches (not measured in this run)" if name in NCU_DRAM_BYTES else None,
                    "algorithmic_bytes": NCU_ALGORITHMIC_BYTES.get(name),
                    "paper_level_integer_count": int_view}

    # ---- per-model leg: one model per kernel template at 4096^3, three launches each after three warm-ups, L2 flushed ----
    per_model, dot_line = None, None
    if not args.skip_extras and not is_dot and world == 1 and not args.no_per_model:
        from paper_2511_10909_b200 import workloads as wl
        size = args.per_model_size
        pm_peaks_needed = set()
        rows, cache = [], {}
        for pk in PER_MODEL:
            ck = (pk[1], pk[2])
            if ck not in cache:
                cache.clear()
                cache[ck] = {k: to_dev(v) for k, v in wl.normal_inputs(pk[1], pk[2], size, size, size, seed=5).items()}
            t = cache[ck]
            mdl = mmasim.Model(*pk)
            pkw = dict(sfa=t["sfa"], sfb=t["sfb"]) if "sfa" in t else {}
            out = mmasim.gemm(mdl, t["A"], t["B"], t["C"], K=size, **pkw)
            for _ in range(2):          # the host generated this model's inputs for seconds: let the clocks come back up
                mmasim.gemm(mdl, t["A"], t["B"], t["C"], out=out, K=size, **pkw)
            torch.cuda.synchronize()
            kern = mmasim.last_kernel()
            best, tot = None, 0.0
            for _ in range(3):
                flush.zero_()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                mmasim.gemm(mdl, t["A"], t["B"], t["C"], out=out, K=size, **pkw)
                e1.record()
                torch.cuda.synchronize()
                ms = e0.elapsed_time(e1)
                tot += ms
                best = ms if best is None else min(best, ms)
            pp, opm = pipe_of(kern, mdl)
            pm_peaks_needed.add(pp)
            rows.append({"model": "-".join(pk), "kernel": kern, "ms": tot / 3, "ms_best": best,
                         "macs_per_s": float(size) ** 3 / (tot / 3 * 1e-3), "_pipe": pp, "_opm": opm})
            del out
        cache.clear()
        peaks.update(measure_pipe_peaks(mmasim, torch, dev, sorted(pm_peaks_needed - set(peaks))))
        per_model = []
        for r in rows:
            v = pipe_view(r.pop("_pipe"), r.pop("_opm"), r["macs_per_s"])
            r.update(pipe=v["pipe"], pipe_ops_per_mac=v["pipe_ops_per_mac"], frac=v["frac"], frac_nominal=v["frac_nominal"])
            per_model.append(r)
        # the HBM-bound probe-style batch (config 4): 2^20 dots of length 32, FP16, both kernel kinds
        dot_line = []
        for dk in (("hopper", "fp16", "fp32"), ("cdna2", "fp16", "fp32")):
            A4, B4, C4 = wl.cfg4("fp16", 32)
            tA, tB, tC = to_dev(A4), to_dev(B4), to_dev(C4)
            mdl = mmasim.Model(*dk)
            o4 = mmasim.dot_batch(mdl, tA, tB, tC)
            torch.cuda.synchronize()
            tot = 0.0
            for _ in range(5):
                flush.zero_()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                mmasim.dot_batch(mdl, tA, tB, tC, out=o4)
                e1.record()
                torch.cuda.synchronize()
                tot += e0.elapsed_time(e1)
            nbytes = (1 << 20) * (2 * 32 * 2 + 8)
            gbs = nbytes / (tot / 5 * 1e-3) / 1e9
            # the same batch as a stream: eight copies of the inputs at different addresses (1.1 GB, nothing is read twice),
            # L2 flushed once, eight launches between one pair of events - launch and event overhead shared by eight batches
            sets = [(tA.clone(), tB.clone(), tC.clone(), torch.empty_like(o4)) for _ in range(8)]
            best_stream = None
            for _ in range(3):
                flush.zero_()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for sA, sB, sC, sO in sets:
                    mmasim.dot_batch(mdl, sA, sB, sC, out=sO)
                e1.record()
                torch.cuda.synchronize()
                us8 = e0.elapsed_time(e1) * 1e3 / len(sets)
                best_stream = us8 if best_stream is None else min(best_stream, us8)
            gbs_stream = nbytes / (best_stream * 1e-6) / 1e9
            dot_line.append({"model": "-".join(dk), "kernel": mmasim.last_kernel(), "dots": 1 << 20, "K": 32, "us": tot / 5 * 1e3,
                             "macs_per_s": (1 << 25) / (tot / 5 * 1e-3), "bound": "hbm", "achieved_gbs": gbs, "peak_gbs": hbm_peak,
                             "frac": gbs / hbm_peak, "peak_source": hbm_src,
                             "stream_of_8": {"us_per_batch": best_stream, "achieved_gbs": gbs_stream, "frac": gbs_stream / hbm_peak}})
            del tA, tB, tC, o4, sets
    if args.skip_extras or is_dot:
        cpu_value, cpu_info = None, {"cores": 0, "sample": "skipped"}
    else:
        cpu_value, cpu_info = oracle_sample_rate(name, inp)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": compute_dtype(kernel_name, model), "data": "synthetic",
        "config": {"workload": f"{name}: {desc}", "model": "-".join(key), "M": M, "N": N, "K": K,
                   "l2": "flushed between timed steps (256 MiB write)", "parallelism": f"replicas x{world} (independent batches, no exchange)"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": args.steps * KERNELS_PER_CALL.get(kernel_name, 1),
        "roofline": roofline,
        "cpu_baseline": {"value": cpu_value, "unit": UNIT, "kind": "oracle", **cpu_info},
        "per_model": per_model, "per_model_size": args.per_model_size if per_model else None, "dot_batch": dot_line,
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def native_difference(torch, key, model, dA, dB, dC, D):
    """Context column of config 5: on how many outputs does the B200's own tensor-core GEMM (cuBLAS through torch.mm /
    torch._scaled_mm, FP32 or FP64 result, C added afterwards in the accumulator type) differ from the model's words?
    The library GEMM is only the other side of this comparison; its summation order is its own business."""
    in_fmt, acc = key[1], key[2]
    try:
        if in_fmt in ("fp16", "bf16", "bf16_1k") and acc == "fp32":
            dt = torch.float16 if in_fmt == "fp16" else torch.bfloat16
            nat = torch.mm(dA.view(dt), dB.view(dt).t(), out_dtype=torch.float32) + dC.view(torch.float32)
            op = "torch.mm(out_dtype=float32) + C"
        elif in_fmt == "tf32":
            old = torch.backends.cuda.matmul.allow_tf32
            torch.backends.cuda.matmul.allow_tf32 = True
            nat = torch.mm(dA.view(torch.float32), dB.view(torch.float32).t()) + dC.view(torch.float32)
            torch.backends.cuda.matmul.allow_tf32 = old
            op = "torch.mm (TF32 allowed) + C"
        elif in_fmt == "fp32":
            old = torch.backends.cuda.matmul.allow_tf32
            torch.backends.cuda.matmul.allow_tf32 = False
            nat = torch.mm(dA.view(torch.float32), dB.view(torch.float32).t()) + dC.view(torch.float32)
            torch.backends.cuda.matmul.allow_tf32 = old
            op = "torch.mm (FP32) + C"
        elif in_fmt == "fp64":
            nat = torch.mm(dA.view(torch.float64), dB.view(torch.float64).t()) + dC.view(torch.float64)
            op = "torch.mm (FP64) + C"
        elif in_fmt in ("e4m3", "e5m2") and acc == "fp32":
            dt = torch.float8_e4m3fn if in_fmt == "e4m3" else torch.float8_e5m2
            one = torch.ones((), dtype=torch.float32, device=dA.device)
            nat = torch._scaled_mm(dA.view(dt), dB.view(dt).t(), scale_a=one, scale_b=one, out_dtype=torch.float32) + dC.view(torch.float32)
            op = "torch._scaled_mm(out_dtype=float32) + C"
        else:
            return {"native_op": None, "native_differs": None}
    except Exception as exc:                                   # an operand combination this torch / cuBLAS does not offer
        return {"native_op": f"unavailable: {type(exc).__name__}", "native_differs": None}
    words = nat.view(torch.int32 if nat.dtype == torch.float32 else torch.int64)
    return {"native_op": op, "native_differs": int((words != D.view(words.dtype)).sum().item()), "outputs": int(D.numel())}


def run_sweep(args):
    """Every registry row at size^3 (config 5 / the per-model headline): MAC/s per model, optional oracle check of
    seeded sampled outputs, one JSON line per model into the output folder (--out-dir) and a summary line on stdout."""
    import torch
    import oracle
    from paper_2511_10909_b200.build import build
    build()
    from paper_2511_10909_b200 import mmasim, workloads as wl
    torch.cuda.set_device(0)
    size = args.size
    M = N = K = size
    keys = sorted(oracle.REGISTRY)
    if args.models:
        keys = [k for k in keys if "-".join(k) in args.models.split(",")]
    out_dir = args.out_dir if os.path.isabs(args.out_dir) else os.path.join(ROOT, args.out_dir)
    os.makedirs(out_dir, exist_ok=True)
    out_path = os.path.join(out_dir, f"sweep_{size}.jsonl")
    cache = {}
    rows = []

    def to_dev(x):
        x = np.ascontiguousarray(x)
        return torch.from_numpy(x.view({1: np.uint8, 2: np.int16, 4: np.int32, 8: np.int64}[x.dtype.itemsize])).cuda()

    with open(out_path, "w") as fh:
        for key in keys:
            ck = (key[1], key[2])
            if ck not in cache:
                cache.clear()
                cache[ck] = wl.normal_inputs(key[1], key[2], M, N, K, seed=5)
            inp = cache[ck]
            model = mmasim.Model(*key)
            dA, dB, dC = to_dev(inp["A"]), to_dev(inp["B"]), to_dev(inp["C"])
            kw = {}
            if "sfa" in inp:
                kw = dict(sfa=to_dev(inp["sfa"]), sfb=to_dev(inp["sfb"]))
            D = mmasim.gemm(model, dA, dB, dC, **kw)            # warm-up
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(args.steps):
                mmasim.gemm(model, dA, dB, dC, out=D, **kw)
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / args.steps
            row = {"model": "-".join(key), "family": model.family, "kernel": mmasim.last_kernel(), "size": size,
                   "ms": ms, "macs_per_s": float(M) * N * K / (ms * 1e-3)}
            if args.native:
                row.update(native_difference(torch, key, model, dA, dB, dC, D))
            if args.check:
                pairs = wl.sample_pairs(M, N, args.check, seed=55)
                A, B = inp["A"], inp["B"]
                if key[1] in ("mxf4", "nvf4"):
                    lo, hi = A & 0xF, A >> 4
                    A = np.stack([lo, hi], axis=-1).reshape(M, K)
                    lo, hi = B & 0xF, B >> 4
                    B = np.stack([lo, hi], axis=-1).reshape(N, K)
                want = oracle.phi_gemm_sampled(oracle.lookup(*key), A, B, inp["C"], pairs, SFA=inp.get("sfa"), SFB=inp.get("sfb"))
                got = D.cpu().numpy()
                got = got.view({2: np.uint16, 4: np.uint32, 8: np.uint64}[got.dtype.itemsize])[pairs[:, 0], pairs[:, 1]].astype(np.uint64)
                row["checked"] = int(args.check)
                row["mismatches"] = int((got != want).sum())
            fh.write(json.dumps(row) + "\n")
            fh.flush()
            rows.append(row)
            del dA, dB, dC, D
    bad = sum(r.get("mismatches", 0) for r in rows)
    print(json.dumps({"sweep": size, "models": len(rows), "mismatching_outputs": bad,
                      "min_macs_per_s": min(r["macs_per_s"] for r in rows), "max_macs_per_s": max(r["macs_per_s"] for r in rows),
                      "file": os.path.relpath(out_path, ROOT)}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3", choices=sorted(WORKLOADS))
    ap.add_argument("--skip-extras", action="store_true",
                    help="skip the end-to-end and CPU-oracle legs (profiler captures only; not a valid bench line)")
    ap.add_argument("--no-per-model", action="store_true", help="skip the per-model and dot_batch legs of the line")
    ap.add_argument("--per-model-size", type=int, default=4096, help="M = N = K of the per-model leg")
    ap.add_argument("--sweep", action="store_true", help="time every registry row at --size^3 (not the bench line)")
    ap.add_argument("--size", type=int, default=4096)
    ap.add_argument("--check", type=int, default=0, help="with --sweep: compare this many seeded sampled outputs per model with the oracle")
    ap.add_argument("--out-dir", default="sweep_out", help="with --sweep: folder of the per-model JSON lines")
    ap.add_argument("--native", action="store_true",
                    help="with --sweep: also count the outputs on which the B200's native tensor-core GEMM (torch.mm / torch._scaled_mm) "
                         "differs from each model (context only)")
    ap.add_argument("--models", default="", help="with --sweep: comma-separated arch-infmt-acc names (default: all)")
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
