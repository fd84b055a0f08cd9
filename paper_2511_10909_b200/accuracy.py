"""Accuracy analysis at GEMM scale (Section 6): deviation of a model's output from the real result A x B + C.

The real result is computed on the GPU in FP64 (the element values widened exactly, the FP64 multiply-add chain of
the library: Phi_FMA with FP64 operands), the deviations are reduced on the GPU by `mmasim_error_stats`.  torch is
used to widen raw words to FP64 tensors and for nothing else.
"""
from __future__ import annotations

from . import mmasim


def widen(fmt: str, words):
    """Raw element words (CUDA integer tensor) -> FP64 tensor of their values."""
    import torch
    if fmt == "fp16":
        return words.view(torch.float16).double()
    if fmt in ("bf16", "bf16_1k"):
        return words.view(torch.bfloat16).double()
    if fmt == "tf32":
        return (words & ~0x1FFF).view(torch.float32).double()
    if fmt == "fp32":
        return words.view(torch.float32).double()
    if fmt == "e4m3":
        return words.view(torch.float8_e4m3fn).double()
    if fmt == "e5m2":
        return words.view(torch.float8_e5m2).double()
    raise ValueError(f"no widening for {fmt}")


def reference_fp64(in_fmt: str, acc: str, A, B, C=None):
    """D_real = A x B^T + C in FP64 (FP64 multiply-add chain in ascending k): an M x N FP64 CUDA tensor."""
    import torch
    fp64 = mmasim.Model("ampere", "fp64", "fp64")
    A64 = widen(in_fmt, A).view(torch.int64)
    B64 = widen(in_fmt, B).view(torch.int64)
    C64 = None if C is None else widen(acc, C).view(torch.int64)
    return mmasim.gemm(fp64, A64, B64, C64).view(torch.float64)


def deviation_stats(model: mmasim.Model, A, B, C=None, ref=None) -> dict:
    """Run the model and reduce delta = D - D_real: count, mean, mean |delta|, rms, share of negative / positive
    deviations, max |delta|, mean relative error."""
    if ref is None:
        ref = reference_fp64(model.in_fmt, model.acc, A, B, C)
    D = mmasim.gemm(model, A, B, C)
    s = mmasim.error_stats(model.acc, D, ref).cpu().tolist()
    n = max(s[0], 1.0)
    return {"count": int(s[0]), "mean": s[1] / n, "mean_abs": s[2] / n, "rms": (s[3] / n) ** 0.5, "negative": s[4] / n,
            "positive": s[5] / n, "max_abs": s[6], "mean_rel": s[7] / n}


def bias_experiment(M: int = 1024, N: int = 1024, K: int = 8, seed: int = 63) -> dict:
    """The experiment of Section 6.2.4 / Figure 3: C ~ N(0,1), A, B ~ 1000 x N(0,1) in FP16, one CDNA3 FP16 block
    chain of length K under TR-FDPA (round-down inside) and under its hypothetical round-to-zero variant."""
    import numpy as np
    import torch
    from . import workloads as wl
    g = wl.rng(seed)
    A = torch.from_numpy(wl.cast((1000.0 * g.standard_normal((M, K))).astype(np.float32), "fp16").view(np.int16)).cuda()
    B = torch.from_numpy(wl.cast((1000.0 * g.standard_normal((N, K))).astype(np.float32), "fp16").view(np.int16)).cuda()
    C = torch.from_numpy(g.standard_normal((M, N)).astype(np.float32).view(np.int32)).cuda()
    ref = reference_fp64("fp16", "fp32", A, B, C)
    rd = deviation_stats(mmasim.Model("cdna3", "fp16", "fp32"), A, B, C, ref)
    rz = deviation_stats(mmasim.Model("cdna3", "fp16", "fp32", inner_round=1), A, B, C, ref)
    return {"RD": rd, "RZ": rz}
