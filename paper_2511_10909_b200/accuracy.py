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


def _words(x, fmt: str):
    """Real numpy array -> CUDA tensor of raw words of ``fmt`` (signed integer view of the storage width)."""
    import numpy as np
    import torch
    from . import workloads as wl
    w = wl.cast(np.asarray(x, dtype=np.float32), fmt)
    return torch.from_numpy(w.view({1: np.uint8, 2: np.int16, 4: np.int32}[w.dtype.itemsize])).cuda()


def asymmetry_count(model: mmasim.Model, A, B, C) -> dict:
    """On how many outputs Phi(-A, B, -C) differs from -Phi(A, B, C) as a value (Section 6.2: asymmetric models), with
    the sign of the difference sum(Phi(A, B, C) + Phi(-A, B, -C)) as the direction of the bias."""
    import torch
    def neg(t):                                            # flip the sign bit of every word
        bits = t.element_size() * 8
        return t ^ (0x80 if t.dtype == torch.uint8 else -(1 << (bits - 1)))
    D = widen(model.acc, mmasim.gemm(model, A, B, C))
    Dn = widen(model.acc, mmasim.gemm(model, neg(A), B, neg(C)))
    ok = torch.isfinite(D) & torch.isfinite(Dn)
    s = torch.where(ok, D + Dn, torch.zeros_like(D))
    return {"count": int(ok.sum()), "asymmetric": int((s != 0).sum()), "mean_sum": float(s.mean())}


def risky_designs(M: int = 512, N: int = 512, K: int = 256, seed: int = 64) -> dict:
    """The rows of Table 10 as statistics at GEMM scale (deviation from the real result A x B + C in FP64; every pair is
    the affected row against the nearest row without the design in question, on the same inputs):
      input_ftz      CDNA2 FP16 (flushes subnormal inputs) against CDNA1 FP16 (exact dot product), A ~ 2^-14 N(0,1);
      small_F        Hopper FP8, F = 13, against the same row with F = 25;
      rz_e8m13       Hopper FP8 with F = 25 and rho = RZ-E8M13 against rho = RZ-FP32;
      rne_fp16       Hopper FP16 with FP16 output against FP32 output, C = 0;
      asymmetry      CDNA3 FP16 / BF16 / FP8 against Hopper FP16: outputs with Phi(-A, B, -C) != -Phi(A, B, C), inputs of
                     Section 6.2.4 (A, B ~ 1000 N(0,1) for the 16-bit types, 16 N(0,1) for FP8; C ~ N(0,1))."""
    import numpy as np
    from . import workloads as wl
    g = wl.rng(seed)
    out = {}
    # input FTZ: most elements of A are FP16 subnormals
    A = _words(g.standard_normal((M, K)) * 2.0 ** -14, "fp16")
    B = _words(g.standard_normal((N, K)), "fp16")
    ref = reference_fp64("fp16", "fp32", A, B)
    out["input_ftz"] = {"cdna2": deviation_stats(mmasim.Model("cdna2", "fp16", "fp32"), A, B, None, ref),
                        "cdna1": deviation_stats(mmasim.Model("cdna1", "fp16", "fp32"), A, B, None, ref)}
    # FP8 rows
    A8 = _words(g.standard_normal((M, K)), "e4m3")
    B8 = _words(g.standard_normal((N, K)), "e4m3")
    C8 = _words(g.standard_normal((M, N)), "fp32")
    ref8 = reference_fp64("e4m3", "fp32", A8, B8, C8)
    out["small_F"] = {"F13": deviation_stats(mmasim.Model("hopper", "e4m3", "fp32", rho="RZ-FP32"), A8, B8, C8, ref8),
                      "F25": deviation_stats(mmasim.Model("hopper", "e4m3", "fp32", rho="RZ-FP32", F=25), A8, B8, C8, ref8)}
    out["rz_e8m13"] = {"RZ-E8M13": deviation_stats(mmasim.Model("hopper", "e4m3", "fp32", F=25), A8, B8, C8, ref8),
                       "RZ-FP32": out["small_F"]["F25"]}
    # FP16 output
    A16 = _words(g.standard_normal((M, K)), "fp16")
    B16 = _words(g.standard_normal((N, K)), "fp16")
    ref16 = reference_fp64("fp16", "fp32", A16, B16)
    out["rne_fp16"] = {"fp16_out": deviation_stats(mmasim.Model("hopper", "fp16", "fp16"), A16, B16, None, ref16),
                       "fp32_out": deviation_stats(mmasim.Model("hopper", "fp16", "fp32"), A16, B16, None, ref16)}
    # asymmetry
    Cn = _words(g.standard_normal((M, N)), "fp32")
    asym = {}
    for arch, fmt, scale in (("cdna3", "fp16", 1000.0), ("cdna3", "bf16", 1000.0), ("cdna3", "e4m3", 16.0), ("hopper", "fp16", 1000.0)):
        Aa = _words(scale * g.standard_normal((M, 64)), fmt)
        Ba = _words(scale * g.standard_normal((N, 64)), fmt)
        asym[f"{arch}-{fmt}"] = asymmetry_count(mmasim.Model(arch, fmt, "fp32"), Aa, Ba, Cn)
    out["asymmetry"] = asym
    return out
