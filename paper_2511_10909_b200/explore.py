"""Workaround and design-space exploration (Sections 6.3 and 7) on top of the library's entry points.

Three experiments, all at GEMM scale on the GPU, each returning the deviation statistics of `accuracy.deviation_stats`
against the FP64 real result:

* `design_sweep`    - hypothetical T-FDPA units: the registry row of a model with other (L_max, F, rho), made by
                      `mmasim_create_model_ex` overrides, to see which parameter buys how much accuracy;
* `chunk_sweep`     - the FP32-promotion workaround for low-precision accumulation with chunk sizes other than 128;
* `fp8_via_fp16`    - the workaround that feeds FP8 data to the FP16 instruction (every E4M3 / E5M2 value is an FP16
                      value): the same architecture's FP16 row evaluated on the widened words.

* `b200_fp8_mma_sync` - what the B200's own warp-level FP8 instruction computes (found with the probes of clfp.py and
                      confirmed bit for bit against `mmasim_hw_mma`): that workaround, in hardware.

torch widens FP8 words to FP16 words; every arithmetic step of a model runs in the library's kernels.
"""
from __future__ import annotations

from . import accuracy, mmasim


def design_sweep(arch: str, in_fmt: str, acc: str, A, B, C=None, l_max=(None,), F=(None,), rho=(None,), ref=None):
    """Deviation statistics of the (arch, in_fmt, acc) row and of its variants with every combination of the given
    L_max, F and rho (None = the table's value).  Returns a list of dicts with the parameters actually used."""
    if ref is None:
        ref = accuracy.reference_fp64(in_fmt, acc, A, B, C)
    out = []
    for L in l_max:
        for f in F:
            for r in rho:
                ov = {}
                if L is not None:
                    ov["l_max"] = L
                if f is not None:
                    ov["F"] = f
                if r is not None:
                    ov["rho"] = r
                m = mmasim.Model(arch, in_fmt, acc, **ov)
                s = accuracy.deviation_stats(m, A, B, C, ref)
                s.update(l_max=m.l_max, F=m.F, rho=m.rho, kernel=mmasim.last_kernel())
                out.append(s)
    return out


def chunk_sweep(model: mmasim.Model, A, B, chunks=(0, 32, 64, 128, 256, 512), row_scale=None, col_scale=None, ref=None):
    """Deviation statistics of the model with FP32 promotion every `k_chunk` elements of K (0 = no promotion: the
    hardware accumulator runs over all of K).  C = +0, as in the workaround; the per-row and per-column scales are
    given together or not at all and enter the real result too."""
    if ref is None:
        ref = accuracy.reference_fp64(model.in_fmt, model.acc, A, B, None)
        if row_scale is not None:
            ref = ref * row_scale.double()[:, None]
        if col_scale is not None:
            ref = ref * col_scale.double()[None, :]
    out = []
    for kc in chunks:
        kw = dict(k_chunk=kc)
        if row_scale is not None:
            kw.update(row_scale=row_scale, col_scale=col_scale)
        D = mmasim.gemm(model, A, B, None, **kw)
        s = _stats(model.acc, D, ref)
        s.update(k_chunk=kc, kernel=mmasim.last_kernel())
        out.append(s)
    return out


def widen_fp8_to_fp16(fmt: str, words):
    """E4M3 / E5M2 bytes -> the FP16 words of the same values (exact: both formats are subsets of FP16)."""
    import torch
    t = {"e4m3": torch.float8_e4m3fn, "e5m2": torch.float8_e5m2}[fmt]
    return words.view(t).to(torch.float16).view(torch.int16)


def fp8_via_fp16(arch: str, fmt: str, A, B, C=None, acc: str = "fp32", ref=None):
    """The FP8 row of `arch` against the same architecture's FP16 row fed with the widened FP8 data."""
    if ref is None:
        ref = accuracy.reference_fp64(fmt, acc, A, B, C)
    native = mmasim.Model(arch, fmt, acc)
    via = mmasim.Model(arch, "fp16", acc)
    s8 = accuracy.deviation_stats(native, A, B, C, ref)
    s8.update(model=repr(native))
    s16 = accuracy.deviation_stats(via, widen_fp8_to_fp16(fmt, A), widen_fp8_to_fp16(fmt, B), C, ref)
    s16.update(model=repr(via))
    return {"native": s8, "via_fp16": s16}


def b200_fp8_mma_sync(fmt: str, A, B, C=None, b_fmt: str | None = None):
    """The B200's `mma.sync.m16n8k32` on E4M3 / E5M2 operands (`b_fmt`: the type of B if it differs from that of A)
    with an FP32 accumulator, chained over K in steps of 32,
    as a composition of the paper's models: per instruction the FP8 values, as FP16, go through the Blackwell FP16 row
    (T-FDPA, L = 16, F = 25, RZ-FP32) in two blocks from a +0 accumulator - first the elements k = 0, 1 mod 4, then
    k = 2, 3 mod 4 with the first block's result as accumulator (the two halves of each 32-bit operand register) - and
    C is added by a separate FP32 addition (RNE; NaN as 0x7FFFFFFF).  That is the FP32-promotion workaround of
    Section 6.3 with chunks of 32, so the library evaluates it with `k_chunk = 32` on widened, reordered operands.
    (With an FP16 accumulator the instruction does the same with the FP16 -> FP16 row and an FP16 addition of C; the
    library has no FP16 promotion, `tests/test_gpu_hw_mma.py` composes that case from two calls and a half addition.)"""
    import torch
    K = A.shape[1]
    if K % 32:
        raise ValueError("K must be a multiple of the instruction's 32")
    order = [32 * q + k for q in range(K // 32) for half in ((0, 1), (2, 3)) for k in range(32) if k % 4 in half]
    p = torch.tensor(order, device=A.device)
    A16 = widen_fp8_to_fp16(fmt, A)[:, p].contiguous()
    B16 = widen_fp8_to_fp16(b_fmt or fmt, B)[:, p].contiguous()
    return mmasim.gemm(mmasim.Model("blackwell", "fp16", "fp32"), A16, B16, C, k_chunk=32)


def _stats(acc: str, D, ref) -> dict:
    s = mmasim.error_stats(acc, D, ref).cpu().tolist()
    n = max(s[0], 1.0)
    return {"count": int(s[0]), "mean": s[1] / n, "mean_abs": s[2] / n, "rms": (s[3] / n) ** 0.5, "negative": s[4] / n,
            "positive": s[5] / n, "max_abs": s[6], "mean_rel": s[7] / n}


def printed_form_difference(arch: str, in_fmt: str, acc: str, A, B, C=None, **kw) -> dict:
    """On how many outputs does the registry row change when the maximum exponent of the fused sum runs over every term,
    as Algorithms 7-11 print it, instead of over the nonzero terms (what the B200's own rows do)?  Runs the row and its
    `literal_emax` override on the same inputs; returns the count, the number of outputs and both results."""
    row = mmasim.gemm(mmasim.Model(arch, in_fmt, acc), A, B, C, **kw)
    lit = mmasim.gemm(mmasim.Model(arch, in_fmt, acc, literal_emax=1), A, B, C, **kw)
    return {"differing": int((row != lit).sum()), "outputs": row.numel(), "row": row, "printed": lit}
