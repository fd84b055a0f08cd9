"""MMA models Phi and the instruction-to-model registry (test infrastructure, CPU oracle).

    phi_ftz_addmul   Algorithm 2          phi_fma   Algorithm 4
    phi_fdpa         Algorithm 5 (chains E-/T-/ST-/GST-/TR-/GTR-FDPA blocks)
    REGISTRY         Tables 3-7 (typed from the paper, not shared with the CUDA library)

Matrices are numpy arrays of raw words: A is M x K, B is N x K (each row of B
is one column of the paper's K x N matrix), C is M x N.  GST inputs are given
one FP4 code per array element here (the packed two-per-byte layout is a
property of the library's interface, not of the model).
"""
from __future__ import annotations

import os
from dataclasses import dataclass
from multiprocessing import get_context

import numpy as np

from .formats import FORMATS
from . import ops

ARCHS = ("volta", "turing", "ampere", "ada", "hopper", "blackwell", "rtx_blackwell",
         "cdna1", "cdna2", "cdna3")


@dataclass(frozen=True)
class Model:
    arch: str
    in_fmt: str            # registry name of the input type (e.g. 'bf16_1k', 'mxe4m3', 'nvf4')
    acc: str               # 'fp32' | 'fp16' | 'fp64'
    family: str            # 'fma' | 'ftz' | 'e' | 't' | 'st' | 'gst' | 'tr' | 'gtr'
    elem: str              # element format of A and B (key of FORMATS)
    L: int = 0             # L_max (FDPA families)
    F: int = 0
    F2: int = 0
    rho: str = ""
    P: int = 0             # FTZ-AddMul group size
    G: int = 0             # GST group size
    k_block: int = 0       # elements per scale factor (ST: 32; GST: 32 or 16)
    scale: str = ""        # scale-factor format
    literal_emax: bool = False   # the maximum exponent over every term, as Algorithms 7-11 print it (not reading R2)


def _build_registry():
    reg = {}

    def add(arch, in_fmt, acc, family, elem, **kw):
        reg[(arch, in_fmt, acc)] = Model(arch, in_fmt, acc, family, elem, **kw)

    def tf(arch, in_fmt, acc, L, F, rho):       # T-FDPA row of Table 4
        add(arch, in_fmt, acc, "t", in_fmt, L=L, F=F, rho=rho)

    # Table 4, Volta and Turing
    tf("volta", "fp16", "fp32", 4, 23, "RZ-FP32")
    tf("volta", "fp16", "fp16", 4, 23, "RNE-FP16")
    tf("turing", "fp16", "fp32", 8, 24, "RZ-FP32")
    tf("turing", "fp16", "fp16", 8, 24, "RNE-FP16")
    # Ampere, Ada Lovelace
    for arch in ("ampere", "ada"):
        tf(arch, "tf32", "fp32", 4, 24, "RZ-FP32")
        tf(arch, "bf16", "fp32", 8, 24, "RZ-FP32")
        tf(arch, "fp16", "fp32", 8, 24, "RZ-FP32")
        tf(arch, "fp16", "fp16", 8, 24, "RNE-FP16")
    for f8 in ("e4m3", "e5m2"):
        tf("ada", f8, "fp32", 16, 13, "RZ-E8M13")
        tf("ada", f8, "fp16", 16, 13, "RNE-FP16")
    # Hopper
    tf("hopper", "tf32", "fp32", 8, 25, "RZ-FP32")
    tf("hopper", "bf16", "fp32", 16, 25, "RZ-FP32")
    tf("hopper", "fp16", "fp32", 16, 25, "RZ-FP32")
    tf("hopper", "fp16", "fp16", 16, 25, "RNE-FP16")
    for f8 in ("e4m3", "e5m2"):
        tf("hopper", f8, "fp32", 32, 13, "RZ-E8M13")
        tf("hopper", f8, "fp16", 32, 13, "RNE-FP16")
    # Blackwell, RTX Blackwell (Table 4 and Table 5)
    for arch in ("blackwell", "rtx_blackwell"):
        tf(arch, "tf32", "fp32", 8, 25, "RZ-FP32")
        tf(arch, "bf16", "fp32", 16, 25, "RZ-FP32")
        tf(arch, "fp16", "fp32", 16, 25, "RZ-FP32")
        tf(arch, "fp16", "fp16", 16, 25, "RNE-FP16")
        for f in ("e4m3", "e5m2", "e3m2", "e2m3", "e2m1"):
            tf(arch, f, "fp32", 32, 25, "RZ-FP32")
            tf(arch, f, "fp16", 32, 25, "RNE-FP16")
            add(arch, "mx" + f, "fp32", "st", f, L=32, F=25, rho="RZ-FP32", k_block=32, scale="e8m0")
        add(arch, "mxf4", "fp32", "gst", "e2m1", L=64, G=16, F=35, rho="RZ-FP32", k_block=32, scale="e8m0")
        add(arch, "nvf4", "fp32", "gst", "e2m1", L=64, G=16, F=35, rho="RZ-FP32", k_block=16, scale="ue4m3")
    # Table 3: every NVIDIA FP64 instruction is a chain of FMAs
    for arch in ("ampere", "ada", "hopper", "blackwell", "rtx_blackwell"):
        add(arch, "fp64", "fp64", "fma", "fp64")
    # Table 6 and Table 7: AMD
    add("cdna1", "fp32", "fp32", "fma", "fp32")
    add("cdna1", "bf16", "fp32", "e", "bf16", L=2)
    add("cdna1", "fp16", "fp32", "e", "fp16", L=4)
    for arch in ("cdna2", "cdna3"):
        add(arch, "fp64", "fp64", "fma", "fp64")
        add(arch, "fp32", "fp32", "fma", "fp32")
    add("cdna2", "bf16", "fp32", "ftz", "bf16", P=2)
    add("cdna2", "bf16_1k", "fp32", "ftz", "bf16", P=4)
    add("cdna2", "fp16", "fp32", "ftz", "fp16", P=4)
    add("cdna3", "tf32", "fp32", "tr", "tf32", L=4, F=24, F2=31, rho="RNE-FP32")
    add("cdna3", "bf16", "fp32", "tr", "bf16", L=8, F=24, F2=31, rho="RNE-FP32")
    add("cdna3", "fp16", "fp32", "tr", "fp16", L=8, F=24, F2=31, rho="RNE-FP32")
    for f8 in ("e4m3", "e5m2"):
        add("cdna3", f8, "fp32", "gtr", f8, L=16, F=24, F2=31, rho="RNE-FP32")
    return reg


REGISTRY = _build_registry()


def printed(m: Model) -> Model:
    """The same registry row with the maximum exponent taken over every term, as Algorithms 7-11 print it."""
    from dataclasses import replace
    return replace(m, literal_emax=True)


def lookup(arch: str, in_fmt: str, acc: str) -> Model:
    return REGISTRY[(arch, in_fmt, acc)]


# ----------------------------------------------------------------------------
# one output element: d = Phi(a, b, c)
# ----------------------------------------------------------------------------
def phi_fma(a, b, c, fmt):
    """Algorithm 4: chain of standard FMAs in ascending k."""
    d = c
    for ak, bk in zip(a, b):
        d = ops.fma(ak, bk, d, fmt)
    return d


def phi_ftz_addmul(a, b, c, fmt, P):
    """Algorithm 2: flush input subnormals to +0; per P products a pairwise FTZ-Add tree, then FTZ-Add into d."""
    fp32 = FORMATS["fp32"]
    a = [ops.flush_subnormal(w, fmt) for w in a]
    b = [ops.flush_subnormal(w, fmt) for w in b]
    d = ops.flush_subnormal(c, fp32)
    K = len(a)
    for k in range(0, K - P + 1, P):
        p = [ops.ftz_mul(a[k + l], b[k + l], fmt) for l in range(P)]
        s = ops.ftz_add(p[0], p[1])
        if P == 4:
            s2 = ops.ftz_add(p[2], p[3])
            s = ops.ftz_add(s, s2)
        d = ops.ftz_add(d, s)
    return d


def _fdpa_block(m: Model, a, b, d, sfa, sfb, k0, L):
    fa = fb = FORMATS[m.elem]
    fc = FORMATS[m.acc]
    if m.family == "t":
        return ops.t_fdpa(a, b, d, fa, fb, fc, m.F, m.rho, literal_emax=m.literal_emax)
    if m.family == "st":
        j = k0 // m.k_block
        return ops.st_fdpa(a, b, d, sfa[j], sfb[j], fa, fb, m.F, m.rho, literal_emax=m.literal_emax)
    if m.family == "gst":
        j0, n = k0 // m.k_block, max(L // m.k_block, 1)
        return ops.gst_fdpa(a, b, d, sfa[j0:j0 + n], sfb[j0:j0 + n], FORMATS[m.scale], m.k_block, m.G, m.F, m.rho,
                            literal_emax=m.literal_emax)
    if m.family == "tr":
        return ops.tr_fdpa(a, b, d, fa, fb, m.F, m.F2, m.rho, literal_emax=m.literal_emax)
    if m.family == "gtr":
        return ops.gtr_fdpa(a, b, d, fa, fb, m.F, m.F2, m.rho, literal_emax=m.literal_emax)
    if m.family == "e":
        return ops.e_fdpa(a, b, d, fa, fb)
    raise ValueError(m.family)


def phi_fdpa(m: Model, a, b, c, sfa=None, sfb=None):
    """Algorithm 5: L = min(K, L_max); d <- FDPA(a[k..k+L), b[k..k+L), d) for k = 0, L, 2L, ..."""
    K = len(a)
    L = min(K, m.L)
    d = c
    for k in range(0, K - L + 1, L):
        d = _fdpa_block(m, a[k:k + L], b[k:k + L], d, sfa, sfb, k, L)
    return d


def phi_dot(m: Model, a, b, c, sfa=None, sfb=None) -> int:
    """d = Phi(a, b, c) for one output element; a, b are sequences of K raw words."""
    if m.family == "fma":
        return phi_fma(a, b, c, FORMATS[m.elem])
    if m.family == "ftz":
        return phi_ftz_addmul(a, b, c, FORMATS[m.elem], m.P)
    return phi_fdpa(m, a, b, c, sfa, sfb)


NAN_CUDA_CORE = 0x7FFFFFFF


def _cuda_core(word: int) -> int:
    """FP32 add / mul on the general compute units: IEEE result, NaN encoded as 0x7FFFFFFF."""
    return NAN_CUDA_CORE if (word & 0x7FFFFFFF) > 0x7F800000 else word


def chunk_promote_dot(m: Model, a, b, c, k_chunk: int, sfa=None, sfb=None) -> int:
    """Software workaround of Sections 2.2 and 6.3 (promotion of partial sums to FP32).

    The paper motivates but does not define it; the definition used here: every
    k_chunk elements of K, the model is run from a +0 accumulator and its result
    is added to an FP32 running sum with an IEEE-754 RNE addition.
    """
    acc = c
    for k in range(0, len(a), k_chunk):
        part = phi_dot(m, a[k:k + k_chunk], b[k:k + k_chunk], 0,
                       None if sfa is None else sfa[k // m.k_block:(k + k_chunk) // m.k_block],
                       None if sfb is None else sfb[k // m.k_block:(k + k_chunk) // m.k_block])
        acc = _cuda_core(ops.ieee_add_f32(acc, part))
    return acc


def dequant(d: int, row_scale: int, col_scale: int) -> int:
    """Epilogue D = fl32(fl32(sa_i * sb_j) * d) with IEEE-754 RNE multiplications (FP32 words)."""
    s = _cuda_core(ops.ieee_mul_f32(row_scale, col_scale))
    return _cuda_core(ops.ieee_mul_f32(s, d))


# ----------------------------------------------------------------------------
# matrix-level drivers
# ----------------------------------------------------------------------------
_G: dict = {}


def _one(i, j):
    g = _G
    m = g["m"]
    a, b = g["rowsA"](i), g["rowsB"](j)
    c = int(g["C"][i, j]) if g["C"] is not None else 0
    sfa = g["sfaRows"](i) if g["SFA"] is not None else None
    sfb = g["sfbRows"](j) if g["SFB"] is not None else None
    if g["k_chunk"]:
        d = chunk_promote_dot(m, a, b, c, g["k_chunk"], sfa, sfb)
    else:
        d = phi_dot(m, a, b, c, sfa, sfb)
    if g["rs"] is not None:
        d = dequant(d, int(g["rs"][i]), int(g["cs"][j]))
    return d


def _work(pairs):
    return [_one(i, j) for i, j in pairs]


def _row_cache(X):
    cache = {}

    def get(i):
        r = cache.get(i)
        if r is None:
            if len(cache) > 4096:
                cache.clear()
            r = cache[i] = X[i].tolist()
        return r
    return get


def phi_gemm_sampled(m: Model, A, B, C, pairs, SFA=None, SFB=None, k_chunk=0,
                     row_scale=None, col_scale=None, processes=None):
    """Output words of D = Phi(A, B, C) at the (i, j) positions in ``pairs`` (list of tuples).

    Runs on ``processes`` worker processes (default: all cores).  Returns a numpy
    array of unsigned 64-bit words in the order of ``pairs``.
    """
    pairs = [(int(i), int(j)) for i, j in pairs]
    _G.update(m=m, rowsA=_row_cache(A), rowsB=_row_cache(B), C=C, SFA=SFA, SFB=SFB,
              sfaRows=_row_cache(SFA) if SFA is not None else None,
              sfbRows=_row_cache(SFB) if SFB is not None else None,
              k_chunk=k_chunk, rs=row_scale, cs=col_scale)
    nproc = processes or os.cpu_count() or 1
    if nproc == 1 or len(pairs) < 64:
        out = _work(pairs)
    else:
        nchunk = min(len(pairs), nproc * 8)
        chunks = [pairs[t::nchunk] for t in range(nchunk)]
        with get_context("fork").Pool(nproc) as pool:
            parts = pool.map(_work, chunks)
        out = [0] * len(pairs)
        for t, part in enumerate(parts):
            out[t::nchunk] = part
    return np.array(out, dtype=np.uint64)


def phi_gemm(m: Model, A, B, C, **kw):
    """Every output word of D = Phi(A, B, C); returns an M x N array of unsigned 64-bit words."""
    M, N = A.shape[0], B.shape[0]
    pairs = [(i, j) for i in range(M) for j in range(N)]
    return phi_gemm_sampled(m, A, B, C, pairs, **kw).reshape(M, N)


def phi_dot_batch(m: Model, A, B, C, processes=None):
    """n independent dot products: A, B are n x K, C has n words; returns n words."""
    n = A.shape[0]
    _G.update(m=m, A=A, B=B, Cv=C)
    nproc = processes or os.cpu_count() or 1
    if nproc == 1 or n < 64:
        out = _dot_rows((0, n))
    else:
        step = -(-n // (nproc * 4))
        spans = [(s, min(s + step, n)) for s in range(0, n, step)]
        with get_context("fork").Pool(nproc) as pool:
            parts = pool.map(_dot_rows, spans)
        out = [w for part in parts for w in part]
    return np.array(out, dtype=np.uint64)


def _dot_rows(span):
    g = _G
    m, A, B, Cv = g["m"], g["A"], g["B"], g["Cv"]
    lo, hi = span
    Al, Bl, Cl = A[lo:hi].tolist(), B[lo:hi].tolist(), Cv[lo:hi].tolist()
    return [phi_dot(m, a, b, c) for a, b, c in zip(Al, Bl, Cl)]
