"""Seeded synthetic inputs shaped like the paper's workloads (serves the tests, the benchmark and the oracle runs).

This module only *produces input words*: random draws (numpy Philox streams) and casts of real numbers to the
storage formats.  It holds none of the models' arithmetic and is imported by neither the oracle nor the library.

The paper validates on random inputs from common distributions, on ill-conditioned inputs and on random bit
streams (Section 3.1, Step 4) and runs its bias experiment on normal matrices (Section 6.2.4); no public
dataset is involved, so these generators are the workloads themselves, not stand-ins.
"""
from __future__ import annotations

import numpy as np

ELEM_OF = {"bf16_1k": "bf16", "mxe4m3": "e4m3", "mxe5m2": "e5m2", "mxe3m2": "e3m2", "mxe2m3": "e2m3",
           "mxe2m1": "e2m1", "mxf4": "e2m1", "nvf4": "e2m1"}
_SMALL = {"e4m3": (4, 3, 7, "fn"), "e5m2": (5, 2, 15, "ieee"), "e3m2": (3, 2, 3, "none"),
          "e2m3": (2, 3, 1, "none"), "e2m1": (2, 1, 1, "none"), "ue4m3": (4, 3, 7, "fn")}
WORD_DTYPE = {"fp64": np.uint64, "fp32": np.uint32, "tf32": np.uint32, "bf16": np.uint16, "fp16": np.uint16}


def rng(seed: int, stream: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=seed + (stream << 32)))


def elem_format(in_fmt: str) -> str:
    return ELEM_OF.get(in_fmt, in_fmt)


def word_dtype(fmt: str):
    return WORD_DTYPE.get(elem_format(fmt), np.uint8)


# ------------------------------------------------------------------------------------------------------------
# casts (round to nearest even, saturating for the formats without infinity)
# ------------------------------------------------------------------------------------------------------------
def _positive_values(name: str) -> np.ndarray:
    eb, mb, bias, special = _SMALL[name]
    codes = np.arange(1 << (eb + mb))
    field, mant = codes >> mb, codes & ((1 << mb) - 1)
    vals = np.where(field == 0, mant / (1 << mb) * 2.0 ** (1 - bias), (1 + mant / (1 << mb)) * 2.0 ** (field - bias))
    if special == "ieee":
        vals = vals[field < (1 << eb) - 1]
    elif special == "fn":
        vals = vals[:-1]
    return vals


def cast_small(x: np.ndarray, name: str) -> np.ndarray:
    """Nearest-even, saturating cast of finite reals to an 8-bit-or-narrower format; returns uint8 codes."""
    eb, mb, _, _ = _SMALL[name]
    vals = _positive_values(name)
    mag = np.abs(x).astype(np.float64)
    hi = np.clip(np.searchsorted(vals, mag, side="left"), 1, len(vals) - 1)
    lo = hi - 1
    dlo, dhi = mag - vals[lo], vals[hi] - mag
    pick_hi = (dhi < dlo) | ((dhi == dlo) & (hi % 2 == 0))
    code = np.where(pick_hi, hi, lo)
    code = np.where(mag >= vals[-1], len(vals) - 1, code)
    sign = (np.signbit(x)).astype(np.int64) << (eb + mb)
    if name == "ue4m3":
        sign = 0
    return (code | sign).astype(np.uint8)


def cast_bf16(x: np.ndarray) -> np.ndarray:
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    r = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return r.astype(np.uint16)


def cast_tf32(x: np.ndarray) -> np.ndarray:
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    r = (u + 0xFFF + ((u >> 13) & 1)) & ~np.uint64(0x1FFF)
    return r.astype(np.uint32)


def cast(x: np.ndarray, fmt: str) -> np.ndarray:
    """Real array -> raw words of ``fmt`` (an element format name)."""
    fmt = elem_format(fmt)
    if fmt == "fp64":
        return np.ascontiguousarray(x, dtype=np.float64).view(np.uint64)
    if fmt == "fp32":
        return np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    if fmt == "tf32":
        return cast_tf32(x)
    if fmt == "bf16":
        return cast_bf16(x)
    if fmt == "fp16":
        with np.errstate(over="ignore"):
            return np.ascontiguousarray(x).astype(np.float16).view(np.uint16)
    return cast_small(x, fmt)


def small_values(codes: np.ndarray, name: str) -> np.ndarray:
    """Value of each code of a small format (used to build block scales)."""
    eb, mb, _, _ = _SMALL[name]
    vals = _positive_values(name)
    mag = vals[np.minimum(codes & ((1 << (eb + mb)) - 1), len(vals) - 1)]
    return np.where((codes >> (eb + mb)) & 1, -mag, mag) if name != "ue4m3" else mag


def pack_fp4(codes: np.ndarray) -> np.ndarray:
    """Two FP4 codes per byte, element 2i in the low nibble."""
    c = codes.astype(np.uint8)
    return (c[..., 0::2] & 0xF) | ((c[..., 1::2] & 0xF) << 4)


# ------------------------------------------------------------------------------------------------------------
# the five configurations
# ------------------------------------------------------------------------------------------------------------
def cfg1():
    """FP16 256x256x256, entries N(0,1), C = +0 (Volta FP16 -> FP32 model)."""
    g = rng(0)
    A = cast(g.standard_normal((256, 256), dtype=np.float32), "fp16")
    B = cast(g.standard_normal((256, 256), dtype=np.float32), "fp16")
    return A, B, np.zeros((256, 256), dtype=np.uint32)


def cfg2(n: int = 2048):
    """BF16 n^3: random signs, exponents uniform over +-20 binades, random mantissas; C ~ N(0,1) FP32."""
    g = rng(2)

    def mat():
        sign = g.integers(0, 2, (n, n), dtype=np.uint16)
        exp = g.integers(-20, 21, (n, n)).astype(np.int32) + 127
        man = g.integers(0, 128, (n, n), dtype=np.uint16)
        return ((sign << 15) | (exp.astype(np.uint16) << 7) | man).astype(np.uint16)

    A, B = mat(), mat()
    C = g.standard_normal((n, n), dtype=np.float32).view(np.uint32)
    return A, B, C


def cfg3(n: int = 4096):
    """E4M3 n^3: X, Y ~ N(0,1) scaled per row to the E4M3 range (max 448) with FP32 scales; C = +0."""
    g = rng(3)

    def mat():
        X = g.standard_normal((n, n), dtype=np.float32)
        s = (np.abs(X).max(axis=1) / np.float32(448.0)).astype(np.float32)
        return cast_small(X / s[:, None], "e4m3"), s

    A, sa = mat()
    B, sb = mat()
    return A, B, np.zeros((n, n), dtype=np.uint32), sa, sb


def _to_words(x, fmt):
    return cast(x, fmt)


def cfg4(fmt: str, K: int, n: int = 1 << 20):
    """Probe-style batch: n dot products of length K, eight input classes interleaved by index mod 8."""
    g = rng(4, stream={"fp16": 1, "bf16": 2, "tf32": 3}[fmt] * 64 + K)
    ebits, mbits = {"fp16": (5, 10), "bf16": (8, 7), "tf32": (8, 10)}[fmt]
    low = 13 if fmt == "tf32" else 0
    wbits = 1 + ebits + mbits
    dt = word_dtype(fmt)
    xa = g.standard_normal((n, K), dtype=np.float32)
    xb = g.standard_normal((n, K), dtype=np.float32)
    xc = g.standard_normal(n, dtype=np.float32)
    cls = np.arange(n) % 8
    # class 1: N(0,1) + Bernoulli(0.001) * N(0,100)
    m1 = cls == 1
    out = (g.random((n, K)) < 0.001) & m1[:, None]
    xa = np.where(out, xa + 10.0 * g.standard_normal((n, K), dtype=np.float32), xa)
    # class 3: exact cancellation (x, -x) pairs, shuffled along K
    m3 = cls == 3
    half = K // 2
    xa3 = np.concatenate([xa[:, :half], xa[:, :half]], axis=1)
    xb3 = np.concatenate([xb[:, :half], -xb[:, :half]], axis=1)
    perm = np.argsort(g.random((n, K)), axis=1)
    xa3, xb3 = np.take_along_axis(xa3, perm, 1), np.take_along_axis(xb3, perm, 1)
    xa = np.where(m3[:, None], xa3, xa)
    xb = np.where(m3[:, None], xb3, xb)
    A, B = _to_words(xa, fmt).astype(np.uint64), _to_words(xb, fmt).astype(np.uint64)
    C = xc.view(np.uint32).astype(np.uint64)
    emask = np.uint64(((1 << ebits) - 1) << (mbits + low))
    # class 2: subnormal-heavy (exponent field cleared with probability 1/2)
    m2 = (cls == 2)[:, None]
    A = np.where(m2 & (g.random((n, K)) < 0.5), A & ~emask, A)
    B = np.where(m2 & (g.random((n, K)) < 0.5), B & ~emask, B)
    C = np.where((cls == 2) & (g.random(n) < 0.5), C & ~np.uint64(0x7F800000), C)
    # class 4: one element with the largest finite exponent
    m4 = np.flatnonzero(cls == 4)
    slot = g.integers(0, K, m4.size)
    big = np.uint64(((1 << ebits) - 2) << (mbits + low))
    A[m4, slot] = (A[m4, slot] & ~emask) | big
    # class 5: ill-conditioned: second half repeats the first with one mantissa bit flipped and the sign of b flipped
    m5 = (cls == 5)[:, None]
    A5 = np.concatenate([A[:, :half], A[:, :half] ^ np.uint64(1 << low)], axis=1)
    B5 = np.concatenate([B[:, :half], B[:, :half] ^ np.uint64(1 << (wbits - 1 + low))], axis=1)
    A, B = np.where(m5, A5, A), np.where(m5, B5, B)
    C = np.where(cls == 5, C & ~np.uint64(0x7F800000) | np.uint64(100 << 23), C)      # small accumulator ~2^-27
    # class 6: infinities and NaNs injected at random slots
    m6 = np.flatnonzero(cls == 6)
    slot = g.integers(0, K, m6.size)
    kind = g.integers(0, 4, m6.size)
    inf = np.uint64(((1 << ebits) - 1) << (mbits + low))
    special = np.where(kind == 0, inf, np.where(kind == 1, inf | np.uint64(1 << (wbits - 1 + low)),
                                                np.where(kind == 2, inf | np.uint64(1 << (mbits - 1 + low)), A[m6, slot])))
    A[m6, slot] = special
    slot_b = g.integers(0, K, m6.size)
    put_b = g.random(m6.size) < 0.3
    B[m6[put_b], slot_b[put_b]] = inf
    c_inf = g.random(m6.size) < 0.2
    C[m6[c_inf]] = np.where(g.random(int(c_inf.sum())) < 0.5, np.uint64(0x7F800000), np.uint64(0xFF800000))
    # class 7: uniformly random bit stream
    m7 = (cls == 7)
    rb = g.integers(0, 1 << 32, (n, K), dtype=np.uint64)
    if fmt != "tf32":
        rb &= np.uint64(0xFFFF)
    A = np.where(m7[:, None], rb, A)
    rb = g.integers(0, 1 << 32, (n, K), dtype=np.uint64)
    if fmt != "tf32":
        rb &= np.uint64(0xFFFF)
    B = np.where(m7[:, None], rb, B)
    C = np.where(m7, g.integers(0, 1 << 32, n, dtype=np.uint64), C)
    return np.ascontiguousarray(A.astype(dt)), np.ascontiguousarray(B.astype(dt)), np.ascontiguousarray(C.astype(np.uint32))


def normal_inputs(in_fmt: str, acc: str, M: int, N: int, K: int, seed: int = 5):
    """A, B ~ N(0,1) cast to the model's input type, C ~ N(0,1) in the accumulator type (config 5 / headline).

    Returns a dict with A, B, C and, for the scaled types, sfa / sfb (one scale byte per k_block elements:
    E8M0 from the block's largest magnitude for the MX types, UE4M3 = amax / 6 for NVFP4).
    FP4 operands of the group-scaled types come packed two per byte.
    """
    g = rng(seed)
    elem = elem_format(in_fmt)
    XA = g.standard_normal((M, K), dtype=np.float32)
    XB = g.standard_normal((N, K), dtype=np.float32)
    XC = g.standard_normal((M, N), dtype=np.float32)
    out = {}
    if acc == "fp64":
        out["C"] = XC.astype(np.float64).view(np.uint64)
    elif acc == "fp16":
        out["C"] = XC.astype(np.float16).view(np.uint16)
    else:
        out["C"] = XC.view(np.uint32)
    if in_fmt in ELEM_OF and in_fmt != "bf16_1k":
        kb = 16 if in_fmt == "nvf4" else 32
        emax_elem = {"e4m3": 8, "e5m2": 15, "e3m2": 4, "e2m3": 2, "e2m1": 2}[elem]

        def scaled(X):
            rows = X.shape[0]
            blocks = X.reshape(rows, K // kb, kb)
            amax = np.maximum(np.abs(blocks).max(axis=2), np.float32(2.0 ** -100))
            if in_fmt == "nvf4":
                sf = cast_small(amax / 6.0, "ue4m3")
                sval = np.maximum(small_values(sf.astype(np.int64), "ue4m3"), 2.0 ** -9)
            else:
                e = np.floor(np.log2(amax)).astype(np.int64) - emax_elem
                sf = np.clip(e + 127, 0, 254).astype(np.uint8)
                sval = 2.0 ** (sf.astype(np.float64) - 127)
            q = cast_small((blocks / sval[:, :, None]).reshape(rows, K), elem)
            return q, sf

        out["A"], out["sfa"] = scaled(XA)
        out["B"], out["sfb"] = scaled(XB)
        if in_fmt in ("mxf4", "nvf4"):
            out["A"], out["B"] = pack_fp4(out["A"]), pack_fp4(out["B"])
    else:
        out["A"], out["B"] = cast(XA, elem), cast(XB, elem)
    return out


def sample_pairs(M: int, N: int, count: int, seed: int):
    """``count`` seeded output positions (i, j) of an M x N result."""
    g = rng(seed, stream=7)
    return np.stack([g.integers(0, M, count), g.integers(0, N, count)], axis=1)


def hw_tiles8(fmt: str, K: int, M: int, nb: int = 16, seed: int = 19, b_fmt: str | None = None):
    """Inputs for a hardware MMA on 8-bit-container types (FP8, FP6, FP4): A (M x K), B (nb x K) codes, C (M x nb) FP32.

    Row classes of A by index mod 4: N(0,1) values cast to the format; uniformly random codes (NaN and infinity codes
    included where the format has them); random codes with about half of the elements +-0; cancelling pairs (x, -x) of
    random finite codes, shuffled along K.  The rows of B take the classes in turn; C mixes N(0,1), zeros, values far
    above and far below the products, and random FP32 bit patterns.
    """
    g = rng(seed, stream=K + 1000 * sum(fmt.encode()))
    b_fmt = b_fmt or fmt

    def mat(rows, f):
        ebits, mbits, _, special = _SMALL[f]
        width = 1 + ebits + mbits
        sign = 1 << (width - 1)
        x = cast_small(g.standard_normal((rows, K)).astype(np.float32) * np.float32(2.0), f)
        codes = g.integers(0, 1 << width, (rows, K)).astype(np.uint8)
        cls = (np.arange(rows) % 4)[:, None]
        x = np.where(cls == 1, codes, x)
        zeros = (g.random((rows, K)) < 0.5)
        x = np.where((cls == 2) & zeros, codes & sign, np.where(cls == 2, codes, x))
        half = K // 2
        fin = codes.copy()
        if special == "ieee":
            top = ((1 << ebits) - 1) << mbits
            fin = np.where((fin & top) == top, fin & ~np.uint8(1 << mbits), fin)          # exponent field below the top one
        elif special == "fn":
            fin = np.where((fin & (sign - 1)) == sign - 1, fin & ~np.uint8(1), fin)      # not the NaN code
        pair = np.concatenate([fin[:, :half], fin[:, :half] ^ np.uint8(sign)], axis=1)
        perm = np.argsort(g.random((rows, K)), axis=1)
        other = np.take_along_axis(np.concatenate([fin[:, half:], fin[:, half:]], axis=1), perm, 1)
        pair = np.take_along_axis(pair, perm, 1)
        x = np.where(cls == 3, pair, x)
        return np.ascontiguousarray(x.astype(np.uint8)), np.ascontiguousarray(other.astype(np.uint8))

    A, _ = mat(M, fmt)
    B, B_other = mat(nb, b_fmt)
    # class 3 of B: the partner of A's pairs is the same column value twice, so that a_k b_k + a_k' b_k' cancels exactly
    B[np.arange(nb) % 4 == 3] = B_other[np.arange(nb) % 4 == 3]
    c = g.standard_normal((M, nb)).astype(np.float32)
    kind = g.integers(0, 8, (M, nb))
    c = np.where(kind == 1, np.float32(0), c)
    c = np.where(kind == 2, c * np.float32(2.0 ** 40), c)
    c = np.where(kind == 3, c * np.float32(2.0 ** -40), c)
    C = c.view(np.uint32).copy()
    bits = g.integers(0, 1 << 32, (M, nb), dtype=np.uint64).astype(np.uint32)
    C = np.where(kind == 4, bits, C)
    return A, B, np.ascontiguousarray(C)


def hw_tiles(fmt: str, acc: str, K: int, M: int, seed: int = 9, nb: int = 8):
    """Inputs for one hardware MMA shape: A (M x K), B (nb x K), C (M x nb) raw words.

    FP16 / BF16 / TF32: the eight input classes of config 4 (row class = row index mod 8; the eight rows of B take
    one class each), plus zero-heavy rows (every 16th row of A has about a third of its elements replaced by +-0).
    FP64: N(0,1) values, every fourth row scaled over +-40 binades.
    """
    g = rng(seed, stream=K)
    if fmt == "fp64":
        def mat(shape):
            x = g.standard_normal(shape)
            wide = (np.arange(shape[0]) % 4 == 3)[:, None]
            x = np.where(wide, x * np.exp2(g.integers(-40, 40, shape)), x)
            return np.ascontiguousarray(x.view(np.uint64))
        return mat((M, K)), mat((nb, K)), mat((M, nb))
    A, _, C1 = cfg4(fmt, K, n=M)
    _, B, _ = cfg4(fmt, K, n=nb)
    zero_rows = np.flatnonzero(np.arange(M) % 16 == 9)
    z = g.random((zero_rows.size, K)) < 0.33
    sign = A.dtype.type(1 << (A.dtype.itemsize * 8 - 1))
    A[zero_rows] = np.where(z, A[zero_rows] & sign, A[zero_rows])
    _, _, C2 = cfg4(fmt, K, n=M * nb)
    C = C2.reshape(M, nb).copy()
    C[np.arange(M) % 16 == 1] = 0                      # a few all-zero accumulator rows
    if acc == "fp16":
        C = (C >> 16).astype(np.uint16)                # the top half of an FP32 word: an arbitrary FP16 word
    return A, B, np.ascontiguousarray(C)
