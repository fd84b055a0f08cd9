"""Pins of the CPU oracle against what the paper prints and what mathematics fixes.

None of these tests touches the CUDA library.  Each pin is chosen so that a
plausible slip in the oracle (wrong sign, dropped term, off-by-one in F, wrong
rounding mode, transposed operand) fails at least one of them.
"""
import ctypes
import ctypes.util
import math
import random
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from oracle import FORMATS, decode, lookup, phi_dot, REGISTRY
from oracle import ops
from oracle.rounding import round_dyadic, rho

from helpers import (exact_word, f32_word, word_f32, f16_word, word_f16, f64_word, word_f64,
                     word_value, read_table)

FP32, FP16 = FORMATS["fp32"], FORMATS["fp16"]


# --------------------------------------------------------------------------
# P1: the paper's Table 8 (worked example of Equation 10)
# --------------------------------------------------------------------------
@pytest.mark.parametrize("arch,in_fmt,acc,expected", read_table("table8_d00.txt"))
@pytest.mark.parametrize("K", [32, 64])
def test_table8(arch, in_fmt, acc, expected, K):
    m = lookup(arch, in_fmt, acc)
    a = [exact_word(m.elem, x) for x in (-2.0 ** 13, -0.5, -0.25, -0.125)] + [0] * (K - 4)
    b = [exact_word(m.elem, x) for x in (2.0 ** 10, 1.0, 1.0, 1.0)] + [0] * (K - 4)
    d = phi_dot(m, a, b, exact_word(acc, 2.0 ** 23))
    assert word_value(acc, d) == float(expected)
    if float(expected) == 0.0:
        assert d == 0          # +0.0


# --------------------------------------------------------------------------
# P2: the d^(i,j)/v tables of Figure 2
# --------------------------------------------------------------------------
def _fig2_expected():
    exp = {}
    for row in read_table("fig2_trees.txt"):
        tree, i, vals = row[0], int(row[1]), [int(x) for x in row[2:]]
        for off, v in enumerate(vals):
            exp[(tree, i, i + 1 + off)] = v
    return exp


FIG2_MODELS = [("a", "cdna1", "fp32", "fp32", 2.0 ** 24, 2.0 ** -4),
               ("a", "ampere", "fp64", "fp64", 2.0 ** 54, 2.0 ** -4),
               ("a", "cdna3", "fp32", "fp32", 2.0 ** 24, 2.0 ** -4),
               ("b", "cdna2", "bf16_1k", "fp32", 2.0 ** 24, 2.0 ** -4),
               ("b", "cdna2", "fp16", "fp32", 2.0 ** 24, 2.0 ** -4),
               ("c", "cdna1", "bf16", "fp32", 2.0 ** 24, 2.0 ** -4),
               ("d", "volta", "fp16", "fp32", 2.0 ** 24, 2.0 ** -4),
               ("d", "cdna3", "bf16", "fp32", 2.0 ** 24, 2.0 ** -4),
               ("d", "ampere", "tf32", "fp32", 2.0 ** 24, 2.0 ** -4)]


@pytest.mark.parametrize("tree,arch,in_fmt,acc,U,v", FIG2_MODELS)
def test_fig2_summation_trees(tree, arch, in_fmt, acc, U, v):
    m = lookup(arch, in_fmt, acc)
    expected = _fig2_expected()
    K = 4
    for i in range(K + 1):
        for j in range(i + 1, K + 1):
            p = [v] * (K + 1)
            p[i], p[j] = U, -U
            # product k = a_k * b_k with a_k = sqrt-ish split so that both factors are representable
            a, b = [], []
            for k in range(K):
                mag = abs(p[k])
                ea = int(math.log2(mag)) // 2
                a.append(exact_word(m.elem, math.copysign(2.0 ** ea, p[k])))
                b.append(exact_word(m.elem, 2.0 ** (int(math.log2(mag)) - ea)))
            d = phi_dot(m, a, b, exact_word(acc, p[K]))
            assert word_value(acc, d) / v == expected[(tree, i, j)], (i, j)


# --------------------------------------------------------------------------
# decode pins: numpy / torch conversions and the OCP value tables
# --------------------------------------------------------------------------
def _decoded_value(fmt, w):
    d = decode(fmt, w)
    if d.cls == oracle.NAN:
        return math.nan
    if d.cls == oracle.INF:
        return -math.inf if d.sign else math.inf
    return math.copysign(d.sig * 2.0 ** (d.exp - fmt.mbits), -1.0 if d.sign else 1.0)


def _same(x, y):
    return (math.isnan(x) and math.isnan(y)) or (x == y and math.copysign(1, x) == math.copysign(1, y))


def test_decode_fp16_bf16_all_codes():
    codes = np.arange(65536, dtype=np.uint16)
    v16 = codes.view(np.float16).astype(np.float64)
    with np.errstate(invalid="ignore"):
        vbf = (codes.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    for w in range(65536):
        assert _same(_decoded_value(FP16, w), float(v16[w]))
        assert _same(_decoded_value(FORMATS["bf16"], w), float(vbf[w]))


def test_decode_fp8_against_torch():
    codes = torch.arange(256, dtype=torch.int32).to(torch.uint8)
    for name, tdt in (("e4m3", torch.float8_e4m3fn), ("e5m2", torch.float8_e5m2)):
        vals = codes.view(tdt).to(torch.float64).tolist()
        for w in range(256):
            assert _same(_decoded_value(FORMATS[name], w), vals[w]), (name, w)


def test_decode_small_formats_value_tables():
    # positive values of the OCP Microscaling element formats, in code order
    e2m1 = [0, 0.5, 1, 1.5, 2, 3, 4, 6]
    e2m3 = [i * 0.125 for i in range(8)] + [1 + i * 0.125 for i in range(8)] + \
           [2 + i * 0.25 for i in range(8)] + [4 + i * 0.5 for i in range(8)]
    e3m2 = [i * 0.0625 for i in range(4)] + [2.0 ** (e - 3) * (1 + m / 4) for e in range(1, 8) for m in range(4)]
    assert max(e2m3) == 7.5 and max(e3m2) == 28.0
    for name, table, sbit in (("e2m1", e2m1, 3), ("e2m3", e2m3, 5), ("e3m2", e3m2, 5)):
        for code, v in enumerate(table):
            assert _decoded_value(FORMATS[name], code) == v
            assert _decoded_value(FORMATS[name], code | (1 << sbit)) == -v
            assert math.copysign(1, _decoded_value(FORMATS[name], code | (1 << sbit))) == -1


def test_decode_scales_and_tf32():
    e8 = FORMATS["e8m0"]
    assert _decoded_value(e8, 127) == 1.0 and _decoded_value(e8, 0) == 2.0 ** -127
    assert _decoded_value(e8, 254) == 2.0 ** 127 and decode(e8, 255).cls == oracle.NAN
    ue = FORMATS["ue4m3"]
    vals = torch.arange(128, dtype=torch.int32).to(torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).tolist()
    for w in range(128):
        assert _same(_decoded_value(ue, w), vals[w])
        assert _same(_decoded_value(ue, w | 0x80), vals[w])      # sign bit ignored
    tf = FORMATS["tf32"]
    rng = random.Random(1)
    for _ in range(2000):
        w = rng.getrandbits(32)
        assert _same(_decoded_value(tf, w), word_f32(w & ~0x1FFF))


# --------------------------------------------------------------------------
# rounding routine against numpy's correctly rounded conversions
# --------------------------------------------------------------------------
def test_round_dyadic_against_numpy():
    rng = random.Random(2)
    for _ in range(20000):
        m = rng.getrandbits(rng.choice([1, 5, 24, 25, 30, 53])) * rng.choice([1, -1])
        e = rng.randint(-190, 140)
        x = math.ldexp(m, e)                                   # exact in float64
        with np.errstate(over="ignore"):
            want32 = int(np.float32(x).view(np.uint32))
            want16 = int(np.float16(x).view(np.uint16)) if abs(e) < 60 else None
        if m == 0:
            want32 = 0
            want16 = 0 if want16 is not None else None
        assert round_dyadic(m, e, 8, 23, 127, "RNE") == want32
        if want16 is not None:
            assert round_dyadic(m, e, 5, 10, 15, "RNE") == want16
        # round toward zero: nearest, stepped back toward zero if it overshot
        if m != 0 and math.isfinite(word_f32(want32)):
            r = np.float32(word_f32(want32))
            if abs(float(r)) > abs(x):
                r = np.nextafter(r, np.float32(0))
            assert round_dyadic(m, e, 8, 23, 127, "RZ") == int(r.view(np.uint32))


def test_rho_overflow_and_e8m13():
    # overflow gives +-inf under every conversion, the round-to-zero ones included (what the B200 returns)
    assert rho("RZ-FP32", 1, 200) == 0x7F800000 and rho("RZ-FP32", -1, 128) == 0xFF800000
    assert rho("RZ-FP32", (1 << 24) - 1, 104) == 0x7F7FFFFF          # the largest finite number is not an overflow
    assert rho("RNE-FP32", 1, 128) == 0x7F800000 and rho("RNE-FP16", -1, 16) == 0xFC00
    assert rho("RZ-E8M13", 1, 128) == 0x7F800000 and rho("RZ-E8M13", (1 << 24) - 1, 104) == 0x7F7FFC00
    assert rho("RZ-FP32", 0, 0) == 0 and rho("RNE-FP16", 0, 5) == 0
    rng = random.Random(3)
    for _ in range(5000):
        w = rng.getrandbits(32) & 0x7FFFFFFF
        if w >= 0x7F800000:
            continue
        d = decode(FP32, w)
        got = rho("RZ-E8M13", d.sig, d.exp - 23)
        assert got == w & ~0x3FF                 # truncating an FP32 word to E8M13 clears 10 mantissa bits
        assert rho("RZ-FP32", d.sig, d.exp - 23) == w
        assert rho("RNE-FP32", -d.sig, d.exp - 23) == (w | 0x80000000 if d.sig else 0)


# --------------------------------------------------------------------------
# IEEE add / mul / fma against numpy and libm
# --------------------------------------------------------------------------
def _rand_f32_word(rng):
    kind = rng.random()
    if kind < 0.1:
        return rng.choice([0, 0x80000000, 0x7F800000, 0xFF800000, 0x7FC00000, 1, 0x80000001, 0x007FFFFF, 0x00800000])
    if kind < 0.3:
        return (rng.getrandbits(1) << 31) | rng.getrandbits(23)             # subnormal
    if kind < 0.6:
        return (rng.getrandbits(1) << 31) | (rng.randint(100, 150) << 23) | rng.getrandbits(23)
    return rng.getrandbits(32)


def _canon(w):
    return 0x7FC00000 if (w & 0x7FFFFFFF) > 0x7F800000 else w


def test_ieee_add_mul_against_numpy():
    rng = random.Random(4)
    xs = np.array([_rand_f32_word(rng) for _ in range(20000)], dtype=np.uint32)
    ys = np.array([_rand_f32_word(rng) for _ in range(20000)], dtype=np.uint32)
    with np.errstate(all="ignore"):
        add = (xs.view(np.float32) + ys.view(np.float32)).view(np.uint32)
        mul = (xs.view(np.float32) * ys.view(np.float32)).view(np.uint32)
    for x, y, s, p in zip(xs.tolist(), ys.tolist(), add.tolist(), mul.tolist()):
        assert ops.ieee_add_f32(x, y) == _canon(s), (hex(x), hex(y))
        assert ops.ieee_mul_f32(x, y) == _canon(p), (hex(x), hex(y))


def test_fma_against_libm():
    libm = ctypes.CDLL(ctypes.util.find_library("m"))
    libm.fmaf.restype = ctypes.c_float
    libm.fmaf.argtypes = [ctypes.c_float] * 3
    libm.fma.restype = ctypes.c_double
    libm.fma.argtypes = [ctypes.c_double] * 3
    rng = random.Random(5)
    for _ in range(20000):
        a, b, c = (_rand_f32_word(rng) for _ in range(3))
        if rng.random() < 0.3:                      # near-cancellation: c ~ -(a*b)
            with np.errstate(all="ignore"):
                c = int((-(np.uint32(a).view(np.float32) * np.uint32(b).view(np.float32))).view(np.uint32))
        want = f32_word(libm.fmaf(word_f32(a), word_f32(b), word_f32(c)))
        assert ops.fma(a, b, c, FP32) == _canon(want), (hex(a), hex(b), hex(c))
    F64 = FORMATS["fp64"]
    for _ in range(20000):
        a, b, c = (rng.getrandbits(64) for _ in range(3))
        if rng.random() < 0.5:
            a = (a & ~(0x7FF << 52)) | (rng.randint(900, 1100) << 52)
            b = (b & ~(0x7FF << 52)) | (rng.randint(900, 1100) << 52)
            c = (c & ~(0x7FF << 52)) | (rng.randint(850, 1200) << 52)
        want = f64_word(libm.fma(word_f64(a), word_f64(b), word_f64(c)))
        if (want & 0x7FFFFFFFFFFFFFFF) > 0x7FF0000000000000:
            want = 0x7FF8000000000000
        assert ops.fma(a, b, c, F64) == want


def test_phi_fma_is_sequential():
    # P10: Phi_FMA equals a left-to-right chain of correctly rounded a*b+d, evaluated with rationals
    rng = np.random.default_rng(6)
    m = lookup("cdna3", "fp32", "fp32")
    for _ in range(200):
        a = rng.standard_normal(16).astype(np.float32)
        b = rng.standard_normal(16).astype(np.float32)
        c = np.float32(rng.standard_normal())
        d = Fraction(float(c))
        for x, y in zip(a.tolist(), b.tolist()):
            exact = Fraction(x) * Fraction(y) + d
            # correctly rounded binary32 of an exact rational: float() of a Fraction is correctly rounded
            # to binary64 only, so round through integers instead
            d = Fraction(_round_fraction_rne(exact, 24, -149))
        got = phi_dot(m, a.view(np.uint32).tolist(), b.view(np.uint32).tolist(), int(c.view(np.uint32)))
        assert Fraction(word_f32(got)) == d


def _round_fraction_rne(x: Fraction, prec: int, emin_quantum: int) -> Fraction:
    """Nearest-even rounding of a rational to ``prec`` significant bits (quantum >= 2**emin_quantum)."""
    if x == 0:
        return x
    e = math.floor(math.log2(abs(x)))
    while Fraction(2) ** e > abs(x):
        e -= 1
    while Fraction(2) ** (e + 1) <= abs(x):
        e += 1
    q = max(e - prec + 1, emin_quantum)
    scaled = x / Fraction(2) ** q
    n = math.floor(scaled)
    r = scaled - n
    if r > Fraction(1, 2) or (r == Fraction(1, 2) and n % 2):
        n += 1
    return n * Fraction(2) ** q


# --------------------------------------------------------------------------
# P11: Phi_FTZ-AddMul against numpy float32 arithmetic + manual flush
# --------------------------------------------------------------------------
def _np_ftz(z):
    z = np.float32(z)
    return np.float32(math.copysign(0.0, float(z))) if abs(float(z)) < 2.0 ** -126 else z


def _np_flush_in(w, fmt):
    if fmt == "fp16":
        x = np.uint16(w).view(np.float16)
        return np.float32(0.0) if (x != 0 and abs(float(x)) < 2.0 ** -14) else np.float32(x)
    x = np.uint32(w << 16).view(np.float32)
    return np.float32(0.0) if (x != 0 and abs(float(x)) < 2.0 ** -126) else x


@pytest.mark.parametrize("arch_fmt,P", [("bf16", 2), ("bf16_1k", 4), ("fp16", 4)])
def test_ftz_addmul_against_numpy(arch_fmt, P):
    m = lookup("cdna2", arch_fmt, "fp32")
    rng = random.Random(7)
    K = 8
    with np.errstate(all="ignore"):
        for t in range(3000):
            if t % 3 == 0:      # exponents near the FP32 flush boundary (bf16) / subnormal inputs (fp16)
                a = [(rng.getrandbits(1) << 15) | (rng.randint(0, 80) << 7 if m.elem == "bf16" else rng.randint(0, 3) << 10) | rng.getrandbits(7)
                     for _ in range(K)]
                b = [(rng.getrandbits(1) << 15) | (rng.randint(40, 130) << 7 if m.elem == "bf16" else rng.randint(0, 3) << 10) | rng.getrandbits(7)
                     for _ in range(K)]
                c = (rng.getrandbits(1) << 31) | (rng.randint(0, 3) << 23) | rng.getrandbits(23)
            else:
                a = [rng.getrandbits(16) for _ in range(K)]
                b = [rng.getrandbits(16) for _ in range(K)]
                c = _rand_f32_word(rng)
            fa = [_np_flush_in(w, m.elem) for w in a]
            fb = [_np_flush_in(w, m.elem) for w in b]
            cf = np.uint32(c).view(np.float32)
            d = np.float32(0.0) if (cf != 0 and abs(float(cf)) < 2.0 ** -126) else cf
            for k in range(0, K, P):
                p = [_np_ftz(fa[k + l] * fb[k + l]) for l in range(P)]
                s = _np_ftz(p[0] + p[1])
                if P == 4:
                    s = _np_ftz(s + _np_ftz(p[2] + p[3]))
                d = _np_ftz(d + s)
            want = _canon(int(np.float32(d).view(np.uint32)))
            assert phi_dot(m, a, b, c) == want, (a, b, hex(c))


def test_ftz_sign_preserving_flush_and_positive_input_flush():
    # Algorithm 1: a subnormal result becomes a zero of the same sign
    tiny_neg = f32_word(-2.0 ** -127)
    assert ops.ftz_add(tiny_neg, 0) == 0x80000000
    assert ops.ftz_add(f32_word(2.0 ** -126), f32_word(-2.0 ** -127)) == 0      # +2^-127 flushed to +0
    # Algorithm 2: a negative subnormal input becomes +0.0, so (-sub) * (-1) contributes +0, not -0 or 2^-24
    m = lookup("cdna2", "fp16", "fp32")
    d = phi_dot(m, [0x8001, 0, 0, 0], [0xBC00, 0, 0, 0], 0x80000000)
    assert d == 0        # (+0 * -1 = -0) + 0 ... pairwise adds give +0; -0 + +0 = +0


# --------------------------------------------------------------------------
# P3: K = 1, c = +0: d = rho(a*b); brute force over every FP8 pair
# --------------------------------------------------------------------------
@pytest.mark.parametrize("fa,fb", [("e4m3", "e4m3"), ("e5m2", "e5m2"), ("e4m3", "e5m2")])
def test_all_fp8_pairs_single_product(fa, fb):
    tdt = {"e4m3": torch.float8_e4m3fn, "e5m2": torch.float8_e5m2}
    codes = torch.arange(256, dtype=torch.int32).to(torch.uint8)
    va = codes.view(tdt[fa]).to(torch.float32)
    vb = codes.view(tdt[fb]).to(torch.float32)
    prod = (va[:, None] * vb[None, :]).contiguous().view(torch.int32).numpy().view(np.uint32)   # exact in FP32
    for x in range(256):
        for y in range(256):
            got = ops.t_fdpa([x], [y], 0, FORMATS[fa], FORMATS[fb], FP32, 25, "RZ-FP32")
            want = int(prod[x, y])
            if (want & 0x7FFFFFFF) > 0x7F800000:
                want = 0x7FFFFFFF                              # NVIDIA canonical NaN
            elif (want & 0x7FFFFFFF) == 0:
                want = 0                                       # exact zero sums give +0
            assert got == want, (x, y)


@pytest.mark.parametrize("name", ["e3m2", "e2m3", "e2m1"])
def test_all_small_format_pairs(name):
    fmt = FORMATS[name]
    n = 1 << (1 + fmt.ebits + fmt.mbits)
    for x in range(n):
        for y in range(n):
            want = _decoded_value(fmt, x) * _decoded_value(fmt, y)
            got = ops.t_fdpa([x], [y], 0, fmt, fmt, FP32, 25, "RZ-FP32")
            assert word_f32(got) == want and (got == 0 or want != 0)


def test_random_fp16_bf16_tf32_single_product():
    rng = random.Random(8)
    for name in ("fp16", "bf16", "tf32"):
        fmt = FORMATS[name]
        for _ in range(5000):
            x = rng.getrandbits(fmt.storage_bits)
            y = rng.getrandbits(fmt.storage_bits)
            vx, vy = _decoded_value(fmt, x), _decoded_value(fmt, y)
            if not (math.isfinite(vx) and math.isfinite(vy)):
                continue
            p = vx * vy                                        # exact in float64 (<= 22 significant bits)
            if p != 0 and not (2.0 ** -126 <= abs(p) < 2.0 ** 128):
                continue                                       # outside the exactly representable FP32 range
            got = ops.t_fdpa([x], [y], 0, fmt, fmt, FP32, 24, "RZ-FP32")
            assert word_f32(got) == p


# --------------------------------------------------------------------------
# P4: K = 1 with a nearby c: a single correctly rounded multiply-add in the mode of rho
# --------------------------------------------------------------------------
def test_single_fma_in_mode_rho():
    rng = random.Random(9)
    fmt = FORMATS["fp16"]
    for _ in range(5000):
        x = (rng.getrandbits(1) << 15) | (rng.randint(10, 20) << 10) | rng.getrandbits(10)
        y = (rng.getrandbits(1) << 15) | (rng.randint(10, 20) << 10) | rng.getrandbits(10)
        p = word_f16(x) * word_f16(y)                                   # exact in float64
        c = np.float32(p * rng.uniform(-1.5, 1.5))
        exact = p + float(c)                                            # exact in float64 (small gap)
        assert Fraction(exact) == Fraction(p) + Fraction(float(c))
        cw = int(c.view(np.uint32))
        # gap between c and the product is at most a few binades, F >= 23 keeps every bit of both terms
        ec = decode(FP32, cw).exp
        ep = decode(fmt, x).exp + decode(fmt, y).exp
        if abs(ec - ep) > 1:
            continue
        got_rz = ops.t_fdpa([x], [y], cw, fmt, fmt, FP32, 25, "RZ-FP32")
        r = np.float32(exact)
        if abs(float(r)) > abs(exact):
            r = np.nextafter(r, np.float32(0))
        assert got_rz == (int(r.view(np.uint32)) if exact != 0 else 0)
        got_tr = ops.tr_fdpa([x], [y], cw, fmt, fmt, 24, 31)
        want = int(np.float32(exact).view(np.uint32)) if exact != 0 else 0
        assert got_tr == want
        got_e = ops.e_fdpa([x], [y], cw, fmt, fmt)
        assert got_e == want


def test_fp16_accumulator_single_fma():
    rng = random.Random(10)
    fmt = FORMATS["fp16"]
    for _ in range(5000):
        x = (rng.getrandbits(1) << 15) | (rng.randint(12, 18) << 10) | rng.getrandbits(10)
        y = (rng.getrandbits(1) << 15) | (rng.randint(12, 18) << 10) | rng.getrandbits(10)
        c = (rng.getrandbits(1) << 15) | (rng.randint(12, 20) << 10) | rng.getrandbits(10)
        exact = word_f16(x) * word_f16(y) + word_f16(c)                 # exact in float64
        ec = decode(fmt, c).exp
        ep = decode(fmt, x).exp + decode(fmt, y).exp
        if max(ec, ep) - min(ec - 10, ep - 20) > 23:
            continue                                                    # some bit would be truncated at F = 23
        got = ops.t_fdpa([x], [y], c, fmt, fmt, fmt, 23, "RNE-FP16")
        with np.errstate(over="ignore"):
            want = int(np.float16(exact).view(np.uint16)) if exact != 0 else 0
        assert got == want


# --------------------------------------------------------------------------
# P5: unlimited F gives the correctly rounded exact sum; E-FDPA is that with RNE-FP32
# --------------------------------------------------------------------------
def test_unlimited_precision_is_exact_sum():
    rng = np.random.default_rng(11)
    fmt = FORMATS["fp16"]
    for _ in range(2000):
        L = int(rng.choice([2, 4, 8]))
        a = (rng.standard_normal(L) * 2.0 ** rng.integers(-8, 8, L)).astype(np.float16)
        b = (rng.standard_normal(L) * 2.0 ** rng.integers(-8, 8, L)).astype(np.float16)
        c = np.float32(rng.standard_normal() * 2.0 ** rng.integers(-10, 10))
        exact = sum((Fraction(float(x)) * Fraction(float(y)) for x, y in zip(a, b)), Fraction(float(c)))
        aw, bw, cw = a.view(np.uint16).tolist(), b.view(np.uint16).tolist(), int(c.view(np.uint32))
        want = _round_fraction_rne(exact, 24, -149)
        got_e = ops.e_fdpa(aw, bw, cw, fmt, fmt)
        assert Fraction(word_f32(got_e)) == want
        got_inf = ops.t_fdpa(aw, bw, cw, fmt, fmt, FP32, None, "RNE-FP32")
        assert got_inf == got_e
        # math.fsum is a correctly rounded (binary64) sum: when that sum is exact, one more rounding gives FP32
        terms = [float(x) * float(y) for x, y in zip(a, b)] + [float(c)]
        fs = math.fsum(terms)
        if Fraction(fs) == exact and exact != 0:
            assert got_e == int(np.float32(fs).view(np.uint32))


# --------------------------------------------------------------------------
# P6: error bounds of Table 9
# --------------------------------------------------------------------------
@pytest.mark.parametrize("key", [("volta", "fp16", "fp32"), ("ampere", "bf16", "fp32"), ("hopper", "e4m3", "fp32"),
                                 ("blackwell", "e5m2", "fp32"), ("hopper", "fp16", "fp16")])
def test_fused_sum_error_bound(key):
    m = lookup(*key)
    fmt, fc = FORMATS[m.elem], FORMATS[m.acc]
    rng = random.Random(12)
    L = m.L
    for _ in range(1500):
        a = [_rand_finite(rng, fmt) for _ in range(L)]
        b = [_rand_finite(rng, fmt) for _ in range(L)]
        c = _rand_finite(rng, fc)
        da, db, dc = [decode(fmt, w) for w in a], [decode(fmt, w) for w in b], decode(fc, c)
        e_max = max([x.exp + y.exp for x, y in zip(da, db)] + [dc.exp])
        exact = sum((_frac(fmt, x) * _frac(fmt, y) for x, y in zip(a, b)), _frac(fc, c))
        got = ops.t_fdpa(a, b, c, fmt, fmt, fc, m.F, m.rho)
        dg = decode(fc, got)
        if dg.cls != oracle.FINITE or abs(exact) >= Fraction(2) ** (fc.emax + 1):
            continue
        gotv = _frac(fc, got)
        if m.rho == "RZ-E8M13":
            ulp = Fraction(2) ** (max(dg.exp, -126) - 13)
        else:
            ulp = Fraction(2) ** (dg.exp - fc.mbits)
        rounding = ulp / 2 if m.rho.startswith("RNE") else ulp
        # the sum before rounding may sit one binade above the result, hence 2*rounding is never needed:
        assert abs(gotv - exact) <= (L + 1) * Fraction(2) ** (e_max - m.F) + rounding


def _rand_finite(rng, fmt):
    while True:
        w = rng.getrandbits(fmt.storage_bits)
        if fmt.name == "fp32" or fmt.name == "bf16":
            w = (w & ~(0xFF << (fmt.storage_bits - 9))) | (rng.randint(100, 150) << (fmt.storage_bits - 9))
        if decode(fmt, w).cls == oracle.FINITE:
            return w


def _frac(fmt, w):
    d = decode(fmt, w)
    return Fraction((-1) ** d.sign * d.sig) * Fraction(2) ** (d.exp - fmt.mbits)


# --------------------------------------------------------------------------
# P7: symmetry Phi(-A, B, -C) = -Phi(A, B, C); TR-/GTR-FDPA are asymmetric
# --------------------------------------------------------------------------
def _neg(fmt, w):
    return w ^ (1 << (fmt.storage_bits - 1 if fmt.name != "e2m1" and fmt.storage_bits != 8 else fmt.ebits + fmt.mbits))


def _flip(fmt, w):
    return w ^ (1 << (fmt.ebits + fmt.mbits + fmt.low_ignored))


@pytest.mark.parametrize("key", sorted(k for k, m in REGISTRY.items() if m.family not in ("st", "gst")))
def test_symmetry(key):
    m = REGISTRY[key]
    fmt, fc = FORMATS[m.elem], FORMATS[m.acc]
    rng = random.Random(13)
    K = 2 * max(m.L, m.P, 4)
    asym = 0
    for _ in range(150):
        a = [_rand_finite(rng, fmt) for _ in range(K)]
        b = [_rand_finite(rng, fmt) for _ in range(K)]
        c = _rand_finite(rng, fc)
        d1 = phi_dot(m, a, b, c)
        d2 = phi_dot(m, [_flip(fmt, w) for w in a], b, _flip(fc, c))
        z = (1 << (fc.storage_bits - 1)) - 1
        same = (d1 & z) == (d2 & z) and ((d1 ^ d2) >> (fc.storage_bits - 1) == 1 or (d1 & z) == 0)
        if m.family in ("tr", "gtr"):
            asym += not same
        elif m.family == "ftz" and ((d1 & z) == 0):
            pass            # flushed subnormal inputs are +0 for both signs, zero signs may differ
        else:
            assert same, (a, b, c)
    if m.family in ("tr", "gtr"):
        assert asym > 0     # round-down makes the CDNA3 models asymmetric (Section 6.2.4)


def test_tr_fdpa_bias_direction():
    # Section 6.3: large A, B and a small negative C: rounding c down at the products' exponent drags the
    # result toward minus infinity; the hypothetical round-to-zero variant of Section 6.2.4 does not
    fmt = FORMATS["fp16"]
    w = lambda x: exact_word("fp16", x)
    a = [w(1024.0), w(-1024.0)] + [0] * 6
    b = [w(1024.0), w(1024.0)] + [0] * 6               # products +-2^20 cancel; e_max = 20, quantum 2^-4
    c = exact_word("fp32", -(2.0 ** -10))
    assert word_f32(ops.tr_fdpa(a, b, c, fmt, fmt, 24, 31)) == -(2.0 ** -4)
    assert ops.tr_fdpa(a, b, c, fmt, fmt, 24, 31, inner_round="RZ") == 0
    assert ops.tr_fdpa(a, b, c ^ 0x80000000, fmt, fmt, 24, 31) == 0


# --------------------------------------------------------------------------
# P8: the paper's own probes recover L, F and the rounding mode from the black box
# --------------------------------------------------------------------------
def _probe_F(m):
    """FusedSum(U, -U, eps): halve eps until the output differs from eps (Section 3.1, Step 3)."""
    e_u = 8
    U = 2.0 ** e_u
    K = m.L
    eps_e = e_u
    while True:
        eps = 2.0 ** eps_e
        a = [exact_word(m.elem, 2.0 ** 4), exact_word(m.elem, -(2.0 ** 4)), exact_word(m.elem, 2.0 ** (eps_e // 2))] + [0] * (K - 3)
        b = [exact_word(m.elem, 2.0 ** 4), exact_word(m.elem, 2.0 ** 4), exact_word(m.elem, 2.0 ** (eps_e - eps_e // 2))] + [0] * (K - 3)
        d = phi_dot(m, a, b, 0)
        if word_value(m.acc, d) != eps:
            return e_u - eps_e - 1
        eps_e -= 1
        assert eps_e > -40


@pytest.mark.parametrize("key", [("volta", "fp16", "fp32"), ("turing", "fp16", "fp32"), ("hopper", "fp16", "fp32"),
                                 ("ampere", "bf16", "fp32"), ("hopper", "bf16", "fp32")])
def test_probe_recovers_F(key):
    m = lookup(*key)
    assert _probe_F(m) == m.F


def test_probe_recovers_output_rounding():
    # U + 1.5 eps, U + 0.5 eps, -U - 1.5 eps, -U - 0.5 eps (Section 3.1, Step 3) with U held in c and
    # 2 eps = one output ulp at U (FP32 ulp(2^23) = 1, eps = 0.5)
    w = lambda x: exact_word("fp16", x)
    U = 2.0 ** 23 + 1
    for key, want in ((("hopper", "fp16", "fp32"), [U, U, -U, -U]),                 # RZ
                      (("cdna3", "fp16", "fp32"), [U + 1, U, -U - 1, -U])):         # RN
        m = lookup(*key)
        outs = []
        for s in (1, -1):
            for mult in (1.5, 0.5):
                a = [w(s * mult)] + [0] * (m.L - 1)
                b = [w(0.5)] + [0] * (m.L - 1)
                outs.append(word_f32(phi_dot(m, a, b, f32_word(s * U))))
        assert outs == want
    # ties: U + eps with U even / odd in the last place -> ties-to-even for the RNE model
    m = lookup("cdna3", "fp16", "fp32")
    outs = []
    for Uc in (2.0 ** 23, 2.0 ** 23 + 1, -(2.0 ** 23), -(2.0 ** 23 + 1)):
        a = [w(math.copysign(1.0, Uc))] + [0] * (m.L - 1)
        b = [w(0.5)] + [0] * (m.L - 1)
        outs.append(word_f32(phi_dot(m, a, b, f32_word(Uc))))
    assert outs == [2.0 ** 23, 2.0 ** 23 + 2, -(2.0 ** 23), -(2.0 ** 23 + 2)]


def test_probe_recovers_L():
    # Step 2 probe: p_0 = U, p_j = -U, others v: the v's of the block holding both U and -U are swamped
    for key in (("volta", "fp16", "fp32"), ("turing", "fp16", "fp32"), ("hopper", "fp16", "fp32")):
        m = lookup(*key)
        K = 4 * m.L
        U, v = 2.0 ** 24, 2.0 ** -4
        a = [exact_word("fp16", 2.0 ** 12)] + [exact_word("fp16", 2.0 ** -2)] * (K - 1)
        b = [exact_word("fp16", 2.0 ** 12)] + [exact_word("fp16", 2.0 ** -2)] * (K - 1)
        counts = []
        for j in range(1, K):
            aj = list(a)
            aj[j] = exact_word("fp16", -(2.0 ** 12))
            bj = list(b)
            bj[j] = exact_word("fp16", 2.0 ** 12)
            counts.append(word_f32(phi_dot(m, aj, bj, exact_word("fp32", v))) / v)
        # -U in the first block: everything in that block is swamped, the K - L later products survive
        assert counts[: m.L - 1] == [K - m.L] * (m.L - 1)
        assert counts[m.L - 1] < K - m.L


# --------------------------------------------------------------------------
# P12: special values (Section 4.2)
# --------------------------------------------------------------------------
def test_special_values():
    inf16, ninf16, nan16, one, zero = 0x7C00, 0xFC00, 0x7E00, 0x3C00, 0
    for key in (("hopper", "fp16", "fp32"), ("cdna3", "fp16", "fp32"), ("cdna1", "fp16", "fp32")):
        m = lookup(*key)
        nan_word = 0x7FFFFFFF if m.family == "t" else 0x7FC00000
        pad = [0] * (m.L - 2)
        assert phi_dot(m, [nan16, one] + pad, [one, one] + pad, 0) == nan_word
        assert phi_dot(m, [inf16, one] + pad, [zero, one] + pad, 0) == nan_word           # inf * 0
        assert phi_dot(m, [inf16, ninf16] + pad, [one, one] + pad, 0) == nan_word         # inf - inf
        assert phi_dot(m, [inf16, one] + pad, [one, one] + pad, 0xFF800000) == nan_word   # inf + (-inf in c)
        assert phi_dot(m, [inf16, one] + pad, [0xBC00, one] + pad, 0) == 0xFF800000       # inf * -1
        assert phi_dot(m, [ninf16, ninf16] + pad, [ninf16, one] + pad, 0) == nan_word     # +inf + -inf
        assert phi_dot(m, [one, one] + pad, [one, one] + pad, 0x7F800000) == 0x7F800000
        assert phi_dot(m, [one, one] + pad, [one, one] + pad, 0x7FC00001) == nan_word
    m = lookup("hopper", "fp16", "fp16")
    pad = [0] * (m.L - 1)
    assert phi_dot(m, [nan16] + pad, [one] + pad, 0) == 0x7FFF
    assert phi_dot(m, [0x7BFF] + pad, [0x7BFF] + pad, 0) == 0x7C00                        # RNE-FP16 overflow
    m = lookup("blackwell", "e4m3", "fp32")
    pad = [0] * 31
    assert phi_dot(m, [0x7F] + pad, [0x38] + pad, 0) == 0x7FFFFFFF                        # E4M3 NaN
    assert word_f32(phi_dot(m, [0x7E] + pad, [0x7E] + pad, 0)) == 448.0 * 448.0           # no infinity in E4M3
    # TR-FDPA: a product of magnitude >= 2^128 overflows to infinity before the sum
    m = lookup("cdna3", "bf16", "fp32")
    big = exact_word("bf16", 2.0 ** 100)
    pad = [0] * 7
    assert phi_dot(m, [big] + pad, [big] + pad, 0) == 0x7F800000
    assert phi_dot(m, [big, big] + pad[1:], [big, big ^ 0x8000] + pad[1:], 0) == 0x7FC00000
    # the NVIDIA model of the same input overflows in rho: +inf as well (not the largest finite number)
    m = lookup("hopper", "bf16", "fp32")
    pad = [0] * 15
    assert phi_dot(m, [big] + pad, [big] + pad, 0) == 0x7F800000
    assert phi_dot(m, [big] + pad, [big ^ 0x8000] + pad, 0) == 0xFF800000


# --------------------------------------------------------------------------
# P13: subnormal inputs: flushed by the CDNA2 model, exact under the NVIDIA models
# --------------------------------------------------------------------------
def test_flush_vs_no_flush():
    sub = 0x0200                                           # FP16 subnormal 2^-15
    one = 0x3C00
    K = 16
    a, b = [sub] + [0] * (K - 1), [one] + [0] * (K - 1)
    assert phi_dot(lookup("cdna2", "fp16", "fp32"), a, b, 0) == 0
    for arch in ("volta", "ampere", "hopper", "blackwell", "cdna1", "cdna3"):
        assert word_f32(phi_dot(lookup(arch, "fp16", "fp32"), a, b, 0)) == 2.0 ** -15
    # FP32 subnormal output: kept by every model except CDNA2
    a = [exact_word("bf16", 2.0 ** -126)] + [0] * (K - 1)
    b = [exact_word("bf16", 2.0 ** -10)] + [0] * (K - 1)
    assert phi_dot(lookup("cdna2", "bf16", "fp32"), a, b, 0) == 0
    for arch in ("ampere", "hopper", "cdna1", "cdna3"):
        assert word_f32(phi_dot(lookup(arch, "bf16", "fp32"), a, b, 0)) == 2.0 ** -136


# --------------------------------------------------------------------------
# P14: Hopper FP8 keeps only 13 fractional bits of the accumulator in every block
# --------------------------------------------------------------------------
def test_hopper_fp8_truncates_accumulator():
    m = lookup("hopper", "e4m3", "fp32")
    rng = random.Random(14)
    for _ in range(500):
        c = (rng.getrandbits(1) << 31) | (rng.randint(122, 140) << 23) | rng.getrandbits(23)
        d = phi_dot(m, [0] * 32, [0] * 32, c)
        assert d == c & ~0x3FF


# --------------------------------------------------------------------------
# Zero terms have no exponent: they do not raise e_max (closed forms)
# --------------------------------------------------------------------------
def test_zero_terms_take_no_part_in_e_max():
    m = lookup("hopper", "fp16", "fp32")
    h = lambda x: exact_word("fp16", x)
    # 0 * 2^15 next to a product of 1.5 * 2^-28: with the zero product counted at Exp(0) + Exp(2^15) = 1 the grid would
    # be 2^(1 - 25) and the small product would be truncated away; it must survive exactly
    a = [h(0.0), h(2.0 ** -14)] + [0] * 14
    b = [h(2.0 ** 15), h(1.5 * 2.0 ** -14)] + [0] * 14
    assert word_f32(phi_dot(m, a, b, 0)) == 1.5 * 2.0 ** -28
    # the same with a zero accumulator of either sign, and with a tiny accumulator that must not be flushed
    assert word_f32(phi_dot(m, a, b, 0x80000000)) == 1.5 * 2.0 ** -28
    assert word_f32(phi_dot(m, a, b, f32_word(2.0 ** -40))) == 1.5 * 2.0 ** -28 + 2.0 ** -40
    # A = 0: D = C bit for bit for every finite C whenever F holds the accumulator's 24 bits
    rng = random.Random(22)
    for key in (("volta", "fp16", "fp32"), ("hopper", "bf16", "fp32"), ("blackwell", "e4m3", "fp32"), ("cdna3", "fp16", "fp32"),
                ("cdna3", "e4m3", "fp32"), ("blackwell", "mxe5m2", "fp32")):
        mm = lookup(*key)
        fmt = FORMATS[mm.elem]
        for _ in range(50):
            c = rng.getrandbits(32)
            if (c & 0x7F800000) == 0x7F800000:
                continue
            bvals = [_rand_finite(rng, fmt) for _ in range(mm.L)]
            kw = {}
            if mm.family == "st":
                kw = {"sfa": [rng.randrange(255)], "sfb": [rng.randrange(255)]}
            d = phi_dot(mm, [0] * mm.L, bvals, c, **kw)
            assert d == (c if c & 0x7FFFFFFF else 0), (key, hex(c), hex(d))
    # an all-zero block gives +0
    assert phi_dot(m, [0x8000] * 16, [h(3.0)] * 16, 0x80000000) == 0


# --------------------------------------------------------------------------
# P15: zero padding is neutral; L = min(K, L_max)
# --------------------------------------------------------------------------
@pytest.mark.parametrize("key", [("volta", "fp16", "fp32"), ("hopper", "fp16", "fp32"), ("hopper", "e5m2", "fp32"),
                                 ("cdna3", "fp16", "fp32"), ("cdna1", "fp16", "fp32")])
def test_zero_padding_neutral(key):
    m = lookup(*key)
    fmt = FORMATS[m.elem]
    rng = random.Random(15)
    for _ in range(300):
        K = rng.choice([1, 2, 3]) if m.L > 3 else 1
        a = [_rand_finite(rng, fmt) for _ in range(K)]
        b = [_rand_finite(rng, fmt) for _ in range(K)]
        c = f32_word(rng.gauss(0, 1))
        if m.family == "e" and K % m.L:
            continue
        short = phi_dot(m, a, b, c)                       # L = min(K, L_max) = K
        padded = phi_dot(m, a + [0] * (m.L - K), b + [0] * (m.L - K), c)
        assert short == padded


# --------------------------------------------------------------------------
# ST / GST: scale handling against exact float64 evaluation (no truncation active)
# --------------------------------------------------------------------------
def test_st_fdpa_scales_shift_exponents():
    m = lookup("blackwell", "mxe4m3", "fp32")
    rng = random.Random(16)
    codes = torch.arange(256, dtype=torch.int32).to(torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).tolist()
    checked = 0
    for _ in range(500):
        a = [rng.choice([0x30, 0x38, 0x3C, 0x40, 0xB8, 0xC0, 0x34]) for _ in range(32)]
        b = [rng.choice([0x30, 0x38, 0x3C, 0x40, 0xB8, 0xC0, 0x34]) for _ in range(32)]
        sa, sb = rng.randint(110, 140), rng.randint(110, 140)
        exact = sum(codes[x] * codes[y] for x, y in zip(a, b)) * 2.0 ** (sa - 127) * 2.0 ** (sb - 127)
        c = np.float32(exact * rng.uniform(-1, 1))
        total = exact + float(c)
        got = phi_dot(m, a, b, int(c.view(np.uint32)), [sa], [sb])
        # all terms within a few binades of each other: nothing is truncated at F = 25 except below 2^(emax-25)
        r = np.float32(total)
        if abs(float(r)) > abs(total):
            r = np.nextafter(r, np.float32(0))
        # guard: the lowest bit of every term must sit at or above 2^(e_max - 25)
        f8 = FORMATS["e4m3"]
        e_k = [decode(f8, x).exp + decode(f8, y).exp + sa + sb - 254 for x, y in zip(a, b)]
        e_c = decode(FP32, int(c.view(np.uint32))).exp
        e_max = max(e_k + [e_c])
        if min(e_k) - 6 < e_max - 25 or e_c - 23 < e_max - 25:
            continue
        checked += 1
        assert got == (int(r.view(np.uint32)) if total != 0 else 0)
    assert checked > 100
    assert phi_dot(m, [0x38] * 32, [0x38] * 32, 0, [255], [127]) == 0x7FFFFFFF


@pytest.mark.parametrize("in_fmt,scale_codes", [("mxf4", [125, 126, 127, 128, 129]),
                                                ("nvf4", [0x30, 0x38, 0x3B, 0x41, 0x2C, 0x05])])
def test_gst_fdpa_against_float64(in_fmt, scale_codes):
    m = lookup("blackwell", in_fmt, "fp32")
    e2m1 = [0, 0.5, 1, 1.5, 2, 3, 4, 6]
    if in_fmt == "mxf4":
        sval = {c: 2.0 ** (c - 127) for c in scale_codes}
    else:
        tbl = torch.arange(128, dtype=torch.int32).to(torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).tolist()
        sval = {c: tbl[c] for c in scale_codes}
    rng = random.Random(17)
    nsf = 64 // m.k_block
    for _ in range(500):
        a = [rng.getrandbits(4) for _ in range(64)]
        b = [rng.getrandbits(4) for _ in range(64)]
        sfa = [rng.choice(scale_codes) for _ in range(nsf)]
        sfb = [rng.choice(scale_codes) for _ in range(nsf)]
        val = lambda w: (-1) ** (w >> 3) * e2m1[w & 7]
        total = 0.0
        for k in range(64):
            total += val(a[k]) * val(b[k]) * sval[sfa[k // m.k_block]] * sval[sfb[k // m.k_block]]   # exact in float64
        c = np.float32(rng.gauss(0, 4))
        total += float(c)
        got = phi_dot(m, a, b, int(c.view(np.uint32)), sfa, sfb)
        r = np.float32(total)
        if abs(float(r)) > abs(total):
            r = np.nextafter(r, np.float32(0))
        # F = 35 keeps every bit here: scale exponents span < 8 binades, c is FP32 with 23 fractional bits
        assert got == (int(r.view(np.uint32)) if total != 0 else 0)


def test_gst_group_truncation_at_F35():
    # two groups 2^40 apart: the small one is cut at 2^(e_max - 35)
    m = lookup("blackwell", "mxf4", "fp32")
    a = [0x2] + [0] * 63           # 1.0 in group 0
    b = [0x2] + [0] * 63
    a[32], b[32] = 0x1, 0x1        # 0.25 in group 2 (second scale block)
    got = phi_dot(m, a, b, 0, [127 + 40, 127], [127, 127])
    assert word_f32(got) == 2.0 ** 40          # 0.25 < 2^(40-35): truncated
    got = phi_dot(m, a, b, 0, [127 + 33, 127], [127, 127])
    assert got == f32_word(2.0 ** 33)          # 0.25 = 2^(33-35) is kept in the fixed-point sum, then cut by RZ-FP32
    a[0] = 0xA                      # -1.0: the sum is -2^33 + 0.25; RZ-FP32 -> -(2^33 - 2^9)
    got = phi_dot(m, a, b, 0, [127 + 33, 127], [127, 127])
    assert word_f32(got) == -(2.0 ** 33 - 2.0 ** 9)
    got = phi_dot(m, a, b, 0, [127 + 34, 127], [127, 127])
    assert word_f32(got) == -(2.0 ** 34)       # one binade further the 0.25 falls below 2^(e_max - 35)


# --------------------------------------------------------------------------
# GTR-FDPA: group structure and special truncation
# --------------------------------------------------------------------------
def test_gtr_even_odd_groups():
    fmt = FORMATS["e5m2"]
    m = lookup("cdna3", "e5m2", "fp32")
    w = lambda x: exact_word("e5m2", x)
    # swapping the roles of even and odd slots swaps which small term survives
    a = [w(-2.0 ** 13), w(-0.5), w(-0.25), w(-0.125)] + [0] * 12
    b = [w(2.0 ** 10), w(1.0), w(1.0), w(1.0)] + [0] * 12
    assert word_f32(phi_dot(m, a, b, f32_word(2.0 ** 23))) == -1.0
    a2 = [a[1], a[0], a[3], a[2]] + [0] * 12
    b2 = [b[1], b[0], b[3], b[2]] + [0] * 12
    assert word_f32(phi_dot(m, a2, b2, f32_word(2.0 ** 23))) == -1.0
    # special truncation: c far below E is dropped entirely instead of rounding down to -1 unit
    a = [w(2.0 ** 10)] + [0] * 15
    b = [w(2.0 ** 10)] + [0] * 15
    d = ops.gtr_fdpa(a, b, f32_word(-(2.0 ** -10)), fmt, fmt, 24, 31)
    assert word_f32(d) == 2.0 ** 20            # without the rule RD would give 2^20 - 2^-4
    d = ops.tr_fdpa(a, b, f32_word(-(2.0 ** -10)), fmt, fmt, 24, 31)
    assert word_f32(d) == 2.0 ** 20 - 2.0 ** -4


# --------------------------------------------------------------------------
# registry against the parameter tables typed from the paper
# --------------------------------------------------------------------------
def test_registry_matches_tables():
    rows = read_table("registry_tables.txt")
    assert len(rows) == len(REGISTRY) == 86
    for arch, in_fmt, acc, family, L, F, F2, rho_name, P, G, kb in rows:
        m = REGISTRY[(arch, in_fmt, acc)]
        num = lambda s: 0 if s == "-" else int(s)
        assert (m.family, m.L, m.F, m.F2, m.P, m.G, m.k_block) == (family, num(L), num(F), num(F2), num(P), num(G), num(kb))
        assert m.rho == ("" if rho_name == "-" else rho_name)


def test_chunk_promotion_composition():
    from oracle.models import chunk_promote_dot
    m = lookup("hopper", "e4m3", "fp32")
    rng = random.Random(18)
    a = [rng.getrandbits(8) & 0x77 | (rng.getrandbits(1) << 7) for _ in range(256)]
    b = [rng.getrandbits(8) & 0x77 | (rng.getrandbits(1) << 7) for _ in range(256)]
    c = f32_word(0.3)
    p0 = phi_dot(m, a[:128], b[:128], 0)
    p1 = phi_dot(m, a[128:], b[128:], 0)
    want = np.float32(np.float32(np.float32(0.3) + np.uint32(p0).view(np.float32)) + np.uint32(p1).view(np.float32))
    assert chunk_promote_dot(m, a, b, c, 128) == int(want.view(np.uint32))


# --------------------------------------------------------------------------
# GTR-FDPA Step 4 (Algorithm 11), worked by hand from the printed steps: F = 24, F2 = 31
# --------------------------------------------------------------------------
def test_gtr_step4_T_is_aligned_with_F2_when_c_has_the_larger_exponent():
    fmt = FORMATS["e5m2"]
    w = lambda x: exact_word("e5m2", x)
    # products 2^-14 (slot 0, even group) and 2^-16 (slot 1, odd group); c = 2^10, so E = Exp(c) = 10 > e_max = -14.
    # T = 2^-14 + 2^-16 exactly (Step 3 keeps 24 fractional bits below 2^-14).
    # Step 4: T' = RD_31(T * 2^(e_max - E)) has units of 2^(10-31) = 2^-21: both bits of T survive.
    #         S = 2^10 + 2^-14 + 2^-16, just above the midpoint 2^10 + 2^-14 of the FP32 grid (ulp 2^-13): RNE goes up.
    # Had T been cut at F = 24 fractional bits (units 2^-14), S would be the exact tie and RNE would return 2^10.
    a = [w(2.0 ** -7), w(2.0 ** -8)] + [0] * 14
    b = [w(2.0 ** -7), w(2.0 ** -8)] + [0] * 14
    d = ops.gtr_fdpa(a, b, f32_word(2.0 ** 10), fmt, fmt, 24, 31)
    assert d == f32_word(2.0 ** 10 + 2.0 ** -13)
    # the same with a negative T = -2^-16: RD_31 keeps it exactly, S = 2^10 - 2^-16 rounds (RNE) back to 2^10;
    # with 24 fractional bits RD would give -2^-14 and S = 2^10 - 2^-14, a representable number
    a = [w(-(2.0 ** -8))] + [0] * 15
    b = [w(2.0 ** -8)] + [0] * 15
    d = ops.gtr_fdpa(a, b, f32_word(2.0 ** 10), fmt, fmt, 24, 31)
    assert d == f32_word(2.0 ** 10)
    # a negative T whose only bit lies below 2^-14 but on the F2 grid: -2^-20 is kept, S = 2^10 - 2^-20 -> RNE -> 2^10
    a = [w(-(2.0 ** -10))] + [0] * 15
    b = [w(2.0 ** -10)] + [0] * 15
    assert ops.gtr_fdpa(a, b, f32_word(2.0 ** 10), fmt, fmt, 24, 31) == f32_word(2.0 ** 10)


def test_gtr_step4_special_truncation_threshold_and_round_down_of_c():
    fmt = FORMATS["e5m2"]
    w = lambda x: exact_word("e5m2", x)
    a = [w(2.0 ** 10)] + [0] * 15
    b = [w(2.0 ** 10)] + [0] * 15                          # T = 2^20, e_max = E = 20, units of s_c' are 2^(20-24) = 2^-4
    g = lambda c: word_f32(ops.gtr_fdpa(a, b, f32_word(c), fmt, fmt, 24, 31))
    # Exp(c) = -5 = E - F - 1: not below the threshold; RD_24(-2^-5) = -1 unit = -2^-4 (round down, not toward zero)
    assert g(-(2.0 ** -5)) == 2.0 ** 20 - 2.0 ** -4
    assert g(-(1.75 * 2.0 ** -5)) == 2.0 ** 20 - 2.0 ** -4
    # Exp(c) = -6 = E - F - 2 < E - F - 1: special truncation, s_c' = 0 although RD alone would give -1 unit
    assert g(-(2.0 ** -6)) == 2.0 ** 20
    assert g(-(1.9999999 * 2.0 ** -6)) == 2.0 ** 20
    # positive c of the same sizes rounds down to 0 either way
    assert g(2.0 ** -5) == 2.0 ** 20
    assert g(2.0 ** -6) == 2.0 ** 20
    # Exp(c) = -4 = E - F: one full unit, and one unit plus lower bits (negative: floor takes two units)
    assert g(-(2.0 ** -4)) == 2.0 ** 20 - 2.0 ** -4
    assert g(-(1.5 * 2.0 ** -4)) == 2.0 ** 20 - 2.0 ** -3


def test_gtr_step4_tie_above_power_of_two_goes_to_even():
    fmt = FORMATS["e5m2"]
    w = lambda x: exact_word("e5m2", x)
    a = [w(2.0 ** 10)] + [0] * 15
    b = [w(2.0 ** 10)] + [0] * 15
    d = ops.gtr_fdpa(a, b, f32_word(1.5 * 2.0 ** -4), fmt, fmt, 24, 31)   # s_c' = RD(1.5 units) = 1 unit = 2^-4
    assert word_f32(d) == 2.0 ** 20                                        # 2^20 + 2^-4: tie, even neighbour


# --------------------------------------------------------------------------
# GST-FDPA Step 2 (Algorithm 9): the accumulator term is truncated toward zero like every other term
# --------------------------------------------------------------------------
def test_gst_accumulator_term_is_truncated_toward_zero():
    m = lookup("blackwell", "mxf4", "fp32")
    a = [0x2] + [0] * 63                                    # 1.0 * 1.0 in group 0, block scale 2^20 * 2^0
    b = [0x2] + [0] * 63
    sfa, sfb = [127 + 20, 127], [127, 127]
    # e_max = 20 (the group's scale exponents), unit of the fused sum 2^(20-35) = 2^-15.
    # c = -(1 + 2^-23): RZ_35 drops the 2^-23 bit and leaves -1 (floor would leave -(1 + 2^-15)).
    # S = 2^20 - 1, an FP32 number (ulp 2^-4 below 2^20).  With floor: 2^20 - 1 - 2^-15 -> RZ-FP32 -> 2^20 - 1 - 2^-4.
    c = f32_word(-(1.0 + 2.0 ** -23))
    assert phi_dot(m, a, b, c, sfa, sfb) == f32_word(2.0 ** 20 - 1.0)
    # the mirrored case: RZ of +(1 + 2^-23) is +1 as well
    c = f32_word(1.0 + 2.0 ** -23)
    assert phi_dot(m, a, b, c, sfa, sfb) == f32_word(2.0 ** 20 + 1.0)
    # a negative accumulator entirely below one unit vanishes (floor would subtract a whole unit)
    c = f32_word(-(2.0 ** -16))
    assert phi_dot(m, a, b, c, sfa, sfb) == f32_word(2.0 ** 20)


# --------------------------------------------------------------------------
# dequantisation epilogue: D = fl32(fl32(sa * sb) * d), in that order, NaN as the CUDA cores encode it
# --------------------------------------------------------------------------
def test_dequant_against_numpy_float32():
    from oracle.models import dequant
    rng = np.random.Generator(np.random.Philox(23))
    n = 4000
    sa = rng.standard_normal(n).astype(np.float32) * np.float32(3.0)
    sb = np.exp(rng.standard_normal(n) * 3).astype(np.float32)
    d = (rng.standard_normal(n) * np.exp(rng.standard_normal(n) * 5)).astype(np.float32)
    with np.errstate(all="ignore"):
        want = ((sa * sb) * d).view(np.uint32)
        other = (sa * (sb * d)).view(np.uint32)
    assert int((want != other).sum()) > 200            # the order of the two multiplications matters on these inputs
    for i in range(n):
        got = dequant(int(d[i:i + 1].view(np.uint32)[0]), int(sa[i:i + 1].view(np.uint32)[0]),
                      int(sb[i:i + 1].view(np.uint32)[0]))
        assert got == int(want[i]), i
    # special values: NaN in any position -> 0x7FFFFFFF; inf * 0 -> NaN; inf * finite -> inf with the product's sign;
    # overflow of the first product is not undone by a small d
    inf, nan = f32_word(float("inf")), 0x7FC00001
    one, zero, big, tiny = f32_word(1.0), 0, f32_word(2.0 ** 100), f32_word(2.0 ** -120)
    assert dequant(nan, one, one) == 0x7FFFFFFF
    assert dequant(one, nan, one) == 0x7FFFFFFF
    assert dequant(one, one, 0xFFC00000) == 0x7FFFFFFF
    assert dequant(zero, inf, one) == 0x7FFFFFFF
    assert dequant(f32_word(-2.0), inf, one) == f32_word(float("-inf"))
    assert dequant(tiny, big, big) == inf              # fl32(2^200) = inf first, then inf * 2^-120
    assert dequant(big, big, tiny) == f32_word(2.0 ** 80)
    # subnormal results round to nearest even on the 2^-149 grid
    assert dequant(f32_word(1.5), f32_word(2.0 ** -75), f32_word(2.0 ** -74)) == 2      # 1.5 * 2^-149 -> 2 * 2^-149
    assert dequant(f32_word(2.5), f32_word(2.0 ** -75), f32_word(2.0 ** -74)) == 2      # 2.5 units: tie -> even


# --------------------------------------------------------------------------
# TR-/GTR-FDPA: the second-stage alignment of T rounds DOWN (Algorithm 10 Step 3, Algorithm 11 Step 4)
# --------------------------------------------------------------------------
@pytest.mark.parametrize("family", ["tr", "gtr"])
def test_tr_gtr_T_is_rounded_down_at_F2(family):
    # products -2^-15 and -2^-24, c = 2^10: E = 10, one unit of T' is 2^(10-31) = 2^-21.
    # T = -(64 + 1/8) units: RD gives -65 units (RZ would give -64).  S = 2^10 - 65 * 2^-21 lies beyond the midpoint
    # 2^10 - 2^-15 of the FP32 grid below 2^10 (spacing 2^-14), so RNE-FP32 gives 2^10 - 2^-14; with -64 units S would
    # be that midpoint exactly and round to the even neighbour 2^10.
    name = "fp16" if family == "tr" else "e5m2"
    fmt = FORMATS[name]
    w = lambda x: exact_word(name, x)
    L = 8 if family == "tr" else 16
    a = [w(-(2.0 ** -8)), w(-(2.0 ** -12))] + [0] * (L - 2)
    b = [w(2.0 ** -7), w(2.0 ** -12)] + [0] * (L - 2)
    op = ops.tr_fdpa if family == "tr" else ops.gtr_fdpa
    assert op(a, b, f32_word(2.0 ** 10), fmt, fmt, 24, 31) == f32_word(2.0 ** 10 - 2.0 ** -14)
    # the positive mirror image: RD drops the 1/8 unit, S = 2^10 + 2^-15 is a quarter of the FP32 spacing above 2^10
    # (2^-13) and rounds to 2^10
    a[0], a[1] = w(2.0 ** -8), w(2.0 ** -12)
    assert op(a, b, f32_word(2.0 ** 10), fmt, fmt, 24, 31) == f32_word(2.0 ** 10)


def test_tr_product_overflow_is_an_infinity_before_the_sum():
    # Section 4.2: a TR-FDPA product of magnitude >= 2^128 is an infinity, whatever the other terms would cancel
    fmt = FORMATS["bf16"]
    w = lambda x: exact_word("bf16", x)
    z = [0] * 6
    inf, ninf, nan = f32_word(float("inf")), f32_word(float("-inf")), 0x7FC00000
    # 2^64 * 2^64 = 2^128 exactly: +inf although the second product takes half of it away again
    assert ops.tr_fdpa([w(2.0 ** 64), w(-(2.0 ** 63))] + z, [w(2.0 ** 64), w(2.0 ** 64)] + z, 0, fmt, fmt, 24, 31) == inf
    # +2^128 and -2^128: inf - inf = NaN (the exact sum would be 0)
    assert ops.tr_fdpa([w(2.0 ** 64), w(-(2.0 ** 64))] + z, [w(2.0 ** 64), w(2.0 ** 64)] + z, 0, fmt, fmt, 24, 31) == nan
    assert ops.tr_fdpa([w(-(2.0 ** 64))] + [0] * 7, [w(2.0 ** 64)] + [0] * 7, 0, fmt, fmt, 24, 31) == ninf
    # just below the threshold the product is an ordinary number: (2 - 2^-7) * 2^127 - 2^127 = (1 - 2^-7) * 2^127
    big = w((2.0 - 2.0 ** -7) * 2.0 ** 63)
    d = ops.tr_fdpa([big, w(-(2.0 ** 63))] + z, [w(2.0 ** 64), w(2.0 ** 64)] + z, 0, fmt, fmt, 24, 31)
    assert d == f32_word((1.0 - 2.0 ** -7) * 2.0 ** 127)
    # and a sum of finite products that reaches 2^128 overflows only in the final conversion
    d = ops.tr_fdpa([big, big] + z, [w(2.0 ** 64), w(2.0 ** 64)] + z, 0, fmt, fmt, 24, 31)
    assert d == inf


# --------------------------------------------------------------------------
# zero accumulators have no exponent (the reading the B200 confirms for its FP16 / BF16 rows)
# --------------------------------------------------------------------------
def test_zero_accumulator_takes_no_part_in_e_max():
    # FP16 accumulator +0 (its exponent would be -14): products 2^-25 and 2^-40.  e_max = -25, nothing is cut,
    # S = 2^-25 + 2^-40 is above the midpoint between 0 and the smallest FP16 number 2^-24: RNE-FP16 gives 2^-24.
    # Were the zero counted, units of 2^(-14-25) would drop the 2^-40 and the exact tie would go to the even side, 0.
    m = lookup("blackwell", "fp16", "fp16")
    w = lambda x: f16_word(x)
    a = [w(2.0 ** -12), w(2.0 ** -20)] + [0] * 14
    b = [w(2.0 ** -13), w(2.0 ** -20)] + [0] * 14
    assert phi_dot(m, a, b, 0) == 0x0001
    # FP32 accumulator +0 (its exponent would be -126): +2^-149 and -2^-160 under RZ-FP32.  The exact sum is below
    # 2^-149 and truncates to 0; units of 2^(-126-25) would cut the negative term away first and leave 2^-149.
    m = lookup("blackwell", "bf16", "fp32")
    w = lambda x: exact_word("bf16", x)
    a = [w(2.0 ** -75), w(-(2.0 ** -80))] + [0] * 14
    b = [w(2.0 ** -74), w(2.0 ** -80)] + [0] * 14
    assert phi_dot(m, a, b, 0) == 0
    assert phi_dot(m, a, b, f32_word(-0.0)) == 0
    # TR-FDPA with c = 0: E = e_max; 2^-150 + 2^-160 is above the midpoint of (0, 2^-149) and rounds up
    fmt = FORMATS["bf16"]
    a = [w(2.0 ** -75), w(2.0 ** -80)] + [0] * 6
    b = [w(2.0 ** -75), w(2.0 ** -80)] + [0] * 6
    assert ops.tr_fdpa(a, b, 0, fmt, fmt, 24, 31) == 0x00000001


# --------------------------------------------------------------------------
# GST-FDPA Step 2: group terms are truncated toward zero; zero groups and a zero accumulator have no exponent
# --------------------------------------------------------------------------
def test_gst_negative_group_term_is_truncated_toward_zero():
    m = lookup("blackwell", "mxf4", "fp32")
    a = [0x2] + [0] * 63           # +1.0 in group 0, scaled by 2^36: e_max = 36, one unit of the fused sum is 2
    b = [0x2] + [0] * 63
    a[32], b[32] = 0x1, 0x9        # 0.5 * -0.5 = -0.25 in group 2 (second scale block, scale 1)
    # RZ_35(-0.25 / 2) = 0: S = 2^36.  Rounding down would give -1 unit, 2^36 - 2, and RZ-FP32 then 2^36 - 2^12.
    assert phi_dot(m, a, b, 0, [127 + 36, 127], [127, 127]) == f32_word(2.0 ** 36)


def test_gst_groups_in_e_max_and_zero_accumulator():
    m = lookup("blackwell", "mxf4", "fp32")
    c = f32_word(-1.5 * 2.0 ** -30)
    near_one = f32_word(1.0 - 2.0 ** -24)                  # RZ-FP32 of 1 - 1.5 * 2^-30
    # Block 1 (scale 1) holds 1.0 in group 2.  Block 0 (scale 2^11) in three versions; the words are what the B200's
    # tcgen05.mma returns for these inputs (MXFP4 and, with per-group scales, NVFP4):
    a = [0] * 64
    b = [0] * 64
    a[32], b[32] = 0x2, 0x2
    # (1) all elements of block 0 zero: its groups have no exponent, e_max = 0, unit 2^-35, c is kept
    assert phi_dot(m, a, b, c, [127 + 11, 127], [127, 127]) == near_one
    # (2) products that cancel (1 * 1 + 1 * -1 in both groups): p_g = 0, but the groups count with e_g = 11:
    #     unit 2^(11-35) = 2^-24 and |c| < 2^-24 vanishes
    a2, b2 = a[:], b[:]
    a2[0], b2[0], a2[1], b2[1] = 0x2, 0x2, 0x2, 0xA
    a2[16], b2[16], a2[17], b2[17] = 0x2, 0x2, 0x2, 0xA
    assert phi_dot(m, a2, b2, c, [127 + 11, 127], [127, 127]) == f32_word(1.0)
    # (3) a nonzero group (0.5 * 0.5 * 2^11 = 512) next to an empty one: 513 (c vanishes again)
    a3, b3 = a[:], b[:]
    a3[16], b3[16] = 0x1, 0x1
    assert phi_dot(m, a3, b3, c, [127 + 11, 127], [127, 127]) == f32_word(513.0)
    # the same three with NVFP4 scales (group 0 under 2^7 * 2^4, the others under 1)
    n = lookup("blackwell", "nvf4", "fp32")
    one, sfa, sfb = 0x38, [0x70, 0x38, 0x38, 0x38], [0x58, 0x38, 0x38, 0x38]
    a = [0] * 64
    b = [0] * 64
    a[16], b[16] = 0x2, 0x2
    assert phi_dot(n, a, b, c, sfa, sfb) == near_one
    a2, b2 = a[:], b[:]
    a2[0], b2[0], a2[1], b2[1] = 0x2, 0x2, 0x2, 0xA
    assert phi_dot(n, a2, b2, c, sfa, sfb) == f32_word(1.0)
    a3, b3 = a[:], b[:]
    a3[0], b3[0] = 0x1, 0x1
    assert phi_dot(n, a3, b3, c, sfa, sfb) == f32_word(513.0)
    m = lookup("blackwell", "mxf4", "fp32")
    # c = +0: group 0 gives +0.25 * 2^-147 = 2^-149, group 2 gives -0.25 * 2^-163 = -2^-165.  e_max = -147, both terms are
    # exact, S = 2^-149 - 2^-165 > 0 truncates (RZ-FP32) to +0.  Were the zero accumulator counted with the exponent -126,
    # units of 2^-161 would cut the negative term to 0 first and leave 2^-149.  (The B200's tcgen05.mma returns 0 here
    # and 1 in the control below.)
    a = [0x1] + [0] * 63
    b = [0x1] + [0] * 63
    a[32], b[32] = 0x1, 0x9
    assert phi_dot(m, a, b, 0, [27, 27], [80, 64]) == 0
    # control: with the first group alone the smallest subnormal comes out
    a[32] = 0
    assert phi_dot(m, a, b, 0, [27, 27], [80, 64]) == 1


# --------------------------------------------------------------------------
# the sign of a zero result (values the B200 returns for these inputs, through mma.sync and tcgen05.mma)
# --------------------------------------------------------------------------
def test_zero_results_of_the_nvidia_conversions_are_positive():
    w = lambda x: exact_word("bf16", x)
    m = lookup("blackwell", "bf16", "fp32")
    z = [0] * 15
    # -2^-75 * 2^-75 = -2^-150 is below the smallest FP32 subnormal: RZ-FP32 leaves magnitude zero, and the word is +0
    assert phi_dot(m, [w(-(2.0 ** -75))] + z, [w(2.0 ** -75)] + z, 0) == 0x00000000
    assert phi_dot(m, [w(-(2.0 ** -100))] + z, [w(2.0 ** -100)] + z, f32_word(-0.0)) == 0x00000000
    # one binade up the subnormal survives with its sign
    assert phi_dot(m, [w(-1.5 * 2.0 ** -75)] + z, [w(2.0 ** -74)] + z, 0) == 0x80000001
    # RNE-FP16: -2^-28 and the tie -2^-25 round to zero: +0; -1.5 * 2^-25 rounds to -2^-24
    m = lookup("blackwell", "fp16", "fp16")
    h = f16_word
    assert phi_dot(m, [h(-(2.0 ** -14))] + z, [h(2.0 ** -14)] + z, 0) == 0x0000
    assert phi_dot(m, [h(-(2.0 ** -13))] + z, [h(2.0 ** -12)] + z, 0x8000) == 0x0000
    assert phi_dot(m, [h(-1.5 * 2.0 ** -13)] + z, [h(2.0 ** -12)] + z, 0) == 0x8001
    # RZ-E8M13 (Hopper FP8): an accumulator below the 2^-139 grid with all-zero products converts to +0
    m = lookup("hopper", "e4m3", "fp32")
    assert phi_dot(m, [0] * 32, [0] * 32, f32_word(-(2.0 ** -145))) == 0x00000000
    assert phi_dot(m, [0] * 32, [0] * 32, f32_word(-(2.0 ** -139))) == 0x80000400
    # RNE-FP32 (the AMD models) keeps the sign of an underflowed sum, as IEEE-754 rounding does
    fmt = FORMATS["bf16"]
    assert ops.tr_fdpa([w(-(2.0 ** -100))] + [0] * 7, [w(2.0 ** -100)] + [0] * 7, 0, fmt, fmt, 24, 31) == 0x80000000


def test_gst_group_with_a_zero_scale_factor_has_no_exponent():
    # NVFP4: group 0 has the scale pair (2^7 * 1.0, 0): its term is zero and, unlike an empty group under nonzero scales,
    # it does not raise e_max.  Group 1: 1.0 * 1.0 under scales (1, 1) = 1.  e_max = 0, one unit is 2^-35:
    # c = -1.5 * 2^-36 is 0.75 units and truncates to 0, the result is 1.0; of c = -1.5 * 2^-35 one unit survives, and
    # RZ-FP32 of 1 - 2^-35 is the largest FP32 number below 1.  Had group 0 counted with e_g = 7 - 6, one unit would be
    # 2^-34 and that c would vanish too.  (The B200's tcgen05.mma on NVFP4 operands with zero scale bytes follows this
    # rule: with zero-scale groups counted, 214 of 524288 outputs of a randomized run differed, without them none.)
    m = lookup("blackwell", "nvf4", "fp32")
    a = [0] * 64
    b = [0] * 64
    a[0], b[0] = 0x7, 0x7                # 6 * 6 in group 0, under a zero scale
    a[16], b[16] = 0x2, 0x2              # 1 * 1 in group 1
    one, big = 0x38, 0x70                # UE4M3 codes of 1.0 and 2^7
    sfa, sfb = [big, one, one, one], [0x00, one, one, one]
    assert phi_dot(m, a, b, f32_word(-1.5 * 2.0 ** -36), sfa, sfb) == f32_word(1.0)
    assert phi_dot(m, a, b, f32_word(-1.5 * 2.0 ** -35), sfa, sfb) == f32_word(1.0 - 2.0 ** -24)
    # the same call with a nonzero (tiny) scale in place of the zero one: the group counts, e_max = 7 - 6 = 1 at least
    sfb2 = [0x01, one, one, one]         # 2^-9: the group's value 36 * 2^7 * 2^-9 = 9, e_g = 7 + (-6) = 1
    assert phi_dot(m, a, b, f32_word(-1.5 * 2.0 ** -35), sfa, sfb2) == f32_word(10.0)


def test_printed_form_of_the_maximum_exponent_is_reachable_and_differs_only_on_zero_terms():
    """Algorithms 7-11 print the maximum over every term; reading R2 (decided by the B200) leaves zero terms out.  The
    printed form is an option of the oracle (and an override of the library): on the inputs that separate the two it gives
    the value the printed algorithm gives by hand, and without zero terms both forms agree."""
    from oracle import printed
    m = lookup("hopper", "fp16", "fp32")
    h = lambda x: exact_word("fp16", x)
    a = [h(0.0), h(2.0 ** -14)] + [0] * 14
    b = [h(2.0 ** 15), h(1.5 * 2.0 ** -14)] + [0] * 14
    # printed: the zero product counts with Exp(0) + Exp(2^15) = -14 + 15 = 1, the grid is 2^(1 - 25), and 1.5 * 2^-28 is
    # truncated away; R2: it survives
    assert word_f32(phi_dot(printed(m), a, b, 0)) == 0.0
    assert word_f32(phi_dot(m, a, b, 0)) == 1.5 * 2.0 ** -28
    # a zero accumulator counts with Exp = -126 in the printed form: no effect here (every product exponent is larger) ...
    assert phi_dot(printed(m), [h(3.0)] * 16, [h(0.5)] * 16, 0) == phi_dot(m, [h(3.0)] * 16, [h(0.5)] * 16, 0)
    # TR-FDPA (Algorithm 10): a zero accumulator counted with Exp = -126 makes E = -126, and T is rounded down onto
    # 2^(-126 - 31) before the final rounding.  One product 145/128 * 2^-100 times 226/128 * 2^-51 = 2^-150 (1 + 2^-14):
    # exactly (R2: E = e_max) it lies above the tie between 0 and 2^-149 and rounds to 2^-149; rounded down onto 2^-157
    # first it is the tie itself, which RNE sends to the even neighbour 0
    hb = lambda x: exact_word("bf16", x)
    mt = lookup("cdna3", "bf16", "fp32")
    at = [hb(145 / 128 * 2.0 ** -100)] + [0] * 7
    bt = [hb(226 / 128 * 2.0 ** -51)] + [0] * 7
    assert phi_dot(mt, at, bt, 0) == 0x00000001
    assert phi_dot(printed(mt), at, bt, 0) == 0x00000000
    # random inputs without zeros: both forms agree (the option changes nothing but the treatment of zero terms)
    rng = random.Random(31)
    for key in (("ampere", "fp16", "fp32"), ("blackwell", "e4m3", "fp32"), ("cdna3", "fp16", "fp32"), ("cdna3", "e5m2", "fp32")):
        mm = lookup(*key)
        fmt = FORMATS[mm.elem]
        for _ in range(100):
            av, bv = [], []
            while len(av) < mm.L:
                x, y = _rand_finite(rng, fmt), _rand_finite(rng, fmt)
                if (x & ((1 << (fmt.ebits + fmt.mbits)) - 1)) and (y & ((1 << (fmt.ebits + fmt.mbits)) - 1)):
                    av.append(x); bv.append(y)
            c = f32_word(rng.gauss(0.0, 1.0))
            assert phi_dot(mm, av, bv, c) == phi_dot(printed(mm), av, bv, c), key
