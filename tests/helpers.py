"""Word <-> value helpers for tests, built on numpy/struct/torch conversions only
(independent of both the oracle and the CUDA library)."""
import struct
from fractions import Fraction

import numpy as np

GOLDEN = __import__("os").path.join(__import__("os").path.dirname(__file__), "golden")


def f32_word(x: float) -> int:
    return struct.unpack("<I", struct.pack("<f", x))[0]


def word_f32(w: int) -> float:
    return struct.unpack("<f", struct.pack("<I", w & 0xFFFFFFFF))[0]


def f64_word(x: float) -> int:
    return struct.unpack("<Q", struct.pack("<d", x))[0]


def word_f64(w: int) -> float:
    return struct.unpack("<d", struct.pack("<Q", w))[0]


def f16_word(x: float) -> int:
    return int(np.float16(x).view(np.uint16))


def word_f16(w: int) -> float:
    return float(np.uint16(w).view(np.float16))


def exact_word(fmt: str, x: float) -> int:
    """Word of format ``fmt`` whose value is exactly ``x`` (asserts representability)."""
    if fmt == "fp64":
        return f64_word(x)
    w32 = f32_word(x)
    assert word_f32(w32) == x
    if fmt == "fp32":
        return w32
    if fmt == "tf32":
        assert w32 & 0x1FFF == 0
        return w32
    if fmt == "bf16":
        assert w32 & 0xFFFF == 0
        return w32 >> 16
    w16 = f16_word(x)
    assert word_f16(w16) == x, (fmt, x)
    if fmt == "fp16":
        return w16
    if fmt == "e5m2":
        assert w16 & 0xFF == 0
        return w16 >> 8
    raise ValueError(fmt)


def word_value(fmt: str, w: int) -> float:
    if fmt == "fp64":
        return word_f64(w)
    if fmt == "fp32":
        return word_f32(w)
    if fmt == "fp16":
        return word_f16(w)
    raise ValueError(fmt)


def float_to_fraction(x: float) -> Fraction:
    return Fraction(x)


def read_table(name):
    rows = []
    with open(f"{GOLDEN}/{name}") as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if line:
                rows.append(line.split())
    return rows
