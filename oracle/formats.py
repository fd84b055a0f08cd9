"""Number formats of the paper's models and their decoding (test infrastructure).

The paper uses ``SignedSig(x)`` and ``Exp(x)`` (Algorithm 7, Step 1) without
defining them bit by bit.  The reading used here: a finite word with exponent
field ``f`` and mantissa field ``m`` (``mbits`` wide) has

    sig = m + (2**mbits if f != 0 else 0)        (integer significand)
    Exp = max(f, 1) - bias                       (unnormalised exponent)
    value = (-1)**sign * sig * 2**(Exp - mbits)

so a subnormal (and zero) keeps the minimum exponent ``1 - bias`` and a
significand without hidden bit ("exact unnormalized products", Section 4.1,
T-FDPA paragraph).  Encodings follow IEEE-754 (FP64/FP32/FP16, BF16 and TF32 as
truncated FP32) and the OCP FP8 / Microscaling formats (E5M2 IEEE-like; E4M3
with no infinity and the single NaN pattern S.1111.111; FP6/FP4 without
specials; E8M0 = 2**(x-127) with 0xFF = NaN; UE4M3 = E4M3 with the sign bit
ignored).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import NamedTuple

FINITE, INF, NAN = 0, 1, 2


class Dec(NamedTuple):
    """Decoded word: class, sign (0/1), integer significand, unnormalised exponent."""
    cls: int
    sign: int
    sig: int
    exp: int


@dataclass(frozen=True)
class Format:
    name: str
    storage_bits: int      # width of the container word
    ebits: int
    mbits: int
    bias: int
    specials: str          # 'ieee' | 'fn' | 'none' | 'e8m0'
    signed: bool = True
    low_ignored: int = 0   # TF32: the low 13 bits of the 32-bit word carry no information

    @property
    def emin(self) -> int:
        return 1 - self.bias

    @property
    def emax(self) -> int:
        top = (1 << self.ebits) - 1
        return (top - 1 if self.specials == "ieee" else top) - self.bias


FORMATS = {
    "fp64": Format("fp64", 64, 11, 52, 1023, "ieee"),
    "fp32": Format("fp32", 32, 8, 23, 127, "ieee"),
    "tf32": Format("tf32", 32, 8, 10, 127, "ieee", low_ignored=13),
    "bf16": Format("bf16", 16, 8, 7, 127, "ieee"),
    "fp16": Format("fp16", 16, 5, 10, 15, "ieee"),
    "e5m2": Format("e5m2", 8, 5, 2, 15, "ieee"),
    "e4m3": Format("e4m3", 8, 4, 3, 7, "fn"),
    "e3m2": Format("e3m2", 8, 3, 2, 3, "none"),
    "e2m3": Format("e2m3", 8, 2, 3, 1, "none"),
    "e2m1": Format("e2m1", 8, 2, 1, 1, "none"),
    "e8m0": Format("e8m0", 8, 8, 0, 127, "e8m0", signed=False),
    "ue4m3": Format("ue4m3", 8, 4, 3, 7, "fn", signed=False),
}


def decode(fmt: Format, word: int) -> Dec:
    """Split a raw word into (class, sign, sig, Exp) as defined in the module header."""
    if fmt.specials == "e8m0":
        word &= 0xFF
        if word == 0xFF:
            return Dec(NAN, 0, 0, 0)
        return Dec(FINITE, 0, 1, word - fmt.bias)
    w = word >> fmt.low_ignored
    mant = w & ((1 << fmt.mbits) - 1)
    field = (w >> fmt.mbits) & ((1 << fmt.ebits) - 1)
    sign = (w >> (fmt.ebits + fmt.mbits)) & 1 if fmt.signed else 0
    top = (1 << fmt.ebits) - 1
    if fmt.specials == "ieee" and field == top:
        return Dec(NAN if mant else INF, sign, 0, 0)
    if fmt.specials == "fn" and field == top and mant == (1 << fmt.mbits) - 1:
        return Dec(NAN, sign, 0, 0)
    sig = mant | ((1 << fmt.mbits) if field else 0)
    return Dec(FINITE, sign, sig, max(field, 1) - fmt.bias)


def is_subnormal(fmt: Format, word: int) -> bool:
    """True for a nonzero word whose exponent field is zero."""
    d = decode(fmt, word)
    return d.cls == FINITE and d.sig != 0 and d.sig < (1 << fmt.mbits)


def value_as_dyadic(fmt: Format, word: int) -> tuple[int, int]:
    """Finite word -> (m, e) with value == m * 2**e (m signed)."""
    d = decode(fmt, word)
    assert d.cls == FINITE
    m = -d.sig if d.sign else d.sig
    return m, d.exp - fmt.mbits


_DECODERS: dict = {}


def decoder(fmt: Format):
    """A function word -> Dec for ``fmt``; memoised through a full table for containers up to 16 bits."""
    f = _DECODERS.get(fmt.name)
    if f is None:
        if fmt.storage_bits <= 16:
            table = [decode(fmt, w) for w in range(1 << fmt.storage_bits)]
            f = table.__getitem__
        else:
            def f(w, _fmt=fmt):
                return decode(_fmt, w)
        _DECODERS[fmt.name] = f
    return f
