"""Conversion of an exact dyadic value to a floating-point word (test infrastructure).

One routine serves every conversion function of Table 2 (RZ-FP32, RZ-E8M13,
RNE-FP32, RNE-FP16) and the RNE roundings of Algorithms 1, 3 and 6.

Readings where the paper is silent:
* gradual underflow everywhere (only the CDNA2 model flushes, Section 4.1);
* on overflow every conversion gives +-inf, the round-to-zero ones too (they
  do not saturate at the largest finite value: the B200's mma.sync, which the
  Blackwell rows describe, returns +-inf);
* a result of magnitude zero under the NVIDIA conversions (RZ-FP32, RZ-E8M13, RNE-FP16) is +0, also when a negative
  sum underflows (the B200 does so through both of its matrix instructions); RNE-FP32 keeps the sign;
* RZ-E8M13 is an FP32 word whose low 10 mantissa bits are zero: 8 exponent
  bits, 13 mantissa bits, subnormals on a 2**-139 grid.
"""
from __future__ import annotations

# name -> (ebits, mbits, bias, mode, left shift into the container)
RHO = {
    "RZ-FP32": (8, 23, 127, "RZ", 0),
    "RZ-E8M13": (8, 13, 127, "RZ", 10),
    "RNE-FP32": (8, 23, 127, "RNE", 0),
    "RNE-FP16": (5, 10, 15, "RNE", 0),
    "RNE-FP64": (11, 52, 1023, "RNE", 0),
}


def round_dyadic(m: int, e: int, ebits: int, mbits: int, bias: int, mode: str,
                 zero_sign: int = 0) -> int:
    """Round the exact value ``m * 2**e`` (``m`` a signed integer) to a word.

    ``mode`` is 'RZ' (truncate the magnitude) or 'RNE' (nearest, ties to even).
    An exact zero gets the sign ``zero_sign``; a nonzero value that rounds to
    zero keeps its own sign.  The word is returned without any container shift.
    """
    sign_shift = ebits + mbits
    if m == 0:
        return zero_sign << sign_shift
    sign = 1 if m < 0 else 0
    mag = -m if sign else m
    emin = 1 - bias
    top = (1 << ebits) - 1                      # exponent field of inf/NaN
    value_exp = mag.bit_length() - 1 + e        # floor(log2 |value|)
    q = max(value_exp, emin) - mbits            # exponent of one unit in the last place
    sh = e - q
    if sh >= 0:
        n, rem, half = mag << sh, 0, 1
    else:
        n = mag >> -sh
        rem = mag & ((1 << -sh) - 1)
        half = 1 << (-sh - 1)
    if mode == "RNE":
        if rem > half or (rem == half and (n & 1)):
            n += 1
    elif mode != "RZ":
        raise ValueError(mode)
    if n >> (mbits + 1):                        # rounding carried into the next binade
        n >>= 1
        q += 1
    if n >> mbits:                              # normal number
        field = q + mbits + bias
        if field >= top:                        # overflow: +-inf in both modes
            return (sign << sign_shift) | (top << mbits)
        return (sign << sign_shift) | (field << mbits) | (n & ((1 << mbits) - 1))
    return (sign << sign_shift) | n             # subnormal or zero (field 0)


# conversions of the NVIDIA models (T-, ST-, GST-FDPA): a result of magnitude zero is +0 whatever the sign of the sum
ZERO_IS_POSITIVE = {"RZ-FP32", "RZ-E8M13", "RNE-FP16"}


def rho(name: str, m: int, e: int) -> int:
    """Apply the conversion function ``name`` of Table 2 to ``m * 2**e``; exact zero -> +0.

    Under RZ-FP32, RZ-E8M13 and RNE-FP16 a nonzero sum that converts to zero gives +0 as well (the B200 returns +0 for
    a negative sum below the smallest subnormal, through mma.sync and through tcgen05.mma, for FP32 and FP16 outputs);
    RNE-FP32, the conversion of the AMD models, keeps the sign as IEEE-754 rounding does (no hardware pin).
    """
    ebits, mbits, bias, mode, lsh = RHO[name]
    w = round_dyadic(m, e, ebits, mbits, bias, mode)
    if name in ZERO_IS_POSITIVE and (w & ((1 << (ebits + mbits)) - 1)) == 0:
        w = 0
    return w << lsh
