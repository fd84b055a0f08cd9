// Device-side building blocks of the generic (any-model) kernels: number-format decoding, the conversion
// functions of Table 2 and one block of each elementary operation (Algorithms 1, 3, 6-11, Section 4.2).
// The tuned kernels in mmasim_tfdpa_fast.cu specialise the T-FDPA block; everything else runs through here.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>
#include "mmasim_internal.h"

namespace mmasim {

// ---------------------------------------------------------------------------------------------------------
// Decoded element: one 32-bit word.
//   bits  0..11  integer significand (hidden bit included for normal numbers), at most 11 bits here
//   bits 12..13  class: 0 finite, 1 infinity, 2 NaN
//   bit  15      sign
//   bits 16..31  unnormalised exponent Exp = max(field, 1) - bias, as a signed 16-bit integer
// value = (-1)^sign * sig * 2^(Exp - mbits).  Subnormals and zero keep Exp = 1 - bias without hidden bit,
// which is the "exact unnormalized product" convention of Algorithm 7, Step 1.
// ---------------------------------------------------------------------------------------------------------
constexpr uint32_t CLS_FINITE = 0u, CLS_INF = 1u, CLS_NAN = 2u;

__host__ __device__ inline uint32_t dec_pack(uint32_t cls, uint32_t sign, uint32_t sig, int exp) {
    return (sig & 0xFFFu) | (cls << 12) | (sign << 15) | (uint32_t(exp & 0xFFFF) << 16);
}
__device__ __forceinline__ uint32_t dec_sig(uint32_t d) { return d & 0xFFFu; }
__device__ __forceinline__ uint32_t dec_cls(uint32_t d) { return (d >> 12) & 3u; }
__device__ __forceinline__ uint32_t dec_sign(uint32_t d) { return (d >> 15) & 1u; }
__device__ __forceinline__ int dec_exp(uint32_t d) { return int(d) >> 16; }
__device__ __forceinline__ int dec_ssig(uint32_t d) { int s = int(d & 0xFFFu); return (d & 0x8000u) ? -s : s; }

// Decode a raw element of one of the narrow input formats (everything except FP32/FP64 accumulators).
__host__ __device__ inline uint32_t decode_elem(const FmtDesc& f, uint32_t word) {
    if (f.specials == SP_E8M0) {
        word &= 0xFFu;
        if (word == 0xFFu) return dec_pack(CLS_NAN, 0, 0, 0);
        return dec_pack(CLS_FINITE, 0, 1, int(word) - f.bias);
    }
    uint32_t w = word >> f.low_ignored;
    uint32_t mant = w & ((1u << f.mbits) - 1u);
    uint32_t field = (w >> f.mbits) & ((1u << f.ebits) - 1u);
    uint32_t sign = f.is_signed ? ((w >> (f.ebits + f.mbits)) & 1u) : 0u;
    uint32_t top = (1u << f.ebits) - 1u;
    if (f.specials == SP_IEEE && field == top) return dec_pack(mant ? CLS_NAN : CLS_INF, sign, 0, 0);
    if (f.specials == SP_FN && field == top && mant == (1u << f.mbits) - 1u) return dec_pack(CLS_NAN, sign, 0, 0);
    uint32_t sig = mant | (field ? (1u << f.mbits) : 0u);
    int e = int(field ? field : 1u) - f.bias;
    return dec_pack(CLS_FINITE, sign, sig, e);
}

// Accumulator (FP32 or FP16 word) split into class / sign / significand / exponent.
struct AccDec {
    uint32_t cls, sign, sig;
    int exp;
};
__device__ __forceinline__ AccDec decode_acc(uint32_t w, bool fp16) {
    AccDec d;
    if (fp16) {
        uint32_t mant = w & 0x3FFu, field = (w >> 10) & 0x1Fu;
        d.sign = (w >> 15) & 1u;
        d.cls = (field == 0x1Fu) ? (mant ? CLS_NAN : CLS_INF) : CLS_FINITE;
        d.sig = mant | (field ? 0x400u : 0u);
        d.exp = int(field ? field : 1u) - 15;
    } else {
        uint32_t mant = w & 0x7FFFFFu, field = (w >> 23) & 0xFFu;
        d.sign = w >> 31;
        d.cls = (field == 0xFFu) ? (mant ? CLS_NAN : CLS_INF) : CLS_FINITE;
        d.sig = mant | (field ? 0x800000u : 0u);
        d.exp = int(field ? field : 1u) - 127;
    }
    return d;
}

// ---------------------------------------------------------------------------------------------------------
// Table 2: convert the exact value (-1)^sign * mag * 2^e to a word.  mode_rne: nearest-even, else truncation.
// Overflow gives infinity in both modes (truncation does not saturate at the largest finite value).  mag == 0 -> +0.
// `sticky` marks nonzero bits below mag's last bit (only the exact E-FDPA sum needs it).
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t round_pack(uint32_t sign, uint64_t mag, int e, int ebits, int mbits, int bias,
                                               bool mode_rne, bool sticky = false) {
    if (mag == 0) return 0u;
    const int msb = 63 - __clzll((long long)mag);
    const int emin = 1 - bias;
    const int vexp = msb + e;
    int q = (vexp > emin ? vexp : emin) - mbits;   // exponent of the last kept bit
    const int sh = e - q;
    uint64_t n;
    if (sh >= 0) {
        n = mag << sh;                              // msb lands at bit mbits or below: no overflow
    } else {
        const int r = -sh;
        uint64_t rem, half;
        if (r >= 64) {
            n = 0;
            rem = (r == 64) ? mag : (mag ? 1 : 0);  // r > 64: strictly below half
            half = (r == 64) ? (1ull << 63) : ~0ull;
        } else {
            n = mag >> r;
            rem = mag & ((1ull << r) - 1ull);
            half = 1ull << (r - 1);
        }
        if (mode_rne) {
            const bool above = rem > half || (rem == half && sticky);
            const bool tie = rem == half && !sticky;
            if (above || (tie && (n & 1ull))) n += 1;
        }
    }
    if (n >> (mbits + 1)) { n >>= 1; q += 1; }
    const uint32_t top = (1u << ebits) - 1u;
    const uint32_t sbit = sign << (ebits + mbits);
    if (n >> mbits) {
        const int field = q + mbits + bias;
        if (field >= int(top)) return sbit | (top << mbits);
        return sbit | (uint32_t(field) << mbits) | (uint32_t(n) & ((1u << mbits) - 1u));
    }
    return sbit | uint32_t(n);
}

// Under the conversions of the NVIDIA models (RZ-FP32, RZ-E8M13, RNE-FP16) a result of magnitude zero is +0, also when a
// negative sum underflows (what the B200's matrix instructions return); RNE-FP32 keeps the sign.
__device__ __forceinline__ uint32_t positive_zero(uint32_t w, uint32_t magnitude_mask) { return (w & magnitude_mask) ? w : 0u; }

__device__ __forceinline__ uint32_t rho_apply(int rho, int64_t S, int e) {
    const uint32_t sign = S < 0;
    const uint64_t mag = sign ? uint64_t(-S) : uint64_t(S);
    switch (rho) {
        case RHO_RZ_FP32: return positive_zero(round_pack(sign, mag, e, 8, 23, 127, false), 0x7FFFFFFFu);
        case RHO_RZ_E8M13: return positive_zero(round_pack(sign, mag, e, 8, 13, 127, false) << 10, 0x7FFFFFFFu);
        case RHO_RNE_FP32: return round_pack(sign, mag, e, 8, 23, 127, true);
        default: return positive_zero(round_pack(sign, mag, e, 5, 10, 15, true), 0x7FFFu);   // RHO_RNE_FP16
    }
}

// ---------------------------------------------------------------------------------------------------------
// Fixed-point alignment helpers.  rz: truncate the magnitude (sign-magnitude), rd: floor.
// ---------------------------------------------------------------------------------------------------------
// A zero operand stays zero whatever the shift (zero terms reach here with meaningless distances); nonzero operands
// never meet a left shift of 64 or more (every aligned term fits 64 bits by construction).  Left shifts are done on
// the unsigned magnitude / two's-complement bits.
__device__ __forceinline__ int64_t rz_scale(int64_t n, int sh) {
    if (n == 0) return 0;
    const bool neg = n < 0;
    uint64_t m = neg ? 0ull - uint64_t(n) : uint64_t(n);
    if (sh >= 0) m = (sh >= 64) ? 0ull : (m << sh);
    else m = (sh <= -64) ? 0ull : (m >> (-sh));
    return neg ? -int64_t(m) : int64_t(m);
}
__device__ __forceinline__ int64_t rd_scale(int64_t n, int sh) {
    if (n == 0) return 0;
    if (sh >= 0) return (sh >= 64) ? 0ll : int64_t(uint64_t(n) << sh);
    return (sh <= -64) ? (n < 0 ? -1ll : 0ll) : (n >> (-sh));
}

// ---------------------------------------------------------------------------------------------------------
// Section 4.2: special values of one block.  Returns 0 (all finite), 1 (NaN), 2 (+inf), 3 (-inf).
// ---------------------------------------------------------------------------------------------------------
struct Special {
    bool nan = false, pinf = false, ninf = false;
    __device__ __forceinline__ void add_inf(uint32_t sign) { if (sign) ninf = true; else pinf = true; }
    __device__ __forceinline__ void product(uint32_t x, uint32_t y) {
        const uint32_t cx = dec_cls(x), cy = dec_cls(y);
        if ((cx | cy) == 0u) return;
        if (cx == CLS_NAN || cy == CLS_NAN) { nan = true; return; }
        const uint32_t other = (cx == CLS_INF) ? y : x;
        if (dec_cls(other) == CLS_FINITE && dec_sig(other) == 0u) nan = true;      // inf * 0
        else add_inf(dec_sign(x) ^ dec_sign(y));
    }
    __device__ __forceinline__ void acc(const AccDec& c) {
        if (c.cls == CLS_NAN) nan = true;
        else if (c.cls == CLS_INF) add_inf(c.sign);
    }
    __device__ __forceinline__ int result() const {
        if (nan || (pinf && ninf)) return 1;
        return pinf ? 2 : (ninf ? 3 : 0);
    }
};
__device__ __forceinline__ uint32_t special_word(int kind, bool fp16, bool nvidia_nan) {
    if (kind == 1) return fp16 ? (nvidia_nan ? 0x7FFFu : 0x7E00u) : (nvidia_nan ? 0x7FFFFFFFu : 0x7FC00000u);
    const uint32_t s = (kind == 3);
    return fp16 ? ((s << 15) | 0x7C00u) : ((s << 31) | 0x7F800000u);
}

// ---------------------------------------------------------------------------------------------------------
// Algorithm 7 (T-FDPA) and Algorithm 8 (ST-FDPA: scale_exp = Exp(alpha)+Exp(beta) added to every e_k).
// a, b: decoded elements (stride 1), L of them.  c: accumulator word.  Returns the output word.
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t tfdpa_block(const uint32_t* a, const uint32_t* b, int L, uint32_t c,
                                                const DevModel& m, int scale_exp, bool scale_nan) {
    const bool fp16 = m.acc == ACC_F16;
    const AccDec dc = decode_acc(c, fp16);
    Special sp;
    sp.nan = scale_nan;
    sp.acc(dc);
    // a term whose value is zero has no exponent: it takes no part in the maximum
    constexpr int NO_EXP = -100000;
    // (m.literal_emax: every term takes part, as Algorithm 7 prints it)
    int e_max = (dc.sig || m.literal_emax) ? dc.exp : NO_EXP;
    for (int k = 0; k < L; ++k) {                                   // Step 1 exponents, Step 2 maximum
        sp.product(a[k], b[k]);
        const int ek = ((dec_sig(a[k]) && dec_sig(b[k])) || m.literal_emax) ? dec_exp(a[k]) + dec_exp(b[k]) + scale_exp : NO_EXP;
        e_max = ek > e_max ? ek : e_max;
    }
    const int kind = sp.result();
    if (kind) return special_word(kind, fp16, true);
    if (e_max == NO_EXP) return 0u;                                 // every term is zero
    int64_t S = 0;
    const int F = m.F, frac = m.frac;
    for (int k = 0; k < L; ++k) {                                   // Step 2: align, truncate, add
        const int64_t sk = int64_t(dec_ssig(a[k])) * int64_t(dec_ssig(b[k]));
        const int ek = dec_exp(a[k]) + dec_exp(b[k]) + scale_exp;
        S += rz_scale(sk, (ek - e_max) + F - frac);
    }
    const int64_t sc = dc.sign ? -int64_t(dc.sig) : int64_t(dc.sig);
    S += rz_scale(sc, (dc.exp - e_max) + F - (fp16 ? 10 : 23));
    return rho_apply(m.rho, S, e_max - F);                          // Step 3
}

// ---------------------------------------------------------------------------------------------------------
// Algorithm 9 (GST-FDPA).  a, b: decoded FP4 elements, L of them (L multiple of G = 16).
// sfa, sfb: decoded scale factors for this block (L / k_block of each, at least one).
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t gst_block(const uint32_t* a, const uint32_t* b, int L, uint32_t c,
                                              const DevModel& m, const uint32_t* sfa, const uint32_t* sfb) {
    const AccDec dc = decode_acc(c, false);
    Special sp;
    sp.acc(dc);
    const int nsf = L / m.k_block > 0 ? L / m.k_block : 1;
    for (int j = 0; j < nsf; ++j)
        if (dec_cls(sfa[j]) == CLS_NAN || dec_cls(sfb[j]) == CLS_NAN) sp.nan = true;
    const int kind = sp.result();
    if (kind) return special_word(kind, false, true);
    const int ng = L / m.G;
    int64_t s[4];
    int e[4];
    constexpr int NO_EXP = -100000;                                 // a zero accumulator takes no part in the maximum
    int e_max = (dc.sig || m.literal_emax) ? dc.exp : NO_EXP;
    for (int g = 0; g < ng; ++g) {                                  // Step 1
        int p = 0;                                                  // units of 2^-2 (E2M1: Exp >= 0, 1 mantissa bit)
        bool has_product = false;                                   // some a_k * b_k of the group is nonzero
        for (int k = g * m.G; k < (g + 1) * m.G; ++k) {
            p += (dec_ssig(a[k]) * dec_ssig(b[k])) * (1 << (dec_exp(a[k]) + dec_exp(b[k])));
            has_product |= dec_sig(a[k]) != 0u && dec_sig(b[k]) != 0u;
        }
        const int j = (g * m.G) / m.k_block;
        s[g] = int64_t(p) * int64_t(dec_sig(sfa[j])) * int64_t(dec_sig(sfb[j]));
        e[g] = dec_exp(sfa[j]) + dec_exp(sfb[j]);
        // a group of zero products, or under a zero scale factor, has no exponent; one whose products cancel has
        if ((has_product && dec_sig(sfa[j]) && dec_sig(sfb[j])) || m.literal_emax) e_max = e[g] > e_max ? e[g] : e_max;
    }
    if (e_max == NO_EXP) return 0u;
    int64_t S = 0;
    for (int g = 0; g < ng; ++g) S += rz_scale(s[g], (e[g] - e_max) + m.F - m.frac);   // Step 2
    const int64_t sc = dc.sign ? -int64_t(dc.sig) : int64_t(dc.sig);
    S += rz_scale(sc, (dc.exp - e_max) + m.F - 23);
    return rho_apply(m.rho, S, e_max - m.F);                        // Step 3
}

// ---------------------------------------------------------------------------------------------------------
// Algorithm 10 (TR-FDPA) and Algorithm 11 (GTR-FDPA).  A product of magnitude >= 2^128 is an infinity.
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ bool product_overflows(int sk, int ek, int frac) {
    if (sk == 0) return false;
    const int lim = 128 - ek + frac;                 // |sk| * 2^(ek - frac) >= 2^128  <=>  |sk| >= 2^lim
    if (lim <= 0) return true;
    if (lim >= 31) return false;
    return (sk < 0 ? -sk : sk) >= (1 << lim);
}

__device__ __forceinline__ uint32_t tr_block(const uint32_t* a, const uint32_t* b, int L, uint32_t c,
                                             const DevModel& m, bool grouped) {
    const AccDec dc = decode_acc(c, false);
    Special sp;
    sp.acc(dc);
    int e_grp[2] = {-100000, -100000};
    for (int k = 0; k < L; ++k) {
        sp.product(a[k], b[k]);
        if ((dec_cls(a[k]) | dec_cls(b[k])) == 0u) {
            const int sk = dec_ssig(a[k]) * dec_ssig(b[k]);
            const int ek = dec_exp(a[k]) + dec_exp(b[k]);
            if (product_overflows(sk, ek, m.frac)) sp.add_inf(sk < 0);
            const int g = grouped ? (k & 1) : 0;
            if (sk != 0 || m.literal_emax) e_grp[g] = ek > e_grp[g] ? ek : e_grp[g];  // zero products take no part in the maximum (unless as printed)
        }
    }
    const int kind = sp.result();
    if (kind) return special_word(kind, false, false);
    const int F = m.F, F2 = m.F2, frac = m.frac;
    int64_t T_grp[2] = {0, 0};
    for (int k = 0; k < L; ++k) {                                   // truncated fused sum(s) of the products
        const int64_t sk = int64_t(dec_ssig(a[k])) * int64_t(dec_ssig(b[k]));
        const int ek = dec_exp(a[k]) + dec_exp(b[k]);
        const int g = grouped ? (k & 1) : 0;
        T_grp[g] += rz_scale(sk, (ek - e_grp[g]) + F - frac);
    }
    int e_max;
    int64_t T;
    if (grouped) {                                                  // Algorithm 11, Step 3 (an all-zero group has T = 0)
        e_max = e_grp[0] > e_grp[1] ? e_grp[0] : e_grp[1];
        T = rd_scale(T_grp[0], e_grp[0] - e_max) + rd_scale(T_grp[1], e_grp[1] - e_max);
    } else {
        e_max = e_grp[0];
        T = T_grp[0];
    }
    const int64_t sc = dc.sign ? -int64_t(dc.sig) : int64_t(dc.sig);
    if (e_max == -100000) return rho_apply(m.rho, sc, dc.exp - 23);  // every product is zero: the block returns c (or +0)
    const int E = ((dc.sig || m.literal_emax) && dc.exp > e_max) ? dc.exp : e_max;
    int64_t T2, sc2;
    if (m.inner_round == 1) {                                       // hypothetical RZ variant (Section 6.2.4)
        T2 = rz_scale(T, (e_max - E) + F2 - F);
        sc2 = rz_scale(sc, (dc.exp - E) + F - 23);
    } else {
        T2 = rd_scale(T, (e_max - E) + F2 - F);
        sc2 = rd_scale(sc, (dc.exp - E) + F - 23);
    }
    if (grouped && dc.exp < E - F - 1) sc2 = 0;                     // special truncation
    const int64_t S = T2 + sc2 * (int64_t(1) << (F2 - F));
    return rho_apply(m.rho, S, E - F2);
}

// ---------------------------------------------------------------------------------------------------------
// Algorithm 6 (E-FDPA): RNE-FP32 of the exact sum, through a 640-bit fixed-point accumulator pair.
// Bit i of the accumulator has weight 2^(i - EF_BASE).
// ---------------------------------------------------------------------------------------------------------
constexpr int EF_LIMBS = 20;
constexpr int EF_BASE = 320;

__device__ __forceinline__ void ef_add(uint32_t* acc, uint32_t mag, int pos) {
    // acc += mag * 2^pos (pos = bit index of mag's bit 0), mag < 2^24
    const int limb = pos >> 5, off = pos & 31;
    uint64_t v = uint64_t(mag) << off;
    uint64_t carry = 0;
    for (int i = limb; i < EF_LIMBS && (v | carry); ++i) {
        const uint64_t t = uint64_t(acc[i]) + (v & 0xFFFFFFFFull) + carry;
        acc[i] = uint32_t(t);
        carry = t >> 32;
        v >>= 32;
    }
}

__device__ __forceinline__ uint32_t efdpa_block(const uint32_t* a, const uint32_t* b, int L, uint32_t c,
                                                const DevModel& m) {
    const AccDec dc = decode_acc(c, false);
    Special sp;
    sp.acc(dc);
    for (int k = 0; k < L; ++k) sp.product(a[k], b[k]);
    const int kind = sp.result();
    if (kind) return special_word(kind, false, false);
    // Common case: every term lies inside one 62-bit window, so the exact sum fits a 64-bit integer.
    {
        int lo = 1 << 20, hi = -(1 << 20);              // lowest term bit, highest possible term bit
        for (int k = 0; k < L; ++k) {
            const uint32_t mag = dec_sig(a[k]) * dec_sig(b[k]);
            if (mag) {
                const int e = dec_exp(a[k]) + dec_exp(b[k]) - m.frac;
                lo = e < lo ? e : lo;
                hi = e + 22 > hi ? e + 22 : hi;         // products have at most 22 significant bits
            }
        }
        if (dc.sig) {
            const int e = dc.exp - 23;
            lo = e < lo ? e : lo;
            hi = e + 24 > hi ? e + 24 : hi;
        }
        if (hi < lo) return 0u;                          // every term is zero
        if (hi - lo <= 58) {                             // up to five terms: three carry bits on top
            long long S = 0;
            for (int k = 0; k < L; ++k) {
                const long long sk = (long long)dec_ssig(a[k]) * (long long)dec_ssig(b[k]);
                if (sk) S += sk << (dec_exp(a[k]) + dec_exp(b[k]) - m.frac - lo);
            }
            if (dc.sig) S += (dc.sign ? -(long long)dc.sig : (long long)dc.sig) << (dc.exp - 23 - lo);
            const uint32_t sign = S < 0;
            return round_pack(sign, sign ? (unsigned long long)(-S) : (unsigned long long)S, lo, 8, 23, 127, true);
        }
    }
    uint32_t pos[EF_LIMBS], neg[EF_LIMBS];
    for (int i = 0; i < EF_LIMBS; ++i) pos[i] = neg[i] = 0u;
    for (int k = 0; k < L; ++k) {
        const uint32_t mag = dec_sig(a[k]) * dec_sig(b[k]);
        const int e = dec_exp(a[k]) + dec_exp(b[k]) - m.frac + EF_BASE;
        if (mag) ef_add((dec_sign(a[k]) ^ dec_sign(b[k])) ? neg : pos, mag, e);
    }
    if (dc.sig) ef_add(dc.sign ? neg : pos, dc.sig, dc.exp - 23 + EF_BASE);
    // |pos - neg| and its sign
    int cmp = 0;
    for (int i = EF_LIMBS - 1; i >= 0 && cmp == 0; --i) cmp = (pos[i] > neg[i]) - (pos[i] < neg[i]);
    if (cmp == 0) return 0u;
    const uint32_t* hi = cmp > 0 ? pos : neg;
    const uint32_t* lo = cmp > 0 ? neg : pos;
    uint32_t diff[EF_LIMBS];
    int64_t borrow = 0;
    for (int i = 0; i < EF_LIMBS; ++i) {
        int64_t t = int64_t(hi[i]) - int64_t(lo[i]) - borrow;
        borrow = t < 0;
        diff[i] = uint32_t(t);
    }
    int top = EF_LIMBS - 1;
    while (diff[top] == 0u) --top;
    // take the top three limbs as a 64-bit magnitude (>= 33 significant bits) plus a sticky flag
    uint64_t mag;
    int e;
    bool sticky = false;
    if (top == 0) { mag = diff[0]; e = -EF_BASE; }
    else {
        const int lz = __clz(diff[top]);
        const uint32_t l2 = top >= 2 ? diff[top - 2] : 0u;
        mag = (uint64_t(diff[top]) << 32) | diff[top - 1];
        if (lz) mag = (mag << lz) | (l2 >> (32 - lz));
        const uint32_t dropped = lz ? (l2 << lz) : l2;
        sticky = dropped != 0u;
        for (int i = 0; i < top - 2; ++i) sticky |= diff[i] != 0u;
        e = (top - 1) * 32 - lz - EF_BASE;
    }
    return round_pack(cmp < 0, mag, e, 8, 23, 127, true, sticky);
}

// ---------------------------------------------------------------------------------------------------------
// Algorithm 1: FTZ-Add / FTZ-Mul on the FP32 pipe; IEEE arithmetic, then a sign-preserving flush.
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ float ftz_out(float z) {
    return (fabsf(z) < 1.17549435e-38f) ? copysignf(0.0f, z) : z;      // |z| < 2^-126 (false for NaN)
}
__device__ __forceinline__ float ftz_add(float x, float y) { return ftz_out(__fadd_rn(x, y)); }
__device__ __forceinline__ float ftz_mul(float x, float y) { return ftz_out(__fmul_rn(x, y)); }

}  // namespace mmasim
