// Tuned T-FDPA kernel for 8-bit inputs with F = 13 (the Ada / Hopper FP8 rows; Algorithm 5 + Algorithm 7 + Table 2),
// and the staging code it shares with the TR- / GTR-FDPA kernels (mmasim_trfdpa_fast.cu).  The F >= 23 variants and
// ST-FDPA live in mmasim_tfdpa_f64.cuh.
//
// Work decomposition.  A CTA of 256 threads owns a 128 x 64 tile of D; a thread owns an 8 x 4 micro-tile and keeps
// its 32 accumulators decoded in registers for the whole K loop: `cs`, the one's-complement signed significand
// aligned to F fractional bits, and `ce`, the exponent (biased, see below).  K is walked in chunks of 32 elements:
// the CTA loads the raw A / B words of the chunk, decodes every element once into an operand word and an exponent
// word (8-bit formats through a 256-entry table, 16/32-bit formats arithmetically) and stores them k-major in
// shared memory, so that one 16-byte shared load feeds four rows (or columns) of a micro-tile.
//
// Per block of L elements and per output (Algorithm 7):
//   pass 1   e_max = max(Exp(c), max_k(Exp(a_k) + Exp(b_k)))   fused add-max on two 16-bit lanes: half an
//                                                              instruction per term
//   pass 2   S <- S + floor(X_k * 2^-(d_k + g))                one FP32 fused multiply-add per term (see the kernel)
//   then the accumulator term, the sign corrections, normalisation and rho (Table 2) - about 25 instructions.
//
// Sign-magnitude truncation without per-term sign work.  RZ_F truncates the magnitude of each aligned term, while
// a floor (an arithmetic right shift of a two's-complement number, a multiply-add rounding toward minus infinity)
// rounds down.  Negative terms are therefore carried in one's complement: -t is represented by ~t = -t - 1, and the
// number of negative terms of the block (a population count over per-row / per-column sign bit masks) is added back
// once per block.
//  * 8-bit inputs (FP8 / FP6 / FP4): the operands are built so that the integer product itself has that form,
//      X = s * (m << (F - frac + g)) + r,  m = sig_a * sig_b,  s = +-1 the product's sign,  g = mbits_a + 1 guard
//      bits,  0 <= r < 2^g for s = +1 and -2^g <= r <= -1 for s = -1,
//    by A_op = +-sig_a and B_op = (+-sig_b << (F - frac + g)) + sign(b), which gives r = +-sig_a.  Then
//    floor(X * 2^-(d + g)) is floor(m * 2^(F - frac) / 2^d) for positive terms and its one's complement for negative
//    ones.  A term counts as negative when the signs differ and both significands are nonzero.
//  * 16/32-bit inputs (FP16 / BF16 / TF32, TR-FDPA kernels): magnitudes are multiplied and shifted, and one 3-input
//    logic instruction applies sign_a xor sign_b (full-width masks staged beside the operands).  Every term whose sign
//    bits differ counts as negative.
//
// Exponents are staged with a bias of 512 per element (1024 per product / accumulator) so that they are positive
// 16-bit lane values.  A zero element, like a zero accumulator, has no exponent and must never decide e_max: it is
// staged as the word 0, which keeps every sum it enters below every sum of two real exponents.
//
// Everything that is rare takes a slow, by-the-book route: NaN / infinity inputs (the threads rescan the raw words
// of the block and keep sticky NaN / +inf / -inf flags per output, Section 4.2) and results outside the normal range
// of the accumulator format (generic conversion routine).
#pragma once
#include <cuda_fp16.h>
#include "mmasim_device.cuh"

namespace mmasim {
namespace fast {

constexpr int BM = 128, BN = 64, TM = 8, TN = 4, KC = 32, NT = 256;
constexpr int EB = 512;            // bias of a staged element exponent
constexpr int CB = 2 * EB;         // bias of an exponent sum and of the accumulator exponent
constexpr int FP_SHIFT = 8;        // FP32 summation path: the B operands are scaled by 2^-FP_SHIFT (see pass 2)
constexpr int FP_EMAX_CLAMP = 100; // FP32 summation path: largest e_max + g that the sum register's exponent carries

enum ElemKind : int { EK_LUT8 = 0, EK_F16 = 1, EK_BF16 = 2, EK_TF32 = 3 };

template <int EK> struct Elem;
template <> struct Elem<EK_LUT8> { static constexpr int BYTES = 1, TASK = 16, EBITS = 4, MBITS = 3, BIAS = 7, LOW = 0; static constexpr bool SIGNMAG = false; };  // EBITS.. unused: table-decoded
template <> struct Elem<EK_F16> { static constexpr int BYTES = 2, TASK = 8, EBITS = 5, MBITS = 10, BIAS = 15, LOW = 0; static constexpr bool SIGNMAG = true; };
template <> struct Elem<EK_BF16> { static constexpr int BYTES = 2, TASK = 8, EBITS = 8, MBITS = 7, BIAS = 127, LOW = 0; static constexpr bool SIGNMAG = true; };
template <> struct Elem<EK_TF32> { static constexpr int BYTES = 4, TASK = 8, EBITS = 8, MBITS = 10, BIAS = 127, LOW = 13; static constexpr bool SIGNMAG = true; };

struct LutEntry {
    uint32_t op;        // multiplier operand
    uint32_t exp;       // Exp(x) + EB; 0 for zero, infinity and NaN (no exponent)
    uint32_t bits;      // bit 0: sign, bit 16: finite and nonzero
    uint32_t special;   // nonzero for infinity / NaN
};

// Staged operands of one chunk (8-bit element kinds; the 16/32-bit kinds are staged by mmasim_tfdpa_f64.cuh).
template <int EK>
struct Planes {
    uint32_t a_op[KC][BM];          // FP32 words: A_op * 2^Exp(a)
    uint32_t b_op[KC][BN];          // FP32 words: B_op * 2^(Exp(b) - FP_SHIFT)
    uint32_t a_exp2[KC / 2][BM];    // exponents of elements 2p (low half) and 2p + 1 (high half)
    uint32_t b_exp2[KC / 2][BN];
    uint32_t a_sgn[BM], a_nz[BM], b_sgn[BN], b_nz[BN];   // bit k of row r: sign / nonzero of element k of the chunk
};

template <int EK, int NBUF = 2>
struct Smem {
    Planes<EK> pl[NBUF];
    LutEntry lut_a[256];
    LutEntry lut_b[256];
    int special[3];                                   // chunk (by index mod 3) holds an infinity or a NaN
};

__device__ __forceinline__ int asr_clamp(int x, int d) {
    int r;
    asm("shr.s32 %0, %1, %2;" : "=r"(r) : "r"(x), "r"(d));      // amounts above 31 behave as 31 (sign fill)
    return r;
}
__device__ __forceinline__ uint32_t shl_clamp(uint32_t x, int d) {
    uint32_t r;
    asm("shl.b32 %0, %1, %2;" : "=r"(r) : "r"(x), "r"(d));      // amounts above 31 give 0
    return r;
}
__device__ __forceinline__ int msb_index(uint32_t x) {
    int r;
    asm("bfind.u32 %0, %1;" : "=r"(r) : "r"(x));                // -1 for x == 0
    return r;
}
// Accumulator state of one output.
struct Acc {
    int cs;     // one's complement signed significand, F fractional bits relative to 2^(ce - CB)
    int ce;     // Exp(c) + CB; 0 for c = 0
};

template <int F, bool ACC16>
__device__ __forceinline__ Acc acc_from_word(uint32_t w, uint32_t& sp) {
    static_assert(F >= (ACC16 ? 10 : 13), "accumulator significand must not lose bits beyond rho");
    const AccDec d = decode_acc(w, ACC16);
    Acc a;
    if (d.cls != CLS_FINITE) {
        sp |= (d.cls == CLS_NAN) ? 1u : (d.sign ? 4u : 2u);
        a.cs = 0;
        a.ce = 0;
        return a;
    }
    constexpr int MB = ACC16 ? 10 : 23;
    // F < 23 (F = 13): the low bits of an FP32 c fall below every block's truncation point anyway
    const int mag = (F >= MB) ? int(d.sig << (F >= MB ? F - MB : 0)) : int(d.sig >> (F >= MB ? 0 : MB - F));
    a.cs = d.sign ? ~mag : mag;
    a.ce = d.sig ? d.exp + CB : 0;      // a zero accumulator has no exponent: 0 never wins the block maximum
    return a;
}

// Accumulator state back to an output word (exact: the state always holds a representable value).
template <int F, bool ACC16>
__device__ __forceinline__ uint32_t acc_to_word(const Acc& a, uint32_t sp) {
    if (sp) {
        const int kind = ((sp & 1u) || (sp & 6u) == 6u) ? 1 : ((sp & 2u) ? 2 : 3);
        return special_word(kind, ACC16, true);
    }
    constexpr int MB = ACC16 ? 10 : 23;
    const uint32_t sign = a.cs < 0;
    const uint32_t magF = uint32_t(sign ? ~a.cs : a.cs);
    const uint32_t sig = (F >= MB) ? (magF >> (F >= MB ? F - MB : 0)) : (magF << (F >= MB ? 0 : MB - F));
    const uint32_t field = (sig >> MB) ? uint32_t(a.ce - CB + (ACC16 ? 15 : 127)) : 0u;
    return (sign << (ACC16 ? 15 : 31)) | (field << MB) | (sig & ((1u << MB) - 1u));
}

// Slow conversion: any rho, any range.  S is the exact fixed-point sum in units of 2^(e_max - F).
template <int F, int RHO, bool ACC16>
__device__ __noinline__ void rho_slow(long long S, int e_max, Acc& a, uint32_t& sp) {
    const uint32_t w = rho_apply(RHO, S, e_max - F);
    a = acc_from_word<F, ACC16>(w, sp);
}

// Fast conversion of a 32-bit block sum whose result is a normal number (or zero); `vmin` / `vmax` collect the result
// exponents so that the caller can detect, once per block, that some output left the normal range.
template <int F, int RHO>
__device__ __forceinline__ void rho_fast(int S, int emaxb, Acc& a, int& vmin, int& vmax) {
    constexpr bool ACC16 = RHO == RHO_RNE_FP16;
    constexpr bool RNE = RHO == RHO_RNE_FP16 || RHO == RHO_RNE_FP32;
    constexpr int MB = RHO == RHO_RZ_E8M13 ? 13 : (ACC16 ? 10 : 23);
    constexpr int EMINB = (ACC16 ? -14 : -126) + CB;
    const int sg = S >> 31;
    const uint32_t mag = uint32_t(abs(S));
    const int msb = msb_index(mag);
    const uint32_t norm = shl_clamp(mag, 31 - msb);            // leading one at bit 31 (msb <= 30, so bit 0 is free)
    uint32_t sig;
    int ve = emaxb - F + msb;
    if (RNE) {
        const uint32_t n2 = norm >> 1;
        const uint32_t r = (n2 + (((1u << (29 - MB)) - 1u) + ((n2 >> (30 - MB)) & 1u))) >> (30 - MB);
        const uint32_t carry = r >> (MB + 1);
        sig = r >> carry;
        ve += int(carry);
    } else {
        sig = norm >> (31 - MB);
    }
    ve = mag ? ve : EMINB;                                     // an exactly zero sum is +0
    vmin = min(vmin, ve);
    vmax = max(vmax, ve);
    a.ce = mag ? ve : 0;
    a.cs = int(sig << (F - MB)) ^ sg;
}

template <int EK>
__device__ __forceinline__ uint32_t raw_elem(const void* p, int64_t idx) {
    if (Elem<EK>::BYTES == 1) return static_cast<const uint8_t*>(p)[idx];
    if (Elem<EK>::BYTES == 2) return static_cast<const uint16_t*>(p)[idx];
    return static_cast<const uint32_t*>(p)[idx];
}

// Arithmetic decode of one FP16 / BF16 / TF32 word: significand, biased exponent, sign, special flag.
template <int EK>
__device__ __forceinline__ void decode_signmag(uint32_t w, uint32_t& sig, uint32_t& expb, uint32_t& sign, uint32_t& special) {
    using E = Elem<EK>;
    const uint32_t x = w >> E::LOW;
    const uint32_t mant = x & ((1u << E::MBITS) - 1u);
    const uint32_t field = (x >> E::MBITS) & ((1u << E::EBITS) - 1u);
    sign = (x >> (E::MBITS + E::EBITS)) & 1u;
    special = field == ((1u << E::EBITS) - 1u);
    sig = special ? 0u : (mant | (field ? (1u << E::MBITS) : 0u));
    // a zero (and the stand-in of an infinity or NaN) has no exponent: the word 0 lies below every real exponent sum
    expb = sig ? uint32_t(int(field ? field : 1u) - E::BIAS + EB) : 0u;
}

// Decode tables of the 8-bit kinds: entry `tid` of both (256 threads).  The staged operands are the floating-point
// form of the integer operands of the header comment: the operand scaled by 2^Exp, exact in FP32 (at most 4 + 15
// significant bits, exponents far inside the FP32 range).  A zero b is staged as 0 (its terms vanish and are not
// counted as negative): with the zero terms outside e_max nothing bounds sig_a * 2^(Exp(a) + Exp_min(b)) below one
// unit of the sum.
template <int EK, class SM>
__device__ __forceinline__ void init_lut(SM& s, const FmtDesc& fa, const FmtDesc& fb, int pre, int guard, int tid) {
    const uint32_t da = decode_elem(fa, uint32_t(tid)), db = decode_elem(fb, uint32_t(tid));
    const bool fin_a = dec_cls(da) == CLS_FINITE, fin_b = dec_cls(db) == CLS_FINITE;
    const bool nz_a = fin_a && dec_sig(da) != 0u, nz_b = fin_b && dec_sig(db) != 0u;
    LutEntry ea, eb;
    ea.op = __float_as_uint(ldexpf(float(fin_a ? dec_ssig(da) : 0), fin_a ? dec_exp(da) : 0));
    ea.exp = nz_a ? uint32_t(dec_exp(da) + EB) : 0u;             // zero, infinity, NaN: no exponent
    ea.bits = fin_a ? (dec_sign(da) | (uint32_t(nz_a) << 16)) : 0u;
    ea.special = fin_a ? 0u : 1u;
    const int sb = fin_b ? dec_ssig(db) : 0;
    const int ub = dec_sign(db) ? -1 : 1;
    eb.op = nz_b ? __float_as_uint(ldexpf(float(sb * (1 << (pre + guard)) + ub), dec_exp(db) - FP_SHIFT)) : 0u;
    eb.exp = nz_b ? uint32_t(dec_exp(db) + EB) : 0u;
    eb.bits = fin_b ? (dec_sign(db) | (uint32_t(nz_b) << 16)) : 0u;
    eb.special = fin_b ? 0u : 1u;
    s.lut_a[tid] = ea;
    s.lut_b[tid] = eb;
}

// Staging of one chunk of KC elements of K, in two steps so that the global loads of the next chunk can be in flight
// while the current one is being computed: (1) every task loads E::TASK consecutive raw elements of one row of A or B
// into registers, (2) it decodes them into operand / exponent (/ sign mask) words, k-major in shared memory, plus the
// row's sign and nonzero bit masks.
template <int EK>
struct RawChunk {
    static constexpr int TPR = KC / Elem<EK>::TASK;                              // tasks per row
    static constexpr int TASKS = (BM + BN) * TPR;
    static constexpr int PER_THREAD = (TASKS + NT - 1) / NT;
    static constexpr int WORDS = Elem<EK>::TASK * Elem<EK>::BYTES / 4;           // 32-bit words per task
    uint32_t w[PER_THREAD][WORDS];
};

template <int EK>
__device__ __forceinline__ void load_chunk(RawChunk<EK>& raw, const GemmArgs& g, int64_t row0, int64_t col0, int64_t k0, int tid) {
    using E = Elem<EK>;
    using R = RawChunk<EK>;
#pragma unroll
    for (int it = 0; it < R::PER_THREAD; ++it) {
        const int task = it * NT + tid;
        const bool is_a = task < BM * R::TPR;
        const int u = is_a ? task : task - BM * R::TPR;
        const int rows = is_a ? BM : BN;
        const int r = u % rows, h = u / rows;              // consecutive threads take consecutive rows
        const int64_t grow = (is_a ? row0 : col0) + r;
        const bool valid = task < R::TASKS && grow < (is_a ? g.M : g.N);
        const unsigned char* base = static_cast<const unsigned char*>(is_a ? g.A : g.B) +
                                    (grow * (is_a ? g.lda : g.ldb) + k0 + h * E::TASK) * E::BYTES;
#pragma unroll
        for (int q = 0; q < R::WORDS / 4; ++q) {
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (valid) v = reinterpret_cast<const uint4*>(base)[q];
            raw.w[it][4 * q] = v.x; raw.w[it][4 * q + 1] = v.y; raw.w[it][4 * q + 2] = v.z; raw.w[it][4 * q + 3] = v.w;
        }
    }
}

template <int EK, class SM, class PL>
__device__ __forceinline__ void store_chunk(SM& sm, PL& s, const RawChunk<EK>& raw, int flag, int tid) {
    using E = Elem<EK>;
    using R = RawChunk<EK>;
    static_assert(!E::SIGNMAG && E::TASK == 16, "table-decoded 8-bit elements, sixteen per task");
    uint32_t spec = 0u;
#pragma unroll
    for (int it = 0; it < R::PER_THREAD; ++it) {
        const int task = it * NT + tid;
        if (task >= R::TASKS) break;
        const bool is_a = task < BM * R::TPR;
        const int u = is_a ? task : task - BM * R::TPR;
        const int rows = is_a ? BM : BN;
        const int r = u % rows, h = u / rows;
        uint32_t bits = 0u, prev_exp = 0u;
#pragma unroll
        for (int q = 0; q < E::TASK; ++q) {
            const int kk = h * E::TASK + q;
            const uint32_t byte = (raw.w[it][q / 4] >> (8 * (q % 4))) & 0xFFu;
            const LutEntry e = is_a ? sm.lut_a[byte] : sm.lut_b[byte];
            bits += e.bits << q;
            spec |= e.special;
            if (is_a) s.a_op[kk][r] = e.op; else s.b_op[kk][r] = e.op;
            if (q & 1) {
                const uint32_t pair = prev_exp | (e.exp << 16);
                if (is_a) s.a_exp2[kk / 2][r] = pair; else s.b_exp2[kk / 2][r] = pair;
            }
            prev_exp = e.exp;
        }
        // sign and nonzero bits of the task's elements go to bits [h * 16, h * 16 + 16) of the row's masks
        if (is_a) {
            reinterpret_cast<uint16_t*>(&s.a_sgn[r])[h] = uint16_t(bits);
            reinterpret_cast<uint16_t*>(&s.a_nz[r])[h] = uint16_t(bits >> 16);
        } else {
            reinterpret_cast<uint16_t*>(&s.b_sgn[r])[h] = uint16_t(bits);
            reinterpret_cast<uint16_t*>(&s.b_nz[r])[h] = uint16_t(bits >> 16);
        }
    }
    if (spec) atomicOr(&sm.special[flag], 1);
}

template <int EK, int L, int F, int RHO, bool PROMOTE>
__global__ void __launch_bounds__(NT, 2) tfdpa_kernel(DevModel m, GemmArgs g) {
    constexpr bool ACC16 = RHO == RHO_RNE_FP16;
    constexpr int NBLK = KC / L;
    static_assert(KC % L == 0 && L % 2 == 0, "blocks tile the chunk; pass 1 handles pairs of elements");
    // FP32 summation: aligned terms stay below 2^15 and block sums below 2^21, so the whole of pass 2 runs exactly on
    // the FP32 pipe, one instruction per term (see pass 2 below).  The staged planes are small enough for two buffers:
    // the next chunk is decoded while the current one is computed, one barrier per chunk.
    static_assert(!Elem<EK>::SIGNMAG && F <= 13, "8-bit inputs with F <= 13; F >= 23 and ST-FDPA run in mmasim_tfdpa_f64.cuh");
    static_assert(RHO == RHO_RZ_E8M13 || RHO == RHO_RNE_FP16, "rho of the F = 13 rows of Table 4");
    using SM = Smem<EK, 2>;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SM& sm = *reinterpret_cast<SM*>(smem_raw);

    const int tid = threadIdx.x;
    const int tx = tid % 16, ty = tid / 16;
    const int64_t row0 = int64_t(blockIdx.y) * BM, col0 = int64_t(blockIdx.x) * BN;
    const FmtDesc fa = fmt_desc(m.fmt_a), fb = fmt_desc(m.fmt_b);
    const int pre = F - (fa.mbits + fb.mbits);      // left shift that gives a product F fractional bits
    const int guard = fa.mbits + 1;                 // guard bits below the truncation point
    // The staged operands carry the products in the scale 2^(F + g - FP_SHIFT): a real value x appears as x * c_scale.
    const float c_scale = __int_as_float((127 + F + guard - FP_SHIFT) << 23);
    // Exponent sums outside [E_LOW, E_HIGH] (biased by CB) are blocks whose products cannot reach the result: below,
    // every product is zero (a nonzero FP8 product has an exponent of at least -28); above, only an accumulator of
    // 2^100 or more gets there and every product is truncated away.  The result is then the accumulator itself,
    // truncated by rho; the sum register's exponent is clamped so that the arithmetic stays finite.
    constexpr int E_LOW = CB - 100, E_HIGH = CB + FP_EMAX_CLAMP;

    init_lut<EK>(sm, fa, fb, pre, guard, tid);
    if (tid == 0) sm.special[0] = sm.special[1] = sm.special[2] = 0;

    uint32_t cw[TM][TN];                                // the accumulator of each output: a finite FP32 / FP16 word
    uint32_t sp_nan = 0u, sp_pinf = 0u, sp_ninf = 0u;   // per output (bit r * TN + c): NaN / +inf / -inf seen so far
    float promoted[PROMOTE ? TM : 1][PROMOTE ? TN : 1];
#define MMASIM_SP_GET(r, c) ((((sp_nan >> ((r) * TN + (c))) & 1u)) | (((sp_pinf >> ((r) * TN + (c))) & 1u) << 1) | (((sp_ninf >> ((r) * TN + (c))) & 1u) << 2))
#define MMASIM_SP_WORD(r, c, w) (MMASIM_SP_GET(r, c) ? special_word(((MMASIM_SP_GET(r, c) & 1u) || (MMASIM_SP_GET(r, c) & 6u) == 6u) ? 1 : ((MMASIM_SP_GET(r, c) & 2u) ? 2 : 3), ACC16, true) : (w))
#pragma unroll
    for (int r = 0; r < TM; ++r)
#pragma unroll
        for (int c = 0; c < TN; ++c) {
            const int64_t i = row0 + ty * TM + r, j = col0 + tx * TN + c;
            uint32_t w = 0u;
            if (g.C && i < g.M && j < g.N)
                w = ACC16 ? uint32_t(static_cast<const uint16_t*>(g.C)[i * g.ldc + j])
                          : static_cast<const uint32_t*>(g.C)[i * g.ldc + j];
            if (PROMOTE) { promoted[PROMOTE ? r : 0][PROMOTE ? c : 0] = __uint_as_float(w); w = 0u; }
            const AccDec d = decode_acc(w, ACC16);
            if (d.cls != CLS_FINITE) {
                const uint32_t bit = 1u << (r * TN + c);
                if (d.cls == CLS_NAN) sp_nan |= bit; else if (d.sign) sp_ninf |= bit; else sp_pinf |= bit;
                w = 0u;
            }
            cw[r][c] = w;
        }

    RawChunk<EK> raw;
    load_chunk<EK>(raw, g, row0, col0, 0, tid);
    __syncthreads();                                       // tables and flags are ready
    store_chunk<EK>(sm, sm.pl[0], raw, 0, tid);
    if (KC < g.K) load_chunk<EK>(raw, g, row0, col0, KC, tid);
    __syncthreads();
    int chunk = 0;
    for (int64_t k0 = 0; k0 < g.K; k0 += KC, ++chunk) {
        // decode chunk n + 1 into the other buffer (its raw words arrived during the previous iteration), then fetch n + 2
        if (tid == 0) sm.special[(chunk + 2) % 3] = 0;     // last read two barriers ago, next written after the coming one
        if (k0 + KC < g.K) {
            store_chunk<EK>(sm, sm.pl[(chunk + 1) & 1], raw, (chunk + 1) % 3, tid);
            if (k0 + 2 * KC < g.K) load_chunk<EK>(raw, g, row0, col0, k0 + 2 * KC, tid);
        }
        auto& s = sm.pl[chunk & 1];
        const bool chunk_special = sm.special[chunk % 3] != 0;

#pragma unroll 1
        for (int blk = 0; blk < NBLK; ++blk) {
            const int kb = blk * L;
            // ---- rare: the chunk holds an infinity or a NaN: special-value events of this block (Section 4.2).
            // Flags are sticky: once an output is special the finite arithmetic below no longer matters for it.
            if (chunk_special) {
#pragma unroll 1
                for (int r = 0; r < TM; ++r)
#pragma unroll 1
                    for (int c = 0; c < TN; ++c) {
                        const int64_t i = row0 + ty * TM + r, j = col0 + tx * TN + c;
                        if (i >= g.M || j >= g.N) continue;
                        Special ev;
                        for (int kk = kb; kk < kb + L; ++kk) {
                            const uint32_t x = decode_elem(fa, raw_elem<EK>(g.A, i * g.lda + k0 + kk));
                            const uint32_t y = decode_elem(fb, raw_elem<EK>(g.B, j * g.ldb + k0 + kk));
                            ev.product(x, y);
                        }
                        const uint32_t bit = 1u << (r * TN + c);
                        if (ev.nan) sp_nan |= bit;
                        if (ev.pinf) sp_pinf |= bit;
                        if (ev.ninf) sp_ninf |= bit;
                    }
            }

            int S0[TM][TN];         // pass 1: e_max + CB; pass 2: the sum register; then the result word
            int elo = E_HIGH, ehi = E_LOW;
            // ---- pass 1: block maximum of the exponent sums, accumulator included (a zero accumulator has no
            // exponent: 0 never wins); two elements per instruction ----
            {
                uint32_t em2[TM][TN];
#pragma unroll
                for (int r = 0; r < TM; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c) {
                        const uint32_t x = cw[r][c] & (ACC16 ? 0x7FFFu : 0x7FFFFFFFu);
                        const uint32_t rel = max(x >> (ACC16 ? 10 : 23), 1u) + uint32_t(CB - (ACC16 ? 15 : 127));
                        em2[r][c] = x ? rel * 0x10001u : 0u;
                    }
#pragma unroll 4
                for (int kp = kb / 2; kp < (kb + L) / 2; ++kp) {
                    const uint4 ea0 = *reinterpret_cast<const uint4*>(&s.a_exp2[kp][ty * TM]);
                    const uint4 ea1 = *reinterpret_cast<const uint4*>(&s.a_exp2[kp][ty * TM + 4]);
                    const uint4 eb = *reinterpret_cast<const uint4*>(&s.b_exp2[kp][tx * TN]);
                    const uint32_t ea[TM] = {ea0.x, ea0.y, ea0.z, ea0.w, ea1.x, ea1.y, ea1.z, ea1.w};
                    const uint32_t ebv[TN] = {eb.x, eb.y, eb.z, eb.w};
#pragma unroll
                    for (int r = 0; r < TM; ++r)
#pragma unroll
                        for (int c = 0; c < TN; ++c) em2[r][c] = __viaddmax_s16x2(ea[r], ebv[c], em2[r][c]);
                }
#pragma unroll
                for (int r = 0; r < TM; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c) {
                        const int e = max(int(em2[r][c] & 0xFFFFu), int(em2[r][c] >> 16));
                        elo = min(elo, e);
                        ehi = max(ehi, e);
                        S0[r][c] = e;
                    }
            }
            uint32_t keep = 0u;                            // outputs whose products cannot reach the result (rare)
            if (elo < E_LOW || ehi > E_HIGH) {
#pragma unroll
                for (int r = 0; r < TM; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c)
                        if (S0[r][c] < E_LOW || S0[r][c] > E_HIGH) keep |= 1u << (r * TN + c);
            }
            // ---- the sum register: (1.5 * 2^23 + S) * u in FP32, u = 2^(e_max + g - FP_SHIFT) the value of one unit
            // of S in the scale of the staged operands: in [2^23 u, 2^24 u) one ulp is u, so adding a product with
            // rounding toward minus infinity floors it onto the grid of S.  It starts with the accumulator term:
            // c' = c with the lowest mantissa bit set is never on the grid, so a negative c floors to the one's
            // complement of its truncated magnitude (+1 for the sign in the correction below). ----
#pragma unroll
            for (int r = 0; r < TM; ++r)
#pragma unroll
                for (int c = 0; c < TN; ++c) {
                    const int ecl = max(min(S0[r][c], E_HIGH), E_LOW) + guard;
                    const float magic = __int_as_float(((ecl + (150 - CB - FP_SHIFT)) << 23) | 0x00400000);
                    const float cf = ACC16 ? __half2float(__ushort_as_half((unsigned short)cw[r][c])) : __uint_as_float(cw[r][c]);
                    S0[r][c] = __float_as_int(__fmaf_rd(__int_as_float(__float_as_int(cf) | 1), c_scale, magic));
                }
            // ---- pass 2: S * u + (A_op * 2^Exp(a)) * (B_op * 2^(Exp(b) - FP_SHIFT)) = (S + X_k * 2^-(d_k + g)) * u: the
            // fused multiply-add forms it exactly and rounds once, toward minus infinity, onto multiples of u:
            // S <- S + floor(X_k * 2^-(d_k + g)), the one's-complement term of the header comment.  One instruction per
            // term; the alignment scale is the exponent of the sum register. ----
#pragma unroll 4
            for (int kk = kb; kk < kb + L; ++kk) {
                const float4 oa0 = *reinterpret_cast<const float4*>(&s.a_op[kk][ty * TM]);
                const float4 oa1 = *reinterpret_cast<const float4*>(&s.a_op[kk][ty * TM + 4]);
                const float4 ob = *reinterpret_cast<const float4*>(&s.b_op[kk][tx * TN]);
                const float oav[TM] = {oa0.x, oa0.y, oa0.z, oa0.w, oa1.x, oa1.y, oa1.z, oa1.w};
                const float obv[TN] = {ob.x, ob.y, ob.z, ob.w};
#pragma unroll
                for (int r = 0; r < TM; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c)
                        S0[r][c] = __float_as_int(__fmaf_rd(oav[r], obv[c], __int_as_float(S0[r][c])));
            }
            // ---- sign corrections and rho: S = register - constant + (negative terms) + (c < 0), value S * 2^(e_max - F)
            // (exact in FP32: |S| < 2^22), then RZ-E8M13 = the low 10 mantissa bits cleared, or RNE-FP16 = one
            // conversion.  The scale is read from the register's exponent field. ----
            const uint32_t kmask = (L == 32) ? 0xFFFFFFFFu : (((1u << L) - 1u) << kb);
            uint32_t wmax = 0u;
#pragma unroll
            for (int r = 0; r < TM; ++r) {
                const uint32_t sa = s.a_sgn[ty * TM + r];
                const uint32_t nza = s.a_nz[ty * TM + r] & kmask;
#pragma unroll
                for (int c = 0; c < TN; ++c) {
                    const int nneg = __popc((sa ^ s.b_sgn[tx * TN + c]) & nza & s.b_nz[tx * TN + c]);
                    const int bits = S0[r][c];
                    const int fld = bits & 0x7F800000;
                    const int S = bits - (fld | 0x00400000) + nneg + int(cw[r][c] >> (ACC16 ? 15 : 31));
                    const float scale = __int_as_float(fld - ((15 + F + guard) << 23));       // 2^(e_max - F)
                    const float v = __fmul_rn(__int2float_rn(S), scale);
                    uint32_t w;
                    if (ACC16) { w = uint32_t(__half_as_ushort(__float2half_rn(v))); wmax = max(wmax, w & 0x7FFFu); }
                    else w = __float_as_uint(v) & 0xFFFFFC00u;
                    S0[r][c] = int(w);
                }
            }
            if (keep) {                                    // rare: rho of the accumulator alone; an exactly zero sum is +0
#pragma unroll
                for (int r = 0; r < TM; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c)
                        if ((keep >> (r * TN + c)) & 1u) {
                            const uint32_t t = ACC16 ? cw[r][c] : (cw[r][c] & 0xFFFFFC00u);
                            S0[r][c] = int((t & (ACC16 ? 0x7FFFu : 0x7FFFFFFFu)) ? t : 0u);
                        }
            }
            if (ACC16 && wmax >= 0x7C00u) {                // rare: RNE-FP16 overflowed: +-infinity from now on
#pragma unroll
                for (int r = 0; r < TM; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c)
                        if ((uint32_t(S0[r][c]) & 0x7FFFu) == 0x7C00u) {
                            const uint32_t bit = 1u << (r * TN + c);
                            if (!((sp_nan | sp_pinf | sp_ninf) & bit)) { if (uint32_t(S0[r][c]) >> 15) sp_ninf |= bit; else sp_pinf |= bit; }
                            S0[r][c] = 0;
                        }
            }
#pragma unroll
            for (int r = 0; r < TM; ++r)
#pragma unroll
                for (int c = 0; c < TN; ++c) cw[r][c] = uint32_t(S0[r][c]);
        }
        __syncthreads();                                   // the other buffer is complete, this one is free
        // ---- FP32 promotion of the partial sum every k_chunk elements ----
        if (PROMOTE && ((k0 + KC) % g.k_chunk) == 0) {
#pragma unroll
            for (int r = 0; r < TM; ++r)
#pragma unroll
                for (int c = 0; c < TN; ++c) {
                    const float part = __uint_as_float(MMASIM_SP_WORD(r, c, cw[r][c]));
                    float v = __fadd_rn(promoted[PROMOTE ? r : 0][PROMOTE ? c : 0], part);
                    if (v != v) v = __uint_as_float(0x7FFFFFFFu);
                    promoted[PROMOTE ? r : 0][PROMOTE ? c : 0] = v;
                    cw[r][c] = 0u;
                }
            sp_nan = sp_pinf = sp_ninf = 0u;
        }
    }

    // ---- store ----
#pragma unroll
    for (int r = 0; r < TM; ++r)
#pragma unroll
        for (int c = 0; c < TN; ++c) {
            const int64_t i = row0 + ty * TM + r, j = col0 + tx * TN + c;
            if (i >= g.M || j >= g.N) continue;
            uint32_t w = PROMOTE ? __float_as_uint(promoted[PROMOTE ? r : 0][PROMOTE ? c : 0]) : MMASIM_SP_WORD(r, c, cw[r][c]);
            if (g.row_scale) {
                float sc = __fmul_rn(g.row_scale[i], g.col_scale[j]);
                if (sc != sc) sc = __uint_as_float(0x7FFFFFFFu);
                float v = __fmul_rn(sc, __uint_as_float(w));
                if (v != v) v = __uint_as_float(0x7FFFFFFFu);
                w = __float_as_uint(v);
            }
            if (ACC16) static_cast<uint16_t*>(g.D)[i * g.ldd + j] = uint16_t(w);
            else static_cast<uint32_t*>(g.D)[i * g.ldd + j] = w;
        }
#undef MMASIM_SP_GET
#undef MMASIM_SP_WORD
}

template <int EK, int L, int F, int RHO, bool PROMOTE>
cudaError_t launch_one(const DevModel& m, const GemmArgs& g, cudaStream_t stream) {
    const size_t sh = sizeof(Smem<EK, 2>);
    cudaError_t err = cudaFuncSetAttribute(tfdpa_kernel<EK, L, F, RHO, PROMOTE>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(sh));
    if (err != cudaSuccess) return err;
    dim3 grid((unsigned)((g.N + BN - 1) / BN), (unsigned)((g.M + BM - 1) / BM), 1);
    tfdpa_kernel<EK, L, F, RHO, PROMOTE><<<grid, NT, sh, stream>>>(m, g);
    return cudaGetLastError();
}

// With or without FP32 promotion (FP32 accumulators only).
template <int EK, int L, int F, int RHO>
cudaError_t launch_variant(const DevModel& m, const GemmArgs& g, cudaStream_t stream) {
    if (RHO != RHO_RNE_FP16 && g.k_chunk) return launch_one<EK, L, F, RHO, RHO != RHO_RNE_FP16>(m, g, stream);
    return launch_one<EK, L, F, RHO, false>(m, g, stream);
}

// Per element kind: returns cudaErrorInvalidValue when (L, F, rho) has no instantiation.
cudaError_t launch_lut8(const DevModel& m, const GemmArgs& g, cudaStream_t stream);
cudaError_t launch_f16(const DevModel& m, const GemmArgs& g, cudaStream_t stream);
cudaError_t launch_bf16(const DevModel& m, const GemmArgs& g, cudaStream_t stream);
cudaError_t launch_tf32(const DevModel& m, const GemmArgs& g, cudaStream_t stream);
cudaError_t launch_tr(const DevModel& m, const GemmArgs& g, cudaStream_t stream);    // TR-/GTR-FDPA (mmasim_trfdpa_f64.cu)

}  // namespace fast
}  // namespace mmasim
