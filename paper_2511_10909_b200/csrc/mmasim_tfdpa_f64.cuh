// T-FDPA / ST-FDPA (Algorithms 5, 7, 8 + Table 2) for GEMM-sized inputs with the fused summation on the FP64 pipe.
// Used for every variant with F >= 23 (FP16 / BF16 / TF32 inputs on all NVIDIA generations, the Blackwell FP8 / FP6 /
// FP4 and MX rows); F = 13 has its own FP32 form in mmasim_tfdpa_fast.cuh.
//
// One fused multiply-add per term.  Within a block every aligned, truncated term is a multiple of q = 2^(e_max - F),
// and the block sum S * q stays below 2^33 * q.  The accumulator register of an output holds
//     acc = 1.5 * 2^52 * q  +  S * q                                   (a double in [2^52 q, 2^53 q): one ulp = q)
// so that `acc = fma.rm.f64(a_k, b_k, acc)` computes a_k * b_k + acc exactly and rounds it once, toward minus infinity,
// onto the grid of q: S <- S + floor(a_k b_k / q).  The alignment shift by e_max - e_k, the truncation and the
// addition of Algorithm 7 are that single rounding; the per-output scale lives in the accumulator's exponent field and
// costs nothing per term.  The operands are the element values themselves as doubles (exact), staged once per CTA.
//
// RZ_F is sign-magnitude truncation, floor is not: negative terms are made to floor to the one's complement
// -floor(|x|) - 1 of the wanted value by an offset far below the term's own granularity but never zero: the staged
// B operand is b + sign(b) * 2^(Exp(b) - mbits_b - 30).  Every nonzero term whose sign bits differ then floors to
// -floor(|x|) - 1, every other term to floor(|x|), and the number of nonzero sign-differing terms of the block, a
// population count over per-row / per-column sign and nonzero bit masks, is added back once per block, as an integer
// added to the bit pattern of acc.  The accumulator operand c gets the same treatment: its double has bit 0 of the
// mantissa set.  Zero elements (and the stand-ins of infinities and NaNs) are staged as 0: their products vanish.
//
// A term whose value is zero has no exponent and takes no part in e_max: zero elements are staged with the exponent
// word 0, far below every real exponent sum, and a zero c enters the maximum as 0 as well.
//
// rho (Table 2): the accumulator lives between blocks as a double.  RZ-FP32 of a result in the normal range is a mask on
// the double's low word; RNE-FP16 is cvt.rn.f16.f64 and the half converted back.  Zero, subnormal and overflowing results
// are found by one range check on the exponent field and take a rare path (cvt.rz.f32.f64 keeps subnormals; a magnitude of
// 2^128 or more, or a half that rounded to infinity, becomes a sticky infinity).
// e_max is computed as in the integer kernels (fused add-max on two 16-bit lanes); NaN / infinity inputs use the same
// sticky flags and rescan of the raw words (Section 4.2): their staged operands are the zero stand-ins.
#pragma once
#include <cuda_fp16.h>
#include <type_traits>
#include "mmasim_tfdpa_fast.cuh"

namespace mmasim {
namespace fast64 {

using fast::BM;
using fast::BN;
using fast::KC;
using fast::EB;
using fast::CB;
using fast::Elem;
using fast::raw_elem;

// 512 threads own the 128 x 64 tile of D, 4 x 4 outputs each (a warp: 32 x 16, the accumulator tiles of eight FP64 matrix
// instructions): sixteen warps per SM keep the FP64 pipe fed while the per-thread state (accumulators, product exponents
// of the next block, operand fragments) stays within 128 registers.
constexpr int TM = 4, TN = 4, NT = 512;

// The raw words of one chunk, E::TASK consecutive elements of one row of A or B per task (as in the integer kernels).
template <int EK>
struct RawChunk {
    static constexpr int TPR = KC / Elem<EK>::TASK;
    static constexpr int TASKS = (BM + BN) * TPR;
    static constexpr int PER_THREAD = (TASKS + NT - 1) / NT;
    static constexpr int WORDS = Elem<EK>::TASK * Elem<EK>::BYTES / 4;
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

constexpr int G_OFF = 30;          // the B offset sits 30 bits below the element's last significand bit (bit 22 - mbits of a double's low word)

struct LutEntry64 {
    double op;          // staged operand
    uint32_t exp;       // Exp(x) + EB; 0 for zero, infinity and NaN
    uint32_t bits;      // bit 0: sign; bit 1: infinity or NaN; bit 2: nonzero finite
};

// Operand planes are row-major (k contiguous) with a pitch of KP doubles = 288 bytes: the fragment loads of the FP64
// matrix instruction (lane (g, t) reads element (row 8 i + g, k 4 s + t)) then hit sixteen different bank pairs per
// half-warp.  Exponent planes and masks are indexed by the permuted row / column (see perm_row64 / perm_col64), so that
// the four rows and the four columns of a thread are adjacent.
constexpr int KP = KC + 4;
template <int EK, bool ROWMAJOR = false>
struct Planes64;
template <int EK>
struct Planes64<EK, true> {
    static constexpr bool ROW_MAJOR = true;
    double a_d[BM][KP];
    double b_d[BN][KP];
    uint32_t a_exp2[KC / 2][BM];    // [pair p][permuted row]: exponents of elements 2p (low half) and 2p + 1 (high half)
    uint32_t b_exp2[KC / 2][BN];
    uint32_t a_sgn[BM], b_sgn[BN];  // [permuted row]: bit k = sign of element k of the chunk
    uint32_t a_nz[BM], b_nz[BN];    // [permuted row]: bit k = element k is finite and nonzero
};
// The k-major layout of the kernels that still issue one scalar FP64 multiply-add per term (TR-, GTR- and E-FDPA): a
// thread owns rows 4 ty .. 4 ty + 3 and the columns col_of(tx, c); nothing is permuted.
template <int EK>
struct Planes64<EK, false> {
    static constexpr bool ROW_MAJOR = false;
    double a_d[KC][BM];
    double b_d[KC][BN];
    uint32_t a_exp2[KC / 2][BM];
    uint32_t b_exp2[KC / 2][BN];
    uint32_t a_sgn[BM], b_sgn[BN];
    uint32_t a_nz[BM], b_nz[BN];
};

// A warp owns 32 rows x 16 columns of the CTA tile, as four by two accumulator tiles of the 8 x 8 x 4 FP64 matrix
// instruction; a thread's outputs are its share of those tiles: rows g + 8 r (g = lane / 4, r = 0..3) and columns
// 8 (c / 2) + 2 t + c % 2 (t = lane % 4, c = 0..3).  Permuted positions put a thread's rows / columns side by side.
__device__ __forceinline__ int perm_row64(int r) { return (r & ~31) | ((r & 7) << 2) | ((r >> 3) & 3); }
__device__ __forceinline__ int perm_col64(int c) { return (c & ~15) | (((c >> 1) & 3) << 2) | (((c >> 3) & 1) << 1) | (c & 1); }

template <int EK, bool ROWMAJOR = false>
struct Smem64 {
    Planes64<EK, ROWMAJOR> pl[2];   // the chunk being computed and the one being decoded
    LutEntry64 lut_a[Elem<EK>::SIGNMAG ? 1 : 256];
    LutEntry64 lut_b[Elem<EK>::SIGNMAG ? 1 : 256];
    int special[3];                 // chunk (by index mod 3) holds an infinity or a NaN
};

__device__ __forceinline__ double pow2d(int e) { return __hiloint2double((1023 + e) << 20, 0); }

// Staged operand of one finite element sign * sig * 2^(exp - mbits); zero stays zero; see the header comment.
__device__ __forceinline__ double operand_a(uint32_t sign, uint32_t sig, int exp, int mbits) {
    const double mag = __dmul_rn(__uint2double_rn(sig), pow2d(exp - mbits));
    return sign ? -mag : mag;
}
__device__ __forceinline__ double operand_b(uint32_t sign, uint32_t sig, int exp, int mbits) {
    const double mag = sig ? __dadd_rn(__dmul_rn(__uint2double_rn(sig), pow2d(exp - mbits)), pow2d(exp - mbits - G_OFF)) : 0.0;
    return sign ? -mag : mag;
}

template <int EK, class SM>
__device__ __forceinline__ void init_lut64(SM& s, const FmtDesc& fa, const FmtDesc& fb, int tid) {
    if (!Elem<EK>::SIGNMAG && tid < 256) {
        const uint32_t da = decode_elem(fa, uint32_t(tid)), db = decode_elem(fb, uint32_t(tid));
        const bool fin_a = dec_cls(da) == CLS_FINITE, fin_b = dec_cls(db) == CLS_FINITE;
        LutEntry64 ea, eb;
        const uint32_t sga = fin_a ? dec_sig(da) : 0u, sgb = fin_b ? dec_sig(db) : 0u;
        ea.op = operand_a(fin_a ? dec_sign(da) : 0u, sga, fin_a ? dec_exp(da) : 0, fa.mbits);
        ea.exp = sga ? uint32_t(dec_exp(da) + EB) : 0u;
        ea.bits = (fin_a ? dec_sign(da) : 0u) | (fin_a ? 0u : 2u) | (sga ? 4u : 0u);
        eb.op = operand_b(fin_b ? dec_sign(db) : 0u, sgb, fin_b ? dec_exp(db) : 0, fb.mbits);
        eb.exp = sgb ? uint32_t(dec_exp(db) + EB) : 0u;
        eb.bits = (fin_b ? dec_sign(db) : 0u) | (fin_b ? 0u : 2u) | (sgb ? 4u : 0u);
        s.lut_a[tid] = ea;
        s.lut_b[tid] = eb;
    }
}

// Decode the raw words of a chunk into double operands, packed exponent pairs and sign bit masks.
template <int EK, class SM, class PL>
__device__ __forceinline__ void store_chunk64(SM& sm, PL& s, const RawChunk<EK>& raw, int flag, int tid) {
    using E = Elem<EK>;
    using R = RawChunk<EK>;
    uint32_t spec = 0u;
#pragma unroll
    for (int it = 0; it < R::PER_THREAD; ++it) {
        const int task = it * NT + tid;
        if (task >= R::TASKS) break;
        const bool is_a = task < BM * R::TPR;
        const int u = is_a ? task : task - BM * R::TPR;
        const int rows = is_a ? BM : BN;
        const int r = u % rows, h = u / rows;
        const int pr = !PL::ROW_MAJOR ? r : (is_a ? perm_row64(r) : perm_col64(r));
        uint32_t bits = 0u, prev_exp = 0u;
#pragma unroll
        for (int q = 0; q < E::TASK; ++q) {
            const int kk = h * E::TASK + q;
            double op;
            uint32_t expb;
            if (!E::SIGNMAG) {
                const uint32_t byte = (raw.w[it][q / 4] >> (8 * (q % 4))) & 0xFFu;
                const LutEntry64 e = is_a ? sm.lut_a[byte] : sm.lut_b[byte];
                op = e.op;
                expb = e.exp;
                bits += ((e.bits & 1u) | ((e.bits & 4u) << 14)) << q;      // sign in the low half, nonzero in the high half
                spec |= e.bits & 2u;
            } else {
                const uint32_t w = E::BYTES == 2 ? ((raw.w[it][q / 2] >> (16 * (q % 2))) & 0xFFFFu) : raw.w[it][q];
                // A normal number becomes a double by moving its exponent and mantissa fields into place and rebiasing
                // (no arithmetic); the offset of a B operand is then bit 22 - mbits of the low word.  Subnormals take
                // the arithmetic route; zeros, infinities and NaNs are staged as zero without exponent.
                constexpr uint32_t TOP = (1u << E::EBITS) - 1u;
                const uint32_t xx = w >> E::LOW;
                const uint32_t mag = xx & ((1u << (E::EBITS + E::MBITS)) - 1u);
                const uint32_t field = mag >> E::MBITS;
                const uint32_t sign = (xx >> (E::EBITS + E::MBITS)) & 1u;
                uint32_t hi = 0u, lo = 0u, nzbit = 1u;
                expb = 0u;
                if (field - 1u < TOP - 1u) {
                    hi = (mag << (20 - E::MBITS)) + (uint32_t(1023 - E::BIAS) << 20);
                    lo = is_a ? 0u : (1u << (22 - E::MBITS));
                    expb = field + uint32_t(EB - E::BIAS);
                } else if (field == 0u && mag != 0u) {
                    const double v = is_a ? operand_a(0u, mag, 1 - E::BIAS, E::MBITS) : operand_b(0u, mag, 1 - E::BIAS, E::MBITS);
                    hi = uint32_t(__double2hiint(v));
                    lo = uint32_t(__double2loint(v));
                    expb = uint32_t(1 - E::BIAS + EB);
                } else {
                    nzbit = 0u;
                    spec |= uint32_t(field == TOP);
                }
                op = __hiloint2double(int(hi | (sign << 31)), int(lo));
                bits += (sign | (nzbit << 16)) << q;
            }
            if (PL::ROW_MAJOR) { if (is_a) s.a_d[r][kk] = op; else s.b_d[r][kk] = op; }
            else { if (is_a) s.a_d[kk][r] = op; else s.b_d[kk][r] = op; }
            if (q & 1) {
                const uint32_t pair = prev_exp | (expb << 16);
                if (is_a) s.a_exp2[kk / 2][pr] = pair; else s.b_exp2[kk / 2][pr] = pair;
            }
            prev_exp = expb;
        }
        // sign and nonzero bits of the task's elements go to bits [h * TASK, h * TASK + TASK) of the row's masks
        if (E::TASK == 16) {
            if (is_a) { reinterpret_cast<uint16_t*>(&s.a_sgn[pr])[h] = uint16_t(bits); reinterpret_cast<uint16_t*>(&s.a_nz[pr])[h] = uint16_t(bits >> 16); }
            else { reinterpret_cast<uint16_t*>(&s.b_sgn[pr])[h] = uint16_t(bits); reinterpret_cast<uint16_t*>(&s.b_nz[pr])[h] = uint16_t(bits >> 16); }
        } else {
            if (is_a) { reinterpret_cast<uint8_t*>(&s.a_sgn[pr])[h] = uint8_t(bits); reinterpret_cast<uint8_t*>(&s.a_nz[pr])[h] = uint8_t(bits >> 16); }
            else { reinterpret_cast<uint8_t*>(&s.b_sgn[pr])[h] = uint8_t(bits); reinterpret_cast<uint8_t*>(&s.b_nz[pr])[h] = uint8_t(bits >> 16); }
        }
    }
    if (spec) atomicOr(&sm.special[flag], 1);
}

// One operand's share of a chunk of KC = 32 elements of K, decoded for the matrix-instruction kernel: R rows of A (or
// columns of B).  A decode kernel writes these blocks to scratch memory once per GEMM; the main kernel brings them in with
// one bulk copy each.  Layouts as in Planes64<EK, true>; `pe` holds BF16 powers 2^(BASE (Exp - 1)) for the tensor-core
// exponent maximum of the element kinds whose exponent sums fit (FP16 and the 8-bit kinds).
constexpr int PE_STRIDE64 = KC + 8;     // 80 bytes per row: fragment loads hit 32 different banks
template <int R>
struct Blk64 {
    double d[R][KP];
    uint32_t exp2[KC / 2][R];
    uint16_t pe[R][PE_STRIDE64];
    uint32_t sgn[R], nz[R];
    uint8_t sf[R];                  // [permuted row]: the E8M0 scale factor of the row for this block of 32 (ST-FDPA), else 127
    uint32_t special;               // the block holds an infinity or a NaN
    uint32_t max_exp;               // the largest Exp(x) + EB of the block's elements (0: all zero)
    uint32_t pad[2];
};
static_assert(sizeof(Blk64<BM>) % 16 == 0 && sizeof(Blk64<BN>) % 16 == 0, "bulk copies move multiples of 16 bytes");

struct SmemMM {
    Blk64<BM> a[2];
    Blk64<BN> b[2];
    unsigned long long full[2];         // mbarriers: the bulk copies of a buffer have landed
    int error;                          // a bounded wait ran out
};

// Base of the exponent powers by element kinds (see the F = 13 kernel for the argument): a sum of at most 2^(BASE-1)
// terms stays within 2^(BASE-1) of its largest term, and BASE times the spread of the exponent sums has to fit FP32.
//   FP16 x FP16 (sums -28..30): BASE 4, sub-blocks of 8 terms; 8-bit kinds: 8 (E4M3 / FP6 / FP4 only: one accumulation of
//   32), 5 (one E5M2 operand: sub-blocks of 16), 4 (two: sub-blocks of 8); BF16 and TF32 do not fit: BASE 0, add-max pass.
__host__ __device__ constexpr int pe64_shift(int base) { return base == 5 ? 3 : 1; }       // (127 + shift) % base == 0
__host__ __device__ constexpr int pe64_sub(int base) { return base == 8 ? 32 : (base == 5 ? 16 : 8); }

// Decode pass: one CTA of 256 threads decodes one block (R rows x 32 elements) into shared memory and copies it to its
// place dst[tile][chunk].  Rows beyond the matrix decode as zeros.
// EOSPLIT (GTR-FDPA, blocks of 16): inside each block of 16 the operand plane holds the even elements first, then the odd
// ones, so that a matrix instruction sums four elements of one group; exponent pairs and masks keep the order of K.
template <int EK, int R, bool IS_A, int BASE, bool EOSPLIT = false>
__global__ void __launch_bounds__(256) decode64_kernel(DevModel m, const unsigned char* src, int64_t rows, int64_t ld, Blk64<R>* dst,
                                                       const uint8_t* sf = nullptr, int64_t ld_sf = 0) {
    using E = Elem<EK>;
    constexpr int TPR = KC / E::TASK, TASKS = R * TPR, WORDS = E::TASK * E::BYTES / 4;
    extern __shared__ __align__(16) unsigned char dec_smem[];
    LutEntry64* lut = reinterpret_cast<LutEntry64*>(dec_smem);
    Blk64<R>& blk = *reinterpret_cast<Blk64<R>*>(dec_smem + 256 * sizeof(LutEntry64));
    const int tid = threadIdx.x;
    if (!E::SIGNMAG) {
        const FmtDesc f = fmt_desc(IS_A ? m.fmt_a : m.fmt_b);
        const uint32_t dd = decode_elem(f, uint32_t(tid));
        const bool fin = dec_cls(dd) == CLS_FINITE;
        const uint32_t sg = fin ? dec_sig(dd) : 0u;
        LutEntry64 e;
        e.op = IS_A ? operand_a(fin ? dec_sign(dd) : 0u, sg, fin ? dec_exp(dd) : 0, f.mbits)
                    : operand_b(fin ? dec_sign(dd) : 0u, sg, fin ? dec_exp(dd) : 0, f.mbits);
        e.exp = sg ? uint32_t(dec_exp(dd) + EB) : 0u;
        e.bits = (fin ? dec_sign(dd) : 0u) | (fin ? 0u : 2u) | (sg ? 4u : 0u);
        lut[tid] = e;
    }
    if (tid == 0) { blk.special = 0u; blk.max_exp = 0u; blk.pad[0] = blk.pad[1] = 0u; }
    __syncthreads();
    const int64_t k0 = int64_t(blockIdx.x) * KC;
    uint32_t spec = 0u, top_exp = 0u;
    for (int task = tid; task < TASKS; task += 256) {
        const int r = task % R, h = task / R;
        const int pr = IS_A ? perm_row64(r) : perm_col64(r);
        const int64_t grow = int64_t(blockIdx.y) * R + r;
        uint32_t w[WORDS];
#pragma unroll
        for (int q = 0; q < WORDS / 4; ++q) {
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (grow < rows) v = reinterpret_cast<const uint4*>(src + (grow * ld + k0 + h * E::TASK) * E::BYTES)[q];
            w[4 * q] = v.x; w[4 * q + 1] = v.y; w[4 * q + 2] = v.z; w[4 * q + 3] = v.w;
        }
        // ST-FDPA (Algorithm 8): the row's scale factor for this block of 32 multiplies its operands here, exactly (an
        // addition to the exponent field of a nonzero double); exponent planes stay unscaled, the main kernel adds
        // Exp(alpha) + Exp(beta) to the block maximum.  A NaN scale factor stages zeros (the output is NaN by its flag).
        int sc20 = 0;
        bool sc_nan = false;
        if (sf) {
            const uint32_t sbyte = grow < rows ? uint32_t(sf[grow * ld_sf + blockIdx.x]) : 127u;
            sc20 = (int(sbyte) - 127) << 20;
            sc_nan = sbyte == 0xFFu;
        }
        uint32_t bits = 0u, prev_exp = 0u, pw[E::TASK / 2];
#pragma unroll
        for (int q = 0; q < E::TASK; ++q) {
            const int kk = h * E::TASK + q;
            double op;
            uint32_t expb;
            if (!E::SIGNMAG) {
                const uint32_t byte = (w[q / 4] >> (8 * (q % 4))) & 0xFFu;
                const LutEntry64 e = lut[byte];
                op = e.op;
                if (sf) {
                    const int ohi = __double2hiint(op);
                    op = ((ohi & 0x7FFFFFFF) == 0 || sc_nan) ? 0.0 : __hiloint2double(ohi + sc20, __double2loint(op));
                }
                expb = e.exp;
                bits += ((e.bits & 1u) | ((e.bits & 4u) << 14)) << q;
                spec |= e.bits & 2u;
            } else {
                const uint32_t x = E::BYTES == 2 ? ((w[q / 2] >> (16 * (q % 2))) & 0xFFFFu) : w[q];
                constexpr uint32_t TOP = (1u << E::EBITS) - 1u;
                const uint32_t xx = x >> E::LOW;
                const uint32_t mag = xx & ((1u << (E::EBITS + E::MBITS)) - 1u);
                const uint32_t field = mag >> E::MBITS;
                const uint32_t sign = (xx >> (E::EBITS + E::MBITS)) & 1u;
                uint32_t hi = 0u, lo = 0u, nzbit = 1u;
                expb = 0u;
                if (field - 1u < TOP - 1u) {
                    hi = (mag << (20 - E::MBITS)) + (uint32_t(1023 - E::BIAS) << 20);
                    lo = IS_A ? 0u : (1u << (22 - E::MBITS));
                    expb = field + uint32_t(EB - E::BIAS);
                } else if (field == 0u && mag != 0u) {
                    const double v = IS_A ? operand_a(0u, mag, 1 - E::BIAS, E::MBITS) : operand_b(0u, mag, 1 - E::BIAS, E::MBITS);
                    hi = uint32_t(__double2hiint(v));
                    lo = uint32_t(__double2loint(v));
                    expb = uint32_t(1 - E::BIAS + EB);
                } else {
                    nzbit = 0u;
                    spec |= uint32_t(field == TOP);
                }
                op = __hiloint2double(int(hi | (sign << 31)), int(lo));
                bits += (sign | (nzbit << 16)) << q;
            }
            blk.d[r][EOSPLIT ? ((kk & ~15) | ((kk & 1) << 3) | ((kk & 15) >> 1)) : kk] = op;
            // BF16 word of 2^(BASE (Exp - 1)) (the B plane times 2^shift); 0 for an element without exponent
            const uint32_t pe = (BASE && expb) ? uint32_t((127 + (IS_A ? 0 : pe64_shift(BASE)) + BASE * (int(expb) - EB - 1)) << 7) : 0u;
            if (q & 1) {
                blk.exp2[kk / 2][pr] = prev_exp | (expb << 16);
                pw[q / 2] |= pe << 16;
            } else pw[q / 2] = pe;
            prev_exp = expb;
            top_exp = max(top_exp, expb);
        }
#pragma unroll
        for (int q = 0; q < E::TASK / 8; ++q)
            reinterpret_cast<uint4*>(&blk.pe[r][h * E::TASK])[q] = make_uint4(pw[4 * q], pw[4 * q + 1], pw[4 * q + 2], pw[4 * q + 3]);
        if (E::TASK == 16) {
            reinterpret_cast<uint16_t*>(&blk.sgn[pr])[h] = uint16_t(bits); reinterpret_cast<uint16_t*>(&blk.nz[pr])[h] = uint16_t(bits >> 16);
        } else {
            reinterpret_cast<uint8_t*>(&blk.sgn[pr])[h] = uint8_t(bits); reinterpret_cast<uint8_t*>(&blk.nz[pr])[h] = uint8_t(bits >> 16);
        }
    }
    if (spec) atomicOr(&blk.special, 1u);
    if (tid < R) {                                      // the scale factors travel with the block (rows beyond the matrix: 2^0)
        const int64_t grow = int64_t(blockIdx.y) * R + tid;
        blk.sf[IS_A ? perm_row64(tid) : perm_col64(tid)] = (sf && grow < rows) ? sf[grow * ld_sf + blockIdx.x] : uint8_t(127);
    }
    top_exp = __reduce_max_sync(0xFFFFFFFFu, top_exp);
    if ((tid & 31) == 0 && top_exp) atomicMax(&blk.max_exp, top_exp);
    __syncthreads();
    uint4* out = reinterpret_cast<uint4*>(dst + (int64_t(blockIdx.y) * gridDim.x + blockIdx.x));
    const uint4* in = reinterpret_cast<const uint4*>(&blk);
    for (int q = tid; q < int(sizeof(Blk64<R>) / 16); q += 256) out[q] = in[q];
}

// Columns of a thread's micro-tile in the k-major layout: two adjacent pairs, 32 columns apart, so that the sixteen
// threads of a row of the thread grid read 256 contiguous bytes of B operands per 16-byte load.
__device__ __forceinline__ int col_of(int tx, int c) { return (c >> 1) * (BN / 2) + tx * 2 + (c & 1); }

// Largest exponent sum of the products of one block (pass 1 of Algorithm 7 without the accumulator), two elements
// per instruction: lane 0 holds the even elements' maximum, lane 1 the odd ones'.  k-major layout.
template <int L>
__device__ __forceinline__ void product_exponents(const uint32_t* ea_p, const uint32_t* eb_p, uint32_t (&emp)[TM][TN]) {
#pragma unroll
    for (int r = 0; r < TM; ++r)
#pragma unroll
        for (int c = 0; c < TN; ++c) emp[r][c] = 0u;
#pragma unroll
    for (int kp = 0; kp < L / 2; ++kp) {
        const uint4 ea0 = *reinterpret_cast<const uint4*>(ea_p + kp * BM);
        const uint2 eb0 = *reinterpret_cast<const uint2*>(eb_p + kp * BN);
        const uint2 eb1 = *reinterpret_cast<const uint2*>(eb_p + kp * BN + BN / 2);
        const uint32_t ea[TM] = {ea0.x, ea0.y, ea0.z, ea0.w};
        const uint32_t ebv[TN] = {eb0.x, eb0.y, eb1.x, eb1.y};
#pragma unroll
        for (int r = 0; r < TM; ++r)
#pragma unroll
            for (int c = 0; c < TN; ++c) emp[r][c] = __viaddmax_s16x2(ea[r], ebv[c], emp[r][c]);
    }
}

// Multipliers read from the constant bank, so that the compiler keeps integer multiply-adds (which issue beside the
// integer pipe) instead of rewriting them as shifts and additions on it.
static __constant__ int c_mul64[8] = {1 << 20, 16, 1, 0, 1 << 21, 32, 2, int(0x80000000u)};
__device__ __forceinline__ int imad(int a, int b, int c) {
    int d;
    asm("mad.lo.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
// max(|a|, b, c) of three words read as FP32 numbers, in one instruction (the absolute value is an operand modifier).
// For nonnegative words the order of FP32 numbers is the order of the integers; a negative b or c reads as a negative
// number or a NaN and loses either way (the maximum of a NaN and a number is the number).
__device__ __forceinline__ int fmax3_abs(int a, int b, int c) {
    float d;
    asm("{ .reg .f32 t; abs.f32 t, %1; max.f32 %0, t, %2, %3; }" : "=f"(d) : "f"(__int_as_float(a)), "f"(__int_as_float(b)), "f"(__int_as_float(c)));
    return __float_as_int(d);
}
// high word of a * b, plus c: with b = 2^31 a logical shift right by one, with b = 2 the top bit of a
__device__ __forceinline__ uint32_t imad_hi(uint32_t a, int b, uint32_t c) {
    uint32_t d;
    asm("mad.hi.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// The same for the permuted layout: ea_p / eb_p point at the thread's four adjacent (permuted) rows / columns of the
// first pair of the block.
template <int L>
__device__ __forceinline__ void product_exponents_adj(const uint32_t* ea_p, const uint32_t* eb_p, uint32_t (&emp)[TM][TN]) {
#pragma unroll
    for (int kp = 0; kp < L / 2; ++kp) {
        const uint4 ea0 = *reinterpret_cast<const uint4*>(ea_p + kp * BM);
        const uint4 eb0 = *reinterpret_cast<const uint4*>(eb_p + kp * BN);
        const uint32_t ea[TM] = {ea0.x, ea0.y, ea0.z, ea0.w};
        const uint32_t ebv[TN] = {eb0.x, eb0.y, eb0.z, eb0.w};
#pragma unroll
        for (int r = 0; r < TM; ++r)
#pragma unroll
            for (int c = 0; c < TN; ++c) emp[r][c] = __viaddmax_s16x2(ea[r], ebv[c], kp == 0 ? 0u : emp[r][c]);
    }
}

// One CTA per SM, 512 threads, a 4 x 4 micro-tile per thread.  The FP64 pipe is the bound (one fma.rm.f64 per term),
// so everything else is arranged to run beside it: the staged planes are double-buffered (the next chunk is decoded
// between two barriers while its raw words were fetched a chunk earlier), and the product-exponent pass of block
// n + 1 is fused, instruction by instruction, into the multiply-add pass of block n - the integer pipe works in
// the issue slots that the FP64 pipe leaves free.
template <int EK, int L, int RHO, bool PROMOTE, bool ST, int BASE>
__global__ void __launch_bounds__(NT, 1) tfdpa64_kernel(DevModel m, GemmArgs g, const Blk64<BM>* __restrict__ wa,
                                                        const Blk64<BN>* __restrict__ wb) {
    // BASE > 0: the block maximum of the product exponents comes from the tensor cores (a product of powers BASE^Exp on
    // BF16 planes, as in the F = 13 kernel); BASE = 0: from fused add-max instructions on packed exponent pairs.
    static_assert(BASE == 0 || ((BASE == 4 || BASE == 8) && L >= 8), "see pe64_shift / pe64_sub");
    constexpr int LB = BASE == 8 ? 3 : 2;                       // log2(BASE)
    constexpr int KP2 = (1023 + 2 - (127 + 1) / (BASE ? BASE : 1)) << 20;   // P-domain key + KP2 = (e_max + 1023) << 20
    using E = Elem<EK>;
    constexpr bool ACC16 = RHO == RHO_RNE_FP16;
    constexpr int NBLK = KC / L;
    static_assert(RHO == RHO_RZ_FP32 || RHO == RHO_RNE_FP16, "rho is a single conversion from FP64");
    static_assert(KC % L == 0 && L % 4 == 0, "blocks tile the chunk; pass 1 handles pairs of elements");
    static_assert(!ST || L == KC, "ST-FDPA: one scale factor pair per block of 32 (Algorithm 8)");
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SmemMM& sm = *reinterpret_cast<SmemMM*>(smem_raw);

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int wr = warp >> 2, wc = warp & 3, gq = lane >> 2, tq = lane & 3;      // warp grid 4 x 4, warp tile 32 x 16
    const int prow = wr * 32 + gq * 4, pcol = wc * 16 + tq * 4;                  // the thread's first permuted row / column
    auto row_at = [&](int r) { return wr * 32 + gq + 8 * r; };                   // inside the CTA tile
    auto col_at = [&](int c) { return wc * 16 + 8 * (c >> 1) + 2 * tq + (c & 1); };
    const int64_t row0 = int64_t(blockIdx.y) * BM, col0 = int64_t(blockIdx.x) * BN;
    const FmtDesc fa = fmt_desc(m.fmt_a), fb = fmt_desc(m.fmt_b);

    // the decoded blocks of this tile row of A and tile column of B, chunk after chunk, land in two buffers by bulk copies
    const int NCH = int(g.K / KC);
    const Blk64<BM>* src_a = wa + int64_t(blockIdx.y) * NCH;
    const Blk64<BN>* src_b = wb + int64_t(blockIdx.x) * NCH;
    auto issue = [&](int n) {                              // one thread: both copies of chunk n into buffer n & 1
        unsigned long long* bar = &sm.full[n & 1];
        fast::mbar_expect_tx(bar, uint32_t(sizeof(Blk64<BM>) + sizeof(Blk64<BN>)));
        fast::bulk_load(&sm.a[n & 1], src_a + n, uint32_t(sizeof(Blk64<BM>)), bar);
        fast::bulk_load(&sm.b[n & 1], src_b + n, uint32_t(sizeof(Blk64<BN>)), bar);
    };
    if (tid == 0) {
        sm.error = 0;
        fast::mbar_init(&sm.full[0], 1u);
        fast::mbar_init(&sm.full[1], 1u);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        issue(0);
        if (NCH > 1) issue(1);
    }

    // FP32 accumulators live between blocks as doubles ("state"): the value RZ-FP32 produced, exactly, with bit 0 of the
    // low word set so that the next block's addition (rounded toward minus infinity) never finds it on its grid; the
    // conversion function is then a mask on the double's low word and the exponent of c is the double's own field.
    // Results outside the range of normal FP32 numbers (zero, subnormal, overflow) leave the fast path.  FP16
    // accumulators live the same way, as the exact doubles of the rounded halves (normal range 2^-14 .. 2^16).
    constexpr bool DS = true;
    // blocks of at most 8 terms: |S| < 2^(F+1) + L * 2^(F+2) < 2^31, so the sum register's low word, started at 2^31, never
    // carries into the high word
    constexpr bool NARROW = DS && L <= 8;
    constexpr int UNROLL_BLK = (L <= 4 || (L <= 16 && BASE == 0)) ? 2 : 1;  // two blocks per trip of the block loop
    // where it measured faster: blocks of 4, and the long blocks of the add-max kinds (BF16, L = 16)
    constexpr bool KEEP_MH = (NARROW && L <= 4) || (!NARROW && BASE == 0);
    // (a zero of either sign becomes the positive state)
    auto state_of = [](uint32_t w) {
        double d = 0.0;
        if (ACC16) { if (w & 0x7FFFu) d = double(__half2float(__ushort_as_half((unsigned short)w))); }
        else if (w & 0x7FFFFFFFu) d = double(__uint_as_float(w));
        return __hiloint2double(__double2hiint(d), __double2loint(d) | 1);
    };
    auto word_of = [](double st) {
        const double d = __hiloint2double(__double2hiint(st), __double2loint(st) & ~1);
        return ACC16 ? uint32_t(__half_as_ushort(__double2half(d))) : __float_as_uint(__double2float_rz(d));
    };
    // the range of normal numbers of the accumulator's format, as exponent fields of doubles
    constexpr int EXP_LOW = ACC16 ? -14 : -126, EXP_TOP = ACC16 ? 16 : 128;
    double cs[DS ? TM : 1][DS ? TN : 1];
    uint32_t sub_mask = 0u;                             // outputs whose accumulator is a nonzero FP32 subnormal: Exp(c) = -126
    uint32_t cw[TM][TN];                                // the words of C as read (finite ones; the rest become flags)
    uint32_t sp_nan = 0u, sp_pinf = 0u, sp_ninf = 0u;   // per output (bit r * TN + c): NaN / +inf / -inf seen so far
    float promoted[PROMOTE ? TM : 1][PROMOTE ? TN : 1];
#define MMASIM_SP_GET(r, c) ((((sp_nan >> ((r) * TN + (c))) & 1u)) | (((sp_pinf >> ((r) * TN + (c))) & 1u) << 1) | (((sp_ninf >> ((r) * TN + (c))) & 1u) << 2))
#pragma unroll
    for (int r = 0; r < TM; ++r)
#pragma unroll
        for (int c = 0; c < TN; ++c) {
            const int64_t i = row0 + row_at(r), j = col0 + col_at(c);
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
            if (DS) {
                cs[DS ? r : 0][DS ? c : 0] = state_of(w);
                if (ACC16 ? ((w & 0x7C00u) == 0u && (w & 0x03FFu) != 0u) : ((w & 0x7F800000u) == 0u && (w & 0x007FFFFFu) != 0u))
                    sub_mask |= 1u << (r * TN + c);
            }
        }

    __syncthreads();                                    // the barriers are initialised
    uint32_t emp[TM][TN];                               // product exponents of the block that comes next

    for (int chunk = 0; chunk < NCH; ++chunk) {
        const int64_t k0 = int64_t(chunk) * KC;
        // a wait that runs out is recorded and the chunk computed on whatever is there; every thread sees the flag after
        // the barrier at the end of the chunk, and the CTA leaves together without storing anything
        if (!fast::mbar_wait(&sm.full[chunk & 1], uint32_t(chunk >> 1) & 1u)) *reinterpret_cast<volatile int*>(&sm.error) = 1;
        const Blk64<BM>& sa_blk = sm.a[chunk & 1];
        const Blk64<BN>& sb_blk = sm.b[chunk & 1];
        const bool chunk_special = (sa_blk.special | sb_blk.special) != 0u;
        // the first block's product exponents (the other blocks' are taken beside the multiply-adds of their predecessor)
        if (BASE == 0) product_exponents_adj<L>(&sa_blk.exp2[0][prow], &sb_blk.exp2[0][pcol], emp);

        // ST-FDPA (Algorithm 8): Exp(alpha) of this thread's rows and Exp(beta) of its columns for this block of 32, as
        // exponent-field increments.  The staged operands already carry the scale factors (decode pass), so the products,
        // their sum and the accumulator all live in the one scaled domain and only the block maximum needs the sum added.
        static_assert(!ST || BASE > 0, "the scaled rows all take their maximum from the tensor cores");
        int sa_exp[ST ? TM : 1], sb_exp[ST ? TN : 1];
        if (ST) {
            // (the scale bytes came in with the decoded blocks: one 32-bit shared load for the thread's four rows / columns)
            static_assert(TM == 4 && TN == 4, "four scale bytes per load");
            const uint32_t wa4 = *reinterpret_cast<const uint32_t*>(&sa_blk.sf[prow]);
            const uint32_t wb4 = *reinterpret_cast<const uint32_t*>(&sb_blk.sf[pcol]);
            uint32_t scale_nan = 0u;                    // bit r * TN + c: alpha or beta of that output is NaN
#pragma unroll
            for (int r = 0; r < TM; ++r) {
                const uint32_t w = (wa4 >> (8 * r)) & 0xFFu;
                sa_exp[ST ? r : 0] = ((int(w) - 127) << 20) + KP2;   // in place of a double's exponent field, with the key's constant
                if (w == 0xFFu) scale_nan |= ((1u << TN) - 1u) << (r * TN);
            }
#pragma unroll
            for (int c = 0; c < TN; ++c) {
                const uint32_t w = (wb4 >> (8 * c)) & 0xFFu;
                sb_exp[ST ? c : 0] = (int(w) - 127) << 20;
                if (w == 0xFFu) scale_nan |= 0x11111111u << c;
            }
            sp_nan |= scale_nan;                        // a NaN scale factor makes the block result NaN
        }

#pragma unroll UNROLL_BLK
        for (int blk = 0; blk < NBLK; ++blk) {
            const int kb = blk * L;
            // ---- rare: the chunk holds an infinity or a NaN: special-value events of this block (Section 4.2).
            // Flags are sticky: once an output is special the finite arithmetic below no longer matters for it.
            if (chunk_special) {
#pragma unroll 1
                for (int r = 0; r < TM; ++r)
#pragma unroll 1
                    for (int c = 0; c < TN; ++c) {
                        const int64_t i = row0 + row_at(r), j = col0 + col_at(c);
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

            if (BASE) {
                // ---- pass 1 on the tensor cores: P = sum_k pe(a_k) pe(b_k) per sub-block of KSUB terms, the block's P the
                // integer maximum of their words; emp receives the raw words (0: no nonzero product) ----
                constexpr int KSUB = pe64_sub(BASE) < L ? pe64_sub(BASE) : L, NSUB = L / KSUB;
                constexpr int NK = KSUB >= 16 ? KSUB / 16 : 1, AR = KSUB >= 16 ? 4 : 2, BR = KSUB >= 16 ? 2 : 1;
#pragma unroll
                for (int mt = 0; mt < 2; ++mt) {
                    uint32_t P[2][4];
#pragma unroll
                    for (int sub = 0; sub < NSUB; ++sub) {
                        uint32_t af[NK][AR];
                        const int ar = wr * 32 + 16 * mt + gq;
#pragma unroll
                        for (int ks = 0; ks < NK; ++ks) {
                            const int kq = kb + sub * KSUB + 16 * ks + 2 * tq;
                            af[ks][0] = *reinterpret_cast<const uint32_t*>(&sa_blk.pe[ar][kq]);
                            af[ks][1] = *reinterpret_cast<const uint32_t*>(&sa_blk.pe[ar + 8][kq]);
                            if (AR == 4) {
                                af[ks][AR - 2] = *reinterpret_cast<const uint32_t*>(&sa_blk.pe[ar][kq + 8]);
                                af[ks][AR - 1] = *reinterpret_cast<const uint32_t*>(&sa_blk.pe[ar + 8][kq + 8]);
                            }
                        }
#pragma unroll
                        for (int j = 0; j < 2; ++j) {
                            uint32_t bf[NK][BR];
#pragma unroll
                            for (int ks = 0; ks < NK; ++ks) {
                                const int kq = kb + sub * KSUB + 16 * ks + 2 * tq;
                                bf[ks][0] = *reinterpret_cast<const uint32_t*>(&sb_blk.pe[wc * 16 + 8 * j + gq][kq]);
                                if (BR == 2) bf[ks][BR - 1] = *reinterpret_cast<const uint32_t*>(&sb_blk.pe[wc * 16 + 8 * j + gq][kq + 8]);
                            }
                            float d[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                            for (int ks = 0; ks < NK; ++ks) {
                                if (KSUB >= 16)
                                    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                                                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                                                 : "r"(af[ks][0]), "r"(af[ks][1]), "r"(af[ks][AR - 2]), "r"(af[ks][AR - 1]),
                                                   "r"(bf[ks][0]), "r"(bf[ks][BR - 1]));
                                else
                                    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
                                                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                                                 : "r"(af[ks][0]), "r"(af[ks][1]), "r"(bf[ks][0]));
                            }
#pragma unroll
                            for (int i = 0; i < 4; ++i)
                                P[j][i] = sub == 0 ? __float_as_uint(d[i]) : max(P[j][i], __float_as_uint(d[i]));
                        }
                    }
                    // accumulator fragment (rows g, g + 8 of the 16-row tile; columns 2 t, 2 t + 1 of the 8-column tile) ->
                    // the thread's outputs r = 2 mt + (i >> 1), c = 2 j + (i & 1)
#pragma unroll
                    for (int j = 0; j < 2; ++j)
#pragma unroll
                        for (int i = 0; i < 4; ++i) emp[2 * mt + (i >> 1)][2 * j + (i & 1)] = P[j][i];
                }
            }
            // ---- e_max = max(Exp(c), product exponents) and the accumulator term:
            // acc = 1.5 * 2^52 * q + floor(c' / q) * q, c' = c with the lowest mantissa bit of its double set (never on
            // the grid: a negative c floors to the one's complement), then + 1 if c < 0.
            // ST: the staged operands carry the scale factors, the key of the products gets Exp(alpha) + Exp(beta) added.
            double acc[TM][TN];
            int mhi[KEEP_MH ? TM : 1][KEEP_MH ? TN : 1];   // high word of each output's 1.5 * 2^52 * q
            // keys (FP32 accumulators) are exponent fields of doubles in place: (Exp + 1023) << 20.  Products: the larger
            // 16-bit lane of emp (Exp + CB, CB = 1024) or, BASE > 0, the exponent field of P over BASE; c: the state's own
            // field (0 for c = 0: below every real key); a subnormal c counts with Exp = -126 (FP16: -14; rare: patched
            // after the pass over the outputs).
            constexpr int KM = (52 << 20) | 0x00080000;              // + (e_max - F) gives the high word of 1.5 * 2^52 * q
            const int km = KM - (m.F << 20);
            auto start = [&](int r, int c, bool subnormal_c) {
                if (DS) {
                    const double st = cs[DS ? r : 0][DS ? c : 0];
                    const int hi = __double2hiint(st);
                    // the keys keep whatever sits below their exponent fields (mantissa bits of c, the other 16-bit lane): it
                    // decides nothing but ties between equal exponents, and one mask after the maximum removes it
                    int keyc = subnormal_c ? (1023 + EXP_LOW) << 20 : hi & 0x7FFFFFFF;
                    const uint32_t e2 = emp[r][c];
                    int m;
                    if (BASE) {
                        // P = 0 gives a key two binades below the smallest real one, which is wrong only for an even smaller c:
                        // the epilogue repairs that case
                        const int kp = ST ? int(e2 >> (3 + LB)) + sa_exp[ST ? r : 0] + sb_exp[ST ? c : 0]
                                          : imad(int(e2 >> (3 + LB)), c_mul64[2], KP2);
                        m = fmax3_abs(subnormal_c ? keyc : hi, kp, kp);
                    } else {
                        // the two 16-bit lanes (Exp + CB of the even and the odd elements) moved to the exponent field by
                        // multiplications, which run beside the integer pipe
                        const int klo = imad(int(e2), c_mul64[0], -(1 << 20)), khi = imad(int(e2), c_mul64[1], -(1 << 20));
                        m = fmax3_abs(subnormal_c ? keyc : hi, klo, khi);
                    }
                    const int e20 = m & 0x7FF00000;
                    // the +1 of a negative c sits in the constant's low word: one unit of the grid either way.  Short blocks:
                    // the low word starts at 2^31, so that the sign correction of the epilogue is a 32-bit addition
                    const int mlo = NARROW ? int(__funnelshift_l(uint32_t(hi), 0x40000000u, 1)) : int(uint32_t(hi) >> 31);
                    const int mh = imad(e20, c_mul64[2], km);
                    if (KEEP_MH) mhi[KEEP_MH ? r : 0][KEEP_MH ? c : 0] = mh;
                    const double magic = __hiloint2double(mh, mlo);
                    acc[r][c] = __dadd_rd(st, magic);
                }
            };
            auto restart_subnormals = [&](int r0) {     // rare: redo the outputs whose accumulator is an FP32 subnormal
                if (DS && sub_mask) {
#pragma unroll
                    for (int r = r0; r < r0 + 2; ++r)
#pragma unroll
                        for (int c = 0; c < TN; ++c)
                            if ((sub_mask >> (r * TN + c)) & 1u) start(r, c, true);
                }
            };
            // four terms per matrix instruction (mma.sync m8n8k4, FP64, rounding toward minus infinity: a chain of four fused
            // multiply-adds per output, each rounded onto the grid of q) for the rows 2 half, 2 half + 1 of the micro-tile;
            // operand fragments: lane (g, t) holds A[8 r + g][k + t] and B[8 j + g][k + t]
            auto mma_half = [&](int half, int ks) {
                double af[2], bf[TN / 2];
#pragma unroll
                for (int r = 0; r < 2; ++r) af[r] = sa_blk.d[wr * 32 + 8 * (2 * half + r) + gq][kb + ks + tq];
#pragma unroll
                for (int j = 0; j < TN / 2; ++j) bf[j] = sb_blk.d[wc * 16 + 8 * j + gq][kb + ks + tq];
#pragma unroll
                for (int r = 0; r < 2; ++r)
#pragma unroll
                    for (int j = 0; j < TN / 2; ++j)
                        asm volatile("mma.sync.aligned.m8n8k4.row.col.rm.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                                     : "+d"(acc[2 * half + r][2 * j]), "+d"(acc[2 * half + r][2 * j + 1]) : "d"(af[r]), "d"(bf[j]));
            };
            // ---- sign corrections, rho.  An overflow (|v| >= 2^128, or an FP16 result that rounds to infinity) is rare
            // and sticky: the loop only tracks it, the flags are set in a second pass ----
            const uint32_t kmask = (L == 32) ? 0xFFFFFFFFu : (((1u << L) - 1u) << kb);
            bool no_product = false;                    // BASE > 0: some output of the micro-tile has no nonzero product
            // FP32 state: the largest (high word of |v|) - (that of 2^-126), unsigned: a v outside the normal FP32 range -
            // zero and the subnormal range wrap to the top - shows as a value of (that of 2^128) - (that of 2^-126) or more
            constexpr uint32_t LOWHI = uint32_t(1023 + EXP_LOW) << 20, SPANHI = uint32_t(EXP_TOP - EXP_LOW) << 20;
            uint32_t urange = 0u;
            auto block_value = [&](int r, int c) -> double {
                const uint32_t sa = sa_blk.sgn[prow + r], nza = sa_blk.nz[prow + r] & kmask;
                const uint32_t live = nza & sb_blk.nz[pcol + c];
                if (BASE) no_product = no_product || live == 0u;
                const int nneg = __popc((sa ^ sb_blk.sgn[pcol + c]) & live);
                double v;
                if (NARROW) {
                    // the register never leaves its binade: its exponent field is the constant's (KEEP_MH: the high word of
                    // the start's constant is kept instead of masked out of the register again)
                    const int hi = __double2hiint(acc[r][c]);
                    const double magic = __hiloint2double(KEEP_MH ? mhi[KEEP_MH ? r : 0][KEEP_MH ? c : 0] : (hi & 0x7FF00000) | 0x00080000, int(0x80000000u));
                    v = __dsub_rn(__hiloint2double(hi, __double2loint(acc[r][c]) + nneg), magic);
                } else {
                    const long long bits = __double_as_longlong(acc[r][c]) + (long long)nneg;
                    const int hi = int(bits >> 32);
                    const double magic = __hiloint2double(KEEP_MH ? mhi[KEEP_MH ? r : 0][KEEP_MH ? c : 0] : (hi & 0x7FF00000) | 0x00080000, 0);
                    v = __dsub_rn(__longlong_as_double(bits), magic);                 // S * q, exact; +0 when S = 0
                }
                return v;
            };
            double nv[DS && BASE ? TM : 1][DS && BASE ? TN : 1];      // BASE > 0: the old accumulators survive until the repair below
            auto finish = [&](int r, int c) {
                const double v = block_value(r, c);
                if (ACC16) {
                    // RNE-FP16 is the conversion instruction (subnormal range and the overflow to infinity included); the
                    // half as a double again is the next accumulator, and its exponent field says whether it is a normal number
                    double x;
                    asm("cvt.f64.f16 %0, %1;" : "=d"(x) : "h"(__half_as_ushort(__double2half(v))));
                    urange = max(uint32_t(imad(__double2hiint(x), c_mul64[6], int(0u - 2u * LOWHI))), urange);
                    const double st = __hiloint2double(__double2hiint(x), __double2loint(x) | 1);
                    if (BASE) nv[BASE ? r : 0][BASE ? c : 0] = st; else cs[DS ? r : 0][DS ? c : 0] = st;
                } else if (DS) {
                    // (twice the high word: the sign leaves at the top, and a multiply-add is not on the integer pipe)
                    urange = max(uint32_t(imad(__double2hiint(v), c_mul64[6], int(0u - 2u * LOWHI))), urange);
                    // RZ-FP32 of a number in the normal range: the low 29 bits of the double's significand go
                    const double st = __hiloint2double(__double2hiint(v), (__double2loint(v) & int(0xE0000000u)) | 1);
                    if (BASE) nv[BASE ? r : 0][BASE ? c : 0] = st; else cs[DS ? r : 0][DS ? c : 0] = st;
                }
            };

            // ---- the block in two halves of the micro-tile (rows 0, 1 and rows 2, 3), so that the multiply-adds of one half
            // (FP64 pipe) are issued between the integer work of the other: start(A); [multiply-adds(A) | start(B)];
            // [multiply-adds(B) | finish(A), and the product exponents of the next block]; finish(B) ----
            constexpr int NKS = L / 4, PER = 8 / (NKS < 8 ? NKS : 8);
            const bool fuse = BASE == 0 && NBLK > 1 && blk + 1 < NBLK;
#pragma unroll
            for (int o = 0; o < 8; ++o) start(o / TN, o % TN, false);
            restart_subnormals(0);
#pragma unroll
            for (int ksi = 0; ksi < NKS; ++ksi) {
                mma_half(0, 4 * ksi);
#pragma unroll
                for (int q = 0; q < PER; ++q)
                    if (ksi * PER + q < 8) start(2 + (ksi * PER + q) / TN, (ksi * PER + q) % TN, false);
            }
            restart_subnormals(2);
#pragma unroll
            for (int ksi = 0; ksi < NKS; ++ksi) {
                mma_half(1, 4 * ksi);
#pragma unroll
                for (int q = 0; q < PER; ++q)
                    if (ksi * PER + q < 8) finish((ksi * PER + q) / TN, (ksi * PER + q) % TN);
                if (fuse) {                             // the product exponents of the next block (add-max kinds)
                    const uint32_t* ea_p = &sa_blk.exp2[(kb + L) / 2 < KC / 2 ? (kb + L) / 2 : 0][prow];
                    const uint32_t* eb_p = &sb_blk.exp2[(kb + L) / 2 < KC / 2 ? (kb + L) / 2 : 0][pcol];
#pragma unroll
                    for (int kp = 2 * ksi; kp < 2 * ksi + 2; ++kp) {
                        const uint4 ea0 = *reinterpret_cast<const uint4*>(ea_p + kp * BM);
                        const uint4 eb0 = *reinterpret_cast<const uint4*>(eb_p + kp * BN);
                        const uint32_t ea[TM] = {ea0.x, ea0.y, ea0.z, ea0.w};
                        const uint32_t ebv[TN] = {eb0.x, eb0.y, eb0.z, eb0.w};
#pragma unroll
                        for (int r = 0; r < TM; ++r)
#pragma unroll
                            for (int c = 0; c < TN; ++c) emp[r][c] = __viaddmax_s16x2(ea[r], ebv[c], kp == 0 ? 0u : emp[r][c]);
                    }
                }
            }
#pragma unroll
            for (int o = 8; o < 16; ++o) finish(o / TN, o % TN);

            if (DS) {
                bool odd = urange >= 2u * SPANHI;       // some result is not a normal FP32 number
                if (BASE && no_product) {               // rare: no nonzero product: the block returns its accumulator
                    odd = true;
#pragma unroll
                    for (int r = 0; r < TM; ++r)
#pragma unroll
                        for (int c = 0; c < TN; ++c)
                            if ((sa_blk.nz[prow + r] & kmask & sb_blk.nz[pcol + c]) == 0u) nv[BASE ? r : 0][BASE ? c : 0] = cs[DS ? r : 0][DS ? c : 0];
                }
#pragma unroll
                for (int r = 0; r < TM; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c) if (BASE) cs[DS ? r : 0][DS ? c : 0] = nv[BASE ? r : 0][BASE ? c : 0];
                if (odd || sub_mask) {                  // rare: zero, FP32 subnormal or overflow somewhere in the micro-tile
                    sub_mask = 0u;
#pragma unroll
                    for (int r = 0; r < TM; ++r)
#pragma unroll
                        for (int c = 0; c < TN; ++c) {
                            const double st = cs[DS ? r : 0][DS ? c : 0];
                            const double v = __hiloint2double(__double2hiint(st), __double2loint(st) & ~1);
                            const uint32_t bit = 1u << (r * TN + c);
                            if (fabs(v) >= (ACC16 ? 65536.0 : 3.402823669209385e38)) {    // |v| >= 2^128 (FP16: the half is infinity): +-infinity from now on
                                if (!((sp_nan | sp_pinf | sp_ninf) & bit)) { if (v < 0.0) sp_ninf |= bit; else sp_pinf |= bit; }
                                cs[DS ? r : 0][DS ? c : 0] = state_of(0u);
                            } else if (fabs(v) < (ACC16 ? 6.103515625e-05 : 1.1754943508222875e-38)) {   // zero or below the normal range: the word decides
                                const uint32_t w = ACC16 ? uint32_t(__half_as_ushort(__double2half(v))) : __float_as_uint(__double2float_rz(v));
                                cs[DS ? r : 0][DS ? c : 0] = state_of(w);
                                if (w & (ACC16 ? 0x7FFFu : 0x7FFFFFFFu)) sub_mask |= bit;
                            }
                        }
                }
            }
        }
        __syncthreads();                                // everybody has finished with this buffer
        if (*reinterpret_cast<volatile int*>(&sm.error)) break;
        if (tid == 0 && chunk + 2 < NCH) issue(chunk + 2);
        // ---- FP32 promotion of the partial sum every k_chunk elements ----
        if (PROMOTE && ((k0 + KC) % g.k_chunk) == 0) {
#pragma unroll
            for (int r = 0; r < TM; ++r)
#pragma unroll
                for (int c = 0; c < TN; ++c) {
                    const uint32_t sp = MMASIM_SP_GET(r, c);
                    const uint32_t pw = sp ? special_word(((sp & 1u) || (sp & 6u) == 6u) ? 1 : ((sp & 2u) ? 2 : 3), ACC16, true)
                                           : positive_zero(DS ? word_of(cs[DS ? r : 0][DS ? c : 0]) : cw[r][c], 0x7FFFFFFFu);
                    float v = __fadd_rn(promoted[PROMOTE ? r : 0][PROMOTE ? c : 0], __uint_as_float(pw));
                    if (v != v) v = __uint_as_float(0x7FFFFFFFu);
                    promoted[PROMOTE ? r : 0][PROMOTE ? c : 0] = v;
                    cw[r][c] = 0u;
                    if (DS) cs[DS ? r : 0][DS ? c : 0] = state_of(0u);
                }
            sp_nan = sp_pinf = sp_ninf = 0u;
            sub_mask = 0u;
        }
    }

    if (*reinterpret_cast<volatile int*>(&sm.error)) {  // a copy never arrived: count it, give the copies in flight one more
        if (tid == 0) {                                 // bounded wait each, and store nothing
            if (g.copy_timeouts) atomicAdd(g.copy_timeouts, 1u);
            fast::mbar_wait(&sm.full[0], 0u);
            fast::mbar_wait(&sm.full[1], 0u);
        }
        return;
    }
    // ---- store ----
#pragma unroll
    for (int r = 0; r < TM; ++r)
#pragma unroll
        for (int c = 0; c < TN; ++c) {
            const int64_t i = row0 + row_at(r), j = col0 + col_at(c);
            if (i >= g.M || j >= g.N) continue;
            const uint32_t sp = MMASIM_SP_GET(r, c);
            uint32_t w = PROMOTE ? __float_as_uint(promoted[PROMOTE ? r : 0][PROMOTE ? c : 0])
                                 : (sp ? special_word(((sp & 1u) || (sp & 6u) == 6u) ? 1 : ((sp & 2u) ? 2 : 3), ACC16, true)
                                       : positive_zero(DS ? word_of(cs[DS ? r : 0][DS ? c : 0]) : cw[r][c], ACC16 ? 0x7FFFu : 0x7FFFFFFFu));   // a zero result is +0
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
}

template <int EK, int L, int RHO, bool PROMOTE, bool ST, int BASE>
cudaError_t launch_one64b(const DevModel& m, const GemmArgs& g, cudaStream_t stream) {
    const size_t sh = sizeof(SmemMM);
    cudaError_t err = cudaFuncSetAttribute(tfdpa64_kernel<EK, L, RHO, PROMOTE, ST, BASE>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(sh));
    if (err != cudaSuccess) return err;
    const size_t dsh_a = 256 * sizeof(LutEntry64) + sizeof(Blk64<BM>), dsh_b = 256 * sizeof(LutEntry64) + sizeof(Blk64<BN>);
    if ((err = cudaFuncSetAttribute(decode64_kernel<EK, BM, true, BASE>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(dsh_a))) != cudaSuccess) return err;
    if ((err = cudaFuncSetAttribute(decode64_kernel<EK, BN, false, BASE>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(dsh_b))) != cudaSuccess) return err;
    const int64_t tiles_m = (g.M + BM - 1) / BM, tiles_n = (g.N + BN - 1) / BN, nch = g.K / KC;
    // scratch: the decoded blocks of A and B, stream-ordered out of the library's pool and returned to it behind the kernel
    const size_t bytes_a = size_t(tiles_m * nch) * sizeof(Blk64<BM>), bytes_b = size_t(tiles_n * nch) * sizeof(Blk64<BN>);
    cudaMemPool_t pool = nullptr;
    if ((err = scratch_pool(&pool)) != cudaSuccess) return err;
    void* ws = nullptr;
    if ((err = cudaMallocFromPoolAsync(&ws, bytes_a + bytes_b, pool, stream)) != cudaSuccess) return err;
    Blk64<BM>* wa = static_cast<Blk64<BM>*>(ws);
    Blk64<BN>* wb = reinterpret_cast<Blk64<BN>*>(static_cast<unsigned char*>(ws) + bytes_a);
    decode64_kernel<EK, BM, true, BASE><<<dim3((unsigned)nch, (unsigned)tiles_m), 256, dsh_a, stream>>>(
        m, static_cast<const unsigned char*>(g.A), g.M, g.lda, wa, ST ? g.sfa : nullptr, g.ld_sfa);
    decode64_kernel<EK, BN, false, BASE><<<dim3((unsigned)nch, (unsigned)tiles_n), 256, dsh_b, stream>>>(
        m, static_cast<const unsigned char*>(g.B), g.N, g.ldb, wb, ST ? g.sfb : nullptr, g.ld_sfb);
    dim3 grid((unsigned)tiles_n, (unsigned)tiles_m, 1);
    tfdpa64_kernel<EK, L, RHO, PROMOTE, ST, BASE><<<grid, NT, sh, stream>>>(m, g, wa, wb);
    err = cudaGetLastError();
    const cudaError_t err2 = cudaFreeAsync(ws, stream);
    return err != cudaSuccess ? err : err2;
}

// The base of the tensor-core exponent maximum by element kinds: FP16 (blocks of 16) 4; 8-bit kinds 4 with an E5M2
// operand, else 8; BF16, TF32 and blocks of 4 and 8: the add-max pass (for blocks of 8 it is as fast, and two of them
// are unrolled per loop trip).
template <int EK, int L, int RHO, bool PROMOTE, bool ST = false>
cudaError_t launch_one64(const DevModel& m, const GemmArgs& g, cudaStream_t stream) {
    if constexpr (EK == fast::EK_F16 && L >= 16) return launch_one64b<EK, L, RHO, PROMOTE, ST, 4>(m, g, stream);
    else if constexpr (EK == fast::EK_LUT8 && L >= 8) {
        if (m.fmt_a == EF_E5M2 || m.fmt_b == EF_E5M2) return launch_one64b<EK, L, RHO, PROMOTE, ST, 4>(m, g, stream);
        return launch_one64b<EK, L, RHO, PROMOTE, ST, 8>(m, g, stream);
    } else return launch_one64b<EK, L, RHO, PROMOTE, ST, 0>(m, g, stream);
}

// With or without FP32 promotion (FP32 accumulators only).
template <int EK, int L, int RHO, bool ST = false>
cudaError_t launch_variant64(const DevModel& m, const GemmArgs& g, cudaStream_t stream) {
    if (RHO != RHO_RNE_FP16 && g.k_chunk) return launch_one64<EK, L, RHO, RHO != RHO_RNE_FP16, ST>(m, g, stream);
    return launch_one64<EK, L, RHO, false, ST>(m, g, stream);
}

}  // namespace fast64
}  // namespace mmasim
