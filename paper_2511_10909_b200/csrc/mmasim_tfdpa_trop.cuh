// T-FDPA for FP8 inputs with F = 13 (the Ada / Hopper FP8 rows, E4M3 and E5M2 in any combination; Algorithm 5 + 7 +
// Table 2): the sum of a block in an FP32 register, one fused multiply-add per term, and the block's exponent maximum
// taken by the tensor cores.
//
// The sum register.  Aligned terms are below 2^15 and block sums below 2^21, so the fixed-point sum S of Algorithm 7
// fits an FP32 register as (1.5 * 2^23 + S) * u with u = 2^(e_max - F): in [2^23 u, 2^24 u) one ulp is u, so
// fma.rm.f32(a, b, register) forms a * b + register exactly and rounds once, toward minus infinity, onto multiples of
// u - the shift by e_max - e_k, the truncation and the addition of Algorithm 7 in one instruction, the alignment
// distance carried by the register's exponent.  Operands are the element values (A) and the element values with an
// offset 2^-(pre + guard) below the last significand bit (B), so that a negative product is never on the grid and
// floors to the one's complement of its truncated magnitude; a population count over sign / nonzero masks adds the
// number of negative nonzero terms back.  The accumulator enters by one addition rounded toward minus infinity (its
// lowest mantissa bit set, so that a negative c floors likewise; the +1 is added to the register's starting value),
// and the block's value S * u leaves by one exact subtraction of 1.5 * 2^23 * u; rho is a mask (RZ-E8M13) or a
// conversion (RNE-FP16).  The accumulator between blocks is the output word itself.
//
// e_max = max_k (Exp(a_k) + Exp(b_k)) is a (max, +) product.  Powers turn it into an ordinary one: with
// pe(x) = 2^(6 (Exp(x) - 1)) for a nonzero finite x and 0 otherwise (the B plane scaled by 2^5 more),
//     P = sum_k pe(a_k) * pe(b_k)  lies in  2^(6 (e_max + 20) - 127) * [1, 32]  (at most 32 terms, 32 < 2^6),
// so its FP32 exponent field is 6 (e_max + 20) + 0..5 and floor(field / 6) - 20 = e_max exactly, whatever the order,
// rounding or truncation of the summation (terms far below the largest may be dropped, they do not matter).  E4M3
// exponents span 15 values: 6 * (Exp - 1) stays within +-42 and P within the FP32 range; with E5M2 operands the base
// is 2^5 or 2^4 and P is taken over sub-blocks of 16 or 8 terms (see pe_shift below).  P for the 32 x 32 outputs
// of a warp and one block of 32 is sixteen mma.sync.m16n8k16 on BF16 planes of pe values (a power of two is exact in
// BF16), instead of sixteen fused add-max instructions per output; P = 0 (every product zero: no exponent) converts
// to an exponent below every real one.  The division by the base is one high multiply on the bits of P, which leaves
// the result as an FP32 exponent field in place, comparable with the bits of |c| and a mask away from the sum
// register's starting value.
//
// A warp owns 32 rows x 32 columns of the CTA tile (two by four accumulator fragments), and the micro-tile of a thread is
// its share of those fragments: rows g, g + 8, g + 16, g + 24 (g = lane / 4) and columns 8 j + 2 t, 8 j + 2 t + 1
// (t = lane % 4, j = 0..3), so that the maxima arrive in the registers of the thread that needs them.  The operand
// planes are stored with rows and columns permuted accordingly (the four rows of a thread adjacent, its eight
// columns contiguous): three 16-byte shared loads feed the 32 fused multiply-adds of one k, which are issued as
// sixteen packed ones (fma.rm.f32x2: two adjacent columns per instruction).
#pragma once
#include <type_traits>
#include "mmasim_tfdpa_fast.cuh"

namespace mmasim {
namespace trop {

using fast::BM;
using fast::KC;
using fast::NT;
using fast::CB;
using fast::Elem;
using fast::raw_elem;
using fast::mbar_init;
using fast::mbar_expect_tx;
using fast::bulk_load;
using fast::mbar_wait;
using fast::smem_addr;

constexpr int PE_STRIDE = KC + 8;       // BF16 elements per row of a pe plane: 80 bytes, fragment loads hit 32 different banks
constexpr int PE_CENTER = 1;            // pe(x) = 2^(6 (Exp(x) - PE_CENTER)); E4M3: Exp in [-6, 8]
// pe(x) = 2^(BASE (Exp(x) - PE_CENTER)), the B plane times 2^pe_shift so that 127 + pe_shift is a multiple of BASE and
// the exponent field of P is BASE * (e_max + constant) + 0..BASE-1.  A sum of at most 2^(BASE-1) terms stays within a
// factor 2^(BASE-1) of its largest term; the spread of the exponents decides which BASE fits the FP32 range:
//   BASE 8: blocks of up to 32 terms in one accumulation; E4M3 x E4M3 (product exponents -12..16: 8 * 28 = 224 binades,
//           plus the 5 binades a sum of 32 terms can grow; the division by 8 is a shift)
//   BASE 5: sub-blocks of 16 terms; E4M3 x E5M2 (-20..23: 5 * 43 = 215 binades)
//   BASE 4: sub-blocks of 8 terms;  E5M2 x E5M2 (-28..30: 4 * 58 = 232 binades)
// The block maximum is then the integer maximum of the sub-blocks' P words.
__host__ __device__ constexpr int pe_shift(int base) { return base == 8 ? 1 : (base == 5 ? 3 : 1); }
__host__ __device__ constexpr int pe_sub(int base) { return base == 8 ? 32 : (base == 5 ? 16 : 8); }
__host__ __device__ constexpr uint32_t pe_mul(int base) { return base == 5 ? 0x33333334u : 0u; }  // ceil(2^32 / BASE); powers of two shift
constexpr int TW = 8;                   // micro-tile: TH rows x 8 columns

// Geometry by the height TH of the micro-tile.  TH = 4: warps 4 x 2, warp tile 32 x 32, CTA tile 128 x 64.
// TH = 8: warps 2 x 4, warp tile 64 x 32, CTA tile 128 x 128 - sixteen operand words per 64 multiply-adds instead of
// twelve per 32, at the price of 64 accumulator registers (used where nothing else has to live across the K loop).
template <int TH>
struct Geo {
    static_assert(TH == 4 || TH == 8, "two or four accumulator fragments stacked");
    static constexpr int WROWS = 8 * TH;                // rows of a warp tile
    static constexpr int WARPS_R = BM / WROWS, WARPS_C = (NT / 32) / WARPS_R;
    static constexpr int BN = 32 * WARPS_C;
    static constexpr int NB = BN * KC / NT;             // elements of B staged per thread: 8 or 16
};

struct LutEntryT {      // 8 bytes: one shared load per staged element
    uint32_t op;        // staged FP32 operand
    uint32_t y;         // bits 0..14: BF16 word of pe(x); bit 15: infinity / NaN (a pe of -0: harmless in P);
                        // bit 16: sign; bit 24: finite and nonzero
};

// One operand's share of a chunk of KC = 32 elements of K, decoded: R rows of A (or columns of B).  A decode kernel
// writes these blocks to scratch memory once per GEMM; the main kernel brings them in with one bulk copy each.
template <int R>
struct BlkT {
    uint32_t op[KC][R];                 // [k][permuted row]: FP32 operands
    uint16_t pe[R][PE_STRIDE];          // [row][k]: BF16 exponent powers for the tensor cores
    uint32_t sgn[R], nz[R];             // [permuted row]: bit k = sign / nonzero of element k of the chunk
    uint32_t special;                   // nonzero: the block holds an infinity or a NaN
    uint32_t pad[3];
};
static_assert(sizeof(BlkT<128>) % 16 == 0 && sizeof(BlkT<64>) % 16 == 0, "bulk copies move multiples of 16 bytes");

template <int TH>
struct SmemT {
    BlkT<BM> a[2];
    BlkT<Geo<TH>::BN> b[2];
    unsigned long long full[2];         // mbarriers: the bulk copies of a buffer have landed
    int error;                          // a bounded wait ran out
};

// Position of a row / column of the CTA tile inside the permuted planes: the TH rows of a thread (g, g + 8, ...)
// adjacent, its eight columns (8 j + 2 t, 8 j + 2 t + 1) contiguous.
template <int TH>
__device__ __forceinline__ int perm_row(int r) {
    return TH == 4 ? ((r & ~31) | ((r & 7) << 2) | ((r >> 3) & 3)) : ((r & ~63) | ((r & 7) << 3) | ((r >> 3) & 7));
}
__device__ __forceinline__ int perm_col(int c) { return (c & ~31) | (((c >> 1) & 3) << 3) | (((c >> 3) & 3) << 1) | (c & 1); }

template <int BASE>
__device__ __forceinline__ void init_lut_t(LutEntryT* lut_a, LutEntryT* lut_b, const FmtDesc& fa, const FmtDesc& fb, int pre, int guard, int tid) {
    const uint32_t da = decode_elem(fa, uint32_t(tid)), db = decode_elem(fb, uint32_t(tid));
    const bool fin_a = dec_cls(da) == CLS_FINITE, fin_b = dec_cls(db) == CLS_FINITE;
    const bool nz_a = fin_a && dec_sig(da) != 0u, nz_b = fin_b && dec_sig(db) != 0u;
    LutEntryT ea, eb;
    ea.op = __float_as_uint(ldexpf(float(fin_a ? dec_ssig(da) : 0), fin_a ? dec_exp(da) : 0));
    ea.y = (nz_a ? uint32_t((127 + BASE * (dec_exp(da) - PE_CENTER)) << 7) : 0u) | (fin_a ? 0u : 0x8000u) |
           (fin_a ? (dec_sign(da) << 16) | (uint32_t(nz_a) << 24) : 0u);
    const int sb = fin_b ? dec_ssig(db) : 0;
    const int ub = dec_sign(db) ? -1 : 1;
    // a_op * b_op = a * b * (1 + 2^-(pre + guard) / |sig_b|): the true product with the offset that makes a negative one inexact
    eb.op = nz_b ? __float_as_uint(ldexpf(float(sb * (1 << (pre + guard)) + ub), dec_exp(db) - (fa.mbits + fb.mbits + pre + guard))) : 0u;
    eb.y = (nz_b ? uint32_t((127 + pe_shift(BASE) + BASE * (dec_exp(db) - PE_CENTER)) << 7) : 0u) | (fin_b ? 0u : 0x8000u) |
           (fin_b ? (dec_sign(db) << 16) | (uint32_t(nz_b) << 24) : 0u);
    lut_a[tid] = ea;
    lut_b[tid] = eb;
}

// N = 16 or 8 elements of one row: operands k-major, pe words row-major, sign / nonzero bits into the masks.
template <int N, int R>
__device__ __forceinline__ uint32_t stage_row(const LutEntryT* lut, BlkT<R>& s, const uint32_t (&w)[N / 4], int r, int pr, int part) {
    uint32_t* op = &s.op[part * N][pr];
    uint32_t acc = 0u, spec = 0u, pw[N / 2];
#pragma unroll
    for (int q = 0; q < N; q += 2) {
        const uint2 e0 = *reinterpret_cast<const uint2*>(&lut[(w[q / 4] >> (8 * (q % 4))) & 0xFFu]);
        const uint2 e1 = *reinterpret_cast<const uint2*>(&lut[(w[q / 4] >> (8 * (q % 4) + 8)) & 0xFFu]);
        op[q * R] = e0.x;
        op[(q + 1) * R] = e1.x;
        // sign byte -> bits 0.., nonzero byte -> bits 16..
        acc += (__byte_perm(e0.y, 0u, 0x4342) << q) + (__byte_perm(e1.y, 0u, 0x4342) << (q + 1));
        spec |= e0.y | e1.y;
        pw[q / 2] = __byte_perm(e0.y, e1.y, 0x5410);
    }
    uint16_t* pe = &s.pe[r][part * N];
#pragma unroll
    for (int q = 0; q < N / 8; ++q)
        reinterpret_cast<uint4*>(pe)[q] = make_uint4(pw[4 * q], pw[4 * q + 1], pw[4 * q + 2], pw[4 * q + 3]);
    if (N == 16) {
        reinterpret_cast<uint16_t*>(&s.sgn[pr])[part] = uint16_t(acc);
        reinterpret_cast<uint16_t*>(&s.nz[pr])[part] = uint16_t(acc >> 16);
    } else {
        reinterpret_cast<uint8_t*>(&s.sgn[pr])[part] = uint8_t(acc);
        reinterpret_cast<uint8_t*>(&s.nz[pr])[part] = uint8_t(acc >> 16);
    }
    return spec;
}

// Decode pass: one CTA decodes one block (R rows of A or columns of B x 32 elements of K) through a 256-entry table of
// 8-byte entries into shared memory and copies it to its place in the scratch array dst[tile][chunk].  Every thread
// takes 16 (R = 128) or 8 (R = 64) consecutive elements of one row.  Rows beyond the matrix decode as zeros.
static_assert(BM == 128 && KC == 32 && NT == 256, "the task split of the decode pass");
template <int BASE, int R, bool IS_A, int TH>
__global__ void __launch_bounds__(NT) trop_decode_kernel(DevModel m, const unsigned char* src, int64_t rows, int64_t ld, int F,
                                                         BlkT<R>* dst) {
    __shared__ __align__(16) LutEntryT lut_a[256];
    __shared__ __align__(16) LutEntryT lut_b[256];
    __shared__ __align__(16) BlkT<R> blk;
    const int tid = threadIdx.x;
    const FmtDesc fa = fmt_desc(m.fmt_a), fb = fmt_desc(m.fmt_b);
    init_lut_t<BASE>(lut_a, lut_b, fa, fb, F - (fa.mbits + fb.mbits), fa.mbits + 1, tid);
    if (tid == 0) { blk.special = 0u; blk.pad[0] = blk.pad[1] = blk.pad[2] = 0u; }
    constexpr int N = R * KC / NT;                      // elements per thread: 16 or 8
    const int r = tid % R, part = tid / R;
    const int64_t i = int64_t(blockIdx.y) * R + r, k0 = int64_t(blockIdx.x) * KC;
    uint32_t w[N / 4];
    if (N == 16) {
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (i < rows) v = *reinterpret_cast<const uint4*>(src + i * ld + k0 + N * part);
        w[0] = v.x; w[1] = v.y; w[N / 4 - 2] = v.z; w[N / 4 - 1] = v.w;
    } else {
        uint2 v = make_uint2(0u, 0u);
        if (i < rows) v = *reinterpret_cast<const uint2*>(src + i * ld + k0 + N * part);
        w[0] = v.x; w[1] = v.y;
    }
    __syncthreads();
    const uint32_t spec = stage_row<N, R>(IS_A ? lut_a : lut_b, blk, w, r, IS_A ? perm_row<TH>(r) : perm_col(r), part);
    if (spec & 0x8000u) atomicOr(&blk.special, 1u);
    __syncthreads();
    uint4* out = reinterpret_cast<uint4*>(dst + (int64_t(blockIdx.y) * gridDim.x + blockIdx.x));
    const uint4* in = reinterpret_cast<const uint4*>(&blk);
    for (int q = tid; q < int(sizeof(BlkT<R>) / 16); q += NT) out[q] = in[q];
}


template <int EK, int L, int F, int RHO, bool PROMOTE, int BASE, int TH>
__global__ void __launch_bounds__(NT, 2) tfdpa_trop_kernel(DevModel m, GemmArgs g, const BlkT<BM>* __restrict__ wa,
                                                           const BlkT<Geo<TH>::BN>* __restrict__ wb) {
    constexpr bool ACC16 = RHO == RHO_RNE_FP16;
    constexpr int NBLK = KC / L;
    static_assert(KC % L == 0 && L % 16 == 0, "a block is one or two k16 matrix instructions");
    static_assert(BASE == 4 || BASE == 5 || BASE == 8, "see pe_shift");
    constexpr int KSUB = pe_sub(BASE) < L ? pe_sub(BASE) : L, NSUB = L / KSUB;        // terms per accumulation of P
    static_assert(!Elem<EK>::SIGNMAG && F <= 13, "8-bit inputs with F <= 13");
    static_assert(RHO == RHO_RZ_E8M13 || RHO == RHO_RNE_FP16, "rho of the F = 13 rows of Table 4");
    using G = Geo<TH>;
    constexpr int BN = G::BN;
    using mask_t = std::conditional_t<(TH * TW > 32), unsigned long long, uint32_t>;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SmemT<TH>& sm = *reinterpret_cast<SmemT<TH>*>(smem_raw);

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int gq = lane >> 2, tq = lane & 3;
    const int row0 = int(blockIdx.y) * BM, col0 = int(blockIdx.x) * BN;        // M, N < 2^31 (checked by the dispatcher)
    const int wr = warp / G::WARPS_C, wc = warp % G::WARPS_C;                  // the warp's part of the CTA tile
    auto row_of = [&](int h) { return wr * G::WROWS + 16 * (h >> 1) + 8 * (h & 1) + gq; };    // inside the CTA tile
    auto col_of = [&](int x) { return wc * 32 + 8 * (x >> 1) + 2 * tq + (x & 1); };
    const FmtDesc fa = fmt_desc(m.fmt_a), fb = fmt_desc(m.fmt_b);
    const int pre = F - (fa.mbits + fb.mbits);
    const int guard = fa.mbits + 1;
    // Exponents are handled as FP32 exponent fields in place (bits 23..30) with whatever lies below as a fraction:
    //   t1 = floor(bits(P) / BASE) + T1_ADD: field e_max + 127 for the largest product (P = 0: a field below that of
    //        the smallest nonzero product); the division is a high multiply, inexact by 2^-30 at most, and P is never
    //        closer than 1 / BASE to the next multiple;
    //   ca = |c|: field Exp(c) + 127.
    // Sum register: (1.5 * 2^23 + S) * 2^(e_max - F), exponent field e + (23 - F).
    constexpr uint32_t MUL = pe_mul(BASE), T1_ADD = uint32_t(127 - (127 + pe_shift(BASE)) / BASE + 2 * PE_CENTER) << 23;
    constexpr uint32_t FIELD = 0x7F800000u, HALF = 0x00400000u;
    constexpr uint32_t RHO_MASK = ACC16 ? 0xFFFFFFFFu : 0xFFFFFC00u;   // RZ-E8M13 of an FP32 word whose exponent stays
    constexpr uint32_t MAGIC_ADD = (uint32_t(23 - F) << 23) | HALF;
    // Below E_LOW no product is nonzero, above E_HIGH the register would overflow (and every product is far below one
    // unit of the accumulator): the result is rho of the accumulator alone.  Such an output rides through pass 2 as a
    // marker KEEP + payload whose unit exceeds every product, so that a term changes it by -1 or not at all, which the
    // sign correction undoes.  FP16 accumulators are never out of range.
    const uint32_t E_LOW = ACC16 ? 0u : uint32_t(127 + 2 - fa.bias - fb.bias) << 23;
    constexpr uint32_t E_HIGH = (241u << 23) - 1u;
    constexpr uint32_t E_KEEP = 243u << 23, KEEP = E_KEEP + MAGIC_ADD;
    static_assert(F == 13 || ACC16, "the kept word is carried as its upper 22 bits");
    // the decoded blocks of this tile row of A and tile column of B, chunk after chunk, land in two buffers by bulk copies
    const int K = int(g.K), NCH = K / KC;
    const BlkT<BM>* src_a = wa + int64_t(blockIdx.y) * NCH;
    const BlkT<BN>* src_b = wb + int64_t(blockIdx.x) * NCH;
    auto issue = [&](int n) {                              // one thread: both copies of chunk n into buffer n & 1
        unsigned long long* bar = &sm.full[n & 1];
        mbar_expect_tx(bar, uint32_t(sizeof(BlkT<BM>) + sizeof(BlkT<BN>)));
        bulk_load(&sm.a[n & 1], src_a + n, uint32_t(sizeof(BlkT<BM>)), bar);
        bulk_load(&sm.b[n & 1], src_b + n, uint32_t(sizeof(BlkT<BN>)), bar);
    };
    if (tid == 0) {
        sm.error = 0;
        mbar_init(&sm.full[0], 1u);
        mbar_init(&sm.full[1], 1u);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        issue(0);
        if (NCH > 1) issue(1);
    }

    uint32_t cw[TH][TW];
    mask_t sp_nan = 0, sp_pinf = 0, sp_ninf = 0;        // per output (bit h * TW + x)
    float promoted[PROMOTE ? TH : 1][PROMOTE ? TW : 1];
#define MMASIM_SP_GET(h, x) (uint32_t((sp_nan >> ((h) * TW + (x))) & 1u) | (uint32_t((sp_pinf >> ((h) * TW + (x))) & 1u) << 1) | (uint32_t((sp_ninf >> ((h) * TW + (x))) & 1u) << 2))
#define MMASIM_SP_WORD(h, x, w) (MMASIM_SP_GET(h, x) ? special_word(((MMASIM_SP_GET(h, x) & 1u) || (MMASIM_SP_GET(h, x) & 6u) == 6u) ? 1 : ((MMASIM_SP_GET(h, x) & 2u) ? 2 : 3), ACC16, true) : (w))
#pragma unroll
    for (int h = 0; h < TH; ++h)
#pragma unroll
        for (int x = 0; x < TW; ++x) {
            const int64_t i = row0 + row_of(h), j = col0 + col_of(x);
            uint32_t w = 0u;
            if (g.C && i < g.M && j < g.N)
                w = ACC16 ? uint32_t(static_cast<const uint16_t*>(g.C)[i * g.ldc + j])
                          : static_cast<const uint32_t*>(g.C)[i * g.ldc + j];
            if (PROMOTE) { promoted[PROMOTE ? h : 0][PROMOTE ? x : 0] = __uint_as_float(w); w = 0u; }
            const AccDec d = decode_acc(w, ACC16);
            if (d.cls != CLS_FINITE) {
                const mask_t bit = mask_t(1) << (h * TW + x);
                if (d.cls == CLS_NAN) sp_nan |= bit; else if (d.sign) sp_ninf |= bit; else sp_pinf |= bit;
                w = 0u;
            }
            cw[h][x] = w;
        }

    __syncthreads();                                       // the barriers are initialised
    for (int chunk = 0; chunk < NCH; ++chunk) {
        const int k0 = chunk * KC;
        // a wait that runs out is recorded and the chunk computed on whatever is there; every thread sees the flag after
        // the barrier at the end of the chunk, and the CTA leaves together without storing anything
        if (!mbar_wait(&sm.full[chunk & 1], uint32_t(chunk >> 1) & 1u)) *reinterpret_cast<volatile int*>(&sm.error) = 1;
        const BlkT<BM>& sa_blk = sm.a[chunk & 1];
        const BlkT<BN>& sb_blk = sm.b[chunk & 1];
        const bool chunk_special = (sa_blk.special | sb_blk.special) != 0u;

#pragma unroll 1
        for (int blk = 0; blk < NBLK; ++blk) {
            const int kb = blk * L;
            if (chunk_special) {                           // rare: special-value events of this block (Section 4.2)
#pragma unroll 1
                for (int h = 0; h < TH; ++h)
#pragma unroll 1
                    for (int x = 0; x < TW; ++x) {
                        const int64_t i = row0 + row_of(h), j = col0 + col_of(x);
                        if (i >= g.M || j >= g.N) continue;
                        Special ev;
                        for (int kk = kb; kk < kb + L; ++kk) {
                            const uint32_t xa = decode_elem(fa, raw_elem<EK>(g.A, i * g.lda + k0 + kk));
                            const uint32_t yb = decode_elem(fb, raw_elem<EK>(g.B, j * g.ldb + k0 + kk));
                            ev.product(xa, yb);
                        }
                        const mask_t bit = mask_t(1) << (h * TW + x);
                        if (ev.nan) sp_nan |= bit;
                        if (ev.pinf) sp_pinf |= bit;
                        if (ev.ninf) sp_ninf |= bit;
                    }
            }

            // ---- pass 1 on the tensor cores: P = sum_k pe(a_k) pe(b_k), one accumulation per sub-block of KSUB terms,
            // the block's P the integer maximum of their words; one accumulator fragment row (16 x 32 outputs of the
            // warp, two rows of the micro-tile) at a time, followed at once by its sum registers ----
            constexpr int NK = KSUB >= 16 ? KSUB / 16 : 1;                 // matrix instructions per accumulation
            constexpr int AR = KSUB >= 16 ? 4 : 2, BR = KSUB >= 16 ? 2 : 1;
            bool rare = false;
#pragma unroll
            for (int mt = 0; mt < TH / 2; ++mt) {
                uint32_t P[4][4];
#pragma unroll
                for (int sub = 0; sub < NSUB; ++sub) {
                    uint32_t af[NK][AR];
                    const int ar = wr * G::WROWS + 16 * mt + gq;
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
                    for (int j = 0; j < 4; ++j) {
                        uint32_t bf[NK][BR];
#pragma unroll
                        for (int ks = 0; ks < NK; ++ks) {
                            const int kq = kb + sub * KSUB + 16 * ks + 2 * tq;
                            bf[ks][0] = *reinterpret_cast<const uint32_t*>(&sb_blk.pe[wc * 32 + 8 * j + gq][kq]);
                            if (BR == 2) bf[ks][BR - 1] = *reinterpret_cast<const uint32_t*>(&sb_blk.pe[wc * 32 + 8 * j + gq][kq + 8]);
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
                // e = max(exponent of the largest product, exponent of the accumulator), kept in the register of P
                uint32_t out_of_range = 0u;
#pragma unroll
                for (int hh = 0; hh < 2; ++hh)
#pragma unroll
                    for (int x = 0; x < TW; ++x) {
                        const int h = 2 * mt + hh;
                        uint32_t& p = P[x >> 1][2 * hh + (x & 1)];
                        const uint32_t t1 = (BASE == 5 ? __umulhi(p, MUL) : (p >> (BASE == 8 ? 3 : 2))) + T1_ADD;
                        uint32_t e;
                        if (ACC16) {
                            // a subnormal FP16 accumulator has the exponent -14, not that of its leading bit.  BASE 6: the
                            // floor also covers c = 0, harmlessly (every nonzero E4M3 product has an exponent of at least
                            // -12); with E5M2 operands products reach down to 2^-28 and a zero accumulator must not count
                            uint32_t ca = __float_as_uint(__half2float(__ushort_as_half((unsigned short)(cw[h][x] & 0x7FFFu))));
                            if (BASE == 8) e = uint32_t(__vimax3_s32(int(t1), int(ca), int(113u << 23)));
                            else { if (ca) ca = max(ca, 113u << 23); e = max(t1, ca); }
                        } else {
                            // |c| and t1 are positive FP32 patterns: their order as numbers is their order as words, and
                            // the absolute value rides on the instruction
                            e = __float_as_uint(fmaxf(__uint_as_float(t1), fabsf(__uint_as_float(cw[h][x]))));
                            out_of_range = __viaddmax_u32(e, 0u - E_LOW, out_of_range);
                        }
                        p = e;
                    }
                if (!ACC16 && out_of_range > E_HIGH - E_LOW) {     // rare: turn the outputs out of range into markers (see above)
                    rare = true;
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh)
#pragma unroll
                        for (int x = 0; x < TW; ++x) {
                            const int h = 2 * mt + hh;
                            uint32_t& p = P[x >> 1][2 * hh + (x & 1)];
                            if (p - E_LOW > E_HIGH - E_LOW) {
                                const uint32_t c = cw[h][x];
                                const uint32_t kept = (c & 0x7FFFFFFFu) ? (c >> 10) : 0u;      // rho(c); an exactly zero sum is +0
                                p = E_KEEP;
                                cw[h][x] = __float_as_uint(__uint2float_rn(kept) * __uint_as_float(uint32_t(E_KEEP >> 23) + uint32_t(23 - F) - 23u << 23));
                            }
                        }
                }
                // the sum register with the accumulator term: floor((c + tiny) / unit); a negative c is one short
#pragma unroll
                for (int hh = 0; hh < 2; ++hh)
#pragma unroll
                    for (int xp = 0; xp < TW / 2; ++xp) {          // two adjacent columns per packed addition
                        const int h = 2 * mt + hh;
                        uint32_t magic[2], cb[2];
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            const uint32_t e = P[xp][2 * hh + q];
                            const uint32_t c = cw[h][2 * xp + q];
                            magic[q] = (e & FIELD) + MAGIC_ADD + (c >> (ACC16 ? 15 : 31));
                            const float cf = ACC16 ? __half2float(__ushort_as_half((unsigned short)c)) : __uint_as_float(c);
                            cb[q] = __float_as_uint(cf) | 1u;
                        }
                        asm("{\n\t.reg .b64 a, b, r;\n\tmov.b64 a, {%2, %3};\n\tmov.b64 b, {%4, %5};\n\tadd.rm.f32x2 r, a, b;\n\tmov.b64 {%0, %1}, r;\n\t}"
                            : "=r"(cw[h][2 * xp]), "=r"(cw[h][2 * xp + 1]) : "r"(cb[0]), "r"(cb[1]), "r"(magic[0]), "r"(magic[1]));
                    }
            }
            // ---- pass 2: one fused multiply-add per term, rounding toward minus infinity onto the grid of S; two
            // columns of the micro-tile per instruction (fma.rm.f32x2: lanes (a_h, a_h) x (b_x, b_x+1) + (S_h,x, S_h,x+1)) ----
            {
                unsigned long long acc[TH][TW / 2];
#pragma unroll
                for (int h = 0; h < TH; ++h)
#pragma unroll
                    for (int xp = 0; xp < TW / 2; ++xp)
                        asm("mov.b64 %0, {%1, %2};" : "=l"(acc[h][xp]) : "r"(cw[h][2 * xp]), "r"(cw[h][2 * xp + 1]));
#pragma unroll
                for (int kk = kb; kk < kb + L; ++kk) {
                    float oas[TH];
#pragma unroll
                    for (int q = 0; q < TH / 4; ++q) {
                        const float4 oa = *reinterpret_cast<const float4*>(&sa_blk.op[kk][wr * G::WROWS + TH * gq + 4 * q]);
                        oas[4 * q] = oa.x; oas[4 * q + 1] = oa.y; oas[4 * q + 2] = oa.z; oas[4 * q + 3] = oa.w;
                    }
                    const ulonglong2 ob0 = *reinterpret_cast<const ulonglong2*>(&sb_blk.op[kk][wc * 32 + 8 * tq]);
                    const ulonglong2 ob1 = *reinterpret_cast<const ulonglong2*>(&sb_blk.op[kk][wc * 32 + 8 * tq + 4]);
                    const unsigned long long obv[TW / 2] = {ob0.x, ob0.y, ob1.x, ob1.y};
#pragma unroll
                    for (int h = 0; h < TH; ++h) {
                        unsigned long long oav;
                        asm("mov.b64 %0, {%1, %1};" : "=l"(oav) : "f"(oas[h]));
#pragma unroll
                        for (int xp = 0; xp < TW / 2; ++xp)
                            asm("fma.rm.f32x2 %0, %1, %2, %0;" : "+l"(acc[h][xp]) : "l"(oav), "l"(obv[xp]));
                    }
                }
#pragma unroll
                for (int h = 0; h < TH; ++h)
#pragma unroll
                    for (int xp = 0; xp < TW / 2; ++xp)
                        asm("mov.b64 {%0, %1}, %2;" : "=r"(cw[h][2 * xp]), "=r"(cw[h][2 * xp + 1]) : "l"(acc[h][xp]));
            }
            // ---- sign corrections and rho ----
            const uint32_t kmask = (L == 32) ? 0xFFFFFFFFu : (((1u << L) - 1u) << kb);
            uint32_t wmax = 0u;
            uint32_t sbv[TW], nzb[TW];
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const uint4 u = *reinterpret_cast<const uint4*>(&sb_blk.sgn[wc * 32 + 8 * tq + 4 * q]);
                const uint4 v = *reinterpret_cast<const uint4*>(&sb_blk.nz[wc * 32 + 8 * tq + 4 * q]);
                sbv[4 * q] = u.x; sbv[4 * q + 1] = u.y; sbv[4 * q + 2] = u.z; sbv[4 * q + 3] = u.w;
                nzb[4 * q] = v.x; nzb[4 * q + 1] = v.y; nzb[4 * q + 2] = v.z; nzb[4 * q + 3] = v.w;
            }
            auto finish = [&](auto with_markers) {
#pragma unroll
                for (int h = 0; h < TH; ++h) {
                    const uint32_t sa = sa_blk.sgn[wr * G::WROWS + TH * gq + h];
                    const uint32_t nza = sa_blk.nz[wr * G::WROWS + TH * gq + h] & kmask;
                    uint32_t bitsv[TW], vv[TW];
#pragma unroll
                    for (int x = 0; x < TW; ++x)                   // every negative nonzero term fell one unit short:
                        bitsv[x] = cw[h][x] + uint32_t(__popc((sa ^ sbv[x]) & nza & nzb[x]));   // (1.5 * 2^23 + S) * unit
#pragma unroll
                    for (int xp = 0; xp < TW / 2; ++xp)            // S * unit, exact; two columns per packed subtraction
                        asm("{\n\t.reg .b64 a, b, r;\n\tmov.b64 a, {%2, %3};\n\tmov.b64 b, {%4, %5};\n\tsub.rn.f32x2 r, a, b;\n\tmov.b64 {%0, %1}, r;\n\t}"
                            : "=r"(vv[2 * xp]), "=r"(vv[2 * xp + 1])
                            : "r"(bitsv[2 * xp]), "r"(bitsv[2 * xp + 1]), "r"((bitsv[2 * xp] & FIELD) | HALF), "r"((bitsv[2 * xp + 1] & FIELD) | HALF));
#pragma unroll
                    for (int x = 0; x < TW; ++x) {
                        const uint32_t bits = bitsv[x];
                        const float v = __uint_as_float(vv[x]);
                        uint32_t w;
                        if (ACC16) { w = uint32_t(__half_as_ushort(__float2half_rn(v))); wmax = max(wmax, w & 0x7FFFu); }
                        else w = __float_as_uint(v);     // RZ-E8M13 is applied where the word leaves the chain (below): the next
                                                         // block's alignment truncates on a grid at least as coarse
                        if (decltype(with_markers)::value && bits >= KEEP) w = (bits - KEEP) << 10;
                        cw[h][x] = w;
                    }
                }
            };
            if (rare) finish(std::true_type{}); else finish(std::false_type{});
            if (ACC16 && wmax >= 0x7C00u) {                // rare: RNE-FP16 overflowed: +-infinity from now on
#pragma unroll
                for (int h = 0; h < TH; ++h)
#pragma unroll
                    for (int x = 0; x < TW; ++x)
                        if ((cw[h][x] & 0x7FFFu) == 0x7C00u) {
                            const mask_t bit = mask_t(1) << (h * TW + x);
                            if (!((sp_nan | sp_pinf | sp_ninf) & bit)) { if (cw[h][x] >> 15) sp_ninf |= bit; else sp_pinf |= bit; }
                            cw[h][x] = 0u;
                        }
            }
        }
        __syncthreads();                                   // everybody has finished with this buffer
        if (*reinterpret_cast<volatile int*>(&sm.error)) break;
        if (tid == 0 && chunk + 2 < NCH) issue(chunk + 2);
        if (PROMOTE && ((k0 + KC) % int(g.k_chunk)) == 0) {     // FP32 promotion of the partial sum every k_chunk elements
#pragma unroll
            for (int h = 0; h < TH; ++h)
#pragma unroll
                for (int x = 0; x < TW; ++x) {
                    const float part = __uint_as_float(MMASIM_SP_WORD(h, x, positive_zero(cw[h][x] & RHO_MASK, 0x7FFFFFFFu)));
                    float v = __fadd_rn(promoted[PROMOTE ? h : 0][PROMOTE ? x : 0], part);
                    if (v != v) v = __uint_as_float(0x7FFFFFFFu);
                    promoted[PROMOTE ? h : 0][PROMOTE ? x : 0] = v;
                    cw[h][x] = 0u;
                }
            sp_nan = sp_pinf = sp_ninf = 0;
        }
    }

    if (*reinterpret_cast<volatile int*>(&sm.error)) {     // a copy never arrived: count it, give the copies in flight one more
        if (tid == 0) {                                    // bounded wait each, and store nothing
            if (g.copy_timeouts) atomicAdd(g.copy_timeouts, 1u);
            mbar_wait(&sm.full[0], 0u);
            mbar_wait(&sm.full[1], 0u);
        }
        return;
    }
#pragma unroll
    for (int h = 0; h < TH; ++h)
#pragma unroll
        for (int x = 0; x < TW; ++x) {
            const int64_t i = row0 + row_of(h), j = col0 + col_of(x);
            if (i >= g.M || j >= g.N) continue;
            // a chain's last word of magnitude zero is +0 (in between the sign of a zero does not matter: it has no exponent)
            uint32_t w = PROMOTE ? __float_as_uint(promoted[PROMOTE ? h : 0][PROMOTE ? x : 0])
                                 : MMASIM_SP_WORD(h, x, positive_zero(cw[h][x] & RHO_MASK, ACC16 ? 0x7FFFu : 0x7FFFFFFFu));
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

// Where the decoded blocks go: memory of the caller's (given != nullptr, capacity bytes) or, by default, a stream-ordered
// allocation out of the library's pool, returned to it behind the kernel.
struct Scratch {
    void* given = nullptr;
    size_t capacity = 0;
};

template <int TH>
size_t scratch_bytes_one(const GemmArgs& g) {
    constexpr int BN = Geo<TH>::BN;
    const int64_t tiles_m = (g.M + BM - 1) / BM, tiles_n = (g.N + BN - 1) / BN, nch = g.K / KC;
    return size_t(tiles_m * nch) * sizeof(BlkT<BM>) + size_t(tiles_n * nch) * sizeof(BlkT<BN>);
}

template <int EK, int L, int F, int RHO, bool PROMOTE, int BASE, int TH>
cudaError_t launch_one_t(const DevModel& m, const GemmArgs& g, cudaStream_t stream, const Scratch& sc) {
    constexpr int BN = Geo<TH>::BN;
    const size_t sh = sizeof(SmemT<TH>);
    cudaError_t err = cudaFuncSetAttribute(tfdpa_trop_kernel<EK, L, F, RHO, PROMOTE, BASE, TH>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(sh));
    if (err != cudaSuccess) return err;
    const int64_t tiles_m = (g.M + BM - 1) / BM, tiles_n = (g.N + BN - 1) / BN, nch = g.K / KC;
    const size_t bytes_a = size_t(tiles_m * nch) * sizeof(BlkT<BM>), bytes_b = size_t(tiles_n * nch) * sizeof(BlkT<BN>);
    void* ws = sc.given;
    if (ws) {
        if (bytes_a + bytes_b > sc.capacity) return cudaErrorInvalidValue;      // the caller checked: never reached
    } else {
        cudaMemPool_t pool = nullptr;
        if ((err = scratch_pool(&pool)) != cudaSuccess) return err;
        if ((err = cudaMallocFromPoolAsync(&ws, bytes_a + bytes_b, pool, stream)) != cudaSuccess) return err;
    }
    BlkT<BM>* wa = static_cast<BlkT<BM>*>(ws);
    BlkT<BN>* wb = reinterpret_cast<BlkT<BN>*>(static_cast<unsigned char*>(ws) + bytes_a);
    trop_decode_kernel<BASE, BM, true, TH><<<dim3((unsigned)nch, (unsigned)tiles_m), NT, 0, stream>>>(
        m, static_cast<const unsigned char*>(g.A), g.M, g.lda, F, wa);
    trop_decode_kernel<BASE, BN, false, TH><<<dim3((unsigned)nch, (unsigned)tiles_n), NT, 0, stream>>>(
        m, static_cast<const unsigned char*>(g.B), g.N, g.ldb, F, wb);
    dim3 grid((unsigned)tiles_n, (unsigned)tiles_m, 1);
    tfdpa_trop_kernel<EK, L, F, RHO, PROMOTE, BASE, TH><<<grid, NT, sh, stream>>>(m, g, wa, wb);
    err = cudaGetLastError();
    if (sc.given) return err;
    const cudaError_t err2 = cudaFreeAsync(ws, stream);
    return err != cudaSuccess ? err : err2;
}

// The tall micro-tile where the registers allow it: FP32 accumulators without promoted partial sums beside them.
inline bool tall_tile(const DevModel& m, const GemmArgs& g) { return m.rho != RHO_RNE_FP16 && !g.k_chunk; }
inline size_t scratch_bytes(const DevModel& m, const GemmArgs& g) {
    return tall_tile(m, g) ? scratch_bytes_one<8>(g) : scratch_bytes_one<4>(g);
}

template <int EK, int L, int F, int RHO, int BASE>
cudaError_t launch_variant_t(const DevModel& m, const GemmArgs& g, cudaStream_t stream, const Scratch& sc) {
    if constexpr (RHO == RHO_RNE_FP16) {
        return launch_one_t<EK, L, F, RHO, false, BASE, 4>(m, g, stream, sc);
    } else {
        if (g.k_chunk) return launch_one_t<EK, L, F, RHO, true, BASE, 4>(m, g, stream, sc);
        return launch_one_t<EK, L, F, RHO, false, BASE, 8>(m, g, stream, sc);
    }
}

// BASE by the exponent spread of the two element types (see pe_shift): both E4M3, one E5M2, both E5M2.
template <int EK, int L, int F, int RHO>
cudaError_t launch_by_types_t(const DevModel& m, const GemmArgs& g, cudaStream_t stream, const Scratch& sc = Scratch()) {
    const int wide = (m.fmt_a == EF_E5M2) + (m.fmt_b == EF_E5M2);
    if ((m.fmt_a != EF_E4M3 && m.fmt_a != EF_E5M2) || (m.fmt_b != EF_E4M3 && m.fmt_b != EF_E5M2)) return cudaErrorInvalidValue;
    if (wide == 0) return launch_variant_t<EK, L, F, RHO, 8>(m, g, stream, sc);
    if (wide == 1) return launch_variant_t<EK, L, F, RHO, 5>(m, g, stream, sc);
    return launch_variant_t<EK, L, F, RHO, 4>(m, g, stream, sc);
}

}  // namespace trop
}  // namespace mmasim
