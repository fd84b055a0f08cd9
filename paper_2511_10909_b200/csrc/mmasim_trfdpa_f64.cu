// Tuned TR-FDPA (Algorithm 10) and GTR-FDPA (Algorithm 11) kernels: the CDNA3 models.
//
// The truncated fused sum of the products is computed like the T-FDPA kernel of mmasim_tfdpa_f64.cuh does it - same
// tile, staging, one fma.rm.f64 per term into a register that holds 1.5 * 2^52 * q + T * q, q = 2^(e_max - F), with
// the one's-complement treatment of negative terms and the population-count correction - except that
//   * the accumulator is not part of that sum: e_max is the maximum over the (nonzero) products only, and the sum
//     register starts as the bare constant;
//   * GTR-FDPA keeps two sums, of the even and of the odd elements, each with its own maximum exponent - the two
//     16-bit lanes of the packed exponent pass are exactly these two maxima - and merges them with round-down.
// What follows per block and output works on T (read from the low word of the register): T and c are aligned at
// E = max(e_max, Exp(c)) with round-down to F2 and F fractional bits - one fma.rd.f64 and one add.rd.f64 onto the
// grids of 1.5 * 2^52 * 2^(E - F2) and 1.5 * 2^52 * 2^(E - F), every intermediate exact - with the "special
// truncation" of c in GTR-FDPA, and the exact sum is converted with RNE-FP32 by one cvt.  The accumulator between
// blocks is the output word itself.
// A product of magnitude >= 2^128 is an infinity (Section 4.2): whenever a block's e_max could allow that, the thread
// rescans the raw words of the block and records the event like any other infinity.  Zero products have no
// exponent: a group without a nonzero product has T = 0 and an exponent lane that never wins a maximum.
#include "mmasim_tfdpa_f64.cuh"

namespace mmasim {
namespace fast64 {

namespace {

using fast::EK_LUT8;
using fast::EK_F16;
using fast::EK_BF16;
using fast::EK_TF32;

template <int EK, int L, bool GTR>
__global__ void __launch_bounds__(NT, 1) trfdpa64_kernel(DevModel m, GemmArgs g) {
    constexpr int NBLK = KC / L;
    static_assert(KC % L == 0 && L % 2 == 0, "blocks tile the chunk; the exponent pass handles pairs of elements");
    using SM = Smem64<EK>;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SM& sm = *reinterpret_cast<SM*>(smem_raw);

    const int tid = threadIdx.x;
    const int tx = tid % 16, ty = tid / 16;
    const int64_t row0 = int64_t(blockIdx.y) * BM, col0 = int64_t(blockIdx.x) * BN;
    const FmtDesc fa = fmt_desc(m.fmt_a), fb = fmt_desc(m.fmt_b);
    const int F = m.F, F2 = m.F2;
    const int frac = fa.mbits + fb.mbits;
    // high word of 1.5 * 2^52 * 2^(e_max - F) is (e_max + CB) * 2^20 + MAGIC_K
    const int MAGIC_E = 1023 + 52 - F - CB;
    const int MAGIC_K = (MAGIC_E << 20) | 0x00080000;
    constexpr int E_FLOOR = CB - 400;

    init_lut64<EK>(sm, fa, fb, tid);
    if (tid == 0) sm.special[0] = sm.special[1] = sm.special[2] = 0;

    uint32_t cw[TM][TN];                                // the accumulator of each output: a finite FP32 word
    uint32_t sp_nan = 0u, sp_pinf = 0u, sp_ninf = 0u;   // per output (bit r * TN + c): NaN / +inf / -inf seen so far
#pragma unroll
    for (int r = 0; r < TM; ++r)
#pragma unroll
        for (int c = 0; c < TN; ++c) {
            const int64_t i = row0 + ty * TM + r, j = col0 + col_of(tx, c);
            uint32_t w = 0u;
            if (g.C && i < g.M && j < g.N) w = static_cast<const uint32_t*>(g.C)[i * g.ldc + j];
            const AccDec d = decode_acc(w, false);
            if (d.cls != CLS_FINITE) {
                const uint32_t bit = 1u << (r * TN + c);
                if (d.cls == CLS_NAN) sp_nan |= bit; else if (d.sign) sp_ninf |= bit; else sp_pinf |= bit;
                w = 0u;
            }
            cw[r][c] = w;
        }

    RawChunk<EK> raw;
    load_chunk<EK>(raw, g, row0, col0, 0, tid);
    __syncthreads();                                    // tables and flags are ready
    store_chunk64<EK>(sm, sm.pl[0], raw, 0, tid);
    if (KC < g.K) load_chunk<EK>(raw, g, row0, col0, KC, tid);
    __syncthreads();
    uint32_t emp[TM][TN];                               // product exponents of the block that comes next (low lane: even elements)

    int chunk = 0;
    for (int64_t k0 = 0; k0 < g.K; k0 += KC, ++chunk) {
        auto& s = sm.pl[chunk & 1];
        auto& nx = sm.pl[(chunk + 1) & 1];
        // one barrier per chunk, at its end: every warp left the other buffer before the barrier that ended the previous
        // iteration, so it can be filled while slower warps still compute on this one
        if (tid == 0) sm.special[(chunk + 2) % 3] = 0;
        if (k0 + KC < g.K) {
            store_chunk64<EK>(sm, nx, raw, (chunk + 1) % 3, tid);
            if (k0 + 2 * KC < g.K) load_chunk<EK>(raw, g, row0, col0, k0 + 2 * KC, tid);
        }
        const bool chunk_special = sm.special[chunk % 3] != 0;
        // the first block's product exponents (the other blocks' are taken beside the multiply-adds of their predecessor)
        product_exponents<L>(&s.a_exp2[0][ty * TM], &s.b_exp2[0][tx * 2], emp);

#pragma unroll 1
        for (int blk = 0; blk < NBLK; ++blk) {
            const int kb = blk * L;
            // ---- sum registers: the bare constants at the maximum exponents of this block's products ----
            double t0[TM][TN], t1[GTR ? TM : 1][GTR ? TN : 1];
            int emax_all = 0;
#pragma unroll
            for (int r = 0; r < TM; ++r)
#pragma unroll
                for (int c = 0; c < TN; ++c) {
                    // a group without a nonzero product (lane 0) gets E_FLOOR, below every real exponent: its sum stays 0
                    // and the constants derived from its register's exponent stay inside FP64
                    const int lo = int(emp[r][c] & 0xFFFFu), hi = int(emp[r][c] >> 16);
                    if (GTR) {
                        t0[r][c] = __hiloint2double(max(lo, E_FLOOR) * (1 << 20) + MAGIC_K, 0);
                        t1[GTR ? r : 0][GTR ? c : 0] = __hiloint2double(max(hi, E_FLOOR) * (1 << 20) + MAGIC_K, 0);
                    } else {
                        t0[r][c] = __hiloint2double(__vimax3_s32(lo, hi, E_FLOOR) * (1 << 20) + MAGIC_K, 0);
                    }
                    emax_all = max(emax_all, max(lo, hi));
                }
            // ---- rare: infinities / NaNs in the chunk, or products that may reach 2^128: events of this block ----
            if (chunk_special || emax_all - CB >= 126) {
#pragma unroll 1
                for (int r = 0; r < TM; ++r)
#pragma unroll 1
                    for (int c = 0; c < TN; ++c) {
                        const int64_t i = row0 + ty * TM + r, j = col0 + col_of(tx, c);
                        if (i >= g.M || j >= g.N) continue;
                        Special ev;
                        for (int kk = kb; kk < kb + L; ++kk) {
                            const uint32_t x = decode_elem(fa, raw_elem<EK>(g.A, i * g.lda + k0 + kk));
                            const uint32_t y = decode_elem(fb, raw_elem<EK>(g.B, j * g.ldb + k0 + kk));
                            ev.product(x, y);
                            if ((dec_cls(x) | dec_cls(y)) == 0u) {
                                const int sk = dec_ssig(x) * dec_ssig(y);
                                if (product_overflows(sk, dec_exp(x) + dec_exp(y), frac)) ev.add_inf(sk < 0);
                            }
                        }
                        const uint32_t bit = 1u << (r * TN + c);
                        if (ev.nan) sp_nan |= bit;
                        if (ev.pinf) sp_pinf |= bit;
                        if (ev.ninf) sp_ninf |= bit;
                    }
            }
            // ---- one fused multiply-add per term; beside it the product exponents of the block that follows ----
            {
                const double* a_p = &s.a_d[kb][ty * TM];
                const double* b_p = &s.b_d[kb][tx * 2];
                // the next block of this chunk (after the chunk's last block the pass reads its first block again; that
                // result is replaced at the start of the next chunk)
                const uint32_t* ea_p = &s.a_exp2[(kb + L) / 2 < KC / 2 ? (kb + L) / 2 : 0][ty * TM];
                const uint32_t* eb_p = &s.b_exp2[(kb + L) / 2 < KC / 2 ? (kb + L) / 2 : 0][tx * 2];
#pragma unroll
                for (int r = 0; r < TM; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c) emp[r][c] = 0u;
#pragma unroll
                for (int kq = 0; kq < L; ++kq) {
                    double av[TM], bv[TN];
#pragma unroll
                    for (int r = 0; r < TM; r += 2) {
                        const double2 t = *reinterpret_cast<const double2*>(a_p + kq * BM + r);
                        av[r] = t.x; av[r + 1] = t.y;
                    }
                    {
                        const double2 u0 = *reinterpret_cast<const double2*>(b_p + kq * BN);
                        const double2 u1 = *reinterpret_cast<const double2*>(b_p + kq * BN + BN / 2);
                        bv[0] = u0.x; bv[1] = u0.y; bv[2] = u1.x; bv[3] = u1.y;
                    }
                    uint32_t ea[TM], ebv[TN];
                    if ((kq & 1) == 0) {
                        const int kp = kq / 2;
                        const uint4 ea0 = *reinterpret_cast<const uint4*>(ea_p + kp * BM);
                        const uint2 eb0 = *reinterpret_cast<const uint2*>(eb_p + kp * BN);
                        const uint2 eb1 = *reinterpret_cast<const uint2*>(eb_p + kp * BN + BN / 2);
                        ea[0] = ea0.x; ea[1] = ea0.y; ea[2] = ea0.z; ea[3] = ea0.w;
                        ebv[0] = eb0.x; ebv[1] = eb0.y; ebv[2] = eb1.x; ebv[3] = eb1.y;
                    }
#pragma unroll
                    for (int r = 0; r < TM; ++r)
#pragma unroll
                        for (int c = 0; c < TN; ++c) {
                            if (GTR && (kq & 1)) t1[GTR ? r : 0][GTR ? c : 0] = __fma_rd(av[r], bv[c], t1[GTR ? r : 0][GTR ? c : 0]);
                            else t0[r][c] = __fma_rd(av[r], bv[c], t0[r][c]);
                            if ((kq & 1) == 0) emp[r][c] = __viaddmax_s16x2(ea[r], ebv[c], emp[r][c]);
                        }
                }
            }
            // ---- merge (Algorithm 10 Step 3 / Algorithm 11 Step 4) in FP64, where every quantity is exact:
            //   E = max(e_max, Exp(c));  T2 = floor(T 2^(e_max - F) / q2) q2 with q2 = 2^(E - F2): one fma.rd onto the
            //   grid of 1.5 * 2^52 * q2;  sc2 = floor(c / q1) q1 with q1 = 2^(E - F): one add.rd onto 1.5 * 2^52 * q1;
            //   their sum has at most 40 significant bits; RNE-FP32 is one conversion.  An overflow is rare and sticky:
            //   the loop tracks the largest result word, the flags are set in a second pass. ----
            const uint32_t kmask = (L == 32) ? 0xFFFFFFFFu : (((1u << L) - 1u) << kb);
            // exponents as the exponent fields of doubles, in place (bits 20..30 of the high word): x20 = (x + 1023) << 20
            constexpr int EXPF = 0x7FF00000;
            const int k_reg = (52 - F) << 20;              // a sum register's field is that of 2^e_max plus 52 - F
            const int k_m2 = ((52 - F2) << 20) | 0x00080000, k_m1 = (F2 - F) << 20, k_st = F << 20, k_gtr = (F + 1) << 20;
            uint32_t wmax = 0u;
#pragma unroll
            for (int r = 0; r < TM; ++r) {
                const uint32_t sa = s.a_sgn[ty * TM + r], nza = s.a_nz[ty * TM + r] & kmask;
#pragma unroll
                for (int c = 0; c < TN; ++c) {
                    const uint32_t negm = (sa ^ s.b_sgn[col_of(tx, c)]) & nza & s.b_nz[col_of(tx, c)];
                    // the low word of a sum register is T (two's complement, |T| < 2^31), its exponent field gives e_max
                    int T, t20;
                    if (GTR) {
                        const int te = __double2loint(t0[r][c]) + __popc(negm & 0x55555555u);
                        const int to = __double2loint(t1[GTR ? r : 0][GTR ? c : 0]) + __popc(negm & 0xAAAAAAAAu);
                        const int e20 = __double2hiint(t0[r][c]) & EXPF, o20 = __double2hiint(t1[GTR ? r : 0][GTR ? c : 0]) & EXPF;
                        t20 = max(e20, o20);
                        T = fast::asr_clamp(te, (t20 - e20) >> 20) + fast::asr_clamp(to, (t20 - o20) >> 20);      // RD_F of both group sums
                    } else {
                        T = __double2loint(t0[r][c]) + __popc(negm);
                        t20 = __double2hiint(t0[r][c]) & EXPF;
                    }
                    const uint32_t w0 = cw[r][c];
                    const double cd = double(__uint_as_float(w0));
                    int ec20 = max(__double2hiint(cd) & EXPF, (1023 - 126) << 20);      // a subnormal accumulator has the exponent -126
                    if ((w0 & 0x7FFFFFFFu) == 0u) ec20 = 0;                             // a zero accumulator has none
                    const int em20 = t20 - k_reg;                                       // e_max
                    const int E20 = max(em20, ec20);                                    // E = max(e_max, Exp(c))
                    const double scale_t = __hiloint2double(em20 - k_st, 0);            // 2^(e_max - F)
                    const double m2 = __hiloint2double(E20 + k_m2, 0);                  // 1.5 * 2^52 * 2^(E - F2)
                    const double m1 = __hiloint2double(E20 + k_m2 + k_m1, 0);           // 1.5 * 2^52 * 2^(E - F)
                    const double t2 = __dsub_rn(__fma_rd(double(T), scale_t, m2), m2);  // RD_F2
                    double sc2 = __dsub_rn(__dadd_rd(cd, m1), m1);                      // RD_F
                    if (GTR && ec20 < E20 - k_gtr) sc2 = 0.0;                           // special truncation
                    const uint32_t w = __float_as_uint(__double2float_rn(__dadd_rn(t2, sc2)));      // exact sum, then rho
                    wmax = max(wmax, w & 0x7FFFFFFFu);
                    cw[r][c] = w;
                }
            }
            if (wmax >= 0x7F800000u) {                     // rare: RNE-FP32 overflowed: +-infinity from now on
#pragma unroll
                for (int r = 0; r < TM; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c)
                        if ((cw[r][c] & 0x7FFFFFFFu) == 0x7F800000u) {
                            const uint32_t bit = 1u << (r * TN + c);
                            if (!((sp_nan | sp_pinf | sp_ninf) & bit)) { if (cw[r][c] >> 31) sp_ninf |= bit; else sp_pinf |= bit; }
                            cw[r][c] = 0u;
                        }
            }
        }
        __syncthreads();                                // the other buffer is complete, this one is free
    }

#pragma unroll
    for (int r = 0; r < TM; ++r)
#pragma unroll
        for (int c = 0; c < TN; ++c) {
            const int64_t i = row0 + ty * TM + r, j = col0 + col_of(tx, c);
            if (i >= g.M || j >= g.N) continue;
            const uint32_t bit = r * TN + c;
            const uint32_t spv = ((sp_nan >> bit) & 1u) | (((sp_pinf >> bit) & 1u) << 1) | (((sp_ninf >> bit) & 1u) << 2);
            uint32_t w = spv ? special_word(((spv & 1u) || (spv & 6u) == 6u) ? 1 : ((spv & 2u) ? 2 : 3), false, false) : cw[r][c];
            if (g.row_scale) {
                float sc = __fmul_rn(g.row_scale[i], g.col_scale[j]);
                if (sc != sc) sc = __uint_as_float(0x7FFFFFFFu);
                float v = __fmul_rn(sc, __uint_as_float(w));
                if (v != v) v = __uint_as_float(0x7FFFFFFFu);
                w = __float_as_uint(v);
            }
            static_cast<uint32_t*>(g.D)[i * g.ldd + j] = w;
        }
}

template <int EK, int L, bool GTR>
cudaError_t launch_tr_one(const DevModel& m, const GemmArgs& g, cudaStream_t stream) {
    const size_t sh = sizeof(Smem64<EK>);
    cudaError_t err = cudaFuncSetAttribute(trfdpa64_kernel<EK, L, GTR>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(sh));
    if (err != cudaSuccess) return err;
    dim3 grid((unsigned)((g.N + BN - 1) / BN), (unsigned)((g.M + BM - 1) / BM), 1);
    trfdpa64_kernel<EK, L, GTR><<<grid, NT, sh, stream>>>(m, g);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_tr64(const DevModel& m, const GemmArgs& g, cudaStream_t st) {
    if (m.family == FAM_GTR) return launch_tr_one<EK_LUT8, 16, true>(m, g, st);
    if (m.fmt_a == EF_F16) return launch_tr_one<EK_F16, 8, false>(m, g, st);
    if (m.fmt_a == EF_BF16) return launch_tr_one<EK_BF16, 8, false>(m, g, st);
    if (m.fmt_a == EF_TF32) return launch_tr_one<EK_TF32, 4, false>(m, g, st);
    return cudaErrorInvalidValue;
}

}  // namespace fast64

namespace fast {
cudaError_t launch_tr(const DevModel& m, const GemmArgs& g, cudaStream_t st) { return fast64::launch_tr64(m, g, st); }
}  // namespace fast
}  // namespace mmasim
