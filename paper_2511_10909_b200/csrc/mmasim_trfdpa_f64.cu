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
__global__ void __launch_bounds__(NT, 1) trfdpa64_kernel(DevModel m, GemmArgs g, const Blk64<BM>* __restrict__ wa,
                                                         const Blk64<BN>* __restrict__ wb) {
    constexpr int NBLK = KC / L;
    static_assert(KC % L == 0 && L % 4 == 0 && (!GTR || L == 16), "blocks tile the chunk; a matrix instruction takes four terms");
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
    const int F = m.F, F2 = m.F2;
    const int frac = fa.mbits + fb.mbits;
    // high word of 1.5 * 2^52 * 2^(e_max - F) is (e_max + CB) * 2^20 + MAGIC_K
    const int MAGIC_E = 1023 + 52 - F - CB;

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

    // The accumulator of each output lives between blocks as a double holding the FP32 value (exact); its exponent field is
    // Exp(c) in place: zero has the field 0 (no exponent), an FP32 subnormal a field below that of 2^-126 (it counts as -126).
    double cs[TM][TN];
    uint32_t sp_nan = 0u, sp_pinf = 0u, sp_ninf = 0u;   // per output (bit r * TN + c): NaN / +inf / -inf seen so far
#pragma unroll
    for (int r = 0; r < TM; ++r)
#pragma unroll
        for (int c = 0; c < TN; ++c) {
            const int64_t i = row0 + row_at(r), j = col0 + col_at(c);
            uint32_t w = 0u;
            if (g.C && i < g.M && j < g.N) w = static_cast<const uint32_t*>(g.C)[i * g.ldc + j];
            const AccDec d = decode_acc(w, false);
            if (d.cls != CLS_FINITE) {
                const uint32_t bit = 1u << (r * TN + c);
                if (d.cls == CLS_NAN) sp_nan |= bit; else if (d.sign) sp_ninf |= bit; else sp_pinf |= bit;
                w = 0u;
            }
            cs[r][c] = double(__uint_as_float(w));
        }

    __syncthreads();                                    // the barriers are initialised
    uint32_t emp[TM][TN];                               // product exponents of the block that comes next (low lane: even elements)

    for (int chunk = 0; chunk < NCH; ++chunk) {
        const int64_t k0 = int64_t(chunk) * KC;
        // a wait that runs out is recorded and the chunk computed on whatever is there; every thread sees the flag after
        // the barrier at the end of the chunk, and the CTA leaves together without storing anything
        if (!fast::mbar_wait(&sm.full[chunk & 1], uint32_t(chunk >> 1) & 1u)) *reinterpret_cast<volatile int*>(&sm.error) = 1;
        const Blk64<BM>& sa_blk = sm.a[chunk & 1];
        const Blk64<BN>& sb_blk = sm.b[chunk & 1];
        const bool chunk_special = (sa_blk.special | sb_blk.special) != 0u;
        // no product of the chunk reaches 2^126 when the largest exponents of its A and B elements do not add up to it (a
        // bound from the decode pass: crossing it only sends the chunk's blocks through the exact scan below)
        const bool chunk_rare = chunk_special || int(sa_blk.max_exp + sb_blk.max_exp) - CB >= 126;
        // the first block's product exponents (the other blocks' are taken beside the multiply-adds of their predecessor)
        product_exponents_adj<L>(&sa_blk.exp2[0][prow], &sb_blk.exp2[0][pcol], emp);

#pragma unroll (L <= 8 ? 2 : 1)
        for (int blk = 0; blk < NBLK; ++blk) {
            const int kb = blk * L;
            // ---- rare: infinities / NaNs in the chunk, or products that may reach 2^128: events of this block ----
            if (chunk_rare) {
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
            // ---- sum registers: the bare constants at the maximum exponents of this block's products; a group without a
            // nonzero product (lane 0) gets an exponent far below every real one: its sum stays 0 ----
            constexpr int EXPF = 0x7FF00000, HALF = 0x00080000, LOW0 = int(0x80000000u);
            double t0[TM][TN], t1[GTR ? TM : 1][GTR ? TN : 1];
            constexpr bool KEEP_M0 = !GTR && L <= 8;       // short blocks keep the high word of the constant from the start of the block to the merge
            int m0k[KEEP_M0 ? TM : 1][KEEP_M0 ? TN : 1];
            // (the two 16-bit lanes reach the exponent field by multiplications, which issue beside the integer pipe; what is
            // left below the field is masked away; the low word starts at 2^31: |T| < 2^30, so the sign correction of the
            // merge is a 32-bit addition that never carries)
            auto start = [&](int r, int c) {
                const int klo = imad(int(emp[r][c]), c_mul64[0], MAGIC_E << 20), khi = imad(int(emp[r][c]), c_mul64[1], MAGIC_E << 20);
                if (GTR) {
                    t0[r][c] = __hiloint2double((klo & EXPF) | HALF, LOW0);
                    t1[GTR ? r : 0][GTR ? c : 0] = __hiloint2double((khi & EXPF) | HALF, LOW0);
                } else {
                    const int mh = (max(klo, khi) & EXPF) | HALF;
                    if (KEEP_M0) m0k[KEEP_M0 ? r : 0][KEEP_M0 ? c : 0] = mh;
                    t0[r][c] = __hiloint2double(mh, LOW0);
                }
            };
            // four terms per matrix instruction (mma.sync m8n8k4, FP64, rounding toward minus infinity) for the rows
            // 2 half, 2 half + 1 of the micro-tile; lane (g, t) holds A[8 r + g][k + t] and B[8 j + g][k + t].  GTR: the plane
            // holds the eight even elements of the block first, then the eight odd ones.
            auto mma_half = [&](int half, int ks) {
                double af[2], bf[TN / 2];
#pragma unroll
                for (int r = 0; r < 2; ++r) af[r] = sa_blk.d[wr * 32 + 8 * (2 * half + r) + gq][kb + ks + tq];
#pragma unroll
                for (int j = 0; j < TN / 2; ++j) bf[j] = sb_blk.d[wc * 16 + 8 * j + gq][kb + ks + tq];
#pragma unroll
                for (int r = 0; r < 2; ++r)
#pragma unroll
                    for (int j = 0; j < TN / 2; ++j) {
                        if (GTR && ks >= 8)
                            asm volatile("mma.sync.aligned.m8n8k4.row.col.rm.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                                         : "+d"(t1[GTR ? 2 * half + r : 0][GTR ? 2 * j : 0]), "+d"(t1[GTR ? 2 * half + r : 0][GTR ? 2 * j + 1 : 0])
                                         : "d"(af[r]), "d"(bf[j]));
                        else
                            asm volatile("mma.sync.aligned.m8n8k4.row.col.rm.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                                         : "+d"(t0[2 * half + r][2 * j]), "+d"(t0[2 * half + r][2 * j + 1]) : "d"(af[r]), "d"(bf[j]));
                    }
            };
            // ---- merge (Algorithm 10 Step 3 / Algorithm 11 Step 4) in FP64, where every quantity is exact.
            //   E = max(e_max, Exp(c)); T is rounded down onto 2^(E - F2), c onto 2^(E - F).  Whichever of the two exponents
            //   is larger, both roundings can be taken on the one grid qv = 2^max(e_max - F, Exp(c) - F2): the operand that
            //   needs no rounding (T when E = e_max, c when E = Exp(c)) is a multiple of qv anyway.  With Mv = 1.5 * 2^52 * qv:
            //       Z1 = RD(c + Mv);   Z = RD(T q + Z1) = Mv + RD_qv(c) + RD_qv(T q);   v = Z - Mv     (at most 40 bits)
            //   T q is the sum register minus its constant (after the sign correction, added to the register's bit pattern).
            //   RNE-FP32 of v is the conversion instruction (a negative sum that rounds to zero is -0, a magnitude that rounds
            //   to 2^128 becomes infinity), and the conversion back gives the accumulator of the next block.  An infinity is
            //   rare and sticky: the loop tracks the largest magnitude, the flags are set in a second pass. ----
            const uint32_t kmask = (L == 32) ? 0xFFFFFFFFu : (((1u << L) - 1u) << kb);
            // exponents as the exponent fields of doubles, in place (bits 20..30 of the high word): x20 = (x + 1023) << 20
            constexpr uint32_t LOWF = (1023 - 126) << 20;
            const uint32_t k_c = uint32_t(((52 - F2) << 20) | HALF) + 1u;   // (field of Exp(c)) - 1 + k_c: high word of 1.5 * 2^52 * 2^(Exp(c) - F2)
            constexpr uint32_t k_gtr = (53u << 20) + 1u;   // a sum register's field minus Exp(c)'s beyond which c is dropped (GTR)
            float wmax = 0.f;
            auto merge = [&](int r, int c) {
                const uint32_t sa = sa_blk.sgn[prow + r], nza = sa_blk.nz[prow + r] & kmask;
                const uint32_t negm = (sa ^ sb_blk.sgn[pcol + c]) & nza & sb_blk.nz[pcol + c];
                double Y;                                   // T * 2^(e_max - F)
                int m0hi;                                   // high word of the sum register's constant (e_max in place)
                if (GTR) {
                    // both group sums rounded down onto the coarser of their two grids, then added (Algorithm 11 Step 3)
                    const double u0 = t0[r][c], u1 = t1[GTR ? r : 0][GTR ? c : 0];
                    const int e_hi = (__double2hiint(u0) & EXPF) | HALF, o_hi = (__double2hiint(u1) & EXPF) | HALF;
                    m0hi = max(e_hi, o_hi);
                    const double ye = __dsub_rn(__hiloint2double(__double2hiint(u0), __double2loint(u0) + __popc(negm & 0x55555555u)),
                                                __hiloint2double(e_hi, LOW0));
                    const double yo = __dsub_rn(__hiloint2double(__double2hiint(u1), __double2loint(u1) + __popc(negm & 0xAAAAAAAAu)),
                                                __hiloint2double(o_hi, LOW0));
                    const double mm = __hiloint2double(m0hi, 0);
                    Y = __dsub_rn(__dadd_rd(yo, __dadd_rd(ye, mm)), mm);
                } else {
                    const double u0 = t0[r][c];
                    m0hi = KEEP_M0 ? m0k[KEEP_M0 ? r : 0][KEEP_M0 ? c : 0] : (__double2hiint(u0) & EXPF) | HALF;
                    Y = __dsub_rn(__hiloint2double(__double2hiint(u0), __double2loint(u0) + __popc(negm)), __hiloint2double(m0hi, LOW0));
                }
                double st = cs[r][c];
                // the field of Exp(c), minus one: zero wraps to the top and comes back as 0 when the one is added again (inside
                // k_c, k_gtr); a subnormal accumulator counts as -126
                const uint32_t ecm = __viaddmax_u32(uint32_t(__double2hiint(st) & EXPF), 0xFFFFFFFFu, LOWF - 1u);
                if (GTR && int(ecm + k_gtr) < m0hi - HALF) st = 0.0;                // special truncation (Algorithm 11 Step 4)
                const double Mv = __hiloint2double(__viaddmax_s32(int(ecm), int(k_c), m0hi), 0);   // 1.5 * 2^52 * qv
                const double v = __dsub_rn(__dadd_rd(Y, __dadd_rd(st, Mv)), Mv);
                // RNE-FP32 (subnormal range, the sign of a zero and the overflow to infinity included) is the conversion
                // instruction itself; back as a double the result is the next block's accumulator
                const float w = __double2float_rn(v);
                wmax = fmaxf(fabsf(w), wmax);
                cs[r][c] = double(w);
            };

            // ---- the block in two halves of the micro-tile (rows 0, 1 and rows 2, 3): the matrix instructions of one half
            // are issued between the merge of the other and the product exponents of the next block ----
            constexpr int NKS = L / 4, PER = 8 / (NKS < 8 ? NKS : 8);
            const bool fuse = NBLK > 1 && blk + 1 < NBLK;
#pragma unroll
            for (int o = 0; o < 16; ++o) start(o / TN, o % TN);
#pragma unroll
            for (int ksi = 0; ksi < NKS; ++ksi) mma_half(0, 4 * ksi);
#pragma unroll
            for (int ksi = 0; ksi < NKS; ++ksi) {
                mma_half(1, 4 * ksi);
#pragma unroll
                for (int q = 0; q < PER; ++q)
                    if (ksi * PER + q < 8) merge((ksi * PER + q) / TN, (ksi * PER + q) % TN);
                if (fuse) {                             // the product exponents of the next block
                    const uint32_t* ea_p = &sa_blk.exp2[(kb + L) / 2][prow];
                    const uint32_t* eb_p = &sb_blk.exp2[(kb + L) / 2][pcol];
                    if (ksi == 0) {
#pragma unroll
                        for (int r = 0; r < TM; ++r)
#pragma unroll
                            for (int c = 0; c < TN; ++c) emp[r][c] = 0u;
                    }
#pragma unroll
                    for (int kp = 2 * ksi; kp < 2 * ksi + 2; ++kp) {
                        const uint4 ea0 = *reinterpret_cast<const uint4*>(ea_p + kp * BM);
                        const uint4 eb0 = *reinterpret_cast<const uint4*>(eb_p + kp * BN);
                        const uint32_t ea[TM] = {ea0.x, ea0.y, ea0.z, ea0.w};
                        const uint32_t ebv[TN] = {eb0.x, eb0.y, eb0.z, eb0.w};
#pragma unroll
                        for (int r = 0; r < TM; ++r)
#pragma unroll
                            for (int c = 0; c < TN; ++c) emp[r][c] = __viaddmax_s16x2(ea[r], ebv[c], emp[r][c]);
                    }
                }
            }
#pragma unroll
            for (int o = 8; o < 16; ++o) merge(o / TN, o % TN);
            if (wmax > 3.4028234663852886e38f) {            // rare: RNE-FP32 overflowed somewhere: +-infinity from now on
#pragma unroll
                for (int r = 0; r < TM; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c)
                        if (fabs(cs[r][c]) >= 3.402823669209385e38) {
                            const uint32_t bit = 1u << (r * TN + c);
                            if (!((sp_nan | sp_pinf | sp_ninf) & bit)) { if (cs[r][c] < 0.0) sp_ninf |= bit; else sp_pinf |= bit; }
                            cs[r][c] = 0.0;
                        }
            }
        }
        __syncthreads();                                // everybody has finished with this buffer
        if (*reinterpret_cast<volatile int*>(&sm.error)) break;
        if (tid == 0 && chunk + 2 < NCH) issue(chunk + 2);
    }

    if (*reinterpret_cast<volatile int*>(&sm.error)) {  // a copy never arrived: count it, give the copies in flight one more
        if (tid == 0) {                                 // bounded wait each, and store nothing
            if (g.copy_timeouts) atomicAdd(g.copy_timeouts, 1u);
            fast::mbar_wait(&sm.full[0], 0u);
            fast::mbar_wait(&sm.full[1], 0u);
        }
        return;
    }
#pragma unroll
    for (int r = 0; r < TM; ++r)
#pragma unroll
        for (int c = 0; c < TN; ++c) {
            const int64_t i = row0 + row_at(r), j = col0 + col_at(c);
            if (i >= g.M || j >= g.N) continue;
            const uint32_t bit = r * TN + c;
            const uint32_t spv = ((sp_nan >> bit) & 1u) | (((sp_pinf >> bit) & 1u) << 1) | (((sp_ninf >> bit) & 1u) << 2);
            uint32_t w = spv ? special_word(((spv & 1u) || (spv & 6u) == 6u) ? 1 : ((spv & 2u) ? 2 : 3), false, false)
                             : __float_as_uint(__double2float_rn(cs[r][c]));
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
    const size_t sh = sizeof(SmemMM);
    cudaError_t err = cudaFuncSetAttribute(trfdpa64_kernel<EK, L, GTR>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(sh));
    if (err != cudaSuccess) return err;
    const size_t dsh_a = 256 * sizeof(LutEntry64) + sizeof(Blk64<BM>), dsh_b = 256 * sizeof(LutEntry64) + sizeof(Blk64<BN>);
    if ((err = cudaFuncSetAttribute(decode64_kernel<EK, BM, true, 0, GTR>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(dsh_a))) != cudaSuccess) return err;
    if ((err = cudaFuncSetAttribute(decode64_kernel<EK, BN, false, 0, GTR>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(dsh_b))) != cudaSuccess) return err;
    const int64_t tiles_m = (g.M + BM - 1) / BM, tiles_n = (g.N + BN - 1) / BN, nch = g.K / KC;
    // scratch: the decoded blocks of A and B, stream-ordered out of the library's pool and returned to it behind the kernel
    const size_t bytes_a = size_t(tiles_m * nch) * sizeof(Blk64<BM>), bytes_b = size_t(tiles_n * nch) * sizeof(Blk64<BN>);
    cudaMemPool_t pool = nullptr;
    if ((err = scratch_pool(&pool)) != cudaSuccess) return err;
    void* ws = nullptr;
    if ((err = cudaMallocFromPoolAsync(&ws, bytes_a + bytes_b, pool, stream)) != cudaSuccess) return err;
    Blk64<BM>* wa = static_cast<Blk64<BM>*>(ws);
    Blk64<BN>* wb = reinterpret_cast<Blk64<BN>*>(static_cast<unsigned char*>(ws) + bytes_a);
    decode64_kernel<EK, BM, true, 0, GTR><<<dim3((unsigned)nch, (unsigned)tiles_m), 256, dsh_a, stream>>>(
        m, static_cast<const unsigned char*>(g.A), g.M, g.lda, wa);
    decode64_kernel<EK, BN, false, 0, GTR><<<dim3((unsigned)nch, (unsigned)tiles_n), 256, dsh_b, stream>>>(
        m, static_cast<const unsigned char*>(g.B), g.N, g.ldb, wb);
    dim3 grid((unsigned)tiles_n, (unsigned)tiles_m, 1);
    trfdpa64_kernel<EK, L, GTR><<<grid, NT, sh, stream>>>(m, g, wa, wb);
    err = cudaGetLastError();
    const cudaError_t err2 = cudaFreeAsync(ws, stream);
    return err != cudaSuccess ? err : err2;
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
