// Tuned T-FDPA kernels (Algorithm 5 + Algorithm 7 + Table 2) for GEMM-sized inputs.
//
// Work decomposition.  A CTA of 256 threads owns a 128 x 64 tile of D; a thread owns an 8 x 4 micro-tile and keeps
// the 32 accumulators decoded in registers (one's-complement significand aligned to F fractional bits, exponent)
// for the whole K loop.  K is walked in chunks of 32 elements: the CTA loads the raw A / B bytes of the chunk,
// decodes every element once through a 256-entry table into an operand word and an exponent word, and stores
// them k-major in shared memory so that one 16-byte shared load feeds four rows (or columns) of a micro-tile.
//
// Per block of L elements and per output (Algorithm 7):
//   pass 1   e_max = max(Exp(c), max_k(Exp(a_k) + Exp(b_k)))       one fused add-max per term
//   pass 2   X_k   = A_op * B_op                                    one multiply on the FMA pipe
//            d_k   = e_max + g - Exp(a_k) - Exp(b_k)                one 3-input add
//            S    += X_k >> d_k (arithmetic)                        one shift, half a 3-input add
//   then the accumulator term, the sign corrections, normalisation and rho (a few tens of instructions).
//
// Sign-magnitude truncation without per-term sign work.  RZ_F truncates the magnitude of each aligned term, but an
// arithmetic right shift of a two's-complement number rounds toward minus infinity.  Operands are therefore built
// so that the 32-bit product is  X = s * (m << (F - frac + g)) + r  with  m = sig_a * sig_b,  s = +-1 the product's
// sign,  g = (mantissa bits of A) + 1 guard bits and a residue  0 <= r < 2^g  for s = +1,  -2^g <= r <= -1  for
// s = -1:  A_op = +-sig_a,  B_op = (+-sig_b << (F - frac + g)) + sign(b)  gives  r = +-sig_a.  Then
// X >> (d + g) equals  floor(m * 2^(F - frac) / 2^d)  for positive terms and  -floor(...) - 1  for negative ones (the
// one's complement of the truncated magnitude).  Adding the number of negative terms of the block, a population
// count over per-row / per-column sign bit masks, restores the exact sign-magnitude sum.  (A term counts as
// negative when the signs differ and sig_a != 0; with b = +-0 it is -sig_a >> (d + g) = -1, the negative zero.)
//
// Everything that is rare takes a slow, obviously correct route: NaN / infinity inputs (the CTA rescans the raw
// words of the chunk and keeps NaN / +inf / -inf flags per output, Section 4.2), results outside the normal range
// of the accumulator format and the nearest-even conversion to FP16 (the generic conversion routine).
#include "mmasim_device.cuh"

namespace mmasim {
namespace {

constexpr int BM = 128, BN = 64, TM = 8, TN = 4, KC = 32, NT = 256;

struct LutEntry {
    uint32_t op;      // multiplier operand
    int32_t exp;      // Exp(x); zero for non-finite inputs
    uint32_t flags;   // bit 0: sign, bit 1: nonzero significand, bit 2: infinity or NaN
    uint32_t pad;
};

struct Smem {
    uint32_t a_op[KC][BM];
    int32_t a_exp[KC][BM];
    uint32_t b_op[KC][BN];
    int32_t b_exp[KC][BN];
    LutEntry lut_a[256];
    LutEntry lut_b[256];
    uint16_t a_sgn[BM][2], a_nz[BM][2], b_sgn[BN][2];   // bit k of row r: sign / nonzero of element k of the chunk
    int special[2];                                     // chunk (by parity) holds an infinity or a NaN
};

__device__ __forceinline__ int fa_emin(const FmtDesc& f) { return 1 - f.bias; }

__device__ __forceinline__ int asr_clamp(int x, int d) {
    int r;
    asm("shr.s32 %0, %1, %2;" : "=r"(r) : "r"(x), "r"(d));      // amounts above 31 behave as 31 (sign fill)
    return r;
}

// Accumulator state of one output.
struct Acc {
    int cs;     // one's complement signed significand, aligned to F fractional bits relative to 2^ce
    int ce;     // Exp(c)
};

template <int F, bool ACC16>
__device__ __forceinline__ Acc acc_from_word(uint32_t w, uint32_t& sp) {
    const AccDec d = decode_acc(w, ACC16);
    Acc a;
    if (d.cls != CLS_FINITE) {
        sp |= (d.cls == CLS_NAN) ? 1u : (d.sign ? 4u : 2u);
        a.cs = 0;
        a.ce = ACC16 ? -14 : -126;
        return a;
    }
    constexpr int MB = ACC16 ? 10 : 23;
    const int mag = (F >= MB) ? int(d.sig << (F >= MB ? F - MB : 0)) : int(d.sig >> (F >= MB ? 0 : MB - F));
    a.cs = d.sign ? ~mag : mag;
    a.ce = d.exp;
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
    const uint32_t field = (sig >> MB) ? uint32_t(a.ce + (ACC16 ? 15 : 127)) : 0u;
    return (sign << (ACC16 ? 15 : 31)) | (field << MB) | (sig & ((1u << MB) - 1u));
}

// Slow conversion: any rho, any range.  S is the exact fixed-point sum in units of 2^(e_max - F).
template <int F, int RHO, bool ACC16>
__device__ __noinline__ void rho_slow(long long S, int e_max, Acc& a, uint32_t& sp) {
    const uint32_t w = rho_apply(RHO, S, e_max - F);
    a = acc_from_word<F, ACC16>(w, sp);
}

template <int L, int F, int RHO, bool PROMOTE>
__global__ void __launch_bounds__(NT, 2) tfdpa8_kernel(DevModel m, GemmArgs g) {
    constexpr bool ACC16 = RHO == RHO_RNE_FP16;
    constexpr int MB_OUT = RHO == RHO_RZ_E8M13 ? 13 : (ACC16 ? 10 : 23);   // mantissa bits kept by rho
    constexpr int EMIN = ACC16 ? -14 : -126, EMAX = ACC16 ? 15 : 127;
    constexpr bool INLINE_RHO = RHO == RHO_RZ_FP32 || RHO == RHO_RZ_E8M13;
    constexpr int HALF = L / 2;                     // products per 32-bit partial sum when two are needed
    constexpr int NBLK = KC / L;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    Smem& s = *reinterpret_cast<Smem*>(smem_raw);

    const int tid = threadIdx.x;
    const int tx = tid % 16, ty = tid / 16;
    const int64_t row0 = int64_t(blockIdx.y) * BM, col0 = int64_t(blockIdx.x) * BN;
    const FmtDesc fa = fmt_desc(m.fmt_a), fb = fmt_desc(m.fmt_b);
    const int pre = F - (fa.mbits + fb.mbits);      // left shift that gives a product F fractional bits
    const int guard = fa.mbits + 1;                 // guard bits below the truncation point

    // decode tables: entry `tid` of both
    {
        const uint32_t da = decode_elem(fa, uint32_t(tid)), db = decode_elem(fb, uint32_t(tid));
        const bool fin_a = dec_cls(da) == CLS_FINITE, fin_b = dec_cls(db) == CLS_FINITE;
        LutEntry ea, eb;
        ea.op = fin_a ? uint32_t(dec_ssig(da)) : 0u;
        ea.exp = fin_a ? dec_exp(da) : fa_emin(fa);
        ea.flags = (fin_a ? dec_sign(da) | ((dec_sig(da) != 0u) << 1) : 0u) | (fin_a ? 0u : 4u);
        ea.pad = 0u;
        const int sb = fin_b ? dec_ssig(db) : 0;
        const int ub = fin_b ? (dec_sign(db) ? -1 : 1) : 0;     // also for b = +-0: the term is then +-sig_a, a signed zero
        eb.op = uint32_t(sb * (1 << (pre + guard)) + ub);
        eb.exp = fin_b ? dec_exp(db) : fa_emin(fb);
        eb.flags = (fin_b ? dec_sign(db) | ((dec_sig(db) != 0u) << 1) : 0u) | (fin_b ? 0u : 4u);
        eb.pad = 0u;
        s.lut_a[tid] = ea;
        s.lut_b[tid] = eb;
        if (tid == 0) s.special[0] = s.special[1] = 0;
    }

    Acc acc[TM][TN];
    uint32_t sp_nan = 0u, sp_pinf = 0u, sp_ninf = 0u;   // per output (bit r * TN + c): NaN / +inf / -inf seen so far
    float promoted[PROMOTE ? TM : 1][PROMOTE ? TN : 1];
#define SP_GET(r, c) ((((sp_nan >> ((r) * TN + (c))) & 1u)) | (((sp_pinf >> ((r) * TN + (c))) & 1u) << 1) | (((sp_ninf >> ((r) * TN + (c))) & 1u) << 2))
#define SP_OR(r, c, v) do { const uint32_t v_ = (v); sp_nan |= (v_ & 1u) << ((r) * TN + (c)); sp_pinf |= ((v_ >> 1) & 1u) << ((r) * TN + (c)); sp_ninf |= ((v_ >> 2) & 1u) << ((r) * TN + (c)); } while (0)
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
            uint32_t ev = 0u;
            acc[r][c] = acc_from_word<F, ACC16>(w, ev);
            SP_OR(r, c, ev);
        }

    int chunk = 0;
    for (int64_t k0 = 0; k0 < g.K; k0 += KC, ++chunk) {
        __syncthreads();
        // ---- stage the chunk: 16 raw bytes per unit, decoded through the tables ----
        {
            const int r = tid % BM, h = tid / BM;
            uint4 raw = make_uint4(0u, 0u, 0u, 0u);
            if (row0 + r < g.M)
                raw = *reinterpret_cast<const uint4*>(static_cast<const uint8_t*>(g.A) + (row0 + r) * g.lda + k0 + 16 * h);
            const uint32_t wv[4] = {raw.x, raw.y, raw.z, raw.w};
            uint32_t sgn = 0u, nz = 0u, spec = 0u;
#pragma unroll
            for (int q = 0; q < 16; ++q) {
                const LutEntry e = s.lut_a[(wv[q / 4] >> (8 * (q % 4))) & 0xFFu];
                s.a_op[16 * h + q][r] = e.op;
                s.a_exp[16 * h + q][r] = e.exp;
                sgn |= (e.flags & 1u) << q;
                nz |= ((e.flags >> 1) & 1u) << q;
                spec |= e.flags & 4u;
            }
            s.a_sgn[r][h] = uint16_t(sgn);
            s.a_nz[r][h] = uint16_t(nz);
            if (tid < 2 * BN) {
                const int rb = tid % BN, hb = tid / BN;
                uint4 rawb = make_uint4(0u, 0u, 0u, 0u);
                if (col0 + rb < g.N)
                    rawb = *reinterpret_cast<const uint4*>(static_cast<const uint8_t*>(g.B) + (col0 + rb) * g.ldb + k0 + 16 * hb);
                const uint32_t wb[4] = {rawb.x, rawb.y, rawb.z, rawb.w};
                uint32_t sgnb = 0u;
#pragma unroll
                for (int q = 0; q < 16; ++q) {
                    const LutEntry e = s.lut_b[(wb[q / 4] >> (8 * (q % 4))) & 0xFFu];
                    s.b_op[16 * hb + q][rb] = e.op;
                    s.b_exp[16 * hb + q][rb] = e.exp;
                    sgnb |= (e.flags & 1u) << q;
                    spec |= e.flags & 4u;
                }
                s.b_sgn[rb][hb] = uint16_t(sgnb);
            }
            if (spec) atomicOr(&s.special[chunk & 1], 1);
        }
        __syncthreads();

        if (tid == 0) s.special[(chunk + 1) & 1] = 0;
        const bool chunk_special = s.special[chunk & 1] != 0;

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
                            const uint32_t x = decode_elem(fa, static_cast<const uint8_t*>(g.A)[i * g.lda + k0 + kk]);
                            const uint32_t y = decode_elem(fb, static_cast<const uint8_t*>(g.B)[j * g.ldb + k0 + kk]);
                            ev.product(x, y);
                        }
                        const uint32_t bit = 1u << (r * TN + c);
                        if (ev.nan) sp_nan |= bit;
                        if (ev.pinf) sp_pinf |= bit;
                        if (ev.ninf) sp_ninf |= bit;
                    }
            }
            int emax[TM][TN];
            // ---- pass 1: block maximum of the exponent sums, accumulator included ----
#pragma unroll
            for (int r = 0; r < TM; ++r)
#pragma unroll
                for (int c = 0; c < TN; ++c) emax[r][c] = acc[r][c].ce;
#pragma unroll 4
            for (int kk = kb; kk < kb + L; ++kk) {
                const int4 ea0 = *reinterpret_cast<const int4*>(&s.a_exp[kk][ty * TM]);
                const int4 ea1 = *reinterpret_cast<const int4*>(&s.a_exp[kk][ty * TM + 4]);
                const int4 eb = *reinterpret_cast<const int4*>(&s.b_exp[kk][tx * TN]);
                const int ea[TM] = {ea0.x, ea0.y, ea0.z, ea0.w, ea1.x, ea1.y, ea1.z, ea1.w};
                const int ebv[TN] = {eb.x, eb.y, eb.z, eb.w};
#pragma unroll
                for (int r = 0; r < TM; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c) emax[r][c] = __viaddmax_s32(ea[r], ebv[c], emax[r][c]);
            }
            // ---- accumulator term: align at e_max, truncate (one's complement keeps sign-magnitude semantics) ----
            constexpr bool NARROW = F <= 13;                  // (L + 1) terms below 2^(F + 2) fit 32 bits
            constexpr bool TWO_SUMS = !NARROW && L > 16;
            int S0[TM][TN], S1[TWO_SUMS ? TM : 1][TWO_SUMS ? TN : 1];
#pragma unroll
            for (int r = 0; r < TM; ++r)
#pragma unroll
                for (int c = 0; c < TN; ++c) {
                    // one's complement term of c, plus 1 if c is negative (restores the two's complement value)
                    S0[r][c] = asr_clamp(acc[r][c].cs, emax[r][c] - acc[r][c].ce) - (acc[r][c].cs >> 31);
                    if (TWO_SUMS) S1[r][c] = 0;
                    emax[r][c] += guard;               // from here on: e_max + g, the shift base of pass 2
                }
            // ---- pass 2: multiply, align, truncate, add ----
#pragma unroll 2
            for (int kk = kb; kk < kb + L; ++kk) {
                const int4 ea0 = *reinterpret_cast<const int4*>(&s.a_exp[kk][ty * TM]);
                const int4 ea1 = *reinterpret_cast<const int4*>(&s.a_exp[kk][ty * TM + 4]);
                const int4 eb = *reinterpret_cast<const int4*>(&s.b_exp[kk][tx * TN]);
                const int4 oa0 = *reinterpret_cast<const int4*>(&s.a_op[kk][ty * TM]);
                const int4 oa1 = *reinterpret_cast<const int4*>(&s.a_op[kk][ty * TM + 4]);
                const int4 ob = *reinterpret_cast<const int4*>(&s.b_op[kk][tx * TN]);
                const int ea[TM] = {ea0.x, ea0.y, ea0.z, ea0.w, ea1.x, ea1.y, ea1.z, ea1.w};
                const int ebv[TN] = {eb.x, eb.y, eb.z, eb.w};
                const int oa[TM] = {oa0.x, oa0.y, oa0.z, oa0.w, oa1.x, oa1.y, oa1.z, oa1.w};
                const int obv[TN] = {ob.x, ob.y, ob.z, ob.w};
                const bool second = TWO_SUMS && (kk - kb >= HALF);
#pragma unroll
                for (int r = 0; r < TM; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c) {
                        const int X = oa[r] * obv[c];
                        const int d = emax[r][c] - ea[r] - ebv[c];
                        const int t = asr_clamp(X, d);
                        if (second) S1[TWO_SUMS ? r : 0][TWO_SUMS ? c : 0] += t; else S0[r][c] += t;
                    }
            }
            // ---- sign corrections, normalisation, rho ----
            const uint32_t kmask = (L == 32) ? 0xFFFFFFFFu : (((1u << L) - 1u) << kb);
#pragma unroll
            for (int r = 0; r < TM; ++r) {
                const uint32_t sa = *reinterpret_cast<const uint32_t*>(&s.a_sgn[ty * TM + r][0]);
                const uint32_t nza = *reinterpret_cast<const uint32_t*>(&s.a_nz[ty * TM + r][0]) & kmask;
#pragma unroll
                for (int c = 0; c < TN; ++c) {
                    const uint32_t sb = *reinterpret_cast<const uint32_t*>(&s.b_sgn[tx * TN + c][0]);
                    const int nneg = __popc((sa ^ sb) & nza);
                    const int e_max = emax[r][c] - guard;
                    Acc& a = acc[r][c];
                    if (NARROW) {
                        const int S = S0[r][c] + nneg;
                        const int sg = S >> 31;
                        const uint32_t mag = uint32_t((S ^ sg) - sg);
                        const int lz = __clz(int(mag));
                        const int ve = e_max - F + 31 - lz;
                        if (INLINE_RHO && mag != 0u && ve >= EMIN && ve <= EMAX) {
                            const uint32_t sig = (mag << lz) >> (31 - MB_OUT);
                            const int magF = (F >= MB_OUT) ? int(sig << (F >= MB_OUT ? F - MB_OUT : 0)) : int(sig >> (F >= MB_OUT ? 0 : MB_OUT - F));
                            a.cs = magF ^ sg;
                            a.ce = ve;
                        } else {
                            uint32_t ev = 0u;
                            rho_slow<F, RHO, ACC16>((long long)S, e_max, a, ev);
                            if (ev && !SP_GET(r, c)) SP_OR(r, c, ev);   // overflow to infinity (RNE only)
                        }
                    } else {
                        const long long S = (long long)S0[r][c] + (TWO_SUMS ? (long long)S1[TWO_SUMS ? r : 0][TWO_SUMS ? c : 0] : 0ll) + nneg;
                        const long long sg = S >> 63;
                        const unsigned long long mag = (unsigned long long)((S ^ sg) - sg);
                        const int lz = __clzll((long long)mag);
                        const int ve = e_max - F + 63 - lz;
                        if (INLINE_RHO && mag != 0ull && ve >= EMIN && ve <= EMAX) {
                            const uint32_t sig = uint32_t((mag << lz) >> (63 - MB_OUT));
                            const int magF = (F >= MB_OUT) ? int(sig << (F >= MB_OUT ? F - MB_OUT : 0)) : int(sig >> (F >= MB_OUT ? 0 : MB_OUT - F));
                            a.cs = magF ^ int(sg);
                            a.ce = ve;
                        } else {
                            uint32_t ev = 0u;
                            rho_slow<F, RHO, ACC16>(S, e_max, a, ev);
                            if (ev && !SP_GET(r, c)) SP_OR(r, c, ev);   // overflow to infinity (RNE only)
                        }
                    }
                }
            }
        }
        // ---- FP32 promotion of the partial sum every k_chunk elements ----
        if (PROMOTE && ((k0 + KC) % g.k_chunk) == 0) {
#pragma unroll
            for (int r = 0; r < TM; ++r)
#pragma unroll
                for (int c = 0; c < TN; ++c) {
                    const float part = __uint_as_float(acc_to_word<F, ACC16>(acc[r][c], SP_GET(r, c)));
                    float v = __fadd_rn(promoted[PROMOTE ? r : 0][PROMOTE ? c : 0], part);
                    if (v != v) v = __uint_as_float(0x7FFFFFFFu);
                    promoted[PROMOTE ? r : 0][PROMOTE ? c : 0] = v;
                    uint32_t dummy = 0u;
                    acc[r][c] = acc_from_word<F, ACC16>(0u, dummy);
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
            uint32_t w = PROMOTE ? __float_as_uint(promoted[PROMOTE ? r : 0][PROMOTE ? c : 0]) : acc_to_word<F, ACC16>(acc[r][c], SP_GET(r, c));
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
}

template <int L, int F, int RHO, bool PROMOTE>
cudaError_t launch8p(const DevModel& m, const GemmArgs& g, cudaStream_t stream) {
    const size_t sh = sizeof(Smem);
    cudaError_t err = cudaFuncSetAttribute(tfdpa8_kernel<L, F, RHO, PROMOTE>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(sh));
    if (err != cudaSuccess) return err;
    dim3 grid((unsigned)((g.N + BN - 1) / BN), (unsigned)((g.M + BM - 1) / BM), 1);
    tfdpa8_kernel<L, F, RHO, PROMOTE><<<grid, NT, sh, stream>>>(m, g);
    return cudaGetLastError();
}

template <int L, int F, int RHO>
int launch8(const DevModel& m, const GemmArgs& g, cudaStream_t stream) {
    const cudaError_t err = g.k_chunk ? launch8p<L, F, RHO, true>(m, g, stream) : launch8p<L, F, RHO, false>(m, g, stream);
    if (err != cudaSuccess) {
        set_error("tfdpa8 kernel launch failed: %s", cudaGetErrorString(err));
        return MMASIM_ERR_CUDA;
    }
    return MMASIM_OK;
}

bool is8(int f) { return f == EF_E4M3 || f == EF_E5M2 || f == EF_E3M2 || f == EF_E2M3 || f == EF_E2M1; }

}  // namespace

bool fast_tfdpa_supported(const DevModel& m, const GemmArgs& g) {
    if (m.family != FAM_T || g.dot_mode || m.packed4) return false;
    if (!is8(m.fmt_a) || !is8(m.fmt_b)) return false;
    const bool combo = (m.F == 13 && (m.L == 16 || m.L == 32) && (m.rho == RHO_RZ_E8M13 || m.rho == RHO_RNE_FP16)) ||
                       (m.F == 25 && m.L == 32 && (m.rho == RHO_RZ_FP32 || m.rho == RHO_RNE_FP16));
    if (!combo) return false;
    if ((m.rho == RHO_RNE_FP16) != (m.acc == ACC_F16)) return false;
    if (g.K % KC) return false;
    if (g.k_chunk % KC) return false;
    if ((g.lda % 16) || (g.ldb % 16)) return false;                 // 16-byte row starts for the vector loads
    if (g.M > 65535ll * BM) return false;
    return true;
}

int launch_fast_tfdpa(const DevModel& m, const GemmArgs& g, cudaStream_t stream) {
    set_kernel_name("tfdpa8");
    if (m.F == 13 && m.L == 16 && m.rho == RHO_RZ_E8M13) return launch8<16, 13, RHO_RZ_E8M13>(m, g, stream);
    if (m.F == 13 && m.L == 16 && m.rho == RHO_RNE_FP16) return launch8<16, 13, RHO_RNE_FP16>(m, g, stream);
    if (m.F == 13 && m.L == 32 && m.rho == RHO_RZ_E8M13) return launch8<32, 13, RHO_RZ_E8M13>(m, g, stream);
    if (m.F == 13 && m.L == 32 && m.rho == RHO_RNE_FP16) return launch8<32, 13, RHO_RNE_FP16>(m, g, stream);
    if (m.F == 25 && m.L == 32 && m.rho == RHO_RZ_FP32) return launch8<32, 25, RHO_RZ_FP32>(m, g, stream);
    if (m.F == 25 && m.L == 32 && m.rho == RHO_RNE_FP16) return launch8<32, 25, RHO_RNE_FP16>(m, g, stream);
    set_error("no tuned kernel for this model");
    return MMASIM_ERR_UNSUPPORTED;
}

}  // namespace mmasim
