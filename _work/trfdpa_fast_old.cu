// Tuned TR-FDPA (Algorithm 10) and GTR-FDPA (Algorithm 11) kernels: the CDNA3 models.
//
// Same decomposition and staging as the T-FDPA kernel (mmasim_tfdpa_fast.cuh): 128 x 64 tile per CTA, 8 x 4 outputs per
// thread, K in chunks of 32, decoded operands k-major in shared memory, negative terms in one's complement with a
// population-count correction.  What differs from T-FDPA:
//   * the truncated fused sum T covers the L products only (the accumulator is not part of e_max);
//     GTR-FDPA keeps two of them, for the even and the odd elements, each with its own maximum exponent - the two
//     16-bit lanes of the packed exponent pass are exactly these two maxima - and merges them with round-down;
//   * the accumulator enters afterwards at E = max(e_max, Exp(c)): T is rounded down to F2 fractional bits and c to F
//     (arithmetic right shifts of two's-complement values are round-down), with the "special truncation" of c in
//     GTR-FDPA; the sum is converted with RNE-FP32 (64-bit, inline);
//   * zero products have no exponent (their staged exponent words are 0, below every real sum): a group without a
//     nonzero product has T = 0 and an exponent lane that never wins a maximum;
//   * a product of magnitude >= 2^128 is an infinity (Section 4.2): whenever a block's e_max could allow that, the
//     thread rescans the raw words of the block and records the event like any other infinity.
// The accumulators stay live across the product passes, so a thread handles its 8 rows in two halves of 4.
#include "mmasim_tfdpa_fast.cuh"

namespace mmasim {
namespace fast {

namespace {

struct TrAcc {
    int cs;     // signed 24-bit significand (two's complement): value = cs * 2^(ce - CB - 23)
    int ce;     // Exp(c) + CB; 0 for c = 0
};

__device__ __forceinline__ TrAcc tr_from_word(uint32_t w, uint32_t& sp) {
    const AccDec d = decode_acc(w, false);
    TrAcc a;
    if (d.cls != CLS_FINITE) {
        sp |= (d.cls == CLS_NAN) ? 1u : (d.sign ? 4u : 2u);
        a.cs = 0;
        a.ce = 0;
        return a;
    }
    a.cs = d.sign ? -int(d.sig) : int(d.sig);
    a.ce = d.sig ? d.exp + CB : 0;      // a zero accumulator has no exponent: 0 never decides E
    return a;
}

__device__ __forceinline__ uint32_t tr_to_word(const TrAcc& a, uint32_t sp) {
    if (sp) {
        const int kind = ((sp & 1u) || (sp & 6u) == 6u) ? 1 : ((sp & 2u) ? 2 : 3);
        return special_word(kind, false, false);
    }
    const uint32_t sign = a.cs < 0;
    const uint32_t sig = uint32_t(abs(a.cs));
    const uint32_t field = (sig >> 23) ? uint32_t(a.ce - CB + 127) : 0u;
    return (sign << 31) | (field << 23) | (sig & 0x7FFFFFu);
}

__device__ __forceinline__ long long asr64_clamp(long long x, int d) { return x >> (d > 63 ? 63 : d); }

// RNE-FP32 of S * 2^(eb - CB) for a 64-bit S when the result is a normal number or zero; otherwise (vmin / vmax leave
// the normal range) the caller redoes the conversion with the generic routine.
__device__ __forceinline__ void rne32_fast(long long S, int eb, TrAcc& a, int& vmin, int& vmax) {
    const long long sg = S >> 63;
    const unsigned long long mag = (unsigned long long)((S ^ sg) - sg);
    const int msb = 63 - __clzll((long long)mag);                   // -1 for zero
    const unsigned long long norm = msb >= 0 ? (mag << (63 - msb)) : 0ull;
    const unsigned long long n2 = norm >> 1;                        // leading one at bit 62; 24 bits kept, 39 dropped
    const unsigned long long r = (n2 + (((1ull << 38) - 1ull) + ((n2 >> 39) & 1ull))) >> 39;
    const int carry = int(r >> 24);
    const int sig = int(r >> carry);
    int ve = eb + msb + carry;
    ve = mag ? ve : -126 + CB;
    vmin = min(vmin, ve);
    vmax = max(vmax, ve);
    a.ce = mag ? ve : 0;
    a.cs = sg ? -sig : sig;
}

__device__ __noinline__ void rne32_slow(long long S, int e, TrAcc& a, uint32_t& sp) {
    const uint32_t w = rho_apply(RHO_RNE_FP32, S, e);
    a = tr_from_word(w, sp);
}

template <int EK, int L, bool GTR>
__global__ void __launch_bounds__(NT, 2) trfdpa_kernel(DevModel m, GemmArgs g) {
    using E = Elem<EK>;
    constexpr bool SIGNMAG = E::SIGNMAG;
    constexpr int RH = 4;                                   // rows handled per pass over the block
    constexpr int NBLK = KC / L;
    constexpr int EMINB = -126 + CB, EMAXB = 127 + CB;
    static_assert(KC % L == 0 && L % 2 == 0, "blocks tile the chunk; pass 1 handles pairs of elements");
    extern __shared__ __align__(16) unsigned char smem_raw[];
    Smem<EK>& sm = *reinterpret_cast<Smem<EK>*>(smem_raw);
    auto& s = sm.pl[0];

    const int tid = threadIdx.x;
    const int tx = tid % 16, ty = tid / 16;
    const int64_t row0 = int64_t(blockIdx.y) * BM, col0 = int64_t(blockIdx.x) * BN;
    const FmtDesc fa = fmt_desc(m.fmt_a), fb = fmt_desc(m.fmt_b);
    const int F = m.F, F2 = m.F2;
    const int frac = fa.mbits + fb.mbits;
    const int pre = F - frac;
    const int guard = SIGNMAG ? 0 : fa.mbits + 1;
    const int one = int(blockDim.x >> 8);

    init_lut<EK>(sm, fa, fb, pre, guard, tid);
    if (tid == 0) sm.special[0] = sm.special[1] = 0;

    TrAcc acc[TM][TN];
    uint32_t sp_nan = 0u, sp_pinf = 0u, sp_ninf = 0u;
#pragma unroll
    for (int r = 0; r < TM; ++r)
#pragma unroll
        for (int c = 0; c < TN; ++c) {
            const int64_t i = row0 + ty * TM + r, j = col0 + tx * TN + c;
            uint32_t w = 0u;
            if (g.C && i < g.M && j < g.N) w = static_cast<const uint32_t*>(g.C)[i * g.ldc + j];
            uint32_t ev = 0u;
            acc[r][c] = tr_from_word(w, ev);
            sp_nan |= (ev & 1u) << (r * TN + c);
            sp_pinf |= ((ev >> 1) & 1u) << (r * TN + c);
            sp_ninf |= ((ev >> 2) & 1u) << (r * TN + c);
        }

    int chunk = 0;
    for (int64_t k0 = 0; k0 < g.K; k0 += KC, ++chunk) {
        __syncthreads();
        stage_chunk<EK>(sm, g, row0, col0, k0, chunk, pre, tid);
        __syncthreads();
        if (tid == 0) sm.special[(chunk + 1) & 1] = 0;
        const bool chunk_special = sm.special[chunk & 1] != 0;

#pragma unroll 1
        for (int blk = 0; blk < NBLK; ++blk) {
            const int kb = blk * L;
            const uint32_t kmask = (L == 32) ? 0xFFFFFFFFu : (((1u << L) - 1u) << kb);
#pragma unroll
            for (int rh = 0; rh < TM; rh += RH) {
                // ---- pass 1: maximum exponent sum of the products (low lane: even elements, high lane: odd) ----
                uint32_t em2[RH][TN];
#pragma unroll
                for (int r = 0; r < RH; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c) em2[r][c] = 0u;
#pragma unroll 4
                for (int kp = kb / 2; kp < (kb + L) / 2; ++kp) {
                    const uint4 ea = *reinterpret_cast<const uint4*>(&s.a_exp2[kp][ty * TM + rh]);
                    const uint4 eb = *reinterpret_cast<const uint4*>(&s.b_exp2[kp][tx * TN]);
                    const uint32_t eav[RH] = {ea.x, ea.y, ea.z, ea.w};
                    const uint32_t ebv[TN] = {eb.x, eb.y, eb.z, eb.w};
#pragma unroll
                    for (int r = 0; r < RH; ++r)
#pragma unroll
                        for (int c = 0; c < TN; ++c) em2[r][c] = __viaddmax_s16x2(eav[r], ebv[c], em2[r][c]);
                }
                int e_lo[RH][TN], e_hi[GTR ? RH : 1][GTR ? TN : 1];     // e_max + CB (+ guard): all / even, odd
                int emax_all = 0;
#pragma unroll
                for (int r = 0; r < RH; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c) {
                        const int lo = int(em2[r][c] & 0xFFFFu), hi = int(em2[r][c] >> 16);
                        if (GTR) { e_lo[r][c] = lo + guard; e_hi[GTR ? r : 0][GTR ? c : 0] = hi + guard; }
                        else e_lo[r][c] = max(lo, hi) + guard;
                        emax_all = max(emax_all, max(lo, hi));
                    }
                // ---- rare: infinities / NaNs in the chunk, or products that may reach 2^128: events of this block ----
                if (chunk_special || emax_all - CB >= 126) {
#pragma unroll 1
                    for (int r = 0; r < RH; ++r)
#pragma unroll 1
                        for (int c = 0; c < TN; ++c) {
                            const int64_t i = row0 + ty * TM + rh + r, j = col0 + tx * TN + c;
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
                            const uint32_t bit = 1u << ((rh + r) * TN + c);
                            if (ev.nan) sp_nan |= bit;
                            if (ev.pinf) sp_pinf |= bit;
                            if (ev.ninf) sp_ninf |= bit;
                        }
                }
                // ---- pass 2: truncated fused sum(s) of the products ----
                int T0[RH][TN], T1[GTR ? RH : 1][GTR ? TN : 1];
#pragma unroll
                for (int r = 0; r < RH; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c) { T0[r][c] = 0; if (GTR) T1[GTR ? r : 0][GTR ? c : 0] = 0; }
#pragma unroll 2
                for (int kk = kb; kk < kb + L; ++kk) {
                    const bool odd = GTR && (kk & 1);
                    const int4 eb = *reinterpret_cast<const int4*>(&s.b_exp[kk][tx * TN]);
                    const int4 ob = *reinterpret_cast<const int4*>(&s.b_op[kk][tx * TN]);
                    const int4 ea = *reinterpret_cast<const int4*>(&s.a_exp[kk][ty * TM + rh]);
                    const int4 oa = *reinterpret_cast<const int4*>(&s.a_op[kk][ty * TM + rh]);
                    const int ebv[TN] = {eb.x, eb.y, eb.z, eb.w};
                    const int obv[TN] = {ob.x, ob.y, ob.z, ob.w};
                    const int eav[RH] = {ea.x, ea.y, ea.z, ea.w};
                    const int oav[RH] = {oa.x, oa.y, oa.z, oa.w};
                    uint32_t mav[RH] = {0u, 0u, 0u, 0u}, mbv[TN] = {0u, 0u, 0u, 0u};
                    if (SIGNMAG) {
                        const uint4 ma = *reinterpret_cast<const uint4*>(&s.a_msk[SIGNMAG ? kk : 0][ty * TM + rh]);
                        const uint4 mb = *reinterpret_cast<const uint4*>(&s.b_msk[SIGNMAG ? kk : 0][tx * TN]);
                        mav[0] = ma.x; mav[1] = ma.y; mav[2] = ma.z; mav[3] = ma.w;
                        mbv[0] = mb.x; mbv[1] = mb.y; mbv[2] = mb.z; mbv[3] = mb.w;
                    }
#pragma unroll
                    for (int r = 0; r < RH; ++r)
#pragma unroll
                        for (int c = 0; c < TN; ++c) {
                            const int X = oav[r] * obv[c];
                            const int eref = odd ? e_hi[GTR ? r : 0][GTR ? c : 0] : e_lo[r][c];
                            const int d = eref - eav[r] - ebv[c];
                            int t;
                            if (SIGNMAG) t = int(lsr_clamp(uint32_t(X), d) ^ mav[r] ^ mbv[c]);
                            else t = asr_clamp(X, d);
                            if (odd) T1[GTR ? r : 0][GTR ? c : 0] = mad_one(t, one, T1[GTR ? r : 0][GTR ? c : 0]);
                            else T0[r][c] = mad_one(t, one, T0[r][c]);
                        }
                }
                // ---- merge, add the accumulator at E = max(e_max, Exp(c)) with round-down, RNE-FP32 ----
#pragma unroll
                for (int r = 0; r < RH; ++r) {
                    const uint32_t sa = s.a_sgn[ty * TM + rh + r];
                    const uint32_t nza = SIGNMAG ? kmask : (s.a_nz[ty * TM + rh + r] & kmask);
#pragma unroll
                    for (int c = 0; c < TN; ++c) {
                        const uint32_t negm = (sa ^ s.b_sgn[tx * TN + c]) & nza;
                        int T, emaxb;
                        if (GTR) {
                            const int te = T0[r][c] + __popc(negm & 0x55555555u);
                            const int to = T1[GTR ? r : 0][GTR ? c : 0] + __popc(negm & 0xAAAAAAAAu);
                            const int ee = e_lo[r][c] - guard, eo = e_hi[GTR ? r : 0][GTR ? c : 0] - guard;
                            emaxb = max(ee, eo);
                            T = asr_clamp(te, emaxb - ee) + asr_clamp(to, emaxb - eo);      // RD_F of both group sums
                        } else {
                            T = T0[r][c] + __popc(negm);
                            emaxb = e_lo[r][c] - guard;
                        }
                        const TrAcc a = acc[rh + r][c];
                        const int E = max(emaxb, a.ce);
                        const long long T2 = asr64_clamp((long long)T << (F2 - F), E - emaxb);       // RD_F2
                        long long sc2 = asr64_clamp((long long)a.cs << (F - 23), E - a.ce);           // RD_F
                        if (GTR && a.ce < E - F - 1) sc2 = 0;                                         // special truncation
                        const long long S = T2 + (sc2 << (F2 - F));
                        int vmin = EMINB, vmax = EMINB;
                        rne32_fast(S, E - F2, acc[rh + r][c], vmin, vmax);
                        if (vmin < EMINB || vmax > EMAXB) {
                            // the result is subnormal or overflows: by the book
                            uint32_t ev = 0u;
                            rne32_slow(S, E - CB - F2, acc[rh + r][c], ev);
                            const uint32_t bit = 1u << ((rh + r) * TN + c);
                            if (ev && !((sp_nan | sp_pinf | sp_ninf) & bit)) {         // overflow to infinity
                                if (ev & 2u) sp_pinf |= bit;
                                if (ev & 4u) sp_ninf |= bit;
                            }
                        }
                    }
                }
            }
        }
    }

#pragma unroll
    for (int r = 0; r < TM; ++r)
#pragma unroll
        for (int c = 0; c < TN; ++c) {
            const int64_t i = row0 + ty * TM + r, j = col0 + tx * TN + c;
            if (i >= g.M || j >= g.N) continue;
            const uint32_t bit = r * TN + c;
            const uint32_t spv = ((sp_nan >> bit) & 1u) | (((sp_pinf >> bit) & 1u) << 1) | (((sp_ninf >> bit) & 1u) << 2);
            uint32_t w = tr_to_word(acc[r][c], spv);
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
    const size_t sh = sizeof(Smem<EK>);
    cudaError_t err = cudaFuncSetAttribute(trfdpa_kernel<EK, L, GTR>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(sh));
    if (err != cudaSuccess) return err;
    dim3 grid((unsigned)((g.N + BN - 1) / BN), (unsigned)((g.M + BM - 1) / BM), 1);
    trfdpa_kernel<EK, L, GTR><<<grid, NT, sh, stream>>>(m, g);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_tr(const DevModel& m, const GemmArgs& g, cudaStream_t st) {
    if (m.family == FAM_GTR) return launch_tr_one<EK_LUT8, 16, true>(m, g, st);
    if (m.fmt_a == EF_F16) return launch_tr_one<EK_F16, 8, false>(m, g, st);
    if (m.fmt_a == EF_BF16) return launch_tr_one<EK_BF16, 8, false>(m, g, st);
    if (m.fmt_a == EF_TF32) return launch_tr_one<EK_TF32, 4, false>(m, g, st);
    return cudaErrorInvalidValue;
}

}  // namespace fast
}  // namespace mmasim
