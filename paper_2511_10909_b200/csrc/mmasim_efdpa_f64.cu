// Tuned E-FDPA (Algorithm 6) kernel: the CDNA1 FP16 / BF16 models - RNE-FP32 of the EXACT sum c + sum_k a_k b_k of
// a block of L = 4 (FP16) or 2 (BF16) products.
//
// Tile, staging and exponent planes are those of the FP64 T-FDPA kernel (mmasim_tfdpa_f64.cuh).  The exact sum is
// taken in FP64 whenever it fits: every product of two FP16 / BF16 values is exact in a double (22 significant bits),
// and if every term of the block - the products and c - lies inside one window of 50 binades (from the lowest bit of
// the smallest term to the top of the largest), every partial sum of the fused multiply-add chain is exact and the
// one conversion cvt.rn.f32.f64 at the end is the single rounding of Algorithm 6.  The window is checked from the
// staged exponents: per output the maximum and the minimum of Exp(a_k) + Exp(b_k) over the block (fused add-max and
// add-min on two 16-bit lanes) and the exponent of c.  Whatever does not fit - a zero product (its staged exponent
// says nothing about the window), terms further apart than the window, an infinity or a NaN in the chunk or in the
// accumulator - goes through the by-the-book block function on the raw words (exact 640-bit fixed-point sum), which
// also produces and propagates the special values: the accumulator between blocks is the plain output word.
// The B operands of the shared staging carry a small offset in the low word of the double (used by the truncating
// kernels); FP16 and BF16 significands fit the high word, so clearing the low word gives the exact value back.
#include "mmasim_tfdpa_f64.cuh"

namespace mmasim {
namespace fast64 {

namespace {

using fast::EK_F16;
using fast::EK_BF16;

// By the book: decode the L elements of row i of A and row j of B from global memory and run Algorithm 6.
template <int EK, int L>
__device__ __noinline__ uint32_t efdpa_by_the_book(DevModel m, const void* A, const void* B, int64_t ia, int64_t ib, uint32_t c) {
    const FmtDesc fa = fmt_desc(m.fmt_a), fb = fmt_desc(m.fmt_b);
    uint32_t a[L], b[L];
#pragma unroll
    for (int k = 0; k < L; ++k) {
        a[k] = decode_elem(fa, raw_elem<EK>(A, ia + k));
        b[k] = decode_elem(fb, raw_elem<EK>(B, ib + k));
    }
    return efdpa_block(a, b, L, c, m);
}

template <int EK, int L>
__global__ void __launch_bounds__(NT, 1) efdpa64_kernel(DevModel m, GemmArgs g) {
    using E = Elem<EK>;
    constexpr int NBLK = KC / L;
    constexpr int FRAC = 2 * E::MBITS;
    constexpr int WINDOW = 50;                          // top of the largest term minus lowest bit of the smallest, in binades
    static_assert(KC % L == 0 && L % 2 == 0, "blocks tile the chunk; the exponent pass handles pairs of elements");
    using SM = Smem64<EK>;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SM& sm = *reinterpret_cast<SM*>(smem_raw);

    const int tid = threadIdx.x;
    const int tx = tid % 16, ty = tid / 16;
    const int64_t row0 = int64_t(blockIdx.y) * BM, col0 = int64_t(blockIdx.x) * BN;
    const FmtDesc fa = fmt_desc(m.fmt_a), fb = fmt_desc(m.fmt_b);

    init_lut64<EK>(sm, fa, fb, tid);
    if (tid == 0) sm.special[0] = sm.special[1] = sm.special[2] = 0;

    uint32_t cw[TM][TN];                                // the accumulator of each output: the FP32 word, special values included
#pragma unroll
    for (int r = 0; r < TM; ++r)
#pragma unroll
        for (int c = 0; c < TN; ++c) {
            const int64_t i = row0 + ty * TM + r, j = col0 + col_of(tx, c);
            cw[r][c] = (g.C && i < g.M && j < g.N) ? static_cast<const uint32_t*>(g.C)[i * g.ldc + j] : 0u;
        }

    RawChunk<EK> raw;
    load_chunk<EK>(raw, g, row0, col0, 0, tid);
    __syncthreads();                                    // tables and flags are ready
    store_chunk64<EK>(sm, sm.pl[0], raw, 0, tid);
    if (KC < g.K) load_chunk<EK>(raw, g, row0, col0, KC, tid);
    __syncthreads();

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

#pragma unroll 1
        for (int blk = 0; blk < NBLK; ++blk) {
            const int kb = blk * L;
            // ---- largest and smallest exponent sum of the block's products (lanes: even and odd elements) ----
            uint32_t emx[TM][TN], emn[TM][TN];
#pragma unroll
            for (int r = 0; r < TM; ++r)
#pragma unroll
                for (int c = 0; c < TN; ++c) { emx[r][c] = 0u; emn[r][c] = 0x7FFF7FFFu; }
#pragma unroll
            for (int kp = kb / 2; kp < (kb + L) / 2; ++kp) {
                const uint4 ea0 = *reinterpret_cast<const uint4*>(&s.a_exp2[kp][ty * TM]);
                const uint2 eb0 = *reinterpret_cast<const uint2*>(&s.b_exp2[kp][tx * 2]);
                const uint2 eb1 = *reinterpret_cast<const uint2*>(&s.b_exp2[kp][tx * 2 + BN / 2]);
                const uint32_t ea[TM] = {ea0.x, ea0.y, ea0.z, ea0.w};
                const uint32_t ebv[TN] = {eb0.x, eb0.y, eb1.x, eb1.y};
#pragma unroll
                for (int r = 0; r < TM; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c) {
                        emx[r][c] = __viaddmax_s16x2(ea[r], ebv[c], emx[r][c]);
                        emn[r][c] = __viaddmin_s16x2(ea[r], ebv[c], emn[r][c]);
                    }
            }
            // ---- the fused multiply-add chain from c, exact inside the window ----
            double sum[TM][TN];
#pragma unroll
            for (int r = 0; r < TM; ++r)
#pragma unroll
                for (int c = 0; c < TN; ++c) sum[r][c] = double(__uint_as_float(cw[r][c]));
#pragma unroll
            for (int kk = kb; kk < kb + L; ++kk) {
                double av[TM], bv[TN];
#pragma unroll
                for (int r = 0; r < TM; r += 2) {
                    const double2 t = *reinterpret_cast<const double2*>(&s.a_d[kk][ty * TM + r]);
                    av[r] = t.x; av[r + 1] = t.y;
                }
                const double2 u0 = *reinterpret_cast<const double2*>(&s.b_d[kk][tx * 2]);
                const double2 u1 = *reinterpret_cast<const double2*>(&s.b_d[kk][tx * 2 + BN / 2]);
                bv[0] = __hiloint2double(__double2hiint(u0.x), 0); bv[1] = __hiloint2double(__double2hiint(u0.y), 0);
                bv[2] = __hiloint2double(__double2hiint(u1.x), 0); bv[3] = __hiloint2double(__double2hiint(u1.y), 0);
#pragma unroll
                for (int r = 0; r < TM; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c) sum[r][c] = __fma_rn(av[r], bv[c], sum[r][c]);
            }
            // ---- the window test and the rounding; what does not fit keeps its accumulator and is marked ----
            const uint32_t kmask = (((L == 32) ? 0u : (1u << L)) - 1u) << kb;
            uint32_t slow = 0u;                                    // bit r * TN + c: this output goes by the book
#pragma unroll
            for (int r = 0; r < TM; ++r) {
                const uint32_t nza = s.a_nz[ty * TM + r];
#pragma unroll
                for (int c = 0; c < TN; ++c) {
                    const uint32_t w0 = cw[r][c];
                    const uint32_t ca = w0 & 0x7FFFFFFFu;
                    const int hi = max(int(emx[r][c] & 0xFFFFu), int(emx[r][c] >> 16));      // biased by CB
                    const int lo = min(int(emn[r][c] & 0xFFFFu), int(emn[r][c] >> 16));
                    const int ec = int(max(ca >> 23, 1u)) + (CB - 127);
                    // a product is below 2^(e + 2) and a multiple of 2^(e - FRAC); c is below 2^(Exp + 1), a multiple of 2^(Exp - 23)
                    const int top = ca ? max(hi + 2, ec + 1) : hi + 2;
                    const int low = ca ? min(lo - FRAC, ec - 23) : lo - FRAC;
                    const bool all_nonzero = (nza & s.b_nz[col_of(tx, c)] & kmask) == kmask;
                    const bool fits = !chunk_special && all_nonzero && ca < 0x7F800000u && top - low <= WINDOW;
                    slow |= uint32_t(!fits) << (r * TN + c);
                    cw[r][c] = fits ? __float_as_uint(__double2float_rn(sum[r][c])) : w0;
                }
            }
            if (slow) {                                        // rare
#pragma unroll
                for (int r = 0; r < TM; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c)
                        if ((slow >> (r * TN + c)) & 1u) {
                            const int64_t i = row0 + ty * TM + r, j = col0 + col_of(tx, c);
                            cw[r][c] = (i < g.M && j < g.N)
                                           ? efdpa_by_the_book<EK, L>(m, g.A, g.B, i * g.lda + k0 + kb, j * g.ldb + k0 + kb, cw[r][c]) : 0u;
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
            uint32_t w = cw[r][c];
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

template <int EK, int L>
cudaError_t launch_e_one(const DevModel& m, const GemmArgs& g, cudaStream_t stream) {
    const size_t sh = sizeof(Smem64<EK>);
    cudaError_t err = cudaFuncSetAttribute(efdpa64_kernel<EK, L>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(sh));
    if (err != cudaSuccess) return err;
    dim3 grid((unsigned)((g.N + BN - 1) / BN), (unsigned)((g.M + BM - 1) / BM), 1);
    efdpa64_kernel<EK, L><<<grid, NT, sh, stream>>>(m, g);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_e64(const DevModel& m, const GemmArgs& g, cudaStream_t st) {
    if (m.fmt_a == EF_F16 && m.L == 4) return launch_e_one<EK_F16, 4>(m, g, st);
    if (m.fmt_a == EF_BF16 && m.L == 2) return launch_e_one<EK_BF16, 2>(m, g, st);
    return cudaErrorInvalidValue;
}

}  // namespace fast64

namespace fast {
cudaError_t launch_e(const DevModel& m, const GemmArgs& g, cudaStream_t st) { return fast64::launch_e64(m, g, st); }
}  // namespace fast
}  // namespace mmasim
