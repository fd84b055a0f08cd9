// Tuned GST-FDPA kernel (Algorithm 9): the group-scaled FP4 models (MXFP4: E8M0 scale per 32 elements, NVFP4:
// UE4M3 scale per 16 elements; L = 64, G = 16, F = 35, RZ-FP32).
//
// A CTA of 256 threads owns a 128 x 64 tile of D, a thread an 8 x 4 micro-tile (handled in two halves of 4 rows).
// K is walked in chunks of 64 elements = one GST-FDPA block.  Staging turns every packed FP4 code into the
// signed byte 2 * value (values are multiples of 0.5 up to 6, so 2 * value is an integer in [-12, 12]) and stores
// four consecutive elements per 32-bit word, k-major, so that the exact group dot product of Step 1 is four 4-way
// byte dot-product instructions: sum(2a * 2b) = 4 * p_g, an integer with two fractional bits.
// Per block and output: e_max over the exponents Exp(alpha) + Exp(beta) of the groups that hold at least one nonzero
// product under nonzero scale factors and Exp(c) of a nonzero accumulator; every group term
// s_g = p_g * Sig(alpha) * Sig(beta) and the accumulator are aligned at e_max, truncated (magnitude) to F = 35
// fractional bits and added in 64-bit fixed point; RZ-FP32 is applied inline when the result is a normal number,
// otherwise by the generic conversion routine.  NaN scale factors and a NaN / infinite accumulator set sticky
// per-output flags (Section 4.2); FP4 itself has no special values.
#include "mmasim_device.cuh"

namespace mmasim {
namespace {

constexpr int BM = 128, BN = 64, TM = 8, TN = 4, RH = 4, KC = 64, KW = KC / 4, NT = 256;
constexpr int SB = 512;                 // bias of a staged scale exponent
constexpr int CB = 2 * SB;              // bias of an exponent sum and of the accumulator exponent

struct Smem {
    uint32_t a[KW][BM];                 // four elements per word, as signed bytes holding 2 * value
    uint32_t b[KW][BN];
    uint32_t sa[4][BM];                 // per group of the block: (Exp + SB) << 8 | Sig; bit 31: NaN
    uint32_t sb[4][BN];
    uint32_t fa[4][2][BM];              // per group and half of it: bit 4 n + 3 set = element n of the eight is nonzero
    uint32_t fb[4][2][BN];
};

// Signed byte 2 * value of an E2M1 code (bit 3 sign, bits 2..0 magnitude code: 0, .5, 1, 1.5, 2, 3, 4, 6).
__device__ __forceinline__ uint32_t fp4_byte(uint32_t code) {
    const uint32_t mags = 0x0C080604u, mags_lo = 0x03020100u;       // bytes: 12, 8, 6, 4 | 3, 2, 1, 0
    const uint32_t m = ((code & 4u) ? mags : mags_lo) >> (8u * (code & 3u)) & 0xFFu;
    return (code & 8u) ? ((0u - m) & 0xFFu) : m;
}

__device__ __forceinline__ uint32_t decode_scale(uint32_t byte, bool ue4m3) {
    if (ue4m3) {
        const uint32_t x = byte & 0x7Fu;
        if (x == 0x7Fu) return 0x80000000u;
        const uint32_t field = x >> 3, mant = x & 7u;
        const uint32_t sig = mant | (field ? 8u : 0u);
        const int e = int(field ? field : 1u) - 7;
        return (uint32_t(e + SB) << 8) | sig;
    }
    if (byte == 0xFFu) return 0x80000000u;
    return (uint32_t(int(byte) - 127 + SB) << 8) | 1u;
}

template <bool NVF4>
__global__ void __launch_bounds__(NT, 2) gst_kernel(DevModel m, GemmArgs g) {
    constexpr int F = 35;
    constexpr int FRAC = NVF4 ? 8 : 2;              // fractional bits of p_g * Sig(alpha) * Sig(beta)
    constexpr int SPB = NVF4 ? 4 : 2;               // scale factors per block of 64 and row
    constexpr int EMINB = -126 + CB, EMAXB = 127 + CB;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    Smem& s = *reinterpret_cast<Smem*>(smem_raw);

    const int tid = threadIdx.x;
    const int tx = tid % 16, ty = tid / 16;
    const int64_t row0 = int64_t(blockIdx.y) * BM, col0 = int64_t(blockIdx.x) * BN;

    uint32_t cw[TM][TN];
    uint32_t sp_nan = 0u;                           // sticky NaN flags (bit r * TN + c); infinities live in cw itself
#pragma unroll
    for (int r = 0; r < TM; ++r)
#pragma unroll
        for (int c = 0; c < TN; ++c) {
            const int64_t i = row0 + ty * TM + r, j = col0 + tx * TN + c;
            cw[r][c] = (g.C && i < g.M && j < g.N) ? static_cast<const uint32_t*>(g.C)[i * g.ldc + j] : 0u;
        }

    for (int64_t k0 = 0; k0 < g.K; k0 += KC) {
        __syncthreads();
        // ---- stage: 16 bytes (32 elements) per task; 128 * 2 tasks for A, 64 * 2 for B ----
        for (int task = tid; task < (BM + BN) * 2; task += NT) {
            const bool is_a = task < BM * 2;
            const int u = is_a ? task : task - BM * 2;
            const int rows = is_a ? BM : BN;
            const int r = u % rows, h = u / rows;
            const int64_t grow = (is_a ? row0 : col0) + r;
            uint4 raw = make_uint4(0u, 0u, 0u, 0u);
            if (grow < (is_a ? g.M : g.N))
                raw = *reinterpret_cast<const uint4*>(static_cast<const unsigned char*>(is_a ? g.A : g.B) +
                                                      (grow * (is_a ? g.lda : g.ldb) + k0) / 2 + 16 * h);
            const uint32_t wv[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
            for (int w = 0; w < 4; ++w) {
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    uint32_t packed = 0u;
#pragma unroll
                    for (int n = 0; n < 4; ++n) packed |= fp4_byte((wv[w] >> (16 * half + 4 * n)) & 0xFu) << (8 * n);
                    if (is_a) s.a[h * 8 + w * 2 + half][r] = packed; else s.b[h * 8 + w * 2 + half][r] = packed;
                }
                // nonzero flags of the word's eight codes (magnitude bits 0..2 of a nibble not all zero -> bit 3 of the nibble)
                const uint32_t mag = wv[w] & 0x77777777u;
                const uint32_t flags = ((mag + 0x77777777u) | mag) & 0x88888888u;
                if (is_a) s.fa[h * 2 + (w >> 1)][w & 1][r] = flags; else s.fb[h * 2 + (w >> 1)][w & 1][r] = flags;
            }
        }
        for (int idx = tid; idx < (BM + BN) * 4; idx += NT) {
            const bool is_a = idx < BM * 4;
            const int u = is_a ? idx : idx - BM * 4;
            const int rows = is_a ? BM : BN;
            const int r = u % rows, grp = u / rows;                 // group of 16 inside the block
            const int64_t grow = (is_a ? row0 : col0) + r;
            uint32_t byte = NVF4 ? 0x38u : 127u;                    // 1.0 for rows outside the matrix
            if (grow < (is_a ? g.M : g.N)) {
                const int64_t sidx = grow * (is_a ? g.ld_sfa : g.ld_sfb) + (k0 / KC) * SPB + (NVF4 ? grp : grp / 2);
                byte = (is_a ? g.sfa : g.sfb)[sidx];
            }
            const uint32_t dec = decode_scale(byte, NVF4);
            if (is_a) s.sa[grp][r] = dec; else s.sb[grp][r] = dec;
        }
        __syncthreads();

#pragma unroll
        for (int rh = 0; rh < TM; rh += RH) {
            // ---- e_max: the scale exponents of the groups that hold a nonzero product (whatever their dot product: the
            // exponent is that of the scale factors) and the exponent of a nonzero accumulator ----
            int emax[RH][TN];
#pragma unroll
            for (int r = 0; r < RH; ++r)
#pragma unroll
                for (int c = 0; c < TN; ++c) {
                    const uint32_t w = cw[rh + r][c];
                    const uint32_t field = (w >> 23) & 0xFFu;
                    emax[r][c] = (w & 0x7FFFFFFFu) ? int(field ? field : 1u) - 127 + CB : 0;   // Exp(c) + CB (garbage for inf / NaN: unused)
                }
            uint32_t nan_rows = 0u, nan_cols = 0u;
#pragma unroll
            for (int grp = 0; grp < 4; ++grp) {
                const uint4 sa4 = *reinterpret_cast<const uint4*>(&s.sa[grp][ty * TM + rh]);
                const uint4 sb4 = *reinterpret_cast<const uint4*>(&s.sb[grp][tx * TN]);
                const uint32_t sav[RH] = {sa4.x, sa4.y, sa4.z, sa4.w}, sbv[TN] = {sb4.x, sb4.y, sb4.z, sb4.w};
                const uint4 fa0 = *reinterpret_cast<const uint4*>(&s.fa[grp][0][ty * TM + rh]), fa1 = *reinterpret_cast<const uint4*>(&s.fa[grp][1][ty * TM + rh]);
                const uint4 fb0 = *reinterpret_cast<const uint4*>(&s.fb[grp][0][tx * TN]), fb1 = *reinterpret_cast<const uint4*>(&s.fb[grp][1][tx * TN]);
                const uint32_t fa0v[RH] = {fa0.x, fa0.y, fa0.z, fa0.w}, fa1v[RH] = {fa1.x, fa1.y, fa1.z, fa1.w};
                const uint32_t fb0v[TN] = {fb0.x, fb0.y, fb0.z, fb0.w}, fb1v[TN] = {fb1.x, fb1.y, fb1.z, fb1.w};
#pragma unroll
                for (int r = 0; r < RH; ++r) nan_rows |= (sav[r] >> 31) << r;
#pragma unroll
                for (int c = 0; c < TN; ++c) nan_cols |= (sbv[c] >> 31) << c;
#pragma unroll
                for (int r = 0; r < RH; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c) {
                        const int eg = int((sav[r] >> 8) & 0xFFFFu) + int((sbv[c] >> 8) & 0xFFFFu);
                        // a group counts if some product a_k b_k of it is nonzero (even when they cancel) and, for UE4M3
                        // scales, neither scale factor is zero
                        bool live = ((fa0v[r] & fb0v[c]) | (fa1v[r] & fb1v[c])) != 0u;
                        if (NVF4) live = live && (sav[r] & 0xFFu) != 0u && (sbv[c] & 0xFFu) != 0u;
                        emax[r][c] = max(emax[r][c], live ? eg : 0);
                    }
            }
#pragma unroll
            for (int r = 0; r < RH; ++r)
#pragma unroll
                for (int c = 0; c < TN; ++c)
                    if (((nan_rows >> r) | (nan_cols >> c)) & 1u) sp_nan |= 1u << ((rh + r) * TN + c);
            // ---- accumulator term ----
            long long S[RH][TN];
#pragma unroll
            for (int r = 0; r < RH; ++r)
#pragma unroll
                for (int c = 0; c < TN; ++c) {
                    const uint32_t w = cw[rh + r][c];
                    const uint32_t field = (w >> 23) & 0xFFu;
                    const uint32_t sig = (w & 0x7FFFFFu) | (field ? 0x800000u : 0u);
                    const int d = emax[r][c] - (int(field ? field : 1u) - 127 + CB);
                    const unsigned long long t = (d >= 0 && d < 64) ? ((unsigned long long)sig << (F - 23)) >> d : 0ull;
                    S[r][c] = (w >> 31) ? -(long long)t : (long long)t;
                }
            // ---- groups: exact dot product, scale significands, align, truncate, add ----
#pragma unroll 1
            for (int grp = 0; grp < 4; ++grp) {
                int p[RH][TN];
#pragma unroll
                for (int r = 0; r < RH; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c) p[r][c] = 0;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int4 a4 = *reinterpret_cast<const int4*>(&s.a[grp * 4 + j][ty * TM + rh]);
                    const int4 b4 = *reinterpret_cast<const int4*>(&s.b[grp * 4 + j][tx * TN]);
                    const int av[RH] = {a4.x, a4.y, a4.z, a4.w}, bv[TN] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
                    for (int r = 0; r < RH; ++r)
#pragma unroll
                        for (int c = 0; c < TN; ++c) p[r][c] = __dp4a(av[r], bv[c], p[r][c]);
                }
                const uint4 sa4 = *reinterpret_cast<const uint4*>(&s.sa[grp][ty * TM + rh]);
                const uint4 sb4 = *reinterpret_cast<const uint4*>(&s.sb[grp][tx * TN]);
                const uint32_t sav[RH] = {sa4.x, sa4.y, sa4.z, sa4.w}, sbv[TN] = {sb4.x, sb4.y, sb4.z, sb4.w};
#pragma unroll
                for (int r = 0; r < RH; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c) {
                        int sg = p[r][c];
                        if (NVF4) sg = sg * int(sav[r] & 0xFFu) * int(sbv[c] & 0xFFu);
                        const int eg = int((sav[r] >> 8) & 0xFFFFu) + int((sbv[c] >> 8) & 0xFFFFu);
                        const int d = emax[r][c] - eg;
                        const unsigned long long mag = (unsigned long long)(unsigned)abs(sg) << (F - FRAC);
                        const unsigned long long t = (d >= 0 && d < 64) ? (mag >> d) : 0ull;
                        S[r][c] += sg < 0 ? -(long long)t : (long long)t;
                    }
            }
            // ---- RZ-FP32 ----
#pragma unroll
            for (int r = 0; r < RH; ++r)
#pragma unroll
                for (int c = 0; c < TN; ++c) {
                    const uint32_t w = cw[rh + r][c];
                    if (((w >> 23) & 0xFFu) == 0xFFu) continue;               // inf / NaN accumulator stays as it is
                    const long long Sv = S[r][c];
                    const unsigned long long mag = (unsigned long long)(Sv < 0 ? -Sv : Sv);
                    const int msb = 63 - __clzll((long long)mag);
                    const int ve = emax[r][c] - F + msb;                      // biased by CB
                    uint32_t out;
                    if (mag == 0ull) out = 0u;
                    else if (ve >= EMINB && ve <= EMAXB) {
                        const uint32_t sig = uint32_t(msb >= 23 ? (mag >> (msb - 23)) : (mag << (23 - msb)));
                        out = (Sv < 0 ? 0x80000000u : 0u) | (uint32_t(ve - CB + 127) << 23) | (sig & 0x7FFFFFu);
                    } else {
                        out = rho_apply(RHO_RZ_FP32, Sv, emax[r][c] - CB - F);
                    }
                    cw[rh + r][c] = out;
                }
        }
    }

#pragma unroll
    for (int r = 0; r < TM; ++r)
#pragma unroll
        for (int c = 0; c < TN; ++c) {
            const int64_t i = row0 + ty * TM + r, j = col0 + tx * TN + c;
            if (i >= g.M || j >= g.N) continue;
            uint32_t w = cw[r][c];
            if ((sp_nan >> (r * TN + c)) & 1u) w = 0x7FFFFFFFu;
            else if ((w & 0x7FFFFFFFu) > 0x7F800000u) w = 0x7FFFFFFFu;      // NaN accumulator input: canonical NaN
            static_cast<uint32_t*>(g.D)[i * g.ldd + j] = w;
        }
}

}  // namespace

bool fast_gst_supported(const DevModel& m, const GemmArgs& g) {
    if (m.family != FAM_GST || g.dot_mode || g.k_chunk || g.row_scale) return false;
    if (m.L != 64 || m.G != 16 || m.F != 35 || m.rho != RHO_RZ_FP32 || !m.packed4) return false;
    if (g.K % KC) return false;
    if ((g.lda % 32) || (g.ldb % 32)) return false;                 // 16-byte row starts (two elements per byte)
    if (g.M > 65535ll * BM) return false;
    return true;
}

int launch_fast_gst(const DevModel& m, const GemmArgs& g, cudaStream_t stream) {
    set_kernel_name("gstfdpa");
    const size_t sh = sizeof(Smem);
    dim3 grid((unsigned)((g.N + BN - 1) / BN), (unsigned)((g.M + BM - 1) / BM), 1);
    cudaError_t err;
    if (m.scale_fmt == EF_UE4M3) {
        err = cudaFuncSetAttribute(gst_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(sh));
        if (err == cudaSuccess) { gst_kernel<true><<<grid, NT, sh, stream>>>(m, g); err = cudaGetLastError(); }
    } else {
        err = cudaFuncSetAttribute(gst_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(sh));
        if (err == cudaSuccess) { gst_kernel<false><<<grid, NT, sh, stream>>>(m, g); err = cudaGetLastError(); }
    }
    if (err != cudaSuccess) {
        set_error("GST-FDPA kernel launch failed: %s", cudaGetErrorString(err));
        return MMASIM_ERR_CUDA;
    }
    return MMASIM_OK;
}

}  // namespace mmasim
