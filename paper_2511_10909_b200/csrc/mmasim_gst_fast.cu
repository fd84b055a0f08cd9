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
// fractional bits and added.  Alignment, truncation and addition run on the FP64 pipe, where all of it is exact: with
// q = 2^(e_max - F) and M = 1.5 * 2^52 * q carrying the sign of the term,  fma.rz(s_g, 2^(e_g - frac), M)  is
// M + RZ_q(term) - the sum has the term's sign, so rounding toward zero truncates its magnitude - and two exact additions
// move that into the block's sum; s_g becomes a double by one conversion instruction (exact).  Exponents are handled as exponent fields of doubles in place: the staged scale
// words hold (Exp + bias) << 20 with the significand below, the sum of an A word and a B word is the field of
// 2^(Exp(alpha) + Exp(beta)) (with the two significands added below it, masked away after the maximum).  RZ-FP32 is one
// conversion instruction.  Liveness of a group needs its per-element nonzero masks (16 bits per row and group); a row
// group with at least nine nonzero elements meets every such column group in a nonzero product, so a thread whose rows
// and columns are all that dense (every ordinary input) skips the test.  NaN scale factors and a NaN / infinite
// accumulator set sticky per-output flags (Section 4.2); FP4 itself has no special values.
#include "mmasim_device.cuh"

namespace mmasim {
namespace {

constexpr int BM = 128, BN = 64, TM = 8, TN = 4, RH = 4, KC = 64, KW = KC / 4, NT = 256;
constexpr int SB_A = 512, SB_B = 511;   // biases of the staged scale exponents: their sum is the bias of a double

struct Smem {
    uint32_t a[KW][BM];                 // four elements per word, as signed bytes holding 2 * value
    uint32_t b[KW][BN];
    uint32_t sa[4][BM];                 // per group of the block: (Exp + bias) << 20 | Sig; bit 31: NaN; a zero significand
    uint32_t sb[4][BN];                 // (UE4M3 zero) has the exponent field 0: such a group never wins the maximum
    uint32_t fa[2][BM];                 // per pair of groups (2 h, 2 h + 1): bit 16 (g & 1) + n = element n of group g is nonzero
    uint32_t fb[2][BN];
    uint32_t da[2][BM];                 // per pair of groups: both have at least nine nonzero elements
    uint32_t db[2][BN];
};

// Signed byte 2 * value of an E2M1 code (bit 3 sign, bits 2..0 magnitude code: 0, .5, 1, 1.5, 2, 3, 4, 6).
__device__ __forceinline__ uint32_t fp4_byte(uint32_t code) {
    const uint32_t mags = 0x0C080604u, mags_lo = 0x03020100u;       // bytes: 12, 8, 6, 4 | 3, 2, 1, 0
    const uint32_t m = ((code & 4u) ? mags : mags_lo) >> (8u * (code & 3u)) & 0xFFu;
    return (code & 8u) ? ((0u - m) & 0xFFu) : m;
}

__device__ __forceinline__ uint32_t decode_scale(uint32_t byte, bool ue4m3, int bias) {
    if (ue4m3) {
        const uint32_t x = byte & 0x7Fu;
        if (x == 0x7Fu) return 0x80000000u;
        const uint32_t field = x >> 3, mant = x & 7u;
        const uint32_t sig = mant | (field ? 8u : 0u);
        const int e = int(field ? field : 1u) - 7;
        return sig ? (uint32_t(e + bias) << 20) | sig : 0u;
    }
    if (byte == 0xFFu) return 0x80000000u;
    return (uint32_t(int(byte) - 127 + bias) << 20) | 1u;
}

// 8-bit mask of the nonzero codes among the eight nibbles of a word (a code is zero when its magnitude bits 0..2 are)
__device__ __forceinline__ uint32_t nonzero8(uint32_t w) {
    const uint32_t mag = w & 0x77777777u;
    uint32_t x = (((mag + 0x77777777u) | mag) >> 3) & 0x11111111u;     // bit 4 n: code n is nonzero
    x = (x | (x >> 3)) & 0x03030303u;
    x = (x | (x >> 6)) & 0x000F000Fu;
    return (x | (x >> 12)) & 0xFFu;
}
// 16-bit mask for the 16 codes of two words (low word first)
__device__ __forceinline__ uint32_t nonzero16(uint32_t w0, uint32_t w1) { return nonzero8(w0) | (nonzero8(w1) << 8); }

template <bool NVF4>
__global__ void __launch_bounds__(NT, 2) gst_kernel(DevModel m, GemmArgs g) {
    constexpr int F = 35;
    constexpr int FRAC = NVF4 ? 8 : 2;              // fractional bits of p_g * Sig(alpha) * Sig(beta)
    constexpr int SPB = NVF4 ? 4 : 2;               // scale factors per block of 64 and row
    constexpr int EXPF = 0x7FF00000, HALF = 0x00080000;
    constexpr uint32_t LOWF = uint32_t(1023 - 126) << 20;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    Smem& s = *reinterpret_cast<Smem*>(smem_raw);

    const int tid = threadIdx.x;
    const int tx = tid % 16, ty = tid / 16;
    const int64_t row0 = int64_t(blockIdx.y) * BM, col0 = int64_t(blockIdx.x) * BN;

    uint32_t cw[TM][TN];                            // the accumulator of each output: a finite FP32 word
    uint32_t sp_nan = 0u, sp_pinf = 0u, sp_ninf = 0u;   // sticky special values (bit r * TN + c)
#pragma unroll
    for (int r = 0; r < TM; ++r)
#pragma unroll
        for (int c = 0; c < TN; ++c) {
            const int64_t i = row0 + ty * TM + r, j = col0 + tx * TN + c;
            uint32_t w = (g.C && i < g.M && j < g.N) ? static_cast<const uint32_t*>(g.C)[i * g.ldc + j] : 0u;
            if ((w & 0x7F800000u) == 0x7F800000u) {
                const uint32_t bit = 1u << (r * TN + c);
                if (w & 0x007FFFFFu) sp_nan |= bit; else if (w >> 31) sp_ninf |= bit; else sp_pinf |= bit;
                w = 0u;
            }
            cw[r][c] = w;
        }

    for (int64_t k0 = 0; k0 < g.K; k0 += KC) {
        __syncthreads();
        // ---- stage: 16 bytes (32 elements = two groups) per task; 128 * 2 tasks for A, 64 * 2 for B ----
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
            }
            const uint32_t f0 = nonzero16(wv[0], wv[1]), f1 = nonzero16(wv[2], wv[3]);
            const uint32_t dense = (__popc(f0) >= 9 && __popc(f1) >= 9) ? 1u : 0u;
            if (is_a) { s.fa[h][r] = f0 | (f1 << 16); s.da[h][r] = dense; }
            else { s.fb[h][r] = f0 | (f1 << 16); s.db[h][r] = dense; }
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
            const uint32_t dec = decode_scale(byte, NVF4, is_a ? SB_A : SB_B);
            if (is_a) s.sa[grp][r] = dec; else s.sb[grp][r] = dec;
        }
        __syncthreads();

#pragma unroll
        for (int rh = 0; rh < TM; rh += RH) {
            // ---- e_max as the exponent field of a double: the accumulator's (zero: none; FP32 subnormal: -126) and the
            // groups' (the sum of the two scale words; what sits below the field is masked after the maximum) ----
            double cd[RH][TN];
            int key[RH][TN];
#pragma unroll
            for (int r = 0; r < RH; ++r)
#pragma unroll
                for (int c = 0; c < TN; ++c) {
                    cd[r][c] = double(__uint_as_float(cw[rh + r][c]));
                    key[r][c] = int(__viaddmax_u32(uint32_t(__double2hiint(cd[r][c]) & EXPF), 0xFFFFFFFFu, LOWF - 1u) + 1u);
                }
            const uint4 d0 = *reinterpret_cast<const uint4*>(&s.da[0][ty * TM + rh]), d1 = *reinterpret_cast<const uint4*>(&s.da[1][ty * TM + rh]);
            const uint4 e0 = *reinterpret_cast<const uint4*>(&s.db[0][tx * TN]), e1 = *reinterpret_cast<const uint4*>(&s.db[1][tx * TN]);
            // every group with nonzero scale factors holds a nonzero product; otherwise (rare) the per-element masks decide
            const bool all_dense = (d0.x & d0.y & d0.z & d0.w & d1.x & d1.y & d1.z & d1.w & e0.x & e0.y & e0.z & e0.w & e1.x & e1.y & e1.z & e1.w) != 0u;
            uint32_t nan_rows = 0u, nan_cols = 0u;
#pragma unroll
            for (int grp = 0; grp < 4; ++grp) {
                const uint4 sa4 = *reinterpret_cast<const uint4*>(&s.sa[grp][ty * TM + rh]);
                const uint4 sb4 = *reinterpret_cast<const uint4*>(&s.sb[grp][tx * TN]);
                const uint32_t sav[RH] = {sa4.x, sa4.y, sa4.z, sa4.w}, sbv[TN] = {sb4.x, sb4.y, sb4.z, sb4.w};
#pragma unroll
                for (int r = 0; r < RH; ++r) nan_rows |= (sav[r] >> 31) << r;
#pragma unroll
                for (int c = 0; c < TN; ++c) nan_cols |= (sbv[c] >> 31) << c;
                if (all_dense) {
#pragma unroll
                    for (int r = 0; r < RH; ++r)
#pragma unroll
                        for (int c = 0; c < TN; ++c) key[r][c] = __viaddmax_s32(int(sav[r]), int(sbv[c]), key[r][c]);
                } else {
                    const uint4 fa4 = *reinterpret_cast<const uint4*>(&s.fa[grp >> 1][ty * TM + rh]);
                    const uint4 fb4 = *reinterpret_cast<const uint4*>(&s.fb[grp >> 1][tx * TN]);
                    const uint32_t fav[RH] = {fa4.x, fa4.y, fa4.z, fa4.w}, fbv[TN] = {fb4.x, fb4.y, fb4.z, fb4.w};
#pragma unroll
                    for (int r = 0; r < RH; ++r)
#pragma unroll
                        for (int c = 0; c < TN; ++c)
                            if (((fav[r] & fbv[c]) >> (16 * (grp & 1))) & 0xFFFFu) key[r][c] = max(key[r][c], int(sav[r] + sbv[c]));
                }
            }
            if (nan_rows | nan_cols) {
#pragma unroll
                for (int r = 0; r < RH; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c)
                        if (((nan_rows >> r) | (nan_cols >> c)) & 1u) sp_nan |= 1u << ((rh + r) * TN + c);
            }
            // ---- the accumulator term: M' + RZ_q(c), minus M' ----
            double S[RH][TN];
            int mhi[RH][TN];                        // high word of M = 1.5 * 2^52 * 2^(e_max - F)
#pragma unroll
            for (int r = 0; r < RH; ++r)
#pragma unroll
                for (int c = 0; c < TN; ++c) {
                    mhi[r][c] = ((key[r][c] & EXPF) + ((52 - F) << 20)) | HALF;
                    const double Ms = __hiloint2double(mhi[r][c] | (__double2hiint(cd[r][c]) & int(0x80000000u)), 0);
                    S[r][c] = __dsub_rn(__dadd_rz(cd[r][c], Ms), Ms);
                }
            // ---- groups: exact dot product, scale significands, then one fused multiply-add rounding toward zero ----
#pragma unroll 1
            for (int grp = 0; grp < 4; ++grp) {
                int p[RH][TN];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int4 a4 = *reinterpret_cast<const int4*>(&s.a[grp * 4 + j][ty * TM + rh]);
                    const int4 b4 = *reinterpret_cast<const int4*>(&s.b[grp * 4 + j][tx * TN]);
                    const int av[RH] = {a4.x, a4.y, a4.z, a4.w}, bv[TN] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
                    for (int r = 0; r < RH; ++r)
#pragma unroll
                        for (int c = 0; c < TN; ++c) p[r][c] = __dp4a(av[r], bv[c], j == 0 ? 0 : p[r][c]);
                }
                const uint4 sa4 = *reinterpret_cast<const uint4*>(&s.sa[grp][ty * TM + rh]);
                const uint4 sb4 = *reinterpret_cast<const uint4*>(&s.sb[grp][tx * TN]);
                const uint32_t sag[RH] = {sa4.x, sa4.y, sa4.z, sa4.w}, sbg[TN] = {sb4.x, sb4.y, sb4.z, sb4.w};
                int ea20[RH], eb20[TN];             // exponent fields: their sum is the high word of 2^(e_g - frac)
#pragma unroll
                for (int r = 0; r < RH; ++r) ea20[r] = int(sag[r] & uint32_t(EXPF)) - (FRAC << 20);
#pragma unroll
                for (int c = 0; c < TN; ++c) eb20[c] = int(sbg[c] & uint32_t(EXPF));
#pragma unroll
                for (int r = 0; r < RH; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c) {
                        int sg = p[r][c];
                        if (NVF4) sg = sg * int(sag[r] & 0xFFu) * int(sbg[c] & 0xFFu);
                        const double gd = __int2double_rn(sg);                      // exact
                        const double sc = __hiloint2double(ea20[r] + eb20[c], 0);                       // 2^(e_g - frac)
                        const double Ms = __hiloint2double(mhi[r][c] | (sg & int(0x80000000u)), 0);
                        S[r][c] = __dsub_rn(__dadd_rn(S[r][c], __fma_rz(gd, sc, Ms)), Ms);
                    }
            }
            // ---- RZ-FP32 (a zero result is +0); a sum of 2^128 or more is an overflow: infinity from now on ----
            uint32_t wmax = 0u;
#pragma unroll
            for (int r = 0; r < RH; ++r)
#pragma unroll
                for (int c = 0; c < TN; ++c) {
                    const uint32_t w = positive_zero(__float_as_uint(__double2float_rz(S[r][c])), 0x7FFFFFFFu);
                    wmax = max(wmax, w & 0x7FFFFFFFu);
                    cw[rh + r][c] = w;
                }
            if (wmax >= 0x7F7FFFFFu) {                          // rare: the conversion saturates at the largest finite word
#pragma unroll
                for (int r = 0; r < RH; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c)
                        if (fabs(S[r][c]) >= 3.402823669209385e38) {
                            const uint32_t bit = 1u << ((rh + r) * TN + c);
                            if (!((sp_nan | sp_pinf | sp_ninf) & bit)) { if (S[r][c] < 0.0) sp_ninf |= bit; else sp_pinf |= bit; }
                            cw[rh + r][c] = 0u;
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
            uint32_t w = cw[r][c];
            if ((sp_nan >> bit) & 1u) w = 0x7FFFFFFFu;
            else if (((sp_pinf & sp_ninf) >> bit) & 1u) w = 0x7FFFFFFFu;
            else if ((sp_pinf >> bit) & 1u) w = 0x7F800000u;
            else if ((sp_ninf >> bit) & 1u) w = 0xFF800000u;
            static_cast<uint32_t*>(g.D)[i * g.ldd + j] = w;
        }
}

}  // namespace

bool fast_gst_supported(const DevModel& m, const GemmArgs& g) {
    if (m.family != FAM_GST || g.dot_mode || g.k_chunk || g.row_scale || m.literal_emax) return false;
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
