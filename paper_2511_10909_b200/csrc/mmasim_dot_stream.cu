// Streaming kernels for mmasim_dot_batch: n independent dot-product-accumulates d_t = Phi(a_t, b_t, c_t) (Equation 4),
// the shape of the paper's probe vectors (Section 3.1).  One thread owns one dot product and walks its two rows block
// by block with 16-byte loads; nothing is shared between threads, so the kernel is bound by HBM traffic
// (2 * K * element bytes + 8 bytes per dot) as long as the per-term integer work stays below it.
//   T-FDPA (Algorithm 7) for FP16 / BF16 / TF32 inputs, L in {4, 8, 16}, any F, rho in {RZ-FP32, RNE-FP16}
//   Phi_FTZ-AddMul (Algorithm 2) for FP16 / BF16 inputs, P in {2, 4}
// Everything else (8-bit inputs, other families, odd shapes) uses the generic kernels.
#include <cuda_fp16.h>
#include "mmasim_tfdpa_fast.cuh"

namespace mmasim {
namespace {

using fast::Elem;
using fast::EK_F16;
using fast::EK_BF16;
using fast::EK_TF32;

constexpr int DOT_THREADS = 256;

// Load L consecutive elements (L * BYTES is 8, 16, 32 or 64 bytes) as raw words.
template <int EK, int L>
__device__ __forceinline__ void load_block(const void* base, int64_t elem_index, uint32_t (&w)[L]) {
    constexpr int BYTES = Elem<EK>::BYTES;
    const unsigned char* p = static_cast<const unsigned char*>(base) + elem_index * BYTES;
    uint32_t raw[L * BYTES / 4];
    if (L * BYTES == 8) {
        const uint2 v = *reinterpret_cast<const uint2*>(p);
        raw[0] = v.x; raw[1] = v.y;
    } else {
#pragma unroll
        for (int q = 0; q < L * BYTES / 16; ++q) {
            const uint4 v = reinterpret_cast<const uint4*>(p)[q];
            raw[4 * q] = v.x; raw[4 * q + 1] = v.y; raw[4 * q + 2] = v.z; raw[4 * q + 3] = v.w;
        }
    }
#pragma unroll
    for (int k = 0; k < L; ++k) w[k] = BYTES == 2 ? ((raw[k / 2] >> (16 * (k % 2))) & 0xFFFFu) : raw[k];
}

template <int EK, int L, int RHO>
__global__ void __launch_bounds__(DOT_THREADS)
dot_tfdpa_kernel(DevModel m, int64_t n, int64_t K, const void* A, const void* B, const void* C, void* D) {
    constexpr bool ACC16 = RHO == RHO_RNE_FP16;
    constexpr int CB = fast::CB;
    constexpr int EMINB = (ACC16 ? -14 : -126) + CB, EMAXB = (ACC16 ? 15 : 127) + CB;
    const int64_t t = int64_t(blockIdx.x) * DOT_THREADS + threadIdx.x;
    if (t >= n) return;
    const int F = m.F;
    const int pre = F - 2 * Elem<EK>::MBITS;
    const int MB_ACC = ACC16 ? 10 : 23;
    uint32_t cw = 0u;
    if (C) cw = ACC16 ? uint32_t(static_cast<const uint16_t*>(C)[t]) : static_cast<const uint32_t*>(C)[t];

    for (int64_t k0 = 0; k0 < K; k0 += L) {
        uint32_t wa[L], wb[L];
        load_block<EK, L>(A, t * K + k0, wa);
        load_block<EK, L>(B, t * K + k0, wb);
        // Step 1: exact products and exponent sums.  Decoding is branch-free: the hidden bit is min(field, 1), the
        // unnormalised exponent max(field, 1); infinities and NaNs are found by the largest exponent field seen.
        using E = Elem<EK>;
        constexpr uint32_t TOP = (1u << E::EBITS) - 1u, MM = (1u << E::MBITS) - 1u;
        constexpr int SIGN_SHIFT = 31 - (E::MBITS + E::EBITS + E::LOW);   // moves the element's sign bit to bit 31
        int X[L], e[L], sm[L];                            // |product| << pre, exponent sum (field units), sign mask
        uint32_t fmax_seen = 0u;
#pragma unroll
        for (int k = 0; k < L; ++k) {
            const uint32_t xa = wa[k] >> E::LOW, xb = wb[k] >> E::LOW;
            const uint32_t fa = (xa >> E::MBITS) & TOP, fb = (xb >> E::MBITS) & TOP;
            const uint32_t sa = (xa & MM) | (min(fa, 1u) << E::MBITS);
            const uint32_t sb = ((xb & MM) | (min(fb, 1u) << E::MBITS)) << pre;
            X[k] = int(sa * sb);
            e[k] = int(max(fa, 1u) + max(fb, 1u));        // Exp(a) + Exp(b) + 2 * bias
            sm[k] = int((wa[k] ^ wb[k]) << SIGN_SHIFT) >> 31;
            fmax_seen = max(fmax_seen, max(fa, fb));
        }
        const AccDec dc = decode_acc(cw, ACC16);
        if (fmax_seen == TOP || dc.cls != CLS_FINITE) {
            // an infinity or a NaN among the 2L + 1 inputs: Section 4.2 decides the result (classes straight from the raw words)
            bool nan = dc.cls == CLS_NAN, pinf = dc.cls == CLS_INF && !dc.sign, ninf = dc.cls == CLS_INF && dc.sign;
#pragma unroll
            for (int k = 0; k < L; ++k) {
                const uint32_t xa = wa[k] >> E::LOW, xb = wb[k] >> E::LOW;
                const bool spa = ((xa >> E::MBITS) & TOP) == TOP, spb = ((xb >> E::MBITS) & TOP) == TOP;
                if (!(spa | spb)) continue;
                const bool nana = spa && (xa & MM), nanb = spb && (xb & MM);
                const bool za = (xa & ((1u << (E::MBITS + E::EBITS)) - 1u)) == 0u, zb = (xb & ((1u << (E::MBITS + E::EBITS)) - 1u)) == 0u;
                if (nana | nanb | (spa && zb) | (spb && za)) nan = true;          // NaN * x, inf * 0
                else if (((xa ^ xb) >> (E::MBITS + E::EBITS)) & 1u) ninf = true;   // inf * z = inf * sign(z)
                else pinf = true;
            }
            cw = special_word((nan || (pinf && ninf)) ? 1 : (pinf ? 2 : 3), ACC16, true);
            continue;
        }
        // Step 2: maximum exponent, alignment, truncation (sign-magnitude), exact sum.  Exponent sums are kept in field
        // units (biased by 2 * E::BIAS); `ceb` and `emax` below carry the bias CB like everywhere else.
        constexpr int EBIAS = CB - 2 * E::BIAS;           // e[k] + EBIAS = Exp(a) + Exp(b) + CB
        const int ceb = dc.exp + CB;
        int emax = ceb - EBIAS;
#pragma unroll
        for (int k = 0; k < L; ++k) emax = max(emax, e[k]);
        const uint32_t cmag = fast::lsr_clamp(dc.sig << (F >= MB_ACC ? F - MB_ACC : 0), (emax + EBIAS - ceb) + (F >= MB_ACC ? 0 : MB_ACC - F));
        // terms stay below 2^27 (F <= 25): eight of them and the accumulator fit 32 bits, sixteen need two partial sums
        int S0 = dc.sign ? -int(cmag) : int(cmag), S1 = 0;
#pragma unroll
        for (int k = 0; k < L; ++k) {
            const int tk = int(fast::lsr_clamp(uint32_t(X[k]), emax - e[k]));
            const int sk = (tk ^ sm[k]) - sm[k];
            if (L > 8 && k >= L / 2) S1 += sk; else S0 += sk;
        }
        emax += EBIAS;
        const long long S = (long long)S0 + (long long)S1;
        // Step 3: rho
        const bool fits = S == (long long)int(S);
        int vmin = EMINB, vmax = EMINB;
        fast::Acc a;
        if (fits && F >= MB_ACC && RHO != RHO_RZ_E8M13) {
            fast::rho_fast<25, RHO>(int(S), emax + (25 - F), a, vmin, vmax);   // value = S * 2^(e_max - F): rescaled to the F = 25 form
        }
        if (!fits || F < MB_ACC || vmin < EMINB || vmax > EMAXB) {
            cw = rho_apply(RHO, S, emax - CB - F);
        } else {
            cw = fast::acc_to_word<25, ACC16>(a, 0u);
        }
    }
    if (ACC16) static_cast<uint16_t*>(D)[t] = uint16_t(cw);
    else static_cast<uint32_t*>(D)[t] = cw;
}

// Phi_FTZ-AddMul, one dot per thread.
template <int EK, int P>
__global__ void __launch_bounds__(DOT_THREADS)
dot_ftz_kernel(int64_t n, int64_t K, const void* A, const void* B, const void* C, void* D) {
    const int64_t t = int64_t(blockIdx.x) * DOT_THREADS + threadIdx.x;
    if (t >= n) return;
    float d = 0.0f;
    if (C) {
        const uint32_t w = static_cast<const uint32_t*>(C)[t];
        d = ((w & 0x7F800000u) == 0u && (w & 0x007FFFFFu)) ? 0.0f : __uint_as_float(w);     // FlushSubnormal(C)
    }
    constexpr int STEP = 4;                           // elements per load (8 bytes)
    for (int64_t k0 = 0; k0 < K; k0 += STEP) {
        uint32_t wa[STEP], wb[STEP];
        load_block<EK, STEP>(A, t * K + k0, wa);
        load_block<EK, STEP>(B, t * K + k0, wb);
        float a[STEP], b[STEP];
#pragma unroll
        for (int k = 0; k < STEP; ++k) {
            if (EK == EK_BF16) {
                a[k] = ((wa[k] & 0x7F80u) == 0u && (wa[k] & 0x007Fu)) ? 0.0f : __uint_as_float(wa[k] << 16);
                b[k] = ((wb[k] & 0x7F80u) == 0u && (wb[k] & 0x007Fu)) ? 0.0f : __uint_as_float(wb[k] << 16);
            } else {
                a[k] = ((wa[k] & 0x7C00u) == 0u && (wa[k] & 0x03FFu)) ? 0.0f : __half2float(__ushort_as_half((unsigned short)wa[k]));
                b[k] = ((wb[k] & 0x7C00u) == 0u && (wb[k] & 0x03FFu)) ? 0.0f : __half2float(__ushort_as_half((unsigned short)wb[k]));
            }
        }
        if (P == 4) {
            const float s = ftz_add(ftz_add(ftz_mul(a[0], b[0]), ftz_mul(a[1], b[1])), ftz_add(ftz_mul(a[2], b[2]), ftz_mul(a[3], b[3])));
            d = ftz_add(d, s);
        } else {
            d = ftz_add(d, ftz_add(ftz_mul(a[0], b[0]), ftz_mul(a[1], b[1])));
            d = ftz_add(d, ftz_add(ftz_mul(a[2], b[2]), ftz_mul(a[3], b[3])));
        }
    }
    uint32_t w = __float_as_uint(d);
    if (d != d) w = 0x7FC00000u;
    static_cast<uint32_t*>(D)[t] = w;
}

template <int EK, int L>
cudaError_t launch_t(const DevModel& m, const GemmArgs& g, cudaStream_t st) {
    const unsigned blocks = unsigned((g.M + DOT_THREADS - 1) / DOT_THREADS);
    if (m.rho == RHO_RZ_FP32) dot_tfdpa_kernel<EK, L, RHO_RZ_FP32><<<blocks, DOT_THREADS, 0, st>>>(m, g.M, g.K, g.A, g.B, g.C, g.D);
    else dot_tfdpa_kernel<EK, L, RHO_RNE_FP16><<<blocks, DOT_THREADS, 0, st>>>(m, g.M, g.K, g.A, g.B, g.C, g.D);
    return cudaGetLastError();
}

template <int EK>
cudaError_t launch_t_l(const DevModel& m, const GemmArgs& g, int L, cudaStream_t st) {
    switch (L) {
        case 4: return launch_t<EK, 4>(m, g, st);
        case 8: return launch_t<EK, 8>(m, g, st);
        case 16: return launch_t<EK, 16>(m, g, st);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

bool dot_stream_supported(const DevModel& m, const GemmArgs& g) {
    if (!g.dot_mode || m.fmt_a != m.fmt_b) return false;
    const int bytes = fmt_desc(m.fmt_a).storage_bits / 8;
    if (m.family == FAM_T) {
        if (m.fmt_a != EF_F16 && m.fmt_a != EF_BF16 && m.fmt_a != EF_TF32) return false;
        const int L = int(g.K < m.L ? g.K : m.L);
        if (L != 4 && L != 8 && L != 16) return false;
        if (m.rho != RHO_RZ_FP32 && m.rho != RHO_RNE_FP16) return false;
        if ((m.rho == RHO_RNE_FP16) != (m.acc == ACC_F16)) return false;
        if (m.F < 23 || m.F > 25) return false;
        return (g.K * bytes) % (L * bytes >= 16 ? 16 : 8) == 0;     // every row starts on a vector-load boundary
    }
    if (m.family == FAM_FTZ) return (m.fmt_a == EF_F16 || m.fmt_a == EF_BF16) && g.K % 4 == 0;
    return false;
}

int launch_dot_stream(const DevModel& m, const GemmArgs& g, cudaStream_t stream) {
    cudaError_t err = cudaErrorInvalidValue;
    if (m.family == FAM_T) {
        const int L = int(g.K < m.L ? g.K : m.L);
        set_kernel_name("dot_tfdpa");
        if (m.fmt_a == EF_F16) err = launch_t_l<EK_F16>(m, g, L, stream);
        else if (m.fmt_a == EF_BF16) err = launch_t_l<EK_BF16>(m, g, L, stream);
        else err = launch_t_l<EK_TF32>(m, g, L, stream);
    } else {
        set_kernel_name("dot_ftz");
        const unsigned blocks = unsigned((g.M + DOT_THREADS - 1) / DOT_THREADS);
        if (m.fmt_a == EF_F16) dot_ftz_kernel<EK_F16, 4><<<blocks, DOT_THREADS, 0, stream>>>(g.M, g.K, g.A, g.B, g.C, g.D);
        else if (m.P == 4) dot_ftz_kernel<EK_BF16, 4><<<blocks, DOT_THREADS, 0, stream>>>(g.M, g.K, g.A, g.B, g.C, g.D);
        else dot_ftz_kernel<EK_BF16, 2><<<blocks, DOT_THREADS, 0, stream>>>(g.M, g.K, g.A, g.B, g.C, g.D);
        err = cudaGetLastError();
    }
    if (err != cudaSuccess) {
        set_error("dot_batch kernel launch failed: %s", cudaGetErrorString(err));
        return MMASIM_ERR_CUDA;
    }
    return MMASIM_OK;
}

}  // namespace mmasim
