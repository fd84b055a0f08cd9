// Tuned kernels for the models that run on the floating-point pipes:
//   Phi_FMA (Algorithm 4): d <- fma(a_k, b_k, d) in ascending k, FP32 or FP64, IEEE-754 round-to-nearest-even
//   Phi_FTZ-AddMul (Algorithm 2): FTZ-Mul products, pairwise FTZ-Add over groups of P, FTZ-Add into d
// Register-tiled like a classic SGEMM (CTA tile in shared memory, k-major, one micro-tile of accumulators per
// thread), except that the order of operations inside one output is fixed by the model, so there is no split-K and
// no reassociation: every accumulator walks K sequentially.
//
// FTZ-Add / FTZ-Mul use the hardware flush-to-zero mode (`add.rn.ftz.f32`, `mul.rn.ftz.f32`), which flushes
// subnormal results to a zero of the same sign, exactly the last line of Algorithm 1.  "Round, then flush" and the
// hardware's flush coincide here: products of two BF16 / FP16 values have at most 22 significant bits, and sums of
// two normal-or-zero FP32 values below 2^-125 are multiples of 2^-149, so no result is rounded across the 2^-126
// boundary.  Inputs are never subnormal (Algorithm 2 flushes A, B and C to +0 first; every intermediate is flushed).
#include <cuda_fp16.h>
#include "mmasim_internal.h"

namespace mmasim {
namespace {

constexpr int NT = 256, KC = 16;

enum FpMode : int { FP_FMA32 = 0, FP_FMA64 = 1, FP_FTZ_F16 = 2, FP_FTZ_BF16 = 3 };

template <int MODE> struct ModeTraits;
template <> struct ModeTraits<FP_FMA32> { using acc_t = float; using in_t = float; static constexpr int TM = 8, TN = 8, IN_BYTES = 4; };
template <> struct ModeTraits<FP_FMA64> { using acc_t = double; using in_t = double; static constexpr int TM = 4, TN = 8, IN_BYTES = 8; };
template <> struct ModeTraits<FP_FTZ_F16> { using acc_t = float; using in_t = float; static constexpr int TM = 8, TN = 4, IN_BYTES = 2; };
template <> struct ModeTraits<FP_FTZ_BF16> { using acc_t = float; using in_t = float; static constexpr int TM = 8, TN = 4, IN_BYTES = 2; };

__device__ __forceinline__ float add_ftz(float x, float y) {
    float z;
    asm("add.rn.ftz.f32 %0, %1, %2;" : "=f"(z) : "f"(x), "f"(y));
    return z;
}
__device__ __forceinline__ float mul_ftz(float x, float y) {
    float z;
    asm("mul.rn.ftz.f32 %0, %1, %2;" : "=f"(z) : "f"(x), "f"(y));
    return z;
}

// FlushSubnormal of Algorithm 2 followed by the exact conversion to FP32.
__device__ __forceinline__ float load_flushed(uint32_t w, bool bf16) {
    if (bf16) return ((w & 0x7F80u) == 0u && (w & 0x007Fu)) ? 0.0f : __uint_as_float(w << 16);
    return ((w & 0x7C00u) == 0u && (w & 0x03FFu)) ? 0.0f : __half2float(__ushort_as_half((unsigned short)w));
}

template <int MODE, int P>
__global__ void __launch_bounds__(NT, 2) fp_kernel(GemmArgs g) {
    using T = ModeTraits<MODE>;
    using in_t = typename T::in_t;
    using acc_t = typename T::acc_t;
    constexpr int TM = T::TM, TN = T::TN;
    constexpr int BM = 16 * TM, BN = 16 * TN;
    constexpr bool FTZ = MODE == FP_FTZ_F16 || MODE == FP_FTZ_BF16;
    constexpr int EPT = 16 / T::IN_BYTES;                   // elements per 16-byte load
    constexpr int TPR = KC / EPT;                           // loads per row per chunk
    static_assert(KC % EPT == 0 && (!FTZ || KC % P == 0), "chunk layout");
    __shared__ __align__(16) in_t As[KC][BM];
    __shared__ __align__(16) in_t Bs[KC][BN];

    const int tid = threadIdx.x;
    const int tx = tid % 16, ty = tid / 16;
    const int64_t row0 = int64_t(blockIdx.y) * BM, col0 = int64_t(blockIdx.x) * BN;
    // Columns of a thread's micro-tile: groups of V (one 16-byte shared load), 16 * V columns apart, so that the sixteen
    // threads of a row of the thread grid read 256 contiguous bytes per load (no bank conflicts).
    constexpr int V = 16 / int(sizeof(in_t));
    auto col_of = [&](int c) { return (c / V) * (16 * V) + tx * V + (c % V); };

    acc_t d[TM][TN];
#pragma unroll
    for (int r = 0; r < TM; ++r)
#pragma unroll
        for (int c = 0; c < TN; ++c) {
            const int64_t i = row0 + ty * TM + r, j = col0 + col_of(c);
            acc_t v = acc_t(0);
            if (g.C && i < g.M && j < g.N) {
                if (FTZ) {
                    const uint32_t w = static_cast<const uint32_t*>(g.C)[i * g.ldc + j];
                    v = ((w & 0x7F800000u) == 0u && (w & 0x007FFFFFu)) ? 0.0f : __uint_as_float(w);   // FlushSubnormal(C)
                } else {
                    v = static_cast<const acc_t*>(g.C)[i * g.ldc + j];
                }
            }
            d[r][c] = v;
        }

    // The raw 16-byte words of the next chunk are fetched while the current one is computed.
    constexpr int TASKS = (BM + BN) * TPR, PER_THREAD = (TASKS + NT - 1) / NT;
    uint4 raw[PER_THREAD];
    auto fetch = [&](int64_t k0) {
#pragma unroll
        for (int it = 0; it < PER_THREAD; ++it) {
            const int task = it * NT + tid;
            const bool is_a = task < BM * TPR;
            const int u = is_a ? task : task - BM * TPR;
            const int rows = is_a ? BM : BN;
            const int r = u % rows, h = u / rows;
            const int64_t grow = (is_a ? row0 : col0) + r;
            raw[it] = make_uint4(0u, 0u, 0u, 0u);
            if (task < TASKS && grow < (is_a ? g.M : g.N))
                raw[it] = *reinterpret_cast<const uint4*>(static_cast<const unsigned char*>(is_a ? g.A : g.B) +
                                                          (grow * (is_a ? g.lda : g.ldb) + k0 + h * EPT) * T::IN_BYTES);
        }
    };
    fetch(0);
    for (int64_t k0 = 0; k0 < g.K; k0 += KC) {
        __syncthreads();
        // ---- stage: decode the fetched words, stored k-major ----
#pragma unroll
        for (int it = 0; it < PER_THREAD; ++it) {
            const int task = it * NT + tid;
            if (task >= TASKS) break;
            const bool is_a = task < BM * TPR;
            const int u = is_a ? task : task - BM * TPR;
            const int rows = is_a ? BM : BN;
            const int r = u % rows, h = u / rows;
            const uint32_t wv[4] = {raw[it].x, raw[it].y, raw[it].z, raw[it].w};
#pragma unroll
            for (int q = 0; q < EPT; ++q) {
                in_t v;
                if (MODE == FP_FMA32) v = in_t(__uint_as_float(wv[q]));
                else if (MODE == FP_FMA64) v = in_t(__longlong_as_double((long long)((unsigned long long)wv[2 * q] | ((unsigned long long)wv[2 * q + 1] << 32))));
                else v = in_t(load_flushed((wv[q / 2] >> (16 * (q % 2))) & 0xFFFFu, MODE == FP_FTZ_BF16));
                if (is_a) As[h * EPT + q][r] = v; else Bs[h * EPT + q][r] = v;
            }
        }
        __syncthreads();
        if (k0 + KC < g.K) fetch(k0 + KC);

        if (!FTZ) {
            // fully unrolled: with a partial unroll the compiler rotates the accumulators through register moves
            // (two moves per multiply-add in the FP64 kernel)
#pragma unroll
            for (int kk = 0; kk < KC; ++kk) {
                in_t a[TM], b[TN];
#pragma unroll
                for (int r = 0; r < TM; ++r) a[r] = As[kk][ty * TM + r];
#pragma unroll
                for (int c = 0; c < TN; ++c) b[c] = Bs[kk][col_of(c)];
#pragma unroll
                for (int r = 0; r < TM; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c) d[r][c] = fma(a[r], b[c], d[r][c]);   // one rounding (fmaf for float)
            }
        } else {
#pragma unroll 1
            for (int kg = 0; kg < KC; kg += P) {
                float s[TM][TN], u[P == 4 ? TM : 1][P == 4 ? TN : 1];
#pragma unroll
                for (int l = 0; l < P; ++l) {
                    float a[TM], b[TN];
#pragma unroll
                    for (int r = 0; r < TM; ++r) a[r] = float(As[kg + l][ty * TM + r]);
#pragma unroll
                    for (int c = 0; c < TN; ++c) b[c] = float(Bs[kg + l][col_of(c)]);
#pragma unroll
                    for (int r = 0; r < TM; ++r)
#pragma unroll
                        for (int c = 0; c < TN; ++c) {
                            const float p = mul_ftz(a[r], b[c]);
                            if (l == 0) s[r][c] = p;
                            else if (l == 1) s[r][c] = add_ftz(s[r][c], p);
                            else if (l == 2) u[P == 4 ? r : 0][P == 4 ? c : 0] = p;
                            else u[P == 4 ? r : 0][P == 4 ? c : 0] = add_ftz(u[P == 4 ? r : 0][P == 4 ? c : 0], p);
                        }
                }
#pragma unroll
                for (int r = 0; r < TM; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c) {
                        float t = s[r][c];
                        if (P == 4) t = add_ftz(t, u[P == 4 ? r : 0][P == 4 ? c : 0]);
                        d[r][c] = acc_t(add_ftz(float(d[r][c]), t));
                    }
            }
        }
    }

#pragma unroll
    for (int r = 0; r < TM; ++r)
#pragma unroll
        for (int c = 0; c < TN; ++c) {
            const int64_t i = row0 + ty * TM + r, j = col0 + col_of(c);
            if (i >= g.M || j >= g.N) continue;
            const acc_t v = d[r][c];
            if (sizeof(acc_t) == 4) {
                uint32_t w = __float_as_uint(float(v));
                if (v != v) w = 0x7FC00000u;
                static_cast<uint32_t*>(g.D)[i * g.ldd + j] = w;
            } else {
                unsigned long long w = (unsigned long long)__double_as_longlong(double(v));
                if (v != v) w = 0x7FF8000000000000ull;
                static_cast<unsigned long long*>(g.D)[i * g.ldd + j] = w;
            }
        }
}

template <int MODE, int P>
cudaError_t launch_fp(const GemmArgs& g, cudaStream_t stream) {
    using T = ModeTraits<MODE>;
    constexpr int BM = 16 * T::TM, BN = 16 * T::TN;
    dim3 grid((unsigned)((g.N + BN - 1) / BN), (unsigned)((g.M + BM - 1) / BM), 1);
    fp_kernel<MODE, P><<<grid, NT, 0, stream>>>(g);
    return cudaGetLastError();
}

}  // namespace

bool fast_fp_supported(const DevModel& m, const GemmArgs& g) {
    if (g.dot_mode || g.k_chunk || g.row_scale) return false;
    if (m.family != FAM_FMA && m.family != FAM_FTZ) return false;
    const int bytes = fmt_desc(m.fmt_a).storage_bits / 8;
    if (g.K % KC) return false;
    if (((g.lda * bytes) % 16) || ((g.ldb * bytes) % 16)) return false;
    if (g.M > 65535ll * 32) return false;
    return true;
}

int launch_fast_fp(const DevModel& m, const GemmArgs& g, cudaStream_t stream) {
    cudaError_t err;
    if (m.family == FAM_FMA) {
        set_kernel_name(m.acc == ACC_F64 ? "fma_f64" : "fma_f32");
        err = m.acc == ACC_F64 ? launch_fp<FP_FMA64, 2>(g, stream) : launch_fp<FP_FMA32, 2>(g, stream);
    } else {
        set_kernel_name("ftz_addmul");
        if (m.fmt_a == EF_F16) err = launch_fp<FP_FTZ_F16, 4>(g, stream);
        else if (m.P == 4) err = launch_fp<FP_FTZ_BF16, 4>(g, stream);
        else err = launch_fp<FP_FTZ_BF16, 2>(g, stream);
    }
    if (err != cudaSuccess) {
        set_error("floating-point kernel launch failed: %s", cudaGetErrorString(err));
        return MMASIM_ERR_CUDA;
    }
    return MMASIM_OK;
}

}  // namespace mmasim
