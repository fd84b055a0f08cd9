// Tuned kernels for the models that run on the floating-point pipes:
//   Phi_FMA (Algorithm 4): d <- fma(a_k, b_k, d) in ascending k, FP32 or FP64, IEEE-754 round-to-nearest-even (FP64: on
//   the FP64 matrix instruction, see fma64_mma_kernel)
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

enum FpMode : int { FP_FMA32 = 0, FP_FTZ_F16 = 2, FP_FTZ_BF16 = 3 };

template <int MODE> struct ModeTraits;
template <> struct ModeTraits<FP_FMA32> { using acc_t = float; using in_t = float; static constexpr int TM = 8, TN = 8, IN_BYTES = 4; };
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
                else v = in_t(load_flushed((wv[q / 2] >> (16 * (q % 2))) & 0xFFFFu, MODE == FP_FTZ_BF16));
                if (is_a) As[h * EPT + q][r] = v; else Bs[h * EPT + q][r] = v;
            }
        }
        __syncthreads();
        if (k0 + KC < g.K) fetch(k0 + KC);

        if (!FTZ) {
            // fully unrolled: with a partial unroll the compiler rotates the accumulators through register moves
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
            uint32_t w = __float_as_uint(v);
            if (v != v) w = 0x7FC00000u;
            static_cast<uint32_t*>(g.D)[i * g.ldd + j] = w;
        }
}

// ---- Phi_FMA in FP64 on the FP64 matrix instruction ----
// `mma.sync.m8n8k4.f64` is, per output, the chain d <- fma(a_k, b_k, d) over its four k in ascending order, each step
// rounded to nearest even: Phi_FMA itself (Algorithm 4; the B200's instruction agrees with the model bit for bit on every
// input class of Section 3.2).  A warp owns 32 x 32 outputs (sixteen accumulator tiles), eight warps a 128 x 64 tile; the
// raw doubles of A and B reach shared memory by 16-byte asynchronous copies, three chunks of 16 k in flight, rows with
// a pitch of 20 doubles so that the fragment loads (lane (g, t) reads element (row 8 i + g, k 4 s + t)) are conflict-free.
namespace dm {
constexpr int BM = 128, BN = 64, DKC = 16, KP = DKC + 4, DNT = 256, STAGES = 3;
struct Stage {
    double a[BM][KP];
    double b[BN][KP];
};
}  // namespace dm

__global__ void __launch_bounds__(dm::DNT, 2) fma64_mma_kernel(GemmArgs g) {
    using namespace dm;
    extern __shared__ __align__(16) unsigned char dm_smem[];
    Stage* stages = reinterpret_cast<Stage*>(dm_smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int wr = warp >> 1, wc = warp & 1, gq = lane >> 2, tq = lane & 3;
    const int64_t row0 = int64_t(blockIdx.y) * BM, col0 = int64_t(blockIdx.x) * BN;
    const int NCH = int(g.K / DKC);

    double acc[4][4][2];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int64_t r = row0 + wr * 32 + 8 * i + gq, c = col0 + wc * 32 + 8 * j + 2 * tq + e;
                acc[i][j][e] = (g.C && r < g.M && c < g.N) ? static_cast<const double*>(g.C)[r * g.ldc + c] : 0.0;
            }

    // one chunk: 192 rows x 8 segments of 16 bytes, consecutive threads on consecutive segments of a row; rows beyond the
    // matrix are filled with zeros (a copy of size 0)
    auto issue = [&](int n) {
        Stage& s = stages[n % STAGES];
#pragma unroll
        for (int it = 0; it < (BM + BN) * 8 / DNT; ++it) {
            const int task = it * DNT + tid;
            const bool is_a = task < BM * 8;
            const int u = is_a ? task : task - BM * 8;
            const int r = u >> 3, seg = u & 7;
            const int64_t grow = (is_a ? row0 : col0) + r;
            const bool valid = grow < (is_a ? g.M : g.N);
            const double* base = static_cast<const double*>(is_a ? g.A : g.B);
            const double* src = valid ? base + grow * (is_a ? g.lda : g.ldb) + int64_t(n) * DKC + 2 * seg : base;
            const uint32_t dst = uint32_t(__cvta_generic_to_shared(is_a ? &s.a[r][2 * seg] : &s.b[r][2 * seg]));
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(valid ? 16 : 0) : "memory");
        }
    };
    issue(0);
    asm volatile("cp.async.commit_group;" ::: "memory");
    if (NCH > 1) issue(1);
    asm volatile("cp.async.commit_group;" ::: "memory");

    for (int n = 0; n < NCH; ++n) {
        asm volatile("cp.async.wait_group 1;" ::: "memory");    // chunk n has landed (n + 1 may still be in flight)
        __syncthreads();                                        // ... for every thread, and everybody has left chunk n - 1
        if (n + 2 < NCH) issue(n + 2);                          // into the buffer of chunk n - 1
        asm volatile("cp.async.commit_group;" ::: "memory");
        const Stage& s = stages[n % STAGES];
#pragma unroll
        for (int ks = 0; ks < DKC / 4; ++ks) {
            double af[4], bf[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) af[i] = s.a[wr * 32 + 8 * i + gq][4 * ks + tq];
#pragma unroll
            for (int j = 0; j < 4; ++j) bf[j] = s.b[wc * 32 + 8 * j + gq][4 * ks + tq];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    asm volatile("mma.sync.aligned.m8n8k4.row.col.rn.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                                 : "+d"(acc[i][j][0]), "+d"(acc[i][j][1]) : "d"(af[i]), "d"(bf[j]));
        }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");

#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int64_t r = row0 + wr * 32 + 8 * i + gq, c = col0 + wc * 32 + 8 * j + 2 * tq + e;
                if (r >= g.M || c >= g.N) continue;
                const double v = acc[i][j][e];
                unsigned long long w = (unsigned long long)__double_as_longlong(v);
                if (v != v) w = 0x7FF8000000000000ull;
                static_cast<unsigned long long*>(g.D)[r * g.ldd + c] = w;
            }
}

cudaError_t launch_fma64_mma(const GemmArgs& g, cudaStream_t stream) {
    using namespace dm;
    constexpr size_t sh = sizeof(Stage) * STAGES;
    cudaError_t err = cudaFuncSetAttribute(fma64_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(sh));
    if (err != cudaSuccess) return err;
    dim3 grid((unsigned)((g.N + BN - 1) / BN), (unsigned)((g.M + BM - 1) / BM), 1);
    fma64_mma_kernel<<<grid, DNT, sh, stream>>>(g);
    return cudaGetLastError();
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
        err = m.acc == ACC_F64 ? launch_fma64_mma(g, stream) : launch_fp<FP_FMA32, 2>(g, stream);
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
