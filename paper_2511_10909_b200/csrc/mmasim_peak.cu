// Issue-rate micro-benchmarks: the denominators of the integer roofline.  Every thread runs eight chains whose
// operations depend only on earlier operations of the chains, so the instruction mix is exactly what the source
// says; the host divides the operation count by the measured time.
#include "mmasim_internal.h"

namespace mmasim {
namespace {

enum PeakKind : int {
    PK_IADD3 = 0, PK_LOP3, PK_SHF, PK_IMAD, PK_MACMIX, PK_VIADDMAX, PK_VIADDMAX16X2, PK_F2I, PK_FMUL, PK_POPC,
    PK_IMAD_PLUS_ALU, PK_FMUL_PLUS_ALU, PK_IMAD_WIDE, PK_MAC_D1, PK_MAC_D2, PK_DP4A, PK_DFMA, PK_DFMA_PLUS_ALU, PK_FFMA_RM, PK_FFMA2_RM,
    PK_FFMA_RN_X16, PK_FFMA_RN_X32, PK_FFMA_RM_X16, PK_FFMA2_RM_X16, PK_DFMA_RN_X16, PK_DFMA_RN_X32, PK_DFMA_RM_X16, PK_DMMA_RM_K4, PK_DMMA_RM_K16, PK_CVT_F32_F64, PK_CVT_S32_F64, PK_DADD_RM_X16, PK_FFMA2_PLUS_ALU, PK_COUNT
};

template <int KIND>
__device__ __forceinline__ void round8(int (&x)[8], float (&f)[8]) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int j = (i + 1) & 7, k = (i + 3) & 7;
        if (KIND == PK_IADD3) x[i] = x[i] + x[j] + x[k];
        else if (KIND == PK_LOP3) x[i] = (x[i] & x[j]) ^ x[k];
        else if (KIND == PK_SHF) x[i] = __funnelshift_rc(x[i], x[j], x[k]);
        else if (KIND == PK_IMAD) x[i] = x[i] * x[j] + x[k];
        else if (KIND == PK_MACMIX) {           // exponent add, running max, distance, shift, accumulate
            const int e = x[j] + x[k];
            const int m = max(x[i], e);
            x[i] = x[i] + (int)((unsigned)x[j] >> ((m - e) & 31));
        } else if (KIND == PK_VIADDMAX) x[i] = __viaddmax_s32(x[j], x[k], x[i]);
        else if (KIND == PK_VIADDMAX16X2) x[i] = (int)__viaddmax_s16x2((unsigned)x[j], (unsigned)x[k], (unsigned)x[i]);
        else if (KIND == PK_F2I) x[i] = __float2int_rz(__int_as_float(x[i]));
        else if (KIND == PK_FMUL) f[i] = f[i] * f[j];
        else if (KIND == PK_POPC) x[i] = __popc(x[i]) + x[j];
        else if (KIND == PK_IMAD_PLUS_ALU) { x[i] = x[i] * x[j] + x[k]; x[j] = x[j] + x[k] + x[i]; }
        else if (KIND == PK_FMUL_PLUS_ALU) { f[i] = f[i] * f[j]; x[i] = x[i] + x[j] + x[k]; }
        else if (KIND == PK_IMAD_WIDE) {            // 32 x 32 -> 64-bit multiply, both halves consumed
            const long long w = (long long)x[j] * (long long)x[k];
            x[i] ^= int(w) ^ int(w >> 32);
        } else if (KIND == PK_MAC_D1) {             // one emulated term: multiply, distance, shift, accumulate-by-multiply
            const int X = x[j] * x[k];
            const int d = x[i] - x[j] - x[k];
            int t;
            asm("shr.s32 %0, %1, %2;" : "=r"(t) : "r"(X), "r"(d));
            asm("mad.lo.s32 %0, %1, %2, %0;" : "+r"(x[i]) : "r"(t), "r"(x[(i + 5) & 7]));
        } else if (KIND == PK_DP4A) {
            x[i] = __dp4a(x[j], x[k], x[i]);
        } else if (KIND == PK_MAC_D2) {             // one emulated term with pre-shifted operands: wide multiply, funnel shift, accumulate
            const long long w = (long long)x[j] * (long long)x[k];
            const int t = __funnelshift_rc(int(w), int(w >> 32), x[(i + 2) & 7]);
            asm("mad.lo.s32 %0, %1, %2, %0;" : "+r"(x[i]) : "r"(t), "r"(x[(i + 5) & 7]));
        }
    }
}

template <int KIND>
__global__ void __launch_bounds__(256) peak_kernel(int64_t iters, int* sink) {
    int x[8];
    float f[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        x[i] = threadIdx.x * 2654435 + i * 40503 + blockIdx.x;
        f[i] = 1.0f + 1e-7f * float(threadIdx.x + i);
    }
    for (int64_t it = 0; it < iters; it += 8) {
#pragma unroll
        for (int u = 0; u < 8; ++u) round8<KIND>(x, f);
    }
    int r = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) r ^= x[i] ^ __float_as_int(f[i]);
    if (r == 0x12345678) *sink = r;             // practically never true: keeps the chains alive
}

// FP64 fused multiply-add chains (a kernel of its own so that the integer kernels keep their register allocation);
// WITH_ALU adds one independent fused add-max per multiply-add: if the two pipes ran side by side the launch would
// take as long as the slower of the two streams alone, and it takes about their sum instead.
template <bool WITH_ALU>
__global__ void __launch_bounds__(256) peak_kernel_f64(int64_t iters, int* sink) {
    double d[8];
    int x[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) { d[i] = 1.0 + 1e-9 * double(threadIdx.x + i); x[i] = threadIdx.x * 2654435 + i * 40503; }
    for (int64_t it = 0; it < iters; it += 8) {
#pragma unroll
        for (int u = 0; u < 8; ++u)
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                d[i] = fma(d[i], d[(i + 1) & 7], d[(i + 3) & 7]);
                if (WITH_ALU) x[i] = (int)__viaddmax_s16x2((unsigned)x[(i + 1) & 7], (unsigned)x[(i + 3) & 7], (unsigned)x[i]);
            }
    }
    double r = 0.0;
    int q = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) { r += d[i]; q ^= x[i]; }
    if (r == 0.12345 && q == 0x12345678) *sink = 1;
}

// FP32 fused multiply-add rounded toward minus infinity, the instruction of the FP32 summation kernels: scalar form,
// and the packed two-lane form of sm_100 (fma.rm.f32x2), eight independent accumulator chains (pairs) per thread.
template <bool PACKED>
__global__ void __launch_bounds__(256) peak_kernel_f32(int64_t iters, int* sink) {
    float a[8], b[8], c[16];
    unsigned long long a2[8], b2[8], c2[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) { a[i] = 1.0f + 1e-7f * float(threadIdx.x + i); b[i] = 1.0f - 1e-7f * float(threadIdx.x + 2 * i); }
#pragma unroll
    for (int i = 0; i < 16; ++i) c[i] = float(i);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        asm("mov.b64 %0, {%1, %2};" : "=l"(a2[i]) : "f"(a[i]), "f"(a[(i + 1) & 7]));
        asm("mov.b64 %0, {%1, %2};" : "=l"(b2[i]) : "f"(b[i]), "f"(b[(i + 1) & 7]));
        asm("mov.b64 %0, {%1, %2};" : "=l"(c2[i]) : "f"(c[2 * i]), "f"(c[2 * i + 1]));
    }
    for (int64_t it = 0; it < iters; it += 8) {
#pragma unroll
        for (int u = 0; u < 8; ++u)
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (PACKED) asm volatile("fma.rm.f32x2 %0, %1, %2, %0;" : "+l"(c2[i]) : "l"(a2[i]), "l"(b2[u]));
                else c[i] = __fmaf_rd(a[i], b[u], c[i]);
            }
    }
    float r = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        float lo, hi;
        asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(c2[i]));
        r += PACKED ? lo + hi : c[i];
    }
    if (r == 0.12345f) *sink = 1;
}

// Second witness of the floating-point multiply-add rates: NACC independent accumulators per thread, the two
// multiplicands loop-invariant registers (c_i = x * y + c_i: two source registers besides the accumulator, so that no
// operand-fetch conflict hides the pipe's own rate), round-to-nearest or toward minus infinity, FP32 (scalar or the
// packed two-lane instruction) or FP64.  One round = NACC multiply-adds (2 NACC lanes for the packed form).
template <typename T, int NACC, bool RM, bool PACKED>
__global__ void __launch_bounds__(256) peak_kernel_fma(int64_t iters, int* sink) {
    T x[2], c[NACC];
    unsigned long long x2[2], c2[NACC];
    x[0] = T(1) + T(1e-7) * T(threadIdx.x);
    x[1] = T(1) - T(1e-7) * T(threadIdx.x + 3);
#pragma unroll
    for (int i = 0; i < NACC; ++i) c[i] = T(i);
    if (PACKED) {
#pragma unroll
        for (int i = 0; i < 2; ++i) asm("mov.b64 %0, {%1, %1};" : "=l"(x2[i]) : "f"(float(x[i])));
#pragma unroll
        for (int i = 0; i < NACC; ++i) asm("mov.b64 %0, {%1, %2};" : "=l"(c2[i]) : "f"(float(i)), "f"(float(i) + 0.5f));
    }
    for (int64_t it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < NACC; ++i) {
            if (PACKED) asm volatile("fma.rm.f32x2 %0, %1, %2, %0;" : "+l"(c2[i]) : "l"(x2[0]), "l"(x2[1]));
            else if (sizeof(T) == 4) {
                if (RM) asm volatile("fma.rm.f32 %0, %1, %2, %0;" : "+f"(*reinterpret_cast<float*>(&c[i])) : "f"(float(x[0])), "f"(float(x[1])));
                else asm volatile("fma.rn.f32 %0, %1, %2, %0;" : "+f"(*reinterpret_cast<float*>(&c[i])) : "f"(float(x[0])), "f"(float(x[1])));
            } else {
                if (RM) asm volatile("fma.rm.f64 %0, %1, %2, %0;" : "+d"(*reinterpret_cast<double*>(&c[i])) : "d"(double(x[0])), "d"(double(x[1])));
                else asm volatile("fma.rn.f64 %0, %1, %2, %0;" : "+d"(*reinterpret_cast<double*>(&c[i])) : "d"(double(x[0])), "d"(double(x[1])));
            }
        }
    }
    T r = T(0);
#pragma unroll
    for (int i = 0; i < NACC; ++i) {
        if (PACKED) {
            float lo, hi;
            asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(c2[i]));
            r += T(lo + hi);
        } else r += c[i];
    }
    if (r == T(0.12345)) *sink = 1;
}

// The FP64 matrix instruction rounding toward minus infinity (mma.sync m8n8k4 with eight independent accumulator tiles per
// warp, m16n8k16 with four): per thread and round 8 x 8 = 64 and 4 x 64 = 256 multiply-adds.
template <bool K16>
__global__ void __launch_bounds__(256) peak_kernel_dmma(int64_t iters, int* sink) {
    double a[8], b[4], c[8][2];
#pragma unroll
    for (int i = 0; i < 8; ++i) { a[i] = 1.0 + 1e-9 * double(threadIdx.x + i); c[i][0] = double(i); c[i][1] = double(i) + 0.5; }
#pragma unroll
    for (int i = 0; i < 4; ++i) b[i] = 1.0 - 1e-9 * double(threadIdx.x + 2 * i);
    for (int64_t it = 0; it < iters; ++it) {
        if (K16) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
                asm volatile("mma.sync.aligned.m16n8k16.row.col.rm.f64.f64.f64.f64 {%0,%1,%2,%3}, {%4,%5,%6,%7,%8,%9,%10,%11}, {%12,%13,%14,%15}, {%0,%1,%2,%3};"
                             : "+d"(c[2 * i][0]), "+d"(c[2 * i][1]), "+d"(c[2 * i + 1][0]), "+d"(c[2 * i + 1][1])
                             : "d"(a[0]), "d"(a[1]), "d"(a[2]), "d"(a[3]), "d"(a[4]), "d"(a[5]), "d"(a[6]), "d"(a[7]),
                               "d"(b[0]), "d"(b[1]), "d"(b[2]), "d"(b[3]));
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i)
                asm volatile("mma.sync.aligned.m8n8k4.row.col.rm.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                             : "+d"(c[i][0]), "+d"(c[i][1]) : "d"(a[i & 1]), "d"(b[i & 3]));
        }
    }
    double r = 0.0;
#pragma unroll
    for (int i = 0; i < 8; ++i) r += c[i][0] + c[i][1];
    if (r == 0.12345) *sink = 1;
}

// Conversions and additions around the FP64 pipe, sixteen independent chains per thread: MODE 0: FP32 -> FP64 -> FP32
// (cvt.f64.f32, cvt.rn.f32.f64), MODE 1: s32 -> FP64 -> s32 (cvt.rn.f64.s32, cvt.rzi.s32.f64), MODE 2: add.rm.f64.
// One round = 16 chains x (2 conversions | 1 addition).
template <int MODE>
__global__ void __launch_bounds__(256) peak_kernel_cvt(int64_t iters, int* sink) {
    float f[16]; int x[16]; double d[16];
    const double inc = 1.0 + 1e-9 * double(threadIdx.x);
#pragma unroll
    for (int i = 0; i < 16; ++i) { f[i] = 1.0f + float(i + threadIdx.x); x[i] = i + int(threadIdx.x); d[i] = double(i); }
    for (int64_t it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            if (MODE == 0) { double t; asm volatile("cvt.f64.f32 %0, %1;" : "=d"(t) : "f"(f[i])); asm volatile("cvt.rn.f32.f64 %0, %1;" : "=f"(f[i]) : "d"(t)); }
            else if (MODE == 1) { double t; asm volatile("cvt.rn.f64.s32 %0, %1;" : "=d"(t) : "r"(x[i])); asm volatile("cvt.rzi.s32.f64 %0, %1;" : "=r"(x[i]) : "d"(t)); }
            else asm volatile("add.rm.f64 %0, %0, %1;" : "+d"(d[i]) : "d"(inc));
        }
    }
    double r = 0.0;
#pragma unroll
    for (int i = 0; i < 16; ++i) r += double(f[i]) + double(x[i]) + d[i];
    if (r == 0.12345) *sink = 1;
}

// Sixteen packed FP32 multiply-adds (fma.rm.f32x2, loop-invariant multiplicands) and sixteen independent 3-input integer
// additions per round, interleaved: do the two pipes issue side by side?  Counted: the 32 multiply-add lanes per round.
__global__ void __launch_bounds__(256) peak_kernel_ffma2_alu(int64_t iters, int* sink) {
    unsigned long long x2[2], c2[16];
    int y[16];
    const float xa = 1.0f + 1e-7f * float(threadIdx.x), xb = 1.0f - 1e-7f * float(threadIdx.x + 3);
    asm("mov.b64 %0, {%1, %1};" : "=l"(x2[0]) : "f"(xa));
    asm("mov.b64 %0, {%1, %1};" : "=l"(x2[1]) : "f"(xb));
#pragma unroll
    for (int i = 0; i < 16; ++i) { asm("mov.b64 %0, {%1, %2};" : "=l"(c2[i]) : "f"(float(i)), "f"(float(i) + 0.5f)); y[i] = int(threadIdx.x) + i; }
    for (int64_t it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            asm volatile("fma.rm.f32x2 %0, %1, %2, %0;" : "+l"(c2[i]) : "l"(x2[0]), "l"(x2[1]));
            asm volatile("add.s32 %0, %0, %1;" : "+r"(y[i]) : "r"(y[(i + 5) & 15]));
        }
    }
    float r = 0.f;
    int z = 0;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        float lo, hi;
        asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(c2[i]));
        r += lo + hi; z += y[i];
    }
    if (r == 0.12345f || z == 0x12345678) *sink = 1;
}

template <int MODE>
int launch_cvt(int64_t blocks, int64_t iters, void* sink, int32_t* ops_per_round, cudaStream_t stream) {
    *ops_per_round = MODE == 2 ? 16 : 32;
    peak_kernel_cvt<MODE><<<(unsigned)blocks, 256, 0, stream>>>(iters * 8, static_cast<int*>(sink));
    const cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) { set_error("int_peak launch failed: %s", cudaGetErrorString(err)); return MMASIM_ERR_CUDA; }
    return MMASIM_OK;
}

template <bool K16>
int launch_dmma(int64_t blocks, int64_t iters, void* sink, int32_t* ops_per_round, cudaStream_t stream) {
    *ops_per_round = K16 ? 256 : 64;
    peak_kernel_dmma<K16><<<(unsigned)blocks, 256, 0, stream>>>(iters * 8, static_cast<int*>(sink));
    const cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) { set_error("int_peak launch failed: %s", cudaGetErrorString(err)); return MMASIM_ERR_CUDA; }
    return MMASIM_OK;
}

template <typename T, int NACC, bool RM, bool PACKED>
int launch_fma(int64_t blocks, int64_t iters, void* sink, int32_t* ops_per_round, cudaStream_t stream) {
    // the host counts blocks * 256 * iters8 * 8 * ops_per_round operations, iters8 = iters rounded up to a multiple of 8:
    // run iters8 * 8 rounds of NACC multiply-adds and report NACC (lanes: twice that for the packed form) per round
    *ops_per_round = NACC * (PACKED ? 2 : 1);
    peak_kernel_fma<T, NACC, RM, PACKED><<<(unsigned)blocks, 256, 0, stream>>>(iters * 8, static_cast<int*>(sink));
    const cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) { set_error("int_peak launch failed: %s", cudaGetErrorString(err)); return MMASIM_ERR_CUDA; }
    return MMASIM_OK;
}

template <int KIND>
int launch(int64_t blocks, int64_t iters, void* sink, cudaStream_t stream) {
    peak_kernel<KIND><<<(unsigned)blocks, 256, 0, stream>>>(iters, static_cast<int*>(sink));
    const cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) { set_error("int_peak launch failed: %s", cudaGetErrorString(err)); return MMASIM_ERR_CUDA; }
    return MMASIM_OK;
}

}  // namespace

int launch_int_peak(int kind, int64_t blocks, int64_t iters, void* sink, int32_t* ops_per_round, cudaStream_t stream) {
    iters = (iters + 7) / 8 * 8;
    switch (kind) {
        case PK_IADD3: *ops_per_round = 1; return launch<PK_IADD3>(blocks, iters, sink, stream);
        case PK_LOP3: *ops_per_round = 1; return launch<PK_LOP3>(blocks, iters, sink, stream);
        case PK_SHF: *ops_per_round = 1; return launch<PK_SHF>(blocks, iters, sink, stream);
        case PK_IMAD: *ops_per_round = 1; return launch<PK_IMAD>(blocks, iters, sink, stream);
        case PK_MACMIX: *ops_per_round = 5; return launch<PK_MACMIX>(blocks, iters, sink, stream);
        case PK_VIADDMAX: *ops_per_round = 1; return launch<PK_VIADDMAX>(blocks, iters, sink, stream);
        case PK_VIADDMAX16X2: *ops_per_round = 1; return launch<PK_VIADDMAX16X2>(blocks, iters, sink, stream);
        case PK_F2I: *ops_per_round = 1; return launch<PK_F2I>(blocks, iters, sink, stream);
        case PK_FMUL: *ops_per_round = 1; return launch<PK_FMUL>(blocks, iters, sink, stream);
        case PK_POPC: *ops_per_round = 2; return launch<PK_POPC>(blocks, iters, sink, stream);
        case PK_IMAD_PLUS_ALU: *ops_per_round = 2; return launch<PK_IMAD_PLUS_ALU>(blocks, iters, sink, stream);
        case PK_FMUL_PLUS_ALU: *ops_per_round = 2; return launch<PK_FMUL_PLUS_ALU>(blocks, iters, sink, stream);
        case PK_IMAD_WIDE: *ops_per_round = 1; return launch<PK_IMAD_WIDE>(blocks, iters, sink, stream);
        case PK_MAC_D1: *ops_per_round = 1; return launch<PK_MAC_D1>(blocks, iters, sink, stream);
        case PK_MAC_D2: *ops_per_round = 1; return launch<PK_MAC_D2>(blocks, iters, sink, stream);
        case PK_DP4A: *ops_per_round = 1; return launch<PK_DP4A>(blocks, iters, sink, stream);
        case PK_DFMA:
        case PK_DFMA_PLUS_ALU: {
            *ops_per_round = kind == PK_DFMA ? 1 : 2;
            if (kind == PK_DFMA) peak_kernel_f64<false><<<(unsigned)blocks, 256, 0, stream>>>(iters, static_cast<int*>(sink));
            else peak_kernel_f64<true><<<(unsigned)blocks, 256, 0, stream>>>(iters, static_cast<int*>(sink));
            const cudaError_t err = cudaGetLastError();
            if (err != cudaSuccess) { set_error("int_peak launch failed: %s", cudaGetErrorString(err)); return MMASIM_ERR_CUDA; }
            return MMASIM_OK;
        }
        case PK_FFMA_RM:
        case PK_FFMA2_RM: {
            *ops_per_round = kind == PK_FFMA_RM ? 1 : 2;
            if (kind == PK_FFMA_RM) peak_kernel_f32<false><<<(unsigned)blocks, 256, 0, stream>>>(iters, static_cast<int*>(sink));
            else peak_kernel_f32<true><<<(unsigned)blocks, 256, 0, stream>>>(iters, static_cast<int*>(sink));
            const cudaError_t err = cudaGetLastError();
            if (err != cudaSuccess) { set_error("int_peak launch failed: %s", cudaGetErrorString(err)); return MMASIM_ERR_CUDA; }
            return MMASIM_OK;
        }
        case PK_FFMA_RN_X16: return launch_fma<float, 16, false, false>(blocks, iters, sink, ops_per_round, stream);
        case PK_FFMA_RN_X32: return launch_fma<float, 32, false, false>(blocks, iters, sink, ops_per_round, stream);
        case PK_FFMA_RM_X16: return launch_fma<float, 16, true, false>(blocks, iters, sink, ops_per_round, stream);
        case PK_FFMA2_RM_X16: return launch_fma<float, 16, true, true>(blocks, iters, sink, ops_per_round, stream);
        case PK_DFMA_RN_X16: return launch_fma<double, 16, false, false>(blocks, iters, sink, ops_per_round, stream);
        case PK_DFMA_RN_X32: return launch_fma<double, 32, false, false>(blocks, iters, sink, ops_per_round, stream);
        case PK_DFMA_RM_X16: return launch_fma<double, 16, true, false>(blocks, iters, sink, ops_per_round, stream);
        case PK_DMMA_RM_K4: return launch_dmma<false>(blocks, iters, sink, ops_per_round, stream);
        case PK_DMMA_RM_K16: return launch_dmma<true>(blocks, iters, sink, ops_per_round, stream);
        case PK_CVT_F32_F64: return launch_cvt<0>(blocks, iters, sink, ops_per_round, stream);
        case PK_CVT_S32_F64: return launch_cvt<1>(blocks, iters, sink, ops_per_round, stream);
        case PK_DADD_RM_X16: return launch_cvt<2>(blocks, iters, sink, ops_per_round, stream);
        case PK_FFMA2_PLUS_ALU: {
            *ops_per_round = 32;
            peak_kernel_ffma2_alu<<<(unsigned)blocks, 256, 0, stream>>>(iters * 8, static_cast<int*>(sink));
            const cudaError_t err = cudaGetLastError();
            if (err != cudaSuccess) { set_error("int_peak launch failed: %s", cudaGetErrorString(err)); return MMASIM_ERR_CUDA; }
            return MMASIM_OK;
        }
        default: set_error("mmasim_int_peak: unknown kind %d", kind); return MMASIM_ERR_INVALID_ARG;
    }
}

}  // namespace mmasim
