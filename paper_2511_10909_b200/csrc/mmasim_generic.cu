// Generic kernels: any model of the registry, any shape.  One thread owns one output element (or one dot
// product in batch mode) and walks K block by block exactly as Algorithm 5 (or 2, or 4) prescribes; the CTA
// stages decoded A / B rows of the current K chunk in shared memory.  These kernels define the library's
// behaviour for every family; the tuned T-FDPA kernels must agree with them bit for bit.
#include <cuda_fp16.h>
#include "mmasim_device.cuh"

namespace mmasim {

namespace {

constexpr int GEN_THREADS = 256;
constexpr int GEMM_TILE = 16;          // 16 x 16 outputs per CTA in GEMM mode

__device__ __forceinline__ uint32_t load_raw(const void* base, int64_t idx, int storage_bits, bool packed4) {
    if (packed4) {
        const uint8_t byte = static_cast<const uint8_t*>(base)[idx >> 1];
        return (idx & 1) ? (byte >> 4) : (byte & 0xFu);
    }
    switch (storage_bits) {
        case 8: return static_cast<const uint8_t*>(base)[idx];
        case 16: return static_cast<const uint16_t*>(base)[idx];
        default: return static_cast<const uint32_t*>(base)[idx];
    }
}

// rows of the tile this thread works on, and where it stores
struct ThreadMap {
    int a_row, b_row;       // row inside the staged A / B tiles
    int64_t i, j;           // global output coordinates (dot mode: i = dot index, j = 0)
    bool valid;
};

__device__ __forceinline__ ThreadMap thread_map(const GemmArgs& g, int rows) {
    ThreadMap t;
    if (g.dot_mode) {
        t.a_row = t.b_row = threadIdx.x;
        t.i = int64_t(blockIdx.x) * rows + threadIdx.x;
        t.j = 0;
        t.valid = t.i < g.M;
    } else {
        t.a_row = threadIdx.x / GEMM_TILE;
        t.b_row = threadIdx.x % GEMM_TILE;
        t.i = int64_t(blockIdx.y) * GEMM_TILE + t.a_row;
        t.j = int64_t(blockIdx.x) * GEMM_TILE + t.b_row;
        t.valid = t.i < g.M && t.j < g.N;
    }
    return t;
}

__device__ __forceinline__ float canonical_nan_nv(float x) { return (x != x) ? __uint_as_float(0x7FFFFFFFu) : x; }

// ---------------------------------------------------------------------------------------------------------
// FDPA families (E, T, ST, GST, TR, GTR)
// ---------------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(GEN_THREADS)
fdpa_generic_kernel(DevModel m, GemmArgs g, int rows, int KC, int L) {
    extern __shared__ uint32_t smem[];
    const int stride = KC + 1;
    uint32_t* As = smem;
    uint32_t* Bs = As + rows * stride;
    const int nsf_chunk = m.k_block ? (KC + m.k_block - 1) / m.k_block : 0;
    uint32_t* SAs = Bs + rows * stride;
    uint32_t* SBs = SAs + rows * (nsf_chunk + 1);
    const int sstride = nsf_chunk + 1;

    const FmtDesc fa = fmt_desc(m.fmt_a), fb = fmt_desc(m.fmt_b);
    const FmtDesc fs = fmt_desc(m.scale_fmt);
    const ThreadMap t = thread_map(g, rows);
    const int64_t a_row0 = g.dot_mode ? int64_t(blockIdx.x) * rows : int64_t(blockIdx.y) * GEMM_TILE;
    const int64_t b_row0 = g.dot_mode ? a_row0 : int64_t(blockIdx.x) * GEMM_TILE;
    const int64_t a_rows_total = g.M, b_rows_total = g.dot_mode ? g.M : g.N;
    const bool fp16 = m.acc == ACC_F16;

    uint32_t acc = 0u;                 // model accumulator word
    if (t.valid && g.C) {
        const int64_t ci = t.i * g.ldc + t.j;
        acc = fp16 ? uint32_t(static_cast<const uint16_t*>(g.C)[ci]) : static_cast<const uint32_t*>(g.C)[ci];
    }
    float promoted = 0.0f;             // FP32 running sum of the promotion workaround
    if (g.k_chunk) { promoted = __uint_as_float(acc); acc = 0u; }

    for (int64_t k0 = 0; k0 < g.K; k0 += KC) {
        const int kc = int(g.K - k0 < KC ? g.K - k0 : KC);
        __syncthreads();
        for (int idx = threadIdx.x; idx < rows * kc; idx += GEN_THREADS) {
            const int r = idx / kc, kk = idx % kc;
            uint32_t da = 0u, db = 0u;
            if (a_row0 + r < a_rows_total)
                da = load_raw(g.A, (a_row0 + r) * g.lda + k0 + kk, fa.storage_bits, m.packed4);
            if (b_row0 + r < b_rows_total)
                db = load_raw(g.B, (b_row0 + r) * g.ldb + k0 + kk, fb.storage_bits, m.packed4);
            As[r * stride + kk] = decode_elem(fa, da);
            Bs[r * stride + kk] = decode_elem(fb, db);
        }
        if (m.k_block) {
            const int nsf = (kc + m.k_block - 1) / m.k_block;
            const int64_t s0 = k0 / m.k_block;
            for (int idx = threadIdx.x; idx < rows * nsf; idx += GEN_THREADS) {
                const int r = idx / nsf, s = idx % nsf;
                uint32_t wa = 0x7Fu, wb = 0x7Fu;
                if (a_row0 + r < a_rows_total) wa = g.sfa[(a_row0 + r) * g.ld_sfa + s0 + s];
                if (b_row0 + r < b_rows_total) wb = g.sfb[(b_row0 + r) * g.ld_sfb + s0 + s];
                SAs[r * sstride + s] = decode_elem(fs, wa);
                SBs[r * sstride + s] = decode_elem(fs, wb);
            }
        }
        __syncthreads();
        if (!t.valid) continue;
        const uint32_t* a = As + t.a_row * stride;
        const uint32_t* b = Bs + t.b_row * stride;
        for (int kb = 0; kb + L <= kc; kb += L) {
            switch (m.family) {
                case FAM_T:
                    acc = tfdpa_block(a + kb, b + kb, L, acc, m, 0, false);
                    break;
                case FAM_ST: {
                    const uint32_t sa = SAs[t.a_row * sstride + kb / m.k_block];
                    const uint32_t sb = SBs[t.b_row * sstride + kb / m.k_block];
                    const bool nan = dec_cls(sa) == CLS_NAN || dec_cls(sb) == CLS_NAN;
                    acc = tfdpa_block(a + kb, b + kb, L, acc, m, dec_exp(sa) + dec_exp(sb), nan);
                    break;
                }
                case FAM_GST:
                    acc = gst_block(a + kb, b + kb, L, acc, m, SAs + t.a_row * sstride + kb / m.k_block,
                                    SBs + t.b_row * sstride + kb / m.k_block);
                    break;
                case FAM_TR: acc = tr_block(a + kb, b + kb, L, acc, m, false); break;
                case FAM_GTR: acc = tr_block(a + kb, b + kb, L, acc, m, true); break;
                default: acc = efdpa_block(a + kb, b + kb, L, acc, m); break;   // FAM_E
            }
            if (g.k_chunk && ((k0 + kb + L) % g.k_chunk) == 0) {
                promoted = canonical_nan_nv(__fadd_rn(promoted, __uint_as_float(acc)));
                acc = 0u;
            }
        }
    }
    if (!t.valid) return;
    if (g.k_chunk) acc = __float_as_uint(promoted);
    if (g.row_scale) {
        const float s = canonical_nan_nv(__fmul_rn(g.row_scale[t.i], g.col_scale[t.j]));
        acc = __float_as_uint(canonical_nan_nv(__fmul_rn(s, __uint_as_float(acc))));
    }
    const int64_t di = t.i * g.ldd + t.j;
    if (fp16) static_cast<uint16_t*>(g.D)[di] = uint16_t(acc);
    else static_cast<uint32_t*>(g.D)[di] = acc;
}

// ---------------------------------------------------------------------------------------------------------
// Phi_FTZ-AddMul (Algorithm 2) on the FP32 pipe
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ float ftz_load(uint32_t w, bool is_bf16) {
    // FlushSubnormal: a subnormal input becomes +0.0; everything else converts exactly to FP32
    if (is_bf16) {
        if ((w & 0x7F80u) == 0u && (w & 0x007Fu)) return 0.0f;
        return __uint_as_float(w << 16);
    }
    if ((w & 0x7C00u) == 0u && (w & 0x03FFu)) return 0.0f;
    return __half2float(__ushort_as_half((unsigned short)w));
}

__global__ void __launch_bounds__(GEN_THREADS)
ftz_generic_kernel(DevModel m, GemmArgs g, int rows, int KC) {
    extern __shared__ uint32_t smem[];
    const int stride = KC + 1;
    float* As = reinterpret_cast<float*>(smem);
    float* Bs = As + rows * stride;
    const ThreadMap t = thread_map(g, rows);
    const int64_t a_row0 = g.dot_mode ? int64_t(blockIdx.x) * rows : int64_t(blockIdx.y) * GEMM_TILE;
    const int64_t b_row0 = g.dot_mode ? a_row0 : int64_t(blockIdx.x) * GEMM_TILE;
    const int64_t b_rows_total = g.dot_mode ? g.M : g.N;
    const bool is_bf16 = m.fmt_a == EF_BF16;
    float d = 0.0f;
    if (t.valid && g.C) {
        const uint32_t w = static_cast<const uint32_t*>(g.C)[t.i * g.ldc + t.j];
        d = ((w & 0x7F800000u) == 0u && (w & 0x007FFFFFu)) ? 0.0f : __uint_as_float(w);
    }
    const int P = m.P;
    for (int64_t k0 = 0; k0 < g.K; k0 += KC) {
        const int kc = int(g.K - k0 < KC ? g.K - k0 : KC);
        __syncthreads();
        for (int idx = threadIdx.x; idx < rows * kc; idx += GEN_THREADS) {
            const int r = idx / kc, kk = idx % kc;
            uint32_t wa = 0u, wb = 0u;
            if (a_row0 + r < g.M) wa = static_cast<const uint16_t*>(g.A)[(a_row0 + r) * g.lda + k0 + kk];
            if (b_row0 + r < b_rows_total) wb = static_cast<const uint16_t*>(g.B)[(b_row0 + r) * g.ldb + k0 + kk];
            As[r * stride + kk] = ftz_load(wa, is_bf16);
            Bs[r * stride + kk] = ftz_load(wb, is_bf16);
        }
        __syncthreads();
        if (!t.valid) continue;
        const float* a = As + t.a_row * stride;
        const float* b = Bs + t.b_row * stride;
        for (int k = 0; k + P <= kc; k += P) {
            float s = ftz_add(ftz_mul(a[k], b[k]), ftz_mul(a[k + 1], b[k + 1]));
            if (P == 4) s = ftz_add(s, ftz_add(ftz_mul(a[k + 2], b[k + 2]), ftz_mul(a[k + 3], b[k + 3])));
            d = ftz_add(d, s);
        }
    }
    if (!t.valid) return;
    uint32_t w = __float_as_uint(d);
    if (d != d) w = 0x7FC00000u;
    static_cast<uint32_t*>(g.D)[t.i * g.ldd + t.j] = w;
}

// ---------------------------------------------------------------------------------------------------------
// Phi_FMA (Algorithm 4): a chain of IEEE-754 fused multiply-adds in ascending k
// ---------------------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(GEN_THREADS)
fma_generic_kernel(GemmArgs g, int rows, int KC) {
    extern __shared__ uint32_t smem[];
    const int stride = KC + 1;
    T* As = reinterpret_cast<T*>(smem);
    T* Bs = As + rows * stride;
    const ThreadMap t = thread_map(g, rows);
    const int64_t a_row0 = g.dot_mode ? int64_t(blockIdx.x) * rows : int64_t(blockIdx.y) * GEMM_TILE;
    const int64_t b_row0 = g.dot_mode ? a_row0 : int64_t(blockIdx.x) * GEMM_TILE;
    const int64_t b_rows_total = g.dot_mode ? g.M : g.N;
    T d = T(0);
    if (t.valid && g.C) d = static_cast<const T*>(g.C)[t.i * g.ldc + t.j];
    for (int64_t k0 = 0; k0 < g.K; k0 += KC) {
        const int kc = int(g.K - k0 < KC ? g.K - k0 : KC);
        __syncthreads();
        for (int idx = threadIdx.x; idx < rows * kc; idx += GEN_THREADS) {
            const int r = idx / kc, kk = idx % kc;
            As[r * stride + kk] = (a_row0 + r < g.M) ? static_cast<const T*>(g.A)[(a_row0 + r) * g.lda + k0 + kk] : T(0);
            Bs[r * stride + kk] = (b_row0 + r < b_rows_total) ? static_cast<const T*>(g.B)[(b_row0 + r) * g.ldb + k0 + kk] : T(0);
        }
        __syncthreads();
        if (!t.valid) continue;
        const T* a = As + t.a_row * stride;
        const T* b = Bs + t.b_row * stride;
        for (int k = 0; k < kc; ++k) d = fma(a[k], b[k], d);          // fma() on float is fmaf: one rounding
    }
    if (!t.valid) return;
    if (sizeof(T) == 4) {
        uint32_t w = __float_as_uint(float(d));
        if (d != d) w = 0x7FC00000u;
        static_cast<uint32_t*>(g.D)[t.i * g.ldd + t.j] = w;
    } else {
        unsigned long long w = (unsigned long long)__double_as_longlong(double(d));
        if (d != d) w = 0x7FF8000000000000ull;
        static_cast<unsigned long long*>(g.D)[t.i * g.ldd + t.j] = w;
    }
}

}  // namespace

int launch_generic(const DevModel& m, const GemmArgs& g, cudaStream_t stream) {
    const int rows = g.dot_mode ? GEN_THREADS : GEMM_TILE;
    dim3 grid;
    if (g.dot_mode) grid = dim3((unsigned)((g.M + rows - 1) / rows), 1, 1);
    else grid = dim3((unsigned)((g.N + GEMM_TILE - 1) / GEMM_TILE), (unsigned)((g.M + GEMM_TILE - 1) / GEMM_TILE), 1);
    const int kmax = g.dot_mode ? 32 : 128;          // elements of K staged per chunk
    cudaError_t err = cudaSuccess;
    if (m.family == FAM_FMA) {
        const int KC = int(g.K < kmax ? g.K : kmax);
        if (m.acc == ACC_F64) {
            const size_t sh = size_t(2) * rows * (KC + 1) * sizeof(double);
            err = cudaFuncSetAttribute(fma_generic_kernel<double>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
            if (err == cudaSuccess) fma_generic_kernel<double><<<grid, GEN_THREADS, sh, stream>>>(g, rows, KC);
        } else {
            const size_t sh = size_t(2) * rows * (KC + 1) * sizeof(float);
            err = cudaFuncSetAttribute(fma_generic_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
            if (err == cudaSuccess) fma_generic_kernel<float><<<grid, GEN_THREADS, sh, stream>>>(g, rows, KC);
        }
    } else if (m.family == FAM_FTZ) {
        int KC = int(g.K < kmax ? g.K : kmax);
        KC -= KC % m.P;
        const size_t sh = size_t(2) * rows * (KC + 1) * sizeof(float);
        err = cudaFuncSetAttribute(ftz_generic_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
        if (err == cudaSuccess) ftz_generic_kernel<<<grid, GEN_THREADS, sh, stream>>>(m, g, rows, KC);
    } else {
        const int L = int(g.K < m.L ? g.K : m.L);
        int KC = L * (kmax / L > 0 ? kmax / L : 1);
        if (KC > g.K) KC = int(g.K);
        const int nsf_chunk = m.k_block ? (KC + m.k_block - 1) / m.k_block : 0;
        const size_t sh = (size_t(2) * rows * (KC + 1) + size_t(2) * rows * (nsf_chunk + 1)) * sizeof(uint32_t);
        err = cudaFuncSetAttribute(fdpa_generic_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (err == cudaSuccess) fdpa_generic_kernel<<<grid, GEN_THREADS, sh, stream>>>(m, g, rows, KC, L);
    }
    if (err == cudaSuccess) err = cudaGetLastError();
    if (err != cudaSuccess) {
        set_error("generic kernel launch failed: %s", cudaGetErrorString(err));
        return MMASIM_ERR_CUDA;
    }
    return MMASIM_OK;
}

}  // namespace mmasim
