// Streaming kernels for mmasim_dot_batch: n independent dot-product-accumulates d_t = Phi(a_t, b_t, c_t) (Equation 4),
// the shape of the paper's probe vectors (Section 3.1).  One thread owns one dot product; nothing is shared between
// dots, so the kernels are bound by HBM traffic (2 * K * element bytes + 8 bytes per dot).
//   T-FDPA (Algorithm 7) for FP16 / BF16 / TF32 inputs, L in {4, 8, 16}, F in 23..25, rho in {RZ-FP32, RNE-FP16}
//   Phi_FTZ-AddMul (Algorithm 2) for FP16 / BF16 inputs, P in {2, 4}
// Two ways to bring the rows in:
//   staged - rows of 8, 16, 32, 64 or 128 bytes: the CTA's 128 rows of A and of B are one contiguous range each, copied
//            to shared memory with 16-byte asynchronous copies (consecutive threads, consecutive chunks: every
//            sector of a request is used), chunks XOR-swizzled so that each thread then reads its own row without bank
//            conflicts; several CTAs per SM keep the copies of one tile under the arithmetic of another
//   direct - any other row length: each thread reads its row with 16-byte loads
// Everything else (8-bit inputs, other families, odd shapes) uses the generic kernels.
#include <cuda_fp16.h>
#include "mmasim_tfdpa_fast.cuh"

namespace mmasim {
namespace {

using fast::Elem;
using fast::EK_F16;
using fast::EK_BF16;
using fast::EK_TF32;

constexpr int DOT_THREADS = 128;

// ---- where a thread finds its two rows ----
struct GlobalRows {                      // row pointers into global memory
    const unsigned char* a;
    const unsigned char* b;
    __device__ __forceinline__ uint4 ld16(bool second, int byte_off) const {
        return *reinterpret_cast<const uint4*>((second ? b : a) + byte_off);
    }
    __device__ __forceinline__ uint2 ld8(bool second, int byte_off) const {
        return *reinterpret_cast<const uint2*>((second ? b : a) + byte_off);
    }
};
struct StagedRows {                      // this thread's rows inside the staged tile (shared memory, swizzled chunks)
    const unsigned char* a;              // start of the row's chunk group
    const unsigned char* b;
    int swz;                             // XOR applied to the chunk index inside the row
    __device__ __forceinline__ uint4 ld16(bool second, int byte_off) const {
        return *reinterpret_cast<const uint4*>((second ? b : a) + (((byte_off >> 4) ^ swz) << 4));
    }
    __device__ __forceinline__ uint2 ld8(bool second, int byte_off) const {
        return *reinterpret_cast<const uint2*>((second ? b : a) + (((byte_off >> 4) ^ swz) << 4) + (byte_off & 8));
    }
};

// L consecutive elements (L * BYTES is 8, 16, 32 or 64 bytes) as raw 32-bit words (two elements per word for the
// 16-bit formats).
template <int BYTES, int L, class Rows>
__device__ __forceinline__ void load_raw(const Rows& rows, bool second, int elem_index, uint32_t (&raw)[L * BYTES / 4]) {
    if (L * BYTES == 8) {
        const uint2 v = rows.ld8(second, elem_index * BYTES);
        raw[0] = v.x; raw[1] = v.y;
    } else {
#pragma unroll
        for (int q = 0; q < L * BYTES / 16; ++q) {
            const uint4 v = rows.ld16(second, elem_index * BYTES + 16 * q);
            raw[4 * q] = v.x; raw[4 * q + 1] = v.y; raw[4 * q + 2] = v.z; raw[4 * q + 3] = v.w;
        }
    }
}

// Start the copy of one tile's rows of A and B (rows t0 .. t0 + nrows - 1, `row_bytes` each) into one stage of shared
// memory.  Chunk c of row r lands at chunk position c ^ ((r / rows_per_line) % chunks_per_row) of that row,
// rows_per_line = 128 bytes / row_bytes: the eight threads of a quarter warp then read eight different 16-byte
// bank groups.  The caller commits the group and waits for it.
__device__ __forceinline__ void stage_issue(unsigned char* stage, const void* A, const void* B, int64_t t0, int nrows,
                                            int row_bytes) {
    const int tid = threadIdx.x;
    const int lcpr = row_bytes >= 16 ? 31 - __clz(row_bytes >> 4) : 0;      // log2(chunks per row); rows of 8 bytes: two rows per chunk
    const int cmask = (1 << lcpr) - 1;
    const int lrpl = 3 - lcpr;                                              // log2(rows per 128-byte line)
    const int bytes = nrows * row_bytes;
    unsigned char* sa = stage;
    unsigned char* sb = stage + DOT_THREADS * row_bytes;
    const unsigned char* ga = static_cast<const unsigned char*>(A) + t0 * row_bytes;
    const unsigned char* gb = static_cast<const unsigned char*>(B) + t0 * row_bytes;
    for (int g = tid; g < (bytes >> 4); g += DOT_THREADS) {
        int dst = g;
        if (row_bytes >= 16) {
            const int r = g >> lcpr, c = g & cmask;
            dst = (r << lcpr) + (c ^ ((r >> lrpl) & cmask));
        }
        const unsigned da = unsigned(__cvta_generic_to_shared(sa + (dst << 4)));
        const unsigned db = unsigned(__cvta_generic_to_shared(sb + (dst << 4)));
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(da), "l"(ga + (int64_t(g) << 4)) : "memory");
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(db), "l"(gb + (int64_t(g) << 4)) : "memory");
    }
    if ((bytes & 8) && tid == 0) {                                          // 8-byte rows, odd row count: the last row
        *reinterpret_cast<uint2*>(sa + bytes - 8) = *reinterpret_cast<const uint2*>(ga + bytes - 8);
        *reinterpret_cast<uint2*>(sb + bytes - 8) = *reinterpret_cast<const uint2*>(gb + bytes - 8);
    }
}

// This thread's rows inside a stage.
__device__ __forceinline__ StagedRows staged_view(const unsigned char* stage, int row_bytes) {
    const int tid = threadIdx.x;
    const int lcpr = row_bytes >= 16 ? 31 - __clz(row_bytes >> 4) : 0;
    StagedRows rows;
    rows.a = stage + tid * row_bytes;
    rows.b = stage + (DOT_THREADS + tid) * row_bytes;
    rows.swz = (tid >> (3 - lcpr)) & ((1 << lcpr) - 1);
    return rows;
}

// One tile per CTA: copy, wait, compute.  With 32 KB per tile about six CTAs share an SM, and the copies of some run
// under the arithmetic of the others.  (A persistent variant with two stages per CTA was slower: the stages cost
// half of the resident warps.)  `body(rows, t, c)` returns the result word of dot t.
template <bool ACC16, class Body>
__device__ __forceinline__ void staged_tile(unsigned char* smem, int64_t n, int row_bytes, const void* A, const void* B,
                                            const void* C, void* D, Body body) {
    const int64_t t0 = int64_t(blockIdx.x) * DOT_THREADS, t = t0 + threadIdx.x;
    stage_issue(smem, A, B, t0, int(min(int64_t(DOT_THREADS), n - t0)), row_bytes);
    asm volatile("cp.async.commit_group;" ::: "memory");
    uint32_t c = 0u;
    if (C && t < n) c = ACC16 ? uint32_t(static_cast<const uint16_t*>(C)[t]) : static_cast<const uint32_t*>(C)[t];
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    if (t >= n) return;
    const uint32_t w = body(staged_view(smem, row_bytes), t, c);
    if (ACC16) static_cast<uint16_t*>(D)[t] = uint16_t(w);
    else static_cast<uint32_t*>(D)[t] = w;
}

// trunc(p * scale) with the sign of p (RZ_F of Algorithm 7 is sign-magnitude), for |p * scale| < 2^51: the magnitude
// is floored by one fused multiply-add rounding toward minus infinity onto 2^52 (one ulp = 1), the sign is copied
// back on the high word.  (Choosing the rounding direction by the sign instead costs more: the compiler turns the two
// predicated operations into two executed ones plus selects.)
__device__ __forceinline__ double trunc_scaled(double p, double scale, int sign_word) {
    const double n = __fma_rd(fabs(p), scale, 4503599627370496.0) - 4503599627370496.0;
    return __hiloint2double(__double2hiint(n) | (sign_word & int(0x80000000u)), __double2loint(n));
}

// T-FDPA (Algorithm 7) on the FP64 pipe, the chain of Algorithm 5 for one dot product.  A double holds every quantity
// of a block exactly: products of two 11-bit (8-bit) significands, their scaling by 2^(F - e_max) (a power of two, no
// underflow in the FP64 range), the truncated terms (< 2^27) and their sum (< 2^32).  Infinities and NaNs need no
// separate tracking: IEEE arithmetic on the products gives NaN for NaN inputs, inf * 0 and inf - inf, and the
// surviving infinity otherwise, which is the rule of Section 4.2; the block result is replaced by the canonical
// word when the sum is not finite.  Only e_max stays on the integer pipe (two terms per instruction, 16-bit lanes).
template <int EK, int L, int RHO, class Rows>
__device__ __forceinline__ uint32_t tfdpa_dot(const Rows& rows, int K, int F, uint32_t cw) {
    using E = Elem<EK>;
    constexpr bool ACC16 = RHO == RHO_RNE_FP16;
    constexpr int NRAW = L * E::BYTES / 4;
    for (int k0 = 0; k0 < K; k0 += L) {
        uint32_t ra[NRAW], rb[NRAW];
        load_raw<E::BYTES, L>(rows, false, k0, ra);
        load_raw<E::BYTES, L>(rows, true, k0, rb);
        // Step 1: exact products (as FP32 for FP16 inputs, whose products stay inside the FP32 range; as FP64
        // otherwise) and the largest exponent sum Exp(a) + Exp(b), with Exp = max(field, 1) - bias, over the products
        // that are not zero (a zero term has no exponent): lanes of a zero product are masked to 0 before the maximum.
        float pf[E::BYTES == 2 && EK == EK_F16 ? L : 1];
        double pd[EK == EK_F16 ? 1 : L];
        constexpr int NO_EXP = -100000;
        int e_prod;
        if (E::BYTES == 2) {
            constexpr uint32_t EXPM = ((1u << E::EBITS) - 1u) << E::MBITS, ONE = 1u << E::MBITS;
            uint32_t mx = 0u;
#pragma unroll
            for (int q = 0; q < NRAW; ++q) {
                const uint32_t ea = __vmaxu2(ra[q] & (EXPM * 0x10001u), ONE * 0x10001u);
                const uint32_t eb = __vmaxu2(rb[q] & (EXPM * 0x10001u), ONE * 0x10001u);
                // 1 per lane where both elements are nonzero, widened to a lane mask
                const uint32_t live = __vminu2(__vminu2(ra[q] & 0x7FFF7FFFu, rb[q] & 0x7FFF7FFFu), 0x00010001u) * 0xFFFFu;
                mx = __vmaxu2(mx, (ea + eb) & live);      // field sums stay below 2^16: no carry between the lanes
                if (EK == EK_F16) {
                    const float2 fa = __half22float2(*reinterpret_cast<const __half2*>(&ra[q]));
                    const float2 fb = __half22float2(*reinterpret_cast<const __half2*>(&rb[q]));
                    pf[2 * q < L ? 2 * q : 0] = __fmul_rn(fa.x, fb.x);
                    pf[2 * q + 1 < L ? 2 * q + 1 : 0] = __fmul_rn(fa.y, fb.y);
                } else {
                    pd[2 * q < L ? 2 * q : 0] = __dmul_rn(double(__uint_as_float(ra[q] << 16)), double(__uint_as_float(rb[q] << 16)));
                    pd[2 * q + 1 < L ? 2 * q + 1 : 0] = __dmul_rn(double(__uint_as_float(ra[q] & 0xFFFF0000u)), double(__uint_as_float(rb[q] & 0xFFFF0000u)));
                }
            }
            const uint32_t m1 = max(mx & 0xFFFFu, mx >> 16);
            e_prod = m1 ? int(m1 >> E::MBITS) - 2 * E::BIAS : NO_EXP;
        } else {
            uint32_t mx = 0u;
#pragma unroll
            for (int k = 0; k < L; ++k) {
                const uint32_t xa = ra[k] & 0x7FFFE000u, xb = rb[k] & 0x7FFFE000u;
                const uint32_t es = max(xa >> 23, 1u) + max(xb >> 23, 1u);
                mx = max(mx, (xa && xb) ? es : 0u);
                pd[EK == EK_F16 ? 0 : k] = __dmul_rn(double(__uint_as_float(ra[k] & 0xFFFFE000u)), double(__uint_as_float(rb[k] & 0xFFFFE000u)));
            }
            e_prod = mx ? int(mx) - 2 * E::BIAS : NO_EXP;
        }
        const uint32_t cfield = ACC16 ? (cw >> 10) & 0x1Fu : (cw >> 23) & 0xFFu;
        const int e_c = (cw & (ACC16 ? 0x7FFFu : 0x7FFFFFFFu)) ? int(max(cfield, 1u)) - (ACC16 ? 15 : 127) : NO_EXP;
        const double cd = ACC16 ? double(__half2float(__ushort_as_half((unsigned short)cw))) : double(__uint_as_float(cw));

        // Step 2: e_max over the L + 1 terms, alignment and sign-magnitude truncation to F fractional bits, exact sum
        const int emax = max(max(e_prod, e_c), -400);     // every term zero: any exponent will do
        const double scale = __hiloint2double((1023 + F - emax) << 20, 0);
        double S0 = trunc_scaled(cd, scale, __double2hiint(cd)), S1 = 0.0;
#pragma unroll
        for (int k = 0; k < L; ++k) {
            double tk;
            if (EK == EK_F16) tk = trunc_scaled(double(pf[EK == EK_F16 ? k : 0]), scale, __float_as_int(pf[EK == EK_F16 ? k : 0]));
            else tk = trunc_scaled(pd[EK == EK_F16 ? 0 : k], scale, __double2hiint(pd[EK == EK_F16 ? 0 : k]));
            if (k & 1) S1 += tk; else S0 += tk;
        }
        // Step 3: d = rho(S * 2^(e_max - F)).  S (|S| < 2^33) times a power of two is exact in FP64, so rho is one
        // conversion: both overflow to infinity (for RZ-FP32 the test is explicit: cvt.rz saturates), both keep
        // subnormal results; an exact zero is +0.  A sum that is not finite gives the NaN / infinity of Section 4.2.
        const double S = S0 + S1;                         // S1 starts from +0, so an all-zero sum is +0
        const double v = __dmul_rn(S, __hiloint2double((1023 + emax - F) << 20, 0));
        if (ACC16) cw = (v != v) ? 0x7FFFu : uint32_t(__half_as_ushort(__double2half(v)));
        else if (fabs(v) >= 3.402823669209385e38) cw = (__double2hiint(v) < 0 ? 0xFF800000u : 0x7F800000u);   // |v| >= 2^128: overflow
        else cw = (v != v) ? 0x7FFFFFFFu : __float_as_uint(__double2float_rz(v));
    }
    // a chain's last word of magnitude zero is +0, also when a negative sum underflowed (in between the sign of a zero
    // does not matter: a zero accumulator has no exponent and adds nothing)
    return positive_zero(cw, ACC16 ? 0x7FFFu : 0x7FFFFFFFu);
}

template <int EK, int L, int RHO, bool STAGED>
__global__ void __launch_bounds__(DOT_THREADS)
dot_tfdpa_kernel(DevModel m, int64_t n, int64_t K, const void* A, const void* B, const void* C, void* D) {
    constexpr bool ACC16 = RHO == RHO_RNE_FP16;
    extern __shared__ __align__(16) unsigned char dot_smem[];
    const int row_bytes = int(K) * Elem<EK>::BYTES;
    const int F = m.F;
    if (STAGED) {
        staged_tile<ACC16>(dot_smem, n, row_bytes, A, B, C, D, [&](const StagedRows& rows, int64_t, uint32_t c) {
            return tfdpa_dot<EK, L, RHO>(rows, int(K), F, c);
        });
    } else {
        const int64_t t = int64_t(blockIdx.x) * DOT_THREADS + threadIdx.x;
        if (t >= n) return;
        uint32_t cw = 0u;
        if (C) cw = ACC16 ? uint32_t(static_cast<const uint16_t*>(C)[t]) : static_cast<const uint32_t*>(C)[t];
        GlobalRows rows;
        rows.a = static_cast<const unsigned char*>(A) + t * row_bytes;
        rows.b = static_cast<const unsigned char*>(B) + t * row_bytes;
        cw = tfdpa_dot<EK, L, RHO>(rows, int(K), F, cw);
        if (ACC16) static_cast<uint16_t*>(D)[t] = uint16_t(cw);
        else static_cast<uint32_t*>(D)[t] = cw;
    }
}

// FTZ-Add / FTZ-Mul (Algorithm 1) as the hardware's flush-to-zero operations: operands are never subnormal here
// (Algorithm 2 flushes the inputs first and every intermediate is flushed), and no result is rounded across 2^-126
// (products of 16-bit formats have at most 22 significant bits; sums below 2^-125 are multiples of 2^-149).
__device__ __forceinline__ float hw_ftz_add(float x, float y) {
    float z;
    asm("add.rn.ftz.f32 %0, %1, %2;" : "=f"(z) : "f"(x), "f"(y));
    return z;
}
__device__ __forceinline__ float hw_ftz_mul(float x, float y) {
    float z;
    asm("mul.rn.ftz.f32 %0, %1, %2;" : "=f"(z) : "f"(x), "f"(y));
    return z;
}

// Phi_FTZ-AddMul (Algorithm 2) for one dot product; STEP elements per load and operand.
template <int EK, int P, int STEP, class Rows>
__device__ __forceinline__ float ftz_dot(const Rows& rows, int K, float d) {
    for (int k0 = 0; k0 < K; k0 += STEP) {
        uint32_t ra[STEP / 2], rb[STEP / 2];
        load_raw<2, STEP>(rows, false, k0, ra);
        load_raw<2, STEP>(rows, true, k0, rb);
        float a[STEP], b[STEP];
#pragma unroll
        for (int k = 0; k < STEP; ++k) {
            const uint32_t wa = (ra[k / 2] >> (16 * (k % 2))) & 0xFFFFu, wb = (rb[k / 2] >> (16 * (k % 2))) & 0xFFFFu;
            if (EK == EK_BF16) {
                a[k] = ((wa & 0x7F80u) == 0u && (wa & 0x007Fu)) ? 0.0f : __uint_as_float(wa << 16);
                b[k] = ((wb & 0x7F80u) == 0u && (wb & 0x007Fu)) ? 0.0f : __uint_as_float(wb << 16);
            } else {
                a[k] = ((wa & 0x7C00u) == 0u && (wa & 0x03FFu)) ? 0.0f : __half2float(__ushort_as_half((unsigned short)wa));
                b[k] = ((wb & 0x7C00u) == 0u && (wb & 0x03FFu)) ? 0.0f : __half2float(__ushort_as_half((unsigned short)wb));
            }
        }
#pragma unroll
        for (int g = 0; g < STEP; g += 4) {
            if (P == 4) {
                const float s = hw_ftz_add(hw_ftz_add(hw_ftz_mul(a[g], b[g]), hw_ftz_mul(a[g + 1], b[g + 1])), hw_ftz_add(hw_ftz_mul(a[g + 2], b[g + 2]), hw_ftz_mul(a[g + 3], b[g + 3])));
                d = hw_ftz_add(d, s);
            } else {
                d = hw_ftz_add(d, hw_ftz_add(hw_ftz_mul(a[g], b[g]), hw_ftz_mul(a[g + 1], b[g + 1])));
                d = hw_ftz_add(d, hw_ftz_add(hw_ftz_mul(a[g + 2], b[g + 2]), hw_ftz_mul(a[g + 3], b[g + 3])));
            }
        }
    }
    return d;
}

__device__ __forceinline__ float flush_c(uint32_t w) {       // FlushSubnormal(C) of Algorithm 2
    return ((w & 0x7F800000u) == 0u && (w & 0x007FFFFFu)) ? 0.0f : __uint_as_float(w);
}
__device__ __forceinline__ uint32_t ftz_word(float d) { return d != d ? 0x7FC00000u : __float_as_uint(d); }

template <int EK, int P, int STEP, bool STAGED>
__global__ void __launch_bounds__(DOT_THREADS)
dot_ftz_kernel(int64_t n, int64_t K, const void* A, const void* B, const void* C, void* D) {
    extern __shared__ __align__(16) unsigned char dot_smem[];
    const int row_bytes = int(K) * 2;
    if (STAGED) {
        staged_tile<false>(dot_smem, n, row_bytes, A, B, C, D, [&](const StagedRows& rows, int64_t, uint32_t c) {
            return ftz_word(ftz_dot<EK, P, STEP>(rows, int(K), flush_c(c)));
        });
    } else {
        const int64_t t = int64_t(blockIdx.x) * DOT_THREADS + threadIdx.x;
        if (t >= n) return;
        GlobalRows rows;
        rows.a = static_cast<const unsigned char*>(A) + t * row_bytes;
        rows.b = static_cast<const unsigned char*>(B) + t * row_bytes;
        const float d = ftz_dot<EK, P, STEP>(rows, int(K), flush_c(C ? static_cast<const uint32_t*>(C)[t] : 0u));
        static_cast<uint32_t*>(D)[t] = ftz_word(d);
    }
}

// Rows of 8 to 128 bytes (a power of two) are staged through shared memory: 2 * 128 rows per CTA.
bool staged_rows(int64_t row_bytes) {
    return row_bytes == 8 || row_bytes == 16 || row_bytes == 32 || row_bytes == 64 || row_bytes == 128;
}

template <class Kernel, class... Args>
cudaError_t launch_dot(Kernel kernel, bool staged, int64_t n, int64_t row_bytes, cudaStream_t st, Args... args) {
    const unsigned blocks = unsigned((n + DOT_THREADS - 1) / DOT_THREADS);
    const size_t smem = staged ? size_t(2 * DOT_THREADS * row_bytes) : 0;          // the tile's rows of A and of B
    if (smem > 48 * 1024) {
        const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
        if (e != cudaSuccess) return e;
    }
    kernel<<<blocks, DOT_THREADS, smem, st>>>(args...);
    return cudaGetLastError();
}

template <int EK, int L, int RHO>
cudaError_t launch_t_rho(const DevModel& m, const GemmArgs& g, cudaStream_t st) {
    const int64_t rb = g.K * Elem<EK>::BYTES;
    if (staged_rows(rb)) return launch_dot(dot_tfdpa_kernel<EK, L, RHO, true>, true, g.M, rb, st, m, g.M, g.K, g.A, g.B, g.C, g.D);
    return launch_dot(dot_tfdpa_kernel<EK, L, RHO, false>, false, g.M, rb, st, m, g.M, g.K, g.A, g.B, g.C, g.D);
}

template <int EK, int L>
cudaError_t launch_t(const DevModel& m, const GemmArgs& g, cudaStream_t st) {
    if (m.rho == RHO_RZ_FP32) return launch_t_rho<EK, L, RHO_RZ_FP32>(m, g, st);
    return launch_t_rho<EK, L, RHO_RNE_FP16>(m, g, st);
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

template <int EK, int P>
cudaError_t launch_ftz(const GemmArgs& g, cudaStream_t st) {
    const int64_t rb = g.K * 2;
    const bool staged = staged_rows(rb);
    if (g.K % 8 == 0) {
        if (staged) return launch_dot(dot_ftz_kernel<EK, P, 8, true>, true, g.M, rb, st, g.M, g.K, g.A, g.B, g.C, g.D);
        return launch_dot(dot_ftz_kernel<EK, P, 8, false>, false, g.M, rb, st, g.M, g.K, g.A, g.B, g.C, g.D);
    }
    if (staged) return launch_dot(dot_ftz_kernel<EK, P, 4, true>, true, g.M, rb, st, g.M, g.K, g.A, g.B, g.C, g.D);
    return launch_dot(dot_ftz_kernel<EK, P, 4, false>, false, g.M, rb, st, g.M, g.K, g.A, g.B, g.C, g.D);
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
        if (m.fmt_a == EF_F16) err = launch_ftz<EK_F16, 4>(g, stream);
        else if (m.P == 4) err = launch_ftz<EK_BF16, 4>(g, stream);
        else err = launch_ftz<EK_BF16, 2>(g, stream);
    }
    if (err != cudaSuccess) {
        set_error("dot_batch kernel launch failed: %s", cudaGetErrorString(err));
        return MMASIM_ERR_CUDA;
    }
    return MMASIM_OK;
}

}  // namespace mmasim
