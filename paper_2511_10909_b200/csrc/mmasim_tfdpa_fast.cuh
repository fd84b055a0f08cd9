// Definitions shared by the tuned FDPA kernels (Algorithm 5 + Algorithms 7, 8, 10, 11): tile shape, exponent biases,
// element kinds, and the per-kind launchers that mmasim_tfdpa_fast.cu dispatches to.
//
// Work decomposition common to all of them.  A CTA owns a 128 x 64 tile of D and keeps its outputs in registers for
// the whole K loop.  K is walked in chunks of 32 elements: the CTA loads the raw A / B words of the chunk, decodes
// every element once (8-bit formats through a 256-entry table, 16/32-bit formats by bit manipulation) and stores the
// decoded planes k-major in shared memory, double-buffered, so that one 16-byte shared load feeds several rows (or
// columns) of a thread's micro-tile.  Per block of L elements and per output the kernels take e_max over the nonzero
// terms and the accumulator, then spend ONE fused multiply-add per term: the sum lives in a floating-point register
// as (1.5 * 2^p + S) * 2^(e_max - F), so that a multiply-add rounded toward minus infinity aligns, truncates and
// accumulates a term at once.
//
// Sign-magnitude truncation without per-term sign work.  RZ_F truncates the magnitude of each aligned term, while
// a multiply-add rounding toward minus infinity rounds down.  Negative terms are therefore carried in one's
// complement (the B operand carries a small offset that makes every negative product inexact, so that it floors to
// -t - 1), and the number of negative nonzero terms of the block (a population count over per-row / per-column sign
// and nonzero bit masks) is added back once per block.
//
//   mmasim_tfdpa_trop.cuh   F = 13, 8-bit inputs: FP32 registers, e_max on the tensor cores
//   mmasim_tfdpa_f64.cuh    F >= 23 and ST-FDPA: FP64 registers, e_max by fused add-max on 16-bit lanes
//   mmasim_trfdpa_f64.cu    TR- / GTR-FDPA: two FP64 registers per output (even and odd terms)
//   mmasim_efdpa_f64.cu     E-FDPA: the exact sum as a chain of FP64 multiply-adds where it fits a window
//
// Exponents, where staged as integers, carry a bias of 512 per element (1024 per product / accumulator) so that they
// are positive 16-bit lane values; a zero element, like a zero accumulator, has no exponent and is staged as the
// word 0, which keeps every sum it enters below every sum of two real exponents.
//
// Everything that is rare takes a slow, by-the-book route: NaN / infinity inputs (the threads rescan the raw words
// of the block and keep sticky NaN / +inf / -inf flags per output, Section 4.2) and results outside the range the
// registers can carry.
#pragma once
#include <cuda_fp16.h>
#include "mmasim_device.cuh"

namespace mmasim {
namespace fast {

constexpr int BM = 128, BN = 64, KC = 32, NT = 256;
constexpr int EB = 512;            // bias of a staged element exponent
constexpr int CB = 2 * EB;         // bias of an exponent sum and of the accumulator exponent

enum ElemKind : int { EK_LUT8 = 0, EK_F16 = 1, EK_BF16 = 2, EK_TF32 = 3 };

template <int EK> struct Elem;
template <> struct Elem<EK_LUT8> { static constexpr int BYTES = 1, TASK = 16, EBITS = 4, MBITS = 3, BIAS = 7, LOW = 0; static constexpr bool SIGNMAG = false; };  // EBITS.. unused: table-decoded
template <> struct Elem<EK_F16> { static constexpr int BYTES = 2, TASK = 8, EBITS = 5, MBITS = 10, BIAS = 15, LOW = 0; static constexpr bool SIGNMAG = true; };
template <> struct Elem<EK_BF16> { static constexpr int BYTES = 2, TASK = 8, EBITS = 8, MBITS = 7, BIAS = 127, LOW = 0; static constexpr bool SIGNMAG = true; };
template <> struct Elem<EK_TF32> { static constexpr int BYTES = 4, TASK = 8, EBITS = 8, MBITS = 10, BIAS = 127, LOW = 13; static constexpr bool SIGNMAG = true; };

__device__ __forceinline__ int asr_clamp(int x, int d) {
    int r;
    asm("shr.s32 %0, %1, %2;" : "=r"(r) : "r"(x), "r"(d));      // amounts above 31 behave as 31 (sign fill)
    return r;
}

template <int EK>
__device__ __forceinline__ uint32_t raw_elem(const void* p, int64_t idx) {
    if (Elem<EK>::BYTES == 1) return static_cast<const uint8_t*>(p)[idx];
    if (Elem<EK>::BYTES == 2) return static_cast<const uint16_t*>(p)[idx];
    return static_cast<const uint32_t*>(p)[idx];
}

// ---- bulk copies and their barrier: inline PTX ----
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return uint32_t(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(unsigned long long* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, unsigned long long* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(smem_addr(dst)), "l"(src), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}
// Waits for the given phase of the barrier; gives up after a bounded number of polls (each poll itself blocks for a
// bounded, implementation-defined time) and returns false.
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, uint32_t parity) {
    const uint32_t addr = smem_addr(bar);
    for (int spin = 0; spin < (1 << 22); ++spin) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(addr), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}

// A CTA whose bounded wait on a bulk copy ran out (never in a healthy run) stores nothing and counts itself in the
// library's device counter (GemmArgs::copy_timeouts), which mmasim_copy_timeouts() reads.

// Per element kind: returns cudaErrorInvalidValue when (L, F, rho) has no instantiation.
cudaError_t launch_lut8(const DevModel& m, const GemmArgs& g, cudaStream_t stream);
cudaError_t launch_f16(const DevModel& m, const GemmArgs& g, cudaStream_t stream);
cudaError_t launch_bf16(const DevModel& m, const GemmArgs& g, cudaStream_t stream);
cudaError_t launch_tf32(const DevModel& m, const GemmArgs& g, cudaStream_t stream);
// the allocation-free variant of the F = 13 kernel (mmasim_tfdpa_fast_lut8.cu): scratch in a fixed device array
bool noalloc_supported(const DevModel& m);
size_t noalloc_capacity();
size_t noalloc_need(const DevModel& m, const GemmArgs& g);
cudaError_t launch_noalloc(const DevModel& m, const GemmArgs& g, cudaStream_t stream);
cudaError_t launch_tr(const DevModel& m, const GemmArgs& g, cudaStream_t stream);    // TR-/GTR-FDPA (mmasim_trfdpa_f64.cu)
cudaError_t launch_e(const DevModel& m, const GemmArgs& g, cudaStream_t stream);     // E-FDPA (mmasim_efdpa_f64.cu)

}  // namespace fast
}  // namespace mmasim
