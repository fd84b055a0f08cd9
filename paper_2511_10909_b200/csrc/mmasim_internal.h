// Types shared by the host-side registry / API and the device kernels of libmmasim.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>
#include "../../include/mmasim.h"

namespace mmasim {

// Element formats (device-side ids).  The order is private to the library.
enum ElemFmt : int {
    EF_F64 = 0, EF_F32, EF_TF32, EF_BF16, EF_F16, EF_E4M3, EF_E5M2, EF_E3M2, EF_E2M3, EF_E2M1, EF_E8M0, EF_UE4M3,
    EF_COUNT
};
enum Specials : int { SP_IEEE = 0, SP_FN, SP_NONE, SP_E8M0 };

struct FmtDesc {
    int ebits, mbits, bias, specials, is_signed, low_ignored, storage_bits;
};

// IEEE-754 binary64/32/16, BF16 and TF32 as truncated binary32, the OCP FP8 formats (E5M2 IEEE-like, E4M3 with
// no infinity and one NaN pattern), the OCP Microscaling element formats (no specials) and scale formats.
__host__ __device__ inline FmtDesc fmt_desc(int f) {
    switch (f) {
        case EF_F64: return {11, 52, 1023, SP_IEEE, 1, 0, 64};
        case EF_F32: return {8, 23, 127, SP_IEEE, 1, 0, 32};
        case EF_TF32: return {8, 10, 127, SP_IEEE, 1, 13, 32};
        case EF_BF16: return {8, 7, 127, SP_IEEE, 1, 0, 16};
        case EF_F16: return {5, 10, 15, SP_IEEE, 1, 0, 16};
        case EF_E4M3: return {4, 3, 7, SP_FN, 1, 0, 8};
        case EF_E5M2: return {5, 2, 15, SP_IEEE, 1, 0, 8};
        case EF_E3M2: return {3, 2, 3, SP_NONE, 1, 0, 8};
        case EF_E2M3: return {2, 3, 1, SP_NONE, 1, 0, 8};
        case EF_E2M1: return {2, 1, 1, SP_NONE, 1, 0, 8};
        case EF_E8M0: return {8, 0, 127, SP_E8M0, 0, 0, 8};
        default: return {4, 3, 7, SP_FN, 0, 0, 8};   // EF_UE4M3
    }
}

enum Family : int { FAM_FMA = 0, FAM_FTZ, FAM_E, FAM_T, FAM_ST, FAM_GST, FAM_TR, FAM_GTR };
enum Rho : int { RHO_NONE = 0, RHO_RZ_FP32, RHO_RZ_E8M13, RHO_RNE_FP32, RHO_RNE_FP16 };
enum Acc : int { ACC_F32 = 0, ACC_F16, ACC_F64 };

// Everything a kernel needs to know about a model; passed by value as a kernel argument.
struct DevModel {
    int family;
    int fmt_a, fmt_b;     // ElemFmt of A and B elements
    int acc;              // Acc
    int L, F, F2, rho;
    int P, G, k_block, scale_fmt;
    int frac;             // fractional bits of a product term (mbits_a + mbits_b; GST: 2 + 2 * scale mbits)
    int inner_round;      // 0: paper; 1: TR second stage in RZ
    int packed4;          // A and B hold two FP4 codes per byte
    int literal_emax;     // 1: the maximum exponent over every term, as Algorithms 7-11 print it (generic kernels only)
};

// Per-call arguments common to the GEMM-shaped kernels.
struct GemmArgs {
    int64_t M, N, K;
    const void* A;
    const void* B;
    const void* C;
    void* D;
    int64_t lda, ldb, ldc, ldd;   // in elements
    const uint8_t* sfa;
    const uint8_t* sfb;
    int64_t ld_sfa, ld_sfb;       // scale factors per row
    int64_t k_chunk;
    const float* row_scale;
    const float* col_scale;
    int dot_mode;                 // 1: n independent dots (row t of A with row t of B), N is ignored
    unsigned int* copy_timeouts;  // device counter of CTAs whose bounded wait on a bulk copy ran out (may be NULL)
};

}  // namespace mmasim

struct mmasim_model {
    int arch, a_fmt, b_fmt, acc_fmt;   // public enums
    mmasim::DevModel dev;
    mmasim_info info;
};

namespace mmasim {
// mmasim_registry.cpp
bool registry_lookup(int arch, int a_fmt, int b_fmt, int acc_fmt, mmasim_model* out, const char** why);
// mmasim_generic.cu
int launch_generic(const DevModel& m, const GemmArgs& g, cudaStream_t stream);
// mmasim_tfdpa_fast.cu
bool fast_tfdpa_supported(const DevModel& m, const GemmArgs& g);
int launch_fast_tfdpa(const DevModel& m, const GemmArgs& g, cudaStream_t stream);
int launch_gemm_noalloc(const DevModel& m, const GemmArgs& g, cudaStream_t stream);   // status code; sets the error message
// mmasim_fp_fast.cu
bool fast_fp_supported(const DevModel& m, const GemmArgs& g);
int launch_fast_fp(const DevModel& m, const GemmArgs& g, cudaStream_t stream);
// mmasim_gst_fast.cu
bool fast_gst_supported(const DevModel& m, const GemmArgs& g);
int launch_fast_gst(const DevModel& m, const GemmArgs& g, cudaStream_t stream);
// mmasim_dot_stream.cu
bool dot_stream_supported(const DevModel& m, const GemmArgs& g);
int launch_dot_stream(const DevModel& m, const GemmArgs& g, cudaStream_t stream);
// mmasim_hw_mma.cu
int launch_hw_mma(int kind, int64_t M, int64_t K, const void* A, const void* B, const void* C, void* D, cudaStream_t stream);
// mmasim_hw_umma.cu
int launch_hw_umma(int kind, int64_t M, int64_t K, const void* A, const void* B, const void* C, void* D, const void* sfa,
                   const void* sfb, int32_t* status, cudaStream_t stream);
// mmasim_stats.cu
int launch_error_stats(int acc, int64_t n, const void* D, const double* ref, double* stats, cudaStream_t stream);
// mmasim_peak.cu
int launch_int_peak(int kind, int64_t blocks, int64_t iters, void* sink, int32_t* ops_per_round, cudaStream_t stream);
// mmasim_api.cpp
unsigned int* copy_timeout_counter();          // the current device's counter (a device variable of the library; NULL on failure)
cudaError_t scratch_pool(cudaMemPool_t* out);   // the library's own memory pool of the current device (created on first use)
void set_error(const char* fmt, ...);
void set_kernel_name(const char* name);
}  // namespace mmasim
