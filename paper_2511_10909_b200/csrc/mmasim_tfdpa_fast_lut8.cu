// Instantiations of the tuned T-FDPA kernel for 8-bit inputs (FP8 / FP6 / FP4, one element per byte) and of its
// block-scaled variant (ST-FDPA, Algorithm 8).
#include "mmasim_tfdpa_f64.cuh"
#include "mmasim_tfdpa_trop.cuh"
#include <mutex>
namespace mmasim { namespace fast {

namespace {
cudaError_t launch_f13(const DevModel& m, const GemmArgs& g, cudaStream_t st, const trop::Scratch& sc) {
    if (m.L == 16 && m.rho == RHO_RZ_E8M13) return trop::launch_by_types_t<EK_LUT8, 16, 13, RHO_RZ_E8M13>(m, g, st, sc);
    if (m.L == 16 && m.rho == RHO_RNE_FP16) return trop::launch_by_types_t<EK_LUT8, 16, 13, RHO_RNE_FP16>(m, g, st, sc);
    if (m.L == 32 && m.rho == RHO_RZ_E8M13) return trop::launch_by_types_t<EK_LUT8, 32, 13, RHO_RZ_E8M13>(m, g, st, sc);
    if (m.L == 32 && m.rho == RHO_RNE_FP16) return trop::launch_by_types_t<EK_LUT8, 32, 13, RHO_RNE_FP16>(m, g, st, sc);
    return cudaErrorInvalidValue;
}

// Scratch of mmasim_gemm_noalloc: the decoded operand blocks of the F = 13 kernel in a fixed array that every GPU loading
// the library holds until the process ends.  Host code must not use the symbol as a pointer: the device address comes
// from cudaGetSymbolAddress, asked once per device with that device current.
constexpr size_t NOALLOC_BYTES = size_t(32) << 20;
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_BYTES];
constexpr int NOALLOC_MAX_DEVICES = 64;
std::mutex g_noalloc_mutex;
void* g_noalloc_ptr[NOALLOC_MAX_DEVICES] = {};
}  // namespace

size_t noalloc_capacity() { return NOALLOC_BYTES; }

bool noalloc_supported(const DevModel& m) {
    const bool f8 = (m.fmt_a == EF_E4M3 || m.fmt_a == EF_E5M2) && (m.fmt_b == EF_E4M3 || m.fmt_b == EF_E5M2);
    return m.family == FAM_T && f8 && m.F == 13 && (m.L == 16 || m.L == 32) && (m.rho == RHO_RZ_E8M13 || m.rho == RHO_RNE_FP16);
}

size_t noalloc_need(const DevModel& m, const GemmArgs& g) { return trop::scratch_bytes(m, g); }

cudaError_t launch_noalloc(const DevModel& m, const GemmArgs& g, cudaStream_t st) {
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= NOALLOC_MAX_DEVICES) return cudaErrorInvalidDevice;
    void* ptr = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_noalloc_mutex);
        if (!g_noalloc_ptr[dev]) {                      // set-up, once per device, with that device current
            void* p = nullptr;
            err = cudaGetSymbolAddress(&p, g_noalloc_scratch);
            if (err != cudaSuccess) return err;
            g_noalloc_ptr[dev] = p;
        }
        ptr = g_noalloc_ptr[dev];
    }
    trop::Scratch sc;
    sc.given = ptr;
    sc.capacity = NOALLOC_BYTES;
    return launch_f13(m, g, st, sc);
}

cudaError_t launch_lut8(const DevModel& m, const GemmArgs& g, cudaStream_t st) {
    if (m.family == FAM_ST) {
        if (m.F == 25 && m.L == 32 && m.rho == RHO_RZ_FP32) return fast64::launch_variant64<EK_LUT8, 32, RHO_RZ_FP32, true>(m, g, st);
        return cudaErrorInvalidValue;
    }
    if (m.F == 13) return launch_f13(m, g, st, trop::Scratch());   // FP8 x FP8 with F = 13: the exponent maximum on the tensor cores
    if (m.F == 25 && m.L == 32 && m.rho == RHO_RZ_FP32) return fast64::launch_variant64<EK_LUT8, 32, RHO_RZ_FP32>(m, g, st);
    if (m.F == 25 && m.L == 32 && m.rho == RHO_RNE_FP16) return fast64::launch_variant64<EK_LUT8, 32, RHO_RNE_FP16>(m, g, st);
    return cudaErrorInvalidValue;
}
}}
