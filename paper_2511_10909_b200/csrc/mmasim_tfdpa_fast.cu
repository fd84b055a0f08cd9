// Dispatch to the tuned FDPA kernels (T-, ST-, TR-, GTR- and E-FDPA; see mmasim_tfdpa_fast.cuh for what they share).
#include "mmasim_tfdpa_fast.cuh"
#include <mutex>

namespace mmasim {

namespace {

bool is8(int f) { return f == EF_E4M3 || f == EF_E5M2 || f == EF_E3M2 || f == EF_E2M3 || f == EF_E2M1; }

constexpr int KIND_TR = 100, KIND_E = 101;

// 0: no tuned kernel; KIND_TR: the TR-/GTR-FDPA kernel; KIND_E: the E-FDPA kernel; otherwise 1 + element kind of the
// T-FDPA kernel
int kind_of(const DevModel& m) {
    if (m.family == FAM_E) {
        const bool ok = m.fmt_a == m.fmt_b && m.acc == ACC_F32 && ((m.fmt_a == EF_F16 && m.L == 4) || (m.fmt_a == EF_BF16 && m.L == 2));
        return ok ? KIND_E : 0;
    }
    if (m.family == FAM_TR || m.family == FAM_GTR) {
        if (m.F != 24 || m.F2 != 31 || m.rho != RHO_RNE_FP32 || m.inner_round || m.acc != ACC_F32) return 0;
        if (m.family == FAM_GTR) return (is8(m.fmt_a) && is8(m.fmt_b) && m.L == 16) ? KIND_TR : 0;
        if (m.fmt_a != m.fmt_b) return 0;
        const bool ok = (m.fmt_a == EF_F16 && m.L == 8) || (m.fmt_a == EF_BF16 && m.L == 8) || (m.fmt_a == EF_TF32 && m.L == 4);
        return ok ? KIND_TR : 0;
    }
    if ((m.family != FAM_T && m.family != FAM_ST) || m.packed4) return 0;
    if (m.family == FAM_ST) {
        const bool ok = is8(m.fmt_a) && is8(m.fmt_b) && m.F == 25 && m.L == 32 && m.rho == RHO_RZ_FP32 && m.acc == ACC_F32 &&
                        m.k_block == 32 && m.scale_fmt == EF_E8M0;
        return ok ? 1 + fast::EK_LUT8 : 0;
    }
    const bool acc_ok = (m.rho == RHO_RNE_FP16) == (m.acc == ACC_F16) && m.acc != ACC_F64;
    if (!acc_ok) return 0;
    if (is8(m.fmt_a) && is8(m.fmt_b)) {
        const bool combo = (m.F == 13 && (m.L == 16 || m.L == 32) && (m.rho == RHO_RZ_E8M13 || m.rho == RHO_RNE_FP16)) ||
                           (m.F == 25 && m.L == 32 && (m.rho == RHO_RZ_FP32 || m.rho == RHO_RNE_FP16));
        return combo ? 1 + fast::EK_LUT8 : 0;
    }
    if (m.fmt_a != m.fmt_b) return 0;
    if (m.fmt_a == EF_F16) {
        const bool combo = ((m.F == 23 && m.L == 4) || (m.F == 24 && m.L == 8) || (m.F == 25 && m.L == 16)) &&
                           (m.rho == RHO_RZ_FP32 || m.rho == RHO_RNE_FP16);
        return combo ? 1 + fast::EK_F16 : 0;
    }
    if (m.fmt_a == EF_BF16) {
        const bool combo = ((m.F == 24 && m.L == 8) || (m.F == 25 && m.L == 16)) && m.rho == RHO_RZ_FP32;
        return combo ? 1 + fast::EK_BF16 : 0;
    }
    if (m.fmt_a == EF_TF32) {
        const bool combo = ((m.F == 24 && m.L == 4) || (m.F == 25 && m.L == 8)) && m.rho == RHO_RZ_FP32;
        return combo ? 1 + fast::EK_TF32 : 0;
    }
    return 0;
}

}  // namespace

bool fast_tfdpa_supported(const DevModel& m, const GemmArgs& g) {
    const int kind = kind_of(m);
    if (!kind || g.dot_mode || m.literal_emax) return false;
    const int bytes = fmt_desc(m.fmt_a).storage_bits / 8;
    if (g.K % fast::KC) return false;
    if (g.k_chunk % fast::KC) return false;
    if ((kind == KIND_TR || kind == KIND_E) && g.k_chunk) return false;
    if (((g.lda * bytes) % 16) || ((g.ldb * bytes) % 16)) return false;      // 16-byte row starts for the vector loads
    if (g.M > 65535ll * fast::BM) return false;                             // grid.y
    if (g.N > 0x7FFFFFFFll - 128 || g.K > 0x7FFFFFFFll - 64) return false;   // 32-bit tile origins and k offsets in the kernels
    return true;
}

// The counter of bulk-copy timeouts: one word per device in a device variable of the library (nothing is allocated).
namespace {
__device__ unsigned int g_copy_timeouts_word = 0u;
std::mutex g_counter_mutex;
unsigned int* g_counter_ptr[64] = {};
}  // namespace

unsigned int* copy_timeout_counter() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(g_counter_mutex);
    if (!g_counter_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_copy_timeouts_word) != cudaSuccess) return nullptr;
        g_counter_ptr[dev] = static_cast<unsigned int*>(p);
    }
    return g_counter_ptr[dev];
}

int launch_gemm_noalloc(const DevModel& m, const GemmArgs& g, cudaStream_t stream) {
    if (!fast::noalloc_supported(m) || !fast_tfdpa_supported(m, g)) {
        set_error("mmasim_gemm_noalloc serves the FP8 models with F = 13 (Ada and Hopper FP8 rows), K a multiple of 32 and "
                  "16-byte row strides; this call needs another kernel");
        return MMASIM_ERR_UNSUPPORTED;
    }
    const size_t need = fast::noalloc_need(m, g), cap = fast::noalloc_capacity();
    if (need > cap) {
        set_error("mmasim_gemm_noalloc: this problem needs %zu bytes of scratch, the fixed array holds %zu "
                  "(about (ceil(M/128) + ceil(N/128)) * K/32 * 27 KiB); use mmasim_gemm_ex", need, cap);
        return MMASIM_ERR_SHAPE;
    }
    set_kernel_name("tfdpa_lut8_noalloc");
    const cudaError_t err = fast::launch_noalloc(m, g, stream);
    if (err != cudaSuccess) {
        set_error("mmasim_gemm_noalloc: %s", cudaGetErrorString(err));
        return MMASIM_ERR_CUDA;
    }
    return MMASIM_OK;
}

int launch_fast_tfdpa(const DevModel& m, const GemmArgs& g, cudaStream_t stream) {
    cudaError_t err = cudaErrorInvalidValue;
    if (kind_of(m) == KIND_TR) {
        set_kernel_name(m.family == FAM_GTR ? "gtrfdpa" : "trfdpa");
        err = fast::launch_tr(m, g, stream);
    } else if (kind_of(m) == KIND_E) {
        set_kernel_name("efdpa");
        err = fast::launch_e(m, g, stream);
    } else switch (kind_of(m) - 1) {
        case fast::EK_LUT8: set_kernel_name("tfdpa_lut8"); err = fast::launch_lut8(m, g, stream); break;
        case fast::EK_F16: set_kernel_name("tfdpa_f16"); err = fast::launch_f16(m, g, stream); break;
        case fast::EK_BF16: set_kernel_name("tfdpa_bf16"); err = fast::launch_bf16(m, g, stream); break;
        case fast::EK_TF32: set_kernel_name("tfdpa_tf32"); err = fast::launch_tf32(m, g, stream); break;
        default: break;
    }
    if (err != cudaSuccess) {
        set_error("tuned T-FDPA kernel launch failed: %s", cudaGetErrorString(err));
        return MMASIM_ERR_CUDA;
    }
    return MMASIM_OK;
}

}  // namespace mmasim
