// Instantiations of the tuned T-FDPA kernel for BF16 and TF32 inputs.
#include "mmasim_tfdpa_fast.cuh"
namespace mmasim { namespace fast {
cudaError_t launch_bf16(const DevModel& m, const GemmArgs& g, cudaStream_t st) {
    if (m.F == 24 && m.L == 8 && m.rho == RHO_RZ_FP32) return launch_variant<EK_BF16, 8, 24, RHO_RZ_FP32>(m, g, st);
    if (m.F == 25 && m.L == 16 && m.rho == RHO_RZ_FP32) return launch_variant<EK_BF16, 16, 25, RHO_RZ_FP32>(m, g, st);
    return cudaErrorInvalidValue;
}
cudaError_t launch_tf32(const DevModel& m, const GemmArgs& g, cudaStream_t st) {
    if (m.F == 24 && m.L == 4 && m.rho == RHO_RZ_FP32) return launch_variant<EK_TF32, 4, 24, RHO_RZ_FP32>(m, g, st);
    if (m.F == 25 && m.L == 8 && m.rho == RHO_RZ_FP32) return launch_variant<EK_TF32, 8, 25, RHO_RZ_FP32>(m, g, st);
    return cudaErrorInvalidValue;
}
}}
