// Instantiations of the tuned T-FDPA kernel for BF16 and TF32 inputs.
#include "mmasim_tfdpa_f64.cuh"
namespace mmasim { namespace fast {
cudaError_t launch_bf16(const DevModel& m, const GemmArgs& g, cudaStream_t st) {
    if (m.F == 24 && m.L == 8 && m.rho == RHO_RZ_FP32) return fast64::launch_variant64<EK_BF16, 8, RHO_RZ_FP32>(m, g, st);
    if (m.F == 25 && m.L == 16 && m.rho == RHO_RZ_FP32) return fast64::launch_variant64<EK_BF16, 16, RHO_RZ_FP32>(m, g, st);
    return cudaErrorInvalidValue;
}
cudaError_t launch_tf32(const DevModel& m, const GemmArgs& g, cudaStream_t st) {
    if (m.F == 24 && m.L == 4 && m.rho == RHO_RZ_FP32) return fast64::launch_variant64<EK_TF32, 4, RHO_RZ_FP32>(m, g, st);
    if (m.F == 25 && m.L == 8 && m.rho == RHO_RZ_FP32) return fast64::launch_variant64<EK_TF32, 8, RHO_RZ_FP32>(m, g, st);
    return cudaErrorInvalidValue;
}
}}
