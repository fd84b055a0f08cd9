// Instantiations of the tuned T-FDPA kernel for FP16 inputs.
#include "mmasim_tfdpa_f64.cuh"
namespace mmasim { namespace fast {
cudaError_t launch_f16(const DevModel& m, const GemmArgs& g, cudaStream_t st) {
    if (m.F == 23 && m.L == 4 && m.rho == RHO_RZ_FP32) return fast64::launch_variant64<EK_F16, 4, RHO_RZ_FP32>(m, g, st);
    if (m.F == 23 && m.L == 4 && m.rho == RHO_RNE_FP16) return fast64::launch_variant64<EK_F16, 4, RHO_RNE_FP16>(m, g, st);
    if (m.F == 24 && m.L == 8 && m.rho == RHO_RZ_FP32) return fast64::launch_variant64<EK_F16, 8, RHO_RZ_FP32>(m, g, st);
    if (m.F == 24 && m.L == 8 && m.rho == RHO_RNE_FP16) return fast64::launch_variant64<EK_F16, 8, RHO_RNE_FP16>(m, g, st);
    if (m.F == 25 && m.L == 16 && m.rho == RHO_RZ_FP32) return fast64::launch_variant64<EK_F16, 16, RHO_RZ_FP32>(m, g, st);
    if (m.F == 25 && m.L == 16 && m.rho == RHO_RNE_FP16) return fast64::launch_variant64<EK_F16, 16, RHO_RNE_FP16>(m, g, st);
    return cudaErrorInvalidValue;
}
}}
