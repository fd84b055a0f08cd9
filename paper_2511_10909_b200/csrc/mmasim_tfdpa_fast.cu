// Tuned T-FDPA kernels (placeholder dispatch: nothing is claimed yet, every call goes to the generic kernels).
#include "mmasim_internal.h"

namespace mmasim {

bool fast_tfdpa_supported(const DevModel&, const GemmArgs&) { return false; }

int launch_fast_tfdpa(const DevModel&, const GemmArgs&, cudaStream_t) {
    set_error("no tuned kernel for this model");
    return MMASIM_ERR_UNSUPPORTED;
}

}  // namespace mmasim
