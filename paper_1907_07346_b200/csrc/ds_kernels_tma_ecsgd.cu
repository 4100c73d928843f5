// Instantiations of the persistent TMA-staged fused kernel for centralized
// error-compensated SGD (Section 1).
#include "ds_fused_tma_ecsgd.h"
#include "ds_fused_tma_kernel.cuh"

namespace ds {

cudaError_t launch_fused_tma_ecsgd(const LaunchShape& sh, const StepParams& p, cudaStream_t stream) {
    switch (sh.code) {
        case CODE_SIGN: return launch_tma_ecsgd_code<CODE_SIGN>(sh, p, stream);
        case CODE_U1: return launch_tma_ecsgd_code<CODE_U1>(sh, p, stream);
        case CODE_U2: return launch_tma_ecsgd_code<CODE_U2>(sh, p, stream);
        case CODE_U4: return launch_tma_ecsgd_code<CODE_U4>(sh, p, stream);
        case CODE_U8: return launch_tma_ecsgd_code<CODE_U8>(sh, p, stream);
        case CODE_ID32: return launch_tma_ecsgd_code<CODE_ID32>(sh, p, stream);
        case CODE_N2: return launch_tma_ecsgd_code<CODE_N2>(sh, p, stream);
        case CODE_N4: return launch_tma_ecsgd_code<CODE_N4>(sh, p, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace ds
