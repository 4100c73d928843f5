// Instantiations of the persistent TMA-staged fused kernel: norm-matched codes.
#include "ds_fused_tma_kernel.cuh"

namespace ds {

cudaError_t launch_fused_tma_norm(const LaunchShape& sh, const StepParams& p, cudaStream_t stream) {
    switch (sh.code) {
        case CODE_N2: return launch_tma_code<CODE_N2>(sh, p, stream);
        case CODE_N4: return launch_tma_code<CODE_N4>(sh, p, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace ds
