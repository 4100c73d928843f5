// Instantiations of the batch-sweeping fused kernel (direct loads) for norm-matched codes.
#include "ds_wide_fused_kernel.cuh"

namespace ds {

cudaError_t launch_fused_wide_norm(const LaunchShape& sh, const StepParams& p, cudaStream_t stream) {
    switch (sh.code) {
        case CODE_N2: return launch_wide_code<CODE_N2>(sh, p, stream);
        case CODE_N4: return launch_wide_code<CODE_N4>(sh, p, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace ds
