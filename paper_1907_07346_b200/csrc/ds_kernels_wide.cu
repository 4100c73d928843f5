// Instantiations of the fused kernel that sweeps the nodes of a column in batches.
#include "ds_wide_fused_kernel.cuh"

namespace ds {

cudaError_t launch_fused_wide(const LaunchShape& sh, const StepParams& p, cudaStream_t stream) {
    switch (sh.code) {
        case CODE_SIGN: return launch_wide_code<CODE_SIGN>(sh, p, stream);
        case CODE_U1: return launch_wide_code<CODE_U1>(sh, p, stream);
        case CODE_U2: return launch_wide_code<CODE_U2>(sh, p, stream);
        case CODE_U4: return launch_wide_code<CODE_U4>(sh, p, stream);
        case CODE_U8: return launch_wide_code<CODE_U8>(sh, p, stream);
        case CODE_N2: case CODE_N4: return launch_fused_wide_norm(sh, p, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace ds
