// Instantiations of the persistent TMA-staged fused kernel: sign, 1-bit and 2-bit codes.
#include "ds_fused_tma_kernel.cuh"

namespace ds {

cudaError_t launch_fused_tma_sign_u1_u2(const LaunchShape& sh, const StepParams& p, cudaStream_t stream) {
    switch (sh.code) {
        case CODE_SIGN: return launch_tma_code<CODE_SIGN>(sh, p, stream);
        case CODE_U1: return launch_tma_code<CODE_U1>(sh, p, stream);
        case CODE_U2: return launch_tma_code<CODE_U2>(sh, p, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace ds
