// Dispatch of the persistent TMA-staged fused kernel; its instantiations are spread over
// the ds_kernels_tma_*.cu units so that they compile in parallel.
#include "ds_internal.h"

namespace ds {

cudaError_t launch_fused_tma_sign_u1_u2(const LaunchShape& sh, const StepParams& p, cudaStream_t stream);
cudaError_t launch_fused_tma_u4_u8_id(const LaunchShape& sh, const StepParams& p, cudaStream_t stream);
cudaError_t launch_fused_tma_norm(const LaunchShape& sh, const StepParams& p, cudaStream_t stream);

cudaError_t launch_fused_tma(const LaunchShape& sh, const StepParams& p, cudaStream_t stream) {
    switch (sh.code) {
        case CODE_SIGN: case CODE_U1: case CODE_U2: return launch_fused_tma_sign_u1_u2(sh, p, stream);
        case CODE_U4: case CODE_U8: case CODE_ID32: return launch_fused_tma_u4_u8_id(sh, p, stream);
        case CODE_N2: case CODE_N4: return launch_fused_tma_norm(sh, p, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace ds
