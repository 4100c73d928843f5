// Instantiations of the persistent TMA-staged fused kernel: 4-bit and 8-bit codes, identity.
#include "ds_fused_tma_kernel.cuh"

namespace ds {

cudaError_t launch_fused_tma_u4_u8_id(const LaunchShape& sh, const StepParams& p, cudaStream_t stream) {
    switch (sh.code) {
        case CODE_U4: return launch_tma_code<CODE_U4>(sh, p, stream);
        case CODE_U8: return launch_tma_code<CODE_U8>(sh, p, stream);
        case CODE_ID32: return launch_tma_code<CODE_ID32>(sh, p, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace ds
