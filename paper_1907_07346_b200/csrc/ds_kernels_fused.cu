// Instantiations of the column kernel in fused mode (compress + mix in one launch).
#include "ds_column_kernel.cuh"

namespace ds {

cudaError_t launch_column_fused(const LaunchShape& sh, const StepParams& p, cudaStream_t stream) {
    switch (sh.code) {
        case CODE_SIGN: return launch_code<CODE_SIGN, MODE_FUSED>(sh, p, stream);
        case CODE_U1: return launch_code<CODE_U1, MODE_FUSED>(sh, p, stream);
        case CODE_U2: return launch_code<CODE_U2, MODE_FUSED>(sh, p, stream);
        case CODE_U4: return launch_code<CODE_U4, MODE_FUSED>(sh, p, stream);
        case CODE_U8: return launch_code<CODE_U8, MODE_FUSED>(sh, p, stream);
        case CODE_N2: return launch_code<CODE_N2, MODE_FUSED>(sh, p, stream);
        case CODE_N4: return launch_code<CODE_N4, MODE_FUSED>(sh, p, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace ds
