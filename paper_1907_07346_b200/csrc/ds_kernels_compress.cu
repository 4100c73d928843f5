// Instantiations of the column kernel in compress-only mode (first kernel of
// the two-kernel path) and in reduce-only mode (per-node scale).
#include "ds_column_kernel.cuh"

namespace ds {

cudaError_t launch_column_compress(const LaunchShape& sh, const StepParams& p, cudaStream_t stream) {
    switch (sh.code) {
        case CODE_SIGN: return launch_code<CODE_SIGN, MODE_COMPRESS>(sh, p, stream);
        case CODE_U1: return launch_code<CODE_U1, MODE_COMPRESS>(sh, p, stream);
        case CODE_U2: return launch_code<CODE_U2, MODE_COMPRESS>(sh, p, stream);
        case CODE_U4: return launch_code<CODE_U4, MODE_COMPRESS>(sh, p, stream);
        case CODE_U8: return launch_code<CODE_U8, MODE_COMPRESS>(sh, p, stream);
        case CODE_ID32: return launch_code<CODE_ID32, MODE_COMPRESS>(sh, p, stream);
        case CODE_N2: return launch_code<CODE_N2, MODE_COMPRESS>(sh, p, stream);
        case CODE_N4: return launch_code<CODE_N4, MODE_COMPRESS>(sh, p, stream);
        default: return cudaErrorInvalidValue;
    }
}

cudaError_t launch_column_reduce(const LaunchShape& sh, const StepParams& p, cudaStream_t stream) {
    // The partial only depends on whether the scale is an l1 mean or a maximum.
    if (sh.code == CODE_SIGN) return launch_code<CODE_SIGN, MODE_REDUCE>(sh, p, stream);
    return launch_code<CODE_U4, MODE_REDUCE>(sh, p, stream);
}

}  // namespace ds
