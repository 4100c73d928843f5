// Instantiations of the column kernel in reduce-only mode for norm-matched codes
// with one norm per node: the per-(node, tile) sums of v^2 and of level^2, taken
// once the maximum that spans the grid is known.
#include "ds_column_kernel.cuh"

namespace ds {

cudaError_t launch_column_reduce_norm(const LaunchShape& sh, const StepParams& p, cudaStream_t stream) {
    switch (sh.code) {
        case CODE_N2: return launch_code<CODE_N2, MODE_REDUCE>(sh, p, stream);
        case CODE_N4: return launch_code<CODE_N4, MODE_REDUCE>(sh, p, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace ds
