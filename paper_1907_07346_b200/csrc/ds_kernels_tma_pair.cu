// Instantiations of the persistent TMA-staged fused kernel with two nodes per warp.
#include "ds_fused_tma_pair_kernel.cuh"

namespace ds {

template <int CODE, int NOISE>
static cudaError_t launch_pair_one(const LaunchShape& sh, const StepParams& p, cudaStream_t stream) {
    auto kern = ds_fused_tma_pair_kernel<CODE, NOISE>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh.smem);
    if (e != cudaSuccess) return e;
    kern<<<sh.grid, sh.block, sh.smem, stream>>>(p);
    return cudaGetLastError();
}

template <int CODE>
static cudaError_t launch_pair_code(const LaunchShape& sh, const StepParams& p, cudaStream_t stream) {
    switch (sh.noise) {
        case NOISE_NONE: return launch_pair_one<CODE, NOISE_NONE>(sh, p, stream);
        case NOISE_GAUSS: return launch_pair_one<CODE, NOISE_GAUSS>(sh, p, stream);
        case NOISE_T3: return launch_pair_one<CODE, NOISE_T3>(sh, p, stream);
        default: return cudaErrorInvalidValue;
    }
}

cudaError_t launch_fused_tma_pair(const LaunchShape& sh, const StepParams& p, cudaStream_t stream) {
    switch (sh.code) {
        case CODE_SIGN: return launch_pair_code<CODE_SIGN>(sh, p, stream);
        case CODE_U1: return launch_pair_code<CODE_U1>(sh, p, stream);
        case CODE_U2: return launch_pair_code<CODE_U2>(sh, p, stream);
        case CODE_U4: return launch_pair_code<CODE_U4>(sh, p, stream);
        case CODE_U8: return launch_pair_code<CODE_U8>(sh, p, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace ds
