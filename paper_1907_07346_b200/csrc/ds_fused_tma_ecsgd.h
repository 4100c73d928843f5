// Launcher of the fused kernel for centralized error-compensated SGD
// (defined in ds_kernels_tma_ecsgd.cu): 16 elements per lane, blocks of up to
// 512 threads; cudaErrorInvalidValue for other launch shapes.
#pragma once

#include "ds_internal.h"

namespace ds {
cudaError_t launch_fused_tma_ecsgd(const LaunchShape& shape, const StepParams& p, cudaStream_t stream);
}
