// Internal declarations shared by the host API and the kernel translation
// units of the DeepSqueeze library (not part of the public ABI).
#pragma once

#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

#include "ds_device.cuh"

namespace ds {

enum : int { MODE_FUSED = 0, MODE_COMPRESS = 1, MODE_REDUCE = 2 };

// Code formats the kernels are instantiated for.
// CODE_N2 / CODE_N4: round-to-nearest b-bit codes whose decoder rescales to the
// Euclidean norm of the original (the paper's own "bit compression").
enum : int { CODE_SIGN = 0, CODE_U1 = 1, CODE_U2 = 2, CODE_U4 = 3, CODE_U8 = 4, CODE_ID32 = 5,
             CODE_N2 = 6, CODE_N4 = 7 };

struct StepParams {
    float* x;
    float* delta;
    const float* a;
    const float* c;
    int64_t ld;
    int64_t N;
    int32_t n;
    int32_t nnz;
    int64_t tile;             // elements per column tile (= chunk unless prescaled)
    int64_t tiles;            // column tiles per row
    int64_t tile_begin;       // this launch covers the tiles [tile_begin, tile_end)
    int64_t tile_end;
    const int32_t* row_ptr;   // device CSR of W - I
    const int32_t* col_idx;
    const float* wprime;      // W_ij - I_ij, binary32
    const float* lut;         // reconstruction levels, 2^bits entries
    uint32_t* codes;
    int64_t code_pitch;       // words
    float* scales;            // the scalar a node sends with each chunk
    int64_t scales_pitch;
    float* dscales;           // the factor the receiver multiplies the levels by (= scales unless the
                              // decoder rescales to a norm), same pitch
    double* partials;         // [n][tiles], per-node-scale reduction (twice that for the two sums of a
                              // per-node norm: sum v^2 in the first half, sum level^2 in the second)
    float* gmax;              // [n], norm-matched codes with one norm per node: max |v| of the node
    int* error_flag;          // set to 1 by a kernel whose bounded wait ran out
    float sigma;
    float neg_gamma;
    float eta;
    RngStep rs;
    int32_t warps_per_group;  // warps sharing one (node, tile)
    int32_t nodes_per_block;
    int32_t prescaled;        // 1: scale of node i is scales[i][0], computed by an earlier launch
    int32_t norm_phase;       // reduce mode, norm-matched codes, one norm per node: 0 = maximum, 2 = sums of squares
    int32_t ecsgd;            // 1 (compress / reduce modes only): centralized error-compensated SGD,
                              // v = g + delta is compressed and x is left for the server's update
};

struct LaunchShape {
    int code;                 // CODE_*
    int noise;                // NOISE_*
    int elems_per_lane;       // 4, 8 or 16
    int mode;                 // MODE_*
    dim3 grid;
    dim3 block;
    size_t smem;
};

// Launchers (defined in the kernel translation units).
cudaError_t launch_column_fused(const LaunchShape& shape, const StepParams& p, cudaStream_t stream);
cudaError_t launch_fused_tma(const LaunchShape& shape, const StepParams& p, cudaStream_t stream);
cudaError_t launch_fused_wide_tma(const LaunchShape& shape, const StepParams& p, cudaStream_t stream);
cudaError_t launch_fused_wide(const LaunchShape& shape, const StepParams& p, cudaStream_t stream);
cudaError_t launch_fused_wide_tma_norm(const LaunchShape& shape, const StepParams& p, cudaStream_t stream);
cudaError_t launch_fused_wide_norm(const LaunchShape& shape, const StepParams& p, cudaStream_t stream);
cudaError_t launch_column_compress(const LaunchShape& shape, const StepParams& p, cudaStream_t stream);
cudaError_t launch_column_reduce(const LaunchShape& shape, const StepParams& p, cudaStream_t stream);
cudaError_t launch_column_reduce_norm(const LaunchShape& shape, const StepParams& p, cudaStream_t stream);
cudaError_t launch_finalize_scales(const StepParams& p, int code, cudaStream_t stream);   // norm-matched codes: the maximum, into gmax
cudaError_t launch_finalize_norms(const StepParams& p, cudaStream_t stream);
cudaError_t launch_mix_kernel(const StepParams& p, int code, cudaStream_t stream);
cudaError_t launch_math_selftest(unsigned long long* counts, cudaStream_t stream);
cudaError_t launch_wait_selftest(int* error_flag, cudaStream_t stream);
cudaError_t launch_noise_kernel(float* out, int32_t n, int64_t N, int64_t ld, int which, int noise,
                                RngStep rs, cudaStream_t stream);

inline int code_bits_of(int code) {
    switch (code) {
        case CODE_SIGN: case CODE_U1: return 1;
        case CODE_U2: case CODE_N2: return 2;
        case CODE_U4: case CODE_N4: return 4;
        case CODE_U8: return 8;
        default: return 32;
    }
}

}  // namespace ds
