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
    int* error_flag;          // DS_FLAG_* bits: a bounded wait ran out; the checked build refused an index
    float sigma;
    float neg_gamma;
    float eta;
    RngStep rs;
    int32_t warps_per_group;  // warps sharing one (node, tile)
    int32_t nodes_per_block;
    int32_t l2_hints;         // batch-sweeping TMA kernel: bit 0 = inputs evict-first, bit 1 = parked values evict-last
    int32_t prescaled;        // 1: scale of node i is scales[i][0], computed by an earlier launch
    int32_t norm_phase;       // reduce mode, norm-matched codes, one norm per node: 0 = maximum, 2 = sums of squares
    int32_t ecsgd;            // 1 (compress / reduce modes only): centralized error-compensated SGD,
                              // v = g + delta is compressed and x is left for the server's update
};

// Values of the error flag (bits): a bounded wait ran out / the checked build
// refused an out-of-range index.
enum : int { DS_FLAG_TIMEOUT = 1, DS_FLAG_BOUNDS = 2 };

// Checked build (-DDS_DEBUG): before a warp touches its part of a row, the index
// arithmetic behind every access of that part is validated here; a part that
// does not lie inside the row, its code words and its scale slot is NOT
// processed, and the error flag records it (ds_sync then returns
// DS_ERR_BOUNDS).  Nothing traps.  In the normal build this is `true` and
// the compiler removes the call.
//   node       row
//   k_first    first element of the part within the row
//   count      elements of the part that are read and written (the staging
//              copies read count rounded up to 4: padding columns up to ld)
//   code_bits  bits per packed code
//   scale_col  index of the scale the part writes within the row's scales, -1 = none
#ifdef DS_DEBUG
#define DS_CHECKED_BUILD 1
#else
#define DS_CHECKED_BUILD 0
#endif
__device__ __forceinline__ bool ds_part_ok(const StepParams& p, int64_t node, int64_t k_first, int64_t count,
                                           int code_bits, int64_t scale_col) {
#if DS_CHECKED_BUILD
    bool ok = node >= 0 && node < p.n && k_first >= 0 && count >= 0;
    ok = ok && (k_first & 3) == 0;                                   // 128-bit accesses
    ok = ok && k_first + count <= p.N && k_first + ((count + 3) & ~(int64_t)3) <= p.ld;
    ok = ok && (((k_first + count) * code_bits + 31) >> 5) <= p.code_pitch;
    ok = ok && scale_col < p.scales_pitch;
    if (!ok && p.error_flag != nullptr) atomicOr(p.error_flag, (int)DS_FLAG_BOUNDS);
    return ok;
#else
    (void)p; (void)node; (void)k_first; (void)count; (void)code_bits; (void)scale_col;
    return true;
#endif
}
// The same for one slot of the per-(node, tile) partials (`rows` rows of p.tiles slots).
__device__ __forceinline__ bool ds_partial_ok(const StepParams& p, int64_t row, int64_t rows, int64_t col) {
#if DS_CHECKED_BUILD
    const bool ok = row >= 0 && row < rows && col >= 0 && col < p.tiles;
    if (!ok && p.error_flag != nullptr) atomicOr(p.error_flag, (int)DS_FLAG_BOUNDS);
    return ok;
#else
    (void)p; (void)row; (void)rows; (void)col;
    return true;
#endif
}

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
cudaError_t launch_bounds_selftest(const StepParams& p, cudaStream_t stream);
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
