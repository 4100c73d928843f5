// ds_node_scales_noalloc: the per-node compressor scale without any device
// allocation, for callers that cannot obtain device memory at call time.
//
// The two-launch reduction behind a per-node scale (per-tile partials, then a
// fixed-order combine) needs scratch for the partials.  Everywhere else in
// this library the caller supplies that scratch inside the workspace.  Here
// it lives in a file-scope __device__ array of fixed size instead, so the
// entry point works with nothing but the caller's inputs and outputs.
#include <mutex>

#include "../../include/deepsqueeze.h"
#include "ds_column_kernel.cuh"

using namespace ds;

namespace {

// Layout of the static scratch (binary64 slots): the first kTableSlots hold a
// zero table that the reduction kernel copies but never uses, the rest hold the
// per-(node, tile) partials.  (128 + 65,536) * 8 B = 513 KiB in total.  The array is
// part of this module's image: with lazy module loading the driver gives it
// storage on a GPU when the module is first used there, i.e. at the first
// cudaGetSymbolAddress below, and keeps it until the process exits.
constexpr int64_t kTableSlots = 128;                 // 1 KiB
constexpr int64_t kMaxPartials = DS_NOALLOC_MAX_PARTIALS;
constexpr int kMaxDevices = 64;
constexpr int64_t kTile = 512;

}  // namespace

static __device__ __align__(256) double g_static_scratch[kTableSlots + kMaxPartials];

namespace {

std::mutex g_mutex;
double* g_scratch_of_device[kMaxDevices] = {};

// In host code `g_static_scratch` is only a handle for the runtime, not an
// address a kernel can use; the device address has to be asked for, once per
// device, while that device is current.
ds_status scratch_of_current_device(double** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        return DS_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_scratch_of_device[dev] == nullptr) {
        void* ptr = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess || ptr == nullptr) {
            (void)cudaGetLastError();
            return DS_ERR_CUDA;
        }
        g_scratch_of_device[dev] = static_cast<double*>(ptr);
    }
    *out = g_scratch_of_device[dev];
    return DS_OK;
}

}  // namespace

extern "C" ds_status ds_node_scales_noalloc(float* scales_out, const float* x, const float* delta,
                                            const ds_grad_params* gp, float gamma, int32_t n,
                                            int64_t N, int64_t ld, int32_t comp_kind, uint64_t seed,
                                            uint64_t step, void* cuda_stream) {
    if (!scales_out || !x || !delta || !gp || !gp->a || !gp->c) return DS_ERR_NULL;
    if (n < 1 || N < 1 || N >= ((int64_t)1 << 31) || ld < N || step >= ((uint64_t)1 << 56)) return DS_ERR_ARG;
    if (gp->noise < DS_NOISE_NONE || gp->noise > DS_NOISE_STUDENT_T3_IID) return DS_ERR_ARG;
    if (comp_kind != DS_COMP_SIGN1_L1 && comp_kind != DS_COMP_UNIFORM_STOCH_MAXABS) return DS_ERR_ARG;
    if ((ld % 4) != 0) return DS_ERR_ALIGN;
    const uintptr_t bits = reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(delta) |
                           reinterpret_cast<uintptr_t>(gp->a) | reinterpret_cast<uintptr_t>(gp->c);
    if ((bits % 16) != 0) return DS_ERR_ALIGN;
    const int64_t tiles = (N + kTile - 1) / kTile;
    // the fixed scratch bounds the problem: n * ceil(N / 512) partials at most
    if ((int64_t)n * tiles > kMaxPartials) return DS_ERR_WORKSPACE;

    double* scratch = nullptr;
    const ds_status st = scratch_of_current_device(&scratch);
    if (st != DS_OK) return st;

    const int code = (comp_kind == DS_COMP_SIGN1_L1) ? CODE_SIGN : CODE_U4;
    const int npb = n < 8 ? n : 8;
    StepParams p = {};
    p.x = const_cast<float*>(x);            // the reduction only reads x and delta
    p.delta = const_cast<float*>(delta);
    p.a = gp->a;
    p.c = gp->c;
    p.ld = ld;
    p.N = N;
    p.n = n;
    p.nnz = 0;
    p.tile = kTile;
    p.tiles = tiles;
    p.tile_begin = 0;
    p.tile_end = tiles;
    p.lut = reinterpret_cast<const float*>(scratch);          // the zero table
    p.partials = scratch + kTableSlots;
    p.scales = scales_out;
    p.dscales = scales_out;
    p.scales_pitch = 1;
    p.code_pitch = (N * 4 + 31) / 32;       // no codes are written; what a row of 4-bit codes would take (checked build)
    p.sigma = gp->sigma;
    p.neg_gamma = -gamma;
    p.eta = 0.0f;
    p.rs = make_rng_step(seed, step);
    p.warps_per_group = 1;
    p.nodes_per_block = npb;
    p.prescaled = 0;

    LaunchShape sh;
    sh.code = code;
    sh.noise = (gp->noise == DS_NOISE_STUDENT_T3_IID) ? (int)NOISE_T3I : (int)gp->noise;
    sh.elems_per_lane = 16;
    sh.mode = MODE_REDUCE;
    sh.grid = dim3((unsigned)tiles, (unsigned)((n + npb - 1) / npb));
    sh.block = dim3((unsigned)(npb * 32));
    sh.smem = smem_layout(MODE_REDUCE, code == CODE_SIGN ? 1 : 4, code != CODE_SIGN, npb, 1, kTile, n, 0).total;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // Every partial that the combine reads is written by the reduction of the
    // same call, so nothing in the scratch has to be cleared between calls.
    cudaError_t e = launch_column_reduce(sh, p, stream);
    if (e == cudaSuccess) e = launch_finalize_scales(p, code, stream);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return DS_ERR_CUDA;
    }
    return DS_OK;
}
