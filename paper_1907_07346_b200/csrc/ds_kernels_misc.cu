// Mix kernel of the two-kernel path, the per-node scale finaliser and the
// random-stream diagnostic kernel.
#include <algorithm>

#include "ds_fused_tma_kernel.cuh"

namespace ds {

// ---------------------------------------------------------------------------
// Local update of Algorithm 1 from codes in global memory:
//   x'_ik = fma(eta, sum_{j in N(i)} fma(w'_ij, C_jk, .), h_ik),  h = x - gamma g
// was left in x by the compress kernel.  One thread owns four consecutive
// elements of one node; a neighbour's four codes are one piece of a code word.
// ---------------------------------------------------------------------------
template <int CODE>
__global__ void __launch_bounds__(256) ds_mix_kernel(const __grid_constant__ StepParams p) {
    using T = CodeTraits<CODE>;
    __shared__ float lut[256];
    if constexpr (T::kLut) {
        for (int t = threadIdx.x; t < (1 << T::kBits); t += blockDim.x) lut[t] = p.lut[t];
        __syncthreads();
    }
    const int node = blockIdx.y;
    // this launch covers the tiles [tile_begin, tile_end): float4 indices [f_begin, f_end)
    const int64_t f_begin = (p.tile_begin * p.tile) >> 2;
    const int64_t nf4 = min((p.N + 3) >> 2, (p.tile_end * p.tile) >> 2);
    const int e_beg = p.row_ptr[node], e_end = p.row_ptr[node + 1];
    for (int64_t f = f_begin + (int64_t)blockIdx.x * blockDim.x + threadIdx.x; f < nf4;
         f += (int64_t)gridDim.x * blockDim.x) {
        const int64_t k = 4 * f;
        const int nv = (int)min((int64_t)4, p.N - k);
        const int64_t tile_idx = p.prescaled ? 0 : k / p.tile;
        if (DS_CHECKED_BUILD && !ds_part_ok(p, node, k, nv, T::kBits, T::kIdentity ? -1 : tile_idx)) continue;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        for (int e = e_beg; e < e_end; ++e) {
            const int j = p.col_idx[e];
            const float w = p.wprime[e];
            const uint32_t* cj = p.codes + (size_t)j * (size_t)p.code_pitch;
            if constexpr (T::kIdentity) {
                const float* cf = reinterpret_cast<const float*>(cj) + k;
#pragma unroll
                for (int t = 0; t < 4; ++t)
                    if (t < nv) acc[t] = __fmaf_rn(w, cf[t], acc[t]);
            } else {
                const float sj = p.dscales[(size_t)j * (size_t)p.scales_pitch + (size_t)tile_idx];
                const uint32_t word = cj[f / T::kLanesPerWord];
                const uint32_t piece = (word >> ((4 * T::kBits * (int)(f % T::kLanesPerWord)) & 31)) & T::kPieceMask;
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    float cv;
                    if constexpr (T::kSign) {
                        const uint32_t neg = ((~piece >> t) & 1u) << 31;
                        cv = __uint_as_float(__float_as_uint(sj) ^ neg);
                    } else {
                        const uint32_t q = (piece >> (T::kBits * t)) & ((1u << (T::kBits & 31)) - 1u);
                        cv = __fmul_rn(sj, lut[q]);
                    }
                    acc[t] = __fmaf_rn(w, cv, acc[t]);
                }
            }
        }
        float* xp = p.x + (size_t)node * (size_t)p.ld + (size_t)k;
        if (nv == 4) {
            const float4 h = *reinterpret_cast<const float4*>(xp);
            *reinterpret_cast<float4*>(xp) =
                make_float4(__fmaf_rn(p.eta, acc[0], h.x), __fmaf_rn(p.eta, acc[1], h.y),
                            __fmaf_rn(p.eta, acc[2], h.z), __fmaf_rn(p.eta, acc[3], h.w));
        } else {
            for (int t = 0; t < nv; ++t) xp[t] = __fmaf_rn(p.eta, acc[t], xp[t]);
        }
    }
}

cudaError_t launch_mix_kernel(const StepParams& p, int code, cudaStream_t stream) {
    const int64_t nf4 = std::min<int64_t>((p.N + 3) >> 2, (p.tile_end * p.tile) >> 2) - ((p.tile_begin * p.tile) >> 2);
    const int threads = 256;
    int64_t bx = std::max<int64_t>(1, (nf4 + threads - 1) / threads);
    if (bx > 148 * 64) bx = 148 * 64;
    const dim3 grid((unsigned)bx, (unsigned)p.n);
    switch (code) {
        case CODE_SIGN: ds_mix_kernel<CODE_SIGN><<<grid, threads, 0, stream>>>(p); break;
        case CODE_U1: ds_mix_kernel<CODE_U1><<<grid, threads, 0, stream>>>(p); break;
        case CODE_U2: ds_mix_kernel<CODE_U2><<<grid, threads, 0, stream>>>(p); break;
        case CODE_U4: ds_mix_kernel<CODE_U4><<<grid, threads, 0, stream>>>(p); break;
        case CODE_U8: ds_mix_kernel<CODE_U8><<<grid, threads, 0, stream>>>(p); break;
        case CODE_ID32: ds_mix_kernel<CODE_ID32><<<grid, threads, 0, stream>>>(p); break;
        case CODE_N2: ds_mix_kernel<CODE_N2><<<grid, threads, 0, stream>>>(p); break;
        case CODE_N4: ds_mix_kernel<CODE_N4><<<grid, threads, 0, stream>>>(p); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Per-node scale: combine the per-tile partials of one node in a fixed order
// (lane-strided binary64 sums, then a butterfly), apply the scale rule.
// One warp per node.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(32) ds_finalize_scales_kernel(const __grid_constant__ StepParams p,
                                                                const int sign, float* const out,
                                                                const int64_t out_pitch) {
    const int node = blockIdx.x;
    const int lane = threadIdx.x;
    const double* part = p.partials + (size_t)node * (size_t)p.tiles;
    if (DS_CHECKED_BUILD && !ds_partial_ok(p, node, p.n, p.tiles - 1)) return;
    double acc = 0.0;
    for (int64_t t = lane; t < p.tiles; t += 32) acc = sign ? acc + part[t] : fmax(acc, part[t]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const double other = __shfl_xor_sync(0xffffffffu, acc, o);
        acc = sign ? acc + other : fmax(acc, other);
    }
    if (lane == 0) {
        float s;
        if (sign) {
            s = (float)(acc / (double)p.N);
        } else {
            s = (float)acc;
            if (s == 0.0f || !(fabsf(s) <= 3.402823466e+38f)) s = 0.0f;
        }
        out[(size_t)node * (size_t)out_pitch] = s;
    }
}

cudaError_t launch_finalize_scales(const StepParams& p, int code, cudaStream_t stream) {
    // norm-matched codes: this maximum only spans the grid; it goes to gmax, the norms follow
    const bool norm = (code == CODE_N2 || code == CODE_N4);
    ds_finalize_scales_kernel<<<p.n, 32, 0, stream>>>(p, code == CODE_SIGN ? 1 : 0, norm ? p.gmax : p.scales,
                                                      norm ? 1 : p.scales_pitch);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Norm-matched codes, one norm per node (Section 5, "Compression": b bits per
// element plus the Euclidean norm of the tensor): combine the per-tile sums of
// v^2 (first half of the partials) and of level^2 (second half) of one node in
// the same fixed order as above; write the norm that is sent and the factor
// norm / ||levels|| the receivers apply.  One warp per node.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(32) ds_finalize_norms_kernel(const __grid_constant__ StepParams p) {
    const int node = blockIdx.x;
    const int lane = threadIdx.x;
    const double* pv = p.partials + (size_t)node * (size_t)p.tiles;
    const double* pl = p.partials + ((size_t)p.n + (size_t)node) * (size_t)p.tiles;
    if (DS_CHECKED_BUILD && !ds_partial_ok(p, (int64_t)p.n + node, 2 * (int64_t)p.n, p.tiles - 1)) return;
    double sv2 = 0.0, sl2 = 0.0;
    for (int64_t t = lane; t < p.tiles; t += 32) { sv2 += pv[t]; sl2 += pl[t]; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        sv2 += __shfl_xor_sync(0xffffffffu, sv2, o);
        sl2 += __shfl_xor_sync(0xffffffffu, sl2, o);
    }
    if (lane == 0) {
        float nrm, r;
        norm_finish(p.gmax[node], sv2, sl2, nrm, r);
        p.scales[(size_t)node * (size_t)p.scales_pitch] = nrm;
        p.dscales[(size_t)node * (size_t)p.scales_pitch] = r;
    }
}

cudaError_t launch_finalize_norms(const StepParams& p, cudaStream_t stream) {
    ds_finalize_norms_kernel<<<p.n, 32, 0, stream>>>(p);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Diagnostics: the random streams, one value per element.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256) ds_noise_kernel(float* out, int32_t n, int64_t N, int64_t ld,
                                                       int which, int noise, RngStep rs) {
    const int node = blockIdx.y;
    const int64_t nf4 = (N + 3) >> 2;
    for (int64_t f = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; f < nf4;
         f += (int64_t)gridDim.x * blockDim.x) {
        const uint32_t k = (uint32_t)(4 * f);
        float4 z;
        if (which == 1) z = rnd24x4(rs, (uint32_t)node, k);
        else if (noise == NOISE_GAUSS) z = noise4<NOISE_GAUSS>(rs, (uint32_t)node, k);
        else if (noise == NOISE_T3) z = noise4<NOISE_T3>(rs, (uint32_t)node, k);
        else if (noise == NOISE_T3I) z = noise4<NOISE_T3I>(rs, (uint32_t)node, k);
        else z = make_float4(0.f, 0.f, 0.f, 0.f);
        const float zv[4] = {z.x, z.y, z.z, z.w};
        float* o = out + (size_t)node * (size_t)ld + (size_t)(4 * f);
        for (int t = 0; t < 4; ++t)
            if (4 * f + t < N) o[t] = zv[t];
    }
}

cudaError_t launch_noise_kernel(float* out, int32_t n, int64_t N, int64_t ld, int which, int noise,
                                RngStep rs, cudaStream_t stream) {
    const int64_t nf4 = (N + 3) >> 2;
    int64_t bx = (nf4 + 255) / 256;
    if (bx > 148 * 32) bx = 148 * 32;
    ds_noise_kernel<<<dim3((unsigned)bx, (unsigned)n), 256, 0, stream>>>(out, n, N, ld, which, noise, rs);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Self-test of the bounded wait: one warp waits, for at most 20 ms, on an
// mbarrier that nothing ever completes, gives up, and raises the error flag --
// the same give-up path the fused kernel takes when a bulk copy does not
// arrive.  The kernel always terminates.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(32) ds_wait_selftest_kernel(int* error_flag) {
    __shared__ __align__(8) unsigned long long bar_storage;
    const uint32_t bar = smem_u32(&bar_storage);
    if (threadIdx.x == 0) mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncwarp();
    const bool done = mbar_wait_bounded(bar, 0u, 20000000ull);      // 20 ms
    if (!done && threadIdx.x == 0) *error_flag = 1;
}

// ---------------------------------------------------------------------------
// Self-test of the arithmetic shortcuts on every possible argument: the packed
// branch-free logarithm against the scalar compare-and-halve form, and the
// one-correction square root against sqrt.rn.f32, for all j = 1 .. 2^24.
// counts[0] += mismatching logarithms, counts[1] += mismatching roots,
// counts[2] += mismatching roots of the Student-t(3) squared radii.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256) ds_math_selftest_kernel(unsigned long long* counts) {
    unsigned bad_log = 0, bad_sqrt = 0, bad_t3 = 0;
    for (uint32_t j = 1u + blockIdx.x * blockDim.x + threadIdx.x; j <= (1u << 24); j += gridDim.x * blockDim.x) {
        const uint32_t j2 = (j == (1u << 24)) ? 1u : j + 1u;
        const float2 lg = log_u24_x2(j, j2);
        if (__float_as_uint(lg.x) != __float_as_uint(log_u24(j))) ++bad_log;
        if (__float_as_uint(lg.y) != __float_as_uint(log_u24(j2))) ++bad_log;
        const float t = __fmul_rn(-2.0f, lg.x);
        if (__float_as_uint(sqrt_of_minus2log(t)) != __float_as_uint(__fsqrt_rn(t))) ++bad_sqrt;
        const float2 q = t3_radius_sq_x2(j, j2);
        if (__float_as_uint(sqrt_of_minus2log(q.x)) != __float_as_uint(__fsqrt_rn(q.x))) ++bad_t3;
    }
    if (bad_log) atomicAdd(&counts[0], (unsigned long long)bad_log);
    if (bad_sqrt) atomicAdd(&counts[1], (unsigned long long)bad_sqrt);
    if (bad_t3) atomicAdd(&counts[2], (unsigned long long)bad_t3);
}

cudaError_t launch_math_selftest(unsigned long long* counts, cudaStream_t stream) {
    ds_math_selftest_kernel<<<148 * 8, 256, 0, stream>>>(counts);
    return cudaGetLastError();
}

// Self-test of the checked build: asks the checker about a part that starts in the row
// after the last one.  It must refuse it (and raise the flag); nothing is accessed.
__global__ void __launch_bounds__(32) ds_bounds_selftest_kernel(const __grid_constant__ StepParams p) {
    if (threadIdx.x == 0) (void)ds_part_ok(p, p.n, 0, 4, 1, -1);
}

cudaError_t launch_bounds_selftest(const StepParams& p, cudaStream_t stream) {
    ds_bounds_selftest_kernel<<<1, 32, 0, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_wait_selftest(int* error_flag, cudaStream_t stream) {
    ds_wait_selftest_kernel<<<1, 32, 0, stream>>>(error_flag);
    return cudaGetLastError();
}

}  // namespace ds
