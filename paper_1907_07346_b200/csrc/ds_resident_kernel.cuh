// Resident multi-step kernel for small problems: T consecutive iterations of
// Algorithm 1 in ONE launch, with the state on chip between iterations.
//
// Column tiles of 512 elements are independent of one another except for the
// reduction behind a per-node scale, so a thread block can own one tile of all
// n nodes for the whole run: warp i keeps its 512 elements of x_i and delta_i
// in registers, a_i and c_i in shared memory, and global memory is touched at
// the start (load), at the end (store) and for what the nodes "send" (packed
// codes and scales of every iteration).  Per iteration and warp:
//   local step with the noise drawn one iteration ahead; scale (per chunk: a
//   warp reduction; per node: the tile's partial goes to global memory, the
//   block ARRIVES at the one grid-wide barrier of the iteration, draws this
//   iteration's rounding uniforms and the next iteration's noise -- neither
//   depends on the scale -- with their Philox blocks in lockstep, and only then
//   waits; every block combines the partials of all tiles in the fixed order of
//   the per-node finaliser); compression and residual, C[v] to shared memory,
//   block barrier, local update from the neighbours' C[v], block barrier.
// The learning-rate schedule (gamma_t, eta_t) travels in the kernel parameters.
//
// The grid barrier is an arrival counter in the workspace; blocks are
// co-resident because the launch is cooperative.  Its wait is bounded (2 s):
// a block that gives up raises the workspace error flag, and every block
// leaves without storing x and delta.
#pragma once

#include "ds_fused_tma_kernel.cuh"

namespace ds {

constexpr int kResidentMaxSteps = 1024;
constexpr int kResidentTile = 512;
constexpr int kResidentMaxNodes = 16;

struct ResidentParams {
    StepParams p;                         // arrays, graph, tables; gamma, eta and the step fields of rs are unused
    double* partials2;                    // [2][n][tiles], per-node scale only
    unsigned int* barrier;                // arrival counter, zero at launch
    uint64_t step0;
    int32_t T;
    float gammas[kResidentMaxSteps];
    float etas[kResidentMaxSteps];
};

struct ResidentSmemLayout {
    uint32_t ac_off, cval_off, lut_off, rowptr_off, col_off, w_off, flag_off, total;
};

__host__ __device__ inline ResidentSmemLayout resident_smem_layout(int n, int nnz) {
    ResidentSmemLayout L;
    uint32_t off = 0;
    L.ac_off = off;      off += (uint32_t)n * 2u * kResidentTile * 4u;
    L.cval_off = off;    off += (uint32_t)n * kResidentTile * 4u;
    L.lut_off = off;     off += 256u * 4u;
    L.rowptr_off = off;  off += (uint32_t)(n + 1) * 4u;
    L.col_off = off;     off += (uint32_t)nnz * 4u;
    L.w_off = off;       off += (uint32_t)nnz * 4u;
    L.flag_off = off;    off += 16u;
    L.total = (off + 15u) & ~15u;
    return L;
}

__device__ __forceinline__ unsigned int ld_acquire_gpu(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

template <int CODE, int NOISE, int MAXT>
__global__ void __launch_bounds__(MAXT, 1) ds_resident_kernel(const __grid_constant__ ResidentParams rp) {
    using T = CodeTraits<CODE>;
    static_assert(!T::kIdentity && !T::kNorm, "sign and stochastic b-bit codes only");
    constexpr int E = 16, V = 4, SEG = kResidentTile;
    const StepParams& p = rp.p;
    extern __shared__ __align__(128) unsigned char smem[];
    const ResidentSmemLayout L = resident_smem_layout(p.n, p.nnz);
    const int lane = threadIdx.x & 31;
    const int node = threadIdx.x >> 5;                  // one warp per node
    const int64_t col = blockIdx.x;                     // one tile per block
    const int64_t k0 = col * SEG;
    const int64_t remain = p.N - k0;
    int m_len = (int)(remain < SEG ? remain : SEG);
    // checked build: a refused tile is worked on as an empty one (nothing loaded, nothing stored;
    // the block still takes part in the grid barrier)
    bool part_ok = true;
    if (DS_CHECKED_BUILD && !ds_part_ok(p, node, k0, m_len, T::kBits, p.prescaled ? -1 : col)) { part_ok = false; m_len = 0; }

    float* ac = reinterpret_cast<float*>(smem + L.ac_off) + (size_t)node * 2 * SEG;
    float* cval = reinterpret_cast<float*>(smem + L.cval_off);
    float* lut = reinterpret_cast<float*>(smem + L.lut_off);
    int32_t* rptr = reinterpret_cast<int32_t*>(smem + L.rowptr_off);
    int32_t* cj = reinterpret_cast<int32_t*>(smem + L.col_off);
    float* wp = reinterpret_cast<float*>(smem + L.w_off);
    volatile int* flag_sm = reinterpret_cast<volatile int*>(smem + L.flag_off);

    if constexpr (T::kLut)
        for (int t = threadIdx.x; t < (1 << T::kBits); t += blockDim.x) lut[t] = p.lut[t];
    for (int t = threadIdx.x; t <= p.n; t += blockDim.x) rptr[t] = p.row_ptr[t];
    for (int t = threadIdx.x; t < p.nnz; t += blockDim.x) { cj[t] = p.col_idx[t]; wp[t] = p.wprime[t]; }
    if (threadIdx.x == 0) flag_sm[0] = 1;

    // ---- load the tile: x, delta -> registers, a, c -> shared memory ----
    const size_t row = (size_t)node * (size_t)p.ld + (size_t)k0;
    float xr[E], dr[E];
#pragma unroll
    for (int r = 0; r < V; ++r) {
        const int e0 = 4 * (32 * r + lane);
        if (e0 + 3 < m_len) {
            const float4 x4 = ld4(p.x + row + e0), d4 = ld4(p.delta + row + e0);
            xr[4 * r] = x4.x; xr[4 * r + 1] = x4.y; xr[4 * r + 2] = x4.z; xr[4 * r + 3] = x4.w;
            dr[4 * r] = d4.x; dr[4 * r + 1] = d4.y; dr[4 * r + 2] = d4.z; dr[4 * r + 3] = d4.w;
            *reinterpret_cast<float4*>(ac + e0) = ld4(p.a + row + e0);
            *reinterpret_cast<float4*>(ac + SEG + e0) = ld4(p.c + row + e0);
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const bool ok = e0 + j < m_len;
                xr[4 * r + j] = ok ? p.x[row + e0 + j] : 0.0f;
                dr[4 * r + j] = ok ? p.delta[row + e0 + j] : 0.0f;
                ac[e0 + j] = ok ? p.a[row + e0 + j] : 0.0f;
                ac[SEG + e0 + j] = ok ? p.c[row + e0 + j] : 0.0f;
            }
        }
    }
    __syncthreads();

    constexpr float kL = (float)((1u << (T::kBits & 15)) - 1u);
    constexpr float kHalfL = 0.5f * kL;
    constexpr bool kNoise = (NOISE == NOISE_GAUSS || NOISE == NOISE_T3);
    constexpr bool kRnd = T::kLut;
    const uint32_t kbase = (uint32_t)k0 + 4u * (uint32_t)lane;
    bool alive = true;

    // Philox blocks of one node in lockstep, each with its own step and stream
    // (words 2 and 3 of the counter): the rounding uniforms of iteration t are
    // drawn together with the noise of iteration t + 1.
    auto draw = [&](uint64_t step_round, uint64_t step_noise, bool want_noise, float (&zn)[kNoise ? E : 1],
                    float (&mn)[kRnd ? E : 1]) {
        if constexpr (kNoise || kRnd) {
            constexpr int kNz = kNoise ? V : 0;
            constexpr int kRn = kRnd ? V : 0;
            uint32_t c0[kNz + kRn], c1[kNz + kRn], c2[kNz + kRn], c3[kNz + kRn];
#pragma unroll
            for (int r = 0; r < V; ++r) {
                const uint32_t blk = (kbase + 128u * (uint32_t)r) >> 2;
                if constexpr (kNz > 0) {
                    c0[r] = blk; c1[r] = (uint32_t)node; c2[r] = (uint32_t)step_noise;
                    c3[r] = (uint32_t)((step_noise >> 32) << 8) | STREAM_NOISE;
                }
                if constexpr (kRn > 0) {
                    c0[kNz + r] = blk; c1[kNz + r] = (uint32_t)node; c2[kNz + r] = (uint32_t)step_round;
                    c3[kNz + r] = (uint32_t)((step_round >> 32) << 8) | STREAM_ROUND;
                }
            }
#pragma unroll
            for (int q = 0; q < 10; ++q) {
                const uint32_t ka = p.rs.k0[q], kb = p.rs.k1[q];
#pragma unroll
                for (int b = 0; b < kNz + kRn; ++b) {
                    const uint64_t pa = (uint64_t)0xD2511F53u * c0[b];
                    const uint64_t pb = (uint64_t)0xCD9E8D57u * c2[b];
                    const uint32_t n0 = (uint32_t)(pb >> 32) ^ c1[b] ^ ka;
                    const uint32_t n2 = (uint32_t)(pa >> 32) ^ c3[b] ^ kb;
                    c1[b] = (uint32_t)pb;
                    c3[b] = (uint32_t)pa;
                    c0[b] = n0;
                    c2[b] = n2;
                }
            }
#pragma unroll
            for (int r = 0; r < V; ++r) {
                if constexpr (kNz > 0) {
                    if (want_noise) {
                        const float4 z4 = noise_of_block<NOISE>(make_uint4(c0[r], c1[r], c2[r], c3[r]));
                        zn[4 * r + 0] = z4.x; zn[4 * r + 1] = z4.y; zn[4 * r + 2] = z4.z; zn[4 * r + 3] = z4.w;
                    }
                }
                if constexpr (kRn > 0) {
                    mn[4 * r + 0] = __uint2float_rn(c0[kNz + r] >> 8); mn[4 * r + 1] = __uint2float_rn(c1[kNz + r] >> 8);
                    mn[4 * r + 2] = __uint2float_rn(c2[kNz + r] >> 8); mn[4 * r + 3] = __uint2float_rn(c3[kNz + r] >> 8);
                }
            }
        }
    };

    float zn[kNoise ? E : 1], mn[kRnd ? E : 1];
    if constexpr (kNoise) draw(rp.step0, rp.step0, true, zn, mn);       // noise of the first iteration

    for (int t = 0; t < rp.T; ++t) {
        const float neg_gamma = -rp.gammas[t];
        const float eta = rp.etas[t];
        const uint64_t step = rp.step0 + (uint64_t)t;

        // ---- local step, scale partial ----
        float h[E], v[E];
        double sum = 0.0;
        float mx = 0.0f;
#pragma unroll
        for (int r = 0; r < V; ++r) {
            const int e0 = 4 * (32 * r + lane);
            const float4 x4 = make_float4(xr[4 * r], xr[4 * r + 1], xr[4 * r + 2], xr[4 * r + 3]);
            const float4 d4 = make_float4(dr[4 * r], dr[4 * r + 1], dr[4 * r + 2], dr[4 * r + 3]);
            const float4 a4 = *reinterpret_cast<const float4*>(ac + e0);
            const float4 c4 = *reinterpret_cast<const float4*>(ac + SEG + e0);
            float4 z4 = make_float4(0.f, 0.f, 0.f, 0.f);
            if constexpr (kNoise) z4 = make_float4(zn[4 * r + 0], zn[4 * r + 1], zn[4 * r + 2], zn[4 * r + 3]);
            local_step4(x4, d4, a4, c4, z4, p.sigma, neg_gamma, &h[4 * r], &v[4 * r]);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (e0 + j >= m_len) { h[4 * r + j] = 0.0f; v[4 * r + j] = 0.0f; }
                if constexpr (T::kSign) sum += (double)fabsf(v[4 * r + j]);
                else mx = fmaxf(mx, fabsf(v[4 * r + j]));
            }
        }
        double part;
        if constexpr (T::kSign) part = warp_sum(sum);
        else part = (double)__uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(mx)));

        // one scale per node: publish the tile's partial and arrive at the grid barrier ...
        double* mine = rp.partials2 + (size_t)(t & 1) * (size_t)p.n * (size_t)p.tiles;
        if (p.prescaled) {
            if (lane == 0 && part_ok) mine[(size_t)node * (size_t)p.tiles + (size_t)col] = part;
            __syncthreads();
            if (threadIdx.x == 0) {
                __threadfence();
                atomicAdd(rp.barrier, 1u);
            }
        }
        // ... draw what does not depend on the scale while the other blocks arrive:
        // this iteration's rounding uniforms and the next iteration's noise
        draw(step, step + 1u, t + 1 < rp.T, zn, mn);

        float s;
        if (p.prescaled) {
            if (threadIdx.x == 0) {
                const unsigned int target = (unsigned int)(t + 1) * gridDim.x;
                bool ok = ld_acquire_gpu(rp.barrier) >= target;
                if (!ok) {
                    const uint64_t t0 = global_timer_ns();
                    for (uint32_t tries = 0; tries < (1u << 24) && !ok; ++tries) {
                        ok = ld_acquire_gpu(rp.barrier) >= target;
                        if (!ok && global_timer_ns() - t0 > 2000000000ull) break;
                    }
                }
                if (!ok) { flag_sm[0] = 0; *p.error_flag = 1; }
                __threadfence();
            }
            __syncthreads();
            alive = flag_sm[0] != 0;
            if (!alive) break;
            // every block combines the partials of all tiles in the order of the per-node finaliser
            const double* all = mine + (size_t)node * (size_t)p.tiles;
            double acc = 0.0;
            for (int64_t q = lane; q < p.tiles; q += 32) {
                const double other = __ldcg(all + q);
                acc = T::kSign ? acc + other : fmax(acc, other);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const double other = __shfl_xor_sync(0xffffffffu, acc, o);
                acc = T::kSign ? acc + other : fmax(acc, other);
            }
            if constexpr (T::kSign) {
                s = (float)(acc / (double)p.N);
            } else {
                s = (float)acc;
                if (s == 0.0f || !(fabsf(s) <= 3.402823466e+38f)) s = 0.0f;
            }
            if (col == 0 && lane == 0) p.scales[(size_t)node * (size_t)p.scales_pitch] = s;
        } else {
            if constexpr (T::kSign) {
                s = (float)(part / (double)m_len);
            } else {
                s = (float)part;
                if (s == 0.0f || !(fabsf(s) <= 3.402823466e+38f)) s = 0.0f;
            }
            if (lane == 0 && part_ok) p.scales[(size_t)node * (size_t)p.scales_pitch + (size_t)col] = s;
        }

        // ---- compress, residual, pack; C[v] to shared memory ----
        const bool degenerate = (!T::kSign && s == 0.0f);
        const bool fast = T::kLut && s >= 0x1p-60f && s <= 0x1p+60f;
        const float inv_s = fast ? __fdiv_rn(1.0f, s) : 0.0f;
        uint32_t* const codes_lane = p.codes + (size_t)node * (size_t)p.code_pitch +
                                     (size_t)((k0 * T::kBits) >> 5) + lane / T::kLanesPerWord;
        float* const cval_lane = cval + (size_t)node * SEG + 4 * lane;
#pragma unroll
        for (int r = 0; r < V; ++r) {
            const int e0 = 4 * (32 * r + lane);
            uint32_t piece = 0u;
            float cv[4];
            if constexpr (T::kSign) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t bit = (v[4 * r + j] >= 0.0f) ? 1u : 0u;
                    cv[j] = bit ? s : -s;
                    if (e0 + j < m_len) piece |= bit << j;
                }
            } else if (fast) {
                uint32_t q[4];
                quantise_recip2(v[4 * r + 0], v[4 * r + 1], s, inv_s, mn[4 * r + 0], mn[4 * r + 1], kHalfL, (int)kL, q[0], q[1]);
                quantise_recip2(v[4 * r + 2], v[4 * r + 3], s, inv_s, mn[4 * r + 2], mn[4 * r + 3], kHalfL, (int)kL, q[2], q[3]);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    cv[j] = __fmul_rn(s, lut[q[j]]);
                    if (e0 + j < m_len) piece |= q[j] << (T::kBits * j);
                }
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float rj = __fmul_rn(mn[kRnd ? 4 * r + j : 0], 0x1p-24f);
                    const uint32_t q = degenerate ? 0u : quantise(v[4 * r + j], s, rj, kHalfL, (int)kL);
                    cv[j] = __fmul_rn(s, lut[q]);
                    if (e0 + j < m_len) piece |= q << (T::kBits * j);
                }
            }
#pragma unroll
            for (int j = 0; j < 4; ++j)
                dr[4 * r + j] = (e0 + j < m_len) ? __fadd_rn(v[4 * r + j], -cv[j]) : 0.0f;
            *reinterpret_cast<float4*>(cval_lane + 128 * r) = make_float4(cv[0], cv[1], cv[2], cv[3]);
            uint32_t word = piece << ((4 * T::kBits * (lane % T::kLanesPerWord)) & 31);
#pragma unroll
            for (int o = 1; o < T::kLanesPerWord; o <<= 1) word |= __shfl_xor_sync(0xffffffffu, word, o);
            if ((lane % T::kLanesPerWord) == 0 && e0 < m_len) codes_lane[(32 / T::kLanesPerWord) * r] = word;
        }
        __syncthreads();          // C[v] of every node of the tile is in shared memory

        // ---- local update ----
        float acc[E];
#pragma unroll
        for (int q = 0; q < E; ++q) acc[q] = 0.0f;
        for (int e = rptr[node]; e < rptr[node + 1]; ++e) {
            const float w = wp[e];
            const float* cn = cval + (size_t)cj[e] * SEG + 4 * lane;
#pragma unroll
            for (int r = 0; r < V; ++r) {
                const float4 c4 = *reinterpret_cast<const float4*>(cn + 128 * r);
                acc[4 * r + 0] = __fmaf_rn(w, c4.x, acc[4 * r + 0]);
                acc[4 * r + 1] = __fmaf_rn(w, c4.y, acc[4 * r + 1]);
                acc[4 * r + 2] = __fmaf_rn(w, c4.z, acc[4 * r + 2]);
                acc[4 * r + 3] = __fmaf_rn(w, c4.w, acc[4 * r + 3]);
            }
        }
#pragma unroll
        for (int q = 0; q < E; ++q) xr[q] = __fmaf_rn(eta, acc[q], h[q]);
        __syncthreads();          // C[v] may be overwritten by the next iteration
    }

    if (!alive) return;
#pragma unroll
    for (int r = 0; r < V; ++r) {
        const int e0 = 4 * (32 * r + lane);
        const int nv = min(max(m_len - e0, 0), 4);
        if (nv > 0) {
            st_partial(p.x + row + e0, make_float4(xr[4 * r], xr[4 * r + 1], xr[4 * r + 2], xr[4 * r + 3]), nv);
            st_partial(p.delta + row + e0, make_float4(dr[4 * r], dr[4 * r + 1], dr[4 * r + 2], dr[4 * r + 3]), nv);
        }
    }
}

// Launch (cooperative when a per-node scale needs the grid barrier); returns
// cudaErrorCooperativeLaunchTooLarge if the blocks cannot all be resident.
cudaError_t launch_resident(int code, int noise, const ResidentParams& rp, int num_sms, cudaStream_t stream);

}  // namespace ds
