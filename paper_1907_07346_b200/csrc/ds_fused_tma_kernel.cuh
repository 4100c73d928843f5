// Persistent fused kernel with TMA-staged inputs (sm_100a).
//
// One thread block per SM walks over the column tiles.  A group of G warps
// owns one (node, tile); every warp owns a contiguous segment of E*32 elements
// of it and a private shared-memory slot holding that segment of x, delta, a
// and c.  The slot is filled by four bulk asynchronous copies
// (cp.async.bulk global -> shared, completion counted on the warp's own
// mbarrier) that the warp issues for its NEXT tile as soon as it has moved the
// current tile into registers, so the copy of tile t+1 runs under the
// compression and mixing of tile t and no warp waits for DRAM in steady state.
//
// The decoded compression C[v] of the tile is kept in shared memory as
// binary32 (double buffered): the node that produced it has it in registers
// anyway, and each neighbour reads it back with 128-bit shared loads, so the
// local update of Algorithm 1 costs one fma per (element, neighbour).  The
// packed codes and the scales still go to global memory: they are what the
// node "sends".
//
// There is no block-wide barrier per tile: a warp announces "C[v] of my node
// is in shared memory" on that node's mbarrier and waits only for the barriers
// of its node's neighbours, so a block is not held to the pace of its slowest
// warp.
//
// Every wait on an mbarrier is bounded.  A warp whose copy (or neighbour) does
// not arrive gives up, raises the step's error flag and stops storing; from
// then on it only keeps announcing its tiles, so that no other warp waits in
// vain, and every warp that sees the flag does the same.
#pragma once

#include <type_traits>

#include "ds_column_kernel.cuh"

namespace ds {

struct TmaSmemLayout {
    uint32_t slots_off, cval_off, red_off, lut_off, rowptr_off, col_off, w_off, mbar_off, nbar_off, abort_off, total;
    uint32_t seg_bytes;    // bytes of one array segment of one warp
};

__host__ __device__ inline TmaSmemLayout tma_smem_layout(bool has_lut, int E, int nwarps, int G,
                                                         int64_t tile, int n, int nnz) {
    TmaSmemLayout L;
    uint32_t off = 0;
    L.seg_bytes = (uint32_t)E * 32u * 4u;
    L.slots_off = off;   off += (uint32_t)nwarps * 4u * L.seg_bytes;
    L.cval_off = off;    off += 2u * (uint32_t)n * (uint32_t)tile * 4u;
    L.red_off = off;     off += (G > 1) ? 3u * (uint32_t)nwarps * 8u : 0u;   // scale partial and two norm sums per warp
    L.mbar_off = off;    off += (uint32_t)nwarps * 8u;
    L.nbar_off = off;    off += 2u * (uint32_t)n * 8u;      // "C[v] of node j is ready", one per buffer and node
    L.lut_off = off;     off += has_lut ? 256u * 4u : 0u;
    L.rowptr_off = off;  off += (uint32_t)(n + 1) * 4u;
    L.col_off = off;     off += (uint32_t)nnz * 4u;
    L.w_off = off;       off += (uint32_t)nnz * 4u;
    L.abort_off = off;   off += 8u;
    L.total = (off + 127u) & ~127u;
    return L;
}

// ---- thin wrappers over the PTX of mbarriers and bulk copies ----------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0u;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: false if the phase did not complete within `limit_ns` of
// wall-clock time (and at most 2^22 polls).  In steady state the first poll
// succeeds and the timer is never read.  `gave_up` (optional): two flags in
// shared memory that a warp of the block raises when ITS wait ran out; the
// slow path polls them, so that once one warp has given up the others stop
// waiting at once instead of each spending its own full time limit.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity,
                                                  uint64_t limit_ns = 2000000000ull,
                                                  const volatile int* gave_up = nullptr) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    for (uint32_t tries = 0; tries < (1u << 22); ++tries) {
        if (mbar_try_wait(bar, parity)) return true;
        if (gave_up != nullptr && (gave_up[0] | gave_up[1]) != 0) return false;
        if (global_timer_ns() - t0 > limit_ns) return false;
    }
    return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// L2 eviction policies and accesses that carry one.  Inputs that are read exactly once are
// fetched "evict first", so that they do not push out lines that the same kernel re-reads.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void bulk_g2s_hint(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar,
                                              uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy) : "memory");
}
__device__ __forceinline__ void st4_hint(float* p, float4 v, uint64_t policy) {
    asm volatile("st.global.L2::cache_hint.v4.f32 [%0], {%1, %2, %3, %4}, %5;"
                 ::"l"(p), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w), "l"(policy) : "memory");
}
__device__ __forceinline__ float4 ld4_hint(const float* p, uint64_t policy) {
    float4 v;
    asm volatile("ld.global.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p), "l"(policy) : "memory");
    return v;
}
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// EC = true: the iteration of centralized error-compensated SGD (Section 1)
// on the same machinery: the compressed variable is v = g + delta, the value
// kept for the update is x itself, and the launcher passes the weights W (not
// W - I) and -gamma in the place of eta, so that the last phase computes
// x' = fma(-gamma, sum_j W_ij C_j, x).
template <int CODE, int NOISE, int E, int MAXT, bool EC = false>
__global__ void __launch_bounds__(MAXT, 1) ds_fused_tma_kernel(const __grid_constant__ StepParams p) {
    using T = CodeTraits<CODE>;
    constexpr int V = E / 4;
    constexpr int SEG = E * 32;                       // elements per warp segment
    extern __shared__ __align__(128) unsigned char smem[];
    const int G = p.warps_per_group;
    const int nwarps = blockDim.x >> 5;
    const TmaSmemLayout L = tma_smem_layout(T::kLut, E, nwarps, G, p.tile, p.n, p.nnz);
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int node = warp / G;                        // the block holds all n nodes
    const int wg = warp - node * G;
    const int seg0 = wg * SEG;                        // first element of this warp's segment in the tile

    float* lut = reinterpret_cast<float*>(smem + L.lut_off);
    int32_t* rp = reinterpret_cast<int32_t*>(smem + L.rowptr_off);
    int32_t* cj = reinterpret_cast<int32_t*>(smem + L.col_off);
    float* wp = reinterpret_cast<float*>(smem + L.w_off);
    volatile int* abort_sm = reinterpret_cast<volatile int*>(smem + L.abort_off);
    const float* slot = reinterpret_cast<const float*>(smem + L.slots_off + (size_t)warp * 4u * L.seg_bytes);
    const uint32_t slot_addr = smem_u32(slot);
    const float* const slot_lane = slot + 4 * lane;     // this lane's first float4 of each staged array
    const uint32_t bar = smem_u32(smem + L.mbar_off + warp * 8);

    if constexpr (T::kLut)
        for (int t = threadIdx.x; t < (1 << T::kBits); t += blockDim.x) lut[t] = p.lut[t];
        // norm-matched codes: squares of the levels in binary64 (exact), in the unused part of the table
        if constexpr (T::kNorm)
            for (int t = threadIdx.x; t < (1 << T::kBits); t += blockDim.x)
                reinterpret_cast<double*>(lut + 32)[t] = (double)p.lut[t] * (double)p.lut[t];
    for (int t = threadIdx.x; t <= p.n; t += blockDim.x) rp[t] = p.row_ptr[t];
    for (int t = threadIdx.x; t < p.nnz; t += blockDim.x) { cj[t] = p.col_idx[t]; wp[t] = p.wprime[t]; }
    if (threadIdx.x < 2) abort_sm[threadIdx.x] = 0;
    if (lane == 0) mbar_init(bar, 1);
    // one "ready" barrier per C[v] buffer and node, completed by the G warps of the node
    const uint32_t nbar0 = smem_u32(smem + L.nbar_off);
    for (int t = threadIdx.x; t < 2 * p.n; t += blockDim.x) mbar_init(nbar0 + 8u * (uint32_t)t, (uint32_t)G);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();

    // Valid elements of this warp's segment in tile `col`, and the copy that fetches them.
    auto seg_len_of = [&](int64_t col) -> int {
        const int64_t remain = p.N - col * p.tile;
        const int m_len = (int)(remain < p.tile ? remain : p.tile);
        return min(max(m_len - seg0, 0), SEG);
    };
    auto issue = [&](int64_t col) -> bool {
        const int len = seg_len_of(col);
        if (len <= 0) return false;
        if (DS_CHECKED_BUILD && !ds_part_ok(p, node, col * p.tile + seg0, len, T::kBits, -1)) return false;
        if (lane == 0) {
            const uint32_t bytes = (uint32_t)((len + 3) & ~3) * 4u;
            const size_t at = (size_t)node * (size_t)p.ld + (size_t)(col * p.tile) + (size_t)seg0;
            fence_proxy_async();      // earlier generic reads of the slot are ordered before the refill
            constexpr uint32_t kArrays = (NOISE == GRAD_GIVEN) ? 3u : 4u;   // x, delta, g | x, delta, a, c
            mbar_expect_tx(bar, kArrays * bytes);
            bulk_g2s(slot_addr + 0u * L.seg_bytes, p.x + at, bytes, bar);
            bulk_g2s(slot_addr + 1u * L.seg_bytes, p.delta + at, bytes, bar);
            bulk_g2s(slot_addr + 2u * L.seg_bytes, p.a + at, bytes, bar);
            if constexpr (NOISE != GRAD_GIVEN) bulk_g2s(slot_addr + 3u * L.seg_bytes, p.c + at, bytes, bar);
        }
        return true;
    };

    int64_t col = p.tile_begin + blockIdx.x;
    bool pending = (col < p.tile_end) ? issue(col) : false;
    // The gradient noise of a tile depends on nothing that is loaded, so it is
    // drawn one tile AHEAD (after the mixing of the previous tile): phase A then
    // only moves the slot into registers and takes the local step, and the refill
    // of the slot for the next tile is in flight for almost the whole tile time.
    constexpr bool kNoiseAhead = (NOISE == NOISE_GAUSS || NOISE == NOISE_T3);
    float zn[kNoiseAhead ? E : 1];
    // the rounding uniforms of the stochastic quantiser are drawn with it
    constexpr bool kRndAhead = T::kLut && !T::kNorm;
    float mn[kRndAhead ? E : 1];
    auto draw_noise = [&](int64_t c) {
        const uint32_t kbase = (uint32_t)(c * p.tile + seg0) + 4u * (uint32_t)lane;   // element of r = 0
        if constexpr (kNoiseAhead || kRndAhead) {
            // all Philox blocks of the tile (V for the noise, V for the rounding stream,
            // whichever are needed) advance together
            constexpr int kGauss = kNoiseAhead ? V : 0;
            constexpr int kRnd = kRndAhead ? V : 0;
            uint32_t stream[kGauss + kRnd], block[kGauss + kRnd];
            uint4 w[kGauss + kRnd];
#pragma unroll
            for (int r = 0; r < V; ++r) {
                if constexpr (kGauss > 0) { stream[r] = STREAM_NOISE; block[r] = (kbase + 128u * (uint32_t)r) >> 2; }
                if constexpr (kRnd > 0) { stream[kGauss + r] = STREAM_ROUND; block[kGauss + r] = (kbase + 128u * (uint32_t)r) >> 2; }
            }
            rng_blocks<kGauss + kRnd>(p.rs, (uint32_t)node, stream, block, w);
#pragma unroll
            for (int r = 0; r < V; ++r) {
                if constexpr (kGauss > 0) {
                    const float4 z4 = noise_of_block<NOISE>(w[r]);
                    zn[4 * r + 0] = z4.x; zn[4 * r + 1] = z4.y; zn[4 * r + 2] = z4.z; zn[4 * r + 3] = z4.w;
                }
                if constexpr (kRnd > 0) {
                    const uint4 u = w[kGauss + r];
                    mn[4 * r + 0] = __uint2float_rn(u.x >> 8); mn[4 * r + 1] = __uint2float_rn(u.y >> 8);
                    mn[4 * r + 2] = __uint2float_rn(u.z >> 8); mn[4 * r + 3] = __uint2float_rn(u.w >> 8);
                }
            }
        }
    };
    if (col < p.tile_end) draw_noise(col);      // (also when only the rounding stream is needed)
    uint32_t parity = 0;
    int buf = 0;
    uint32_t iter = 0;          // tiles this block has worked on
    bool drain = false;         // after an abort: keep announcing tiles so that no neighbour waits in vain, nothing else
    constexpr float kL = (float)((1u << (T::kBits & 15)) - 1u);
    constexpr float kHalfL = 0.5f * kL;

    for (; col < p.tile_end; col += gridDim.x, ++iter) {
        if (drain) {
            // (the block-wide barriers of the reductions of a multi-warp chunk are still kept)
            if (G > 1 && !T::kIdentity && !p.prescaled) {
                __syncthreads();
                if constexpr (T::kNorm) __syncthreads();
            }
            if (lane == 0) mbar_arrive(nbar0 + 8u * (uint32_t)(buf * p.n + node));
            buf ^= 1;
            continue;
        }
        const int64_t k0 = col * p.tile;
        const int64_t remain = p.N - k0;
        const int m_len = (int)(remain < p.tile ? remain : p.tile);
        const int seg_len = min(max(m_len - seg0, 0), SEG);
        const size_t row = (size_t)node * (size_t)p.ld + (size_t)k0 + (size_t)seg0;
        float* cval = reinterpret_cast<float*>(smem + L.cval_off) + (size_t)buf * p.n * p.tile;

        // ---- wait for this tile's segment --------------------------------
        bool alive = true;
        if (pending) {
            alive = mbar_wait_bounded(bar, parity);
            parity ^= 1u;
            if (!alive) {
                abort_sm[buf] = 1;
                if (lane == 0) *p.error_flag = 1;
            }
        }
        if (DS_CHECKED_BUILD && seg_len > 0 &&
            !ds_part_ok(p, node, k0 + seg0, seg_len, T::kBits, (T::kIdentity || p.prescaled) ? -1 : col)) {
            alive = false;              // refused: the warp stores nothing and the block winds down
            abort_sm[buf] = 1;
        }
        const int live_len = alive ? seg_len : 0;
        const bool full = (live_len == SEG);

        auto tile_body = [&](auto full_tag) -> bool {
            constexpr bool FULL = decltype(full_tag)::value;
            // ---- phase A: slot -> registers, local step, scale partial ---------
            float h[E], v[E];
            double sum = 0.0;
            float mx = 0.0f;
    #pragma unroll
            for (int r = 0; r < V; ++r) {
                const int e0 = 4 * (32 * r + lane);              // offset inside the segment
                const int nv = FULL ? 4 : min(max(live_len - e0, 0), 4);
                if (nv > 0) {
                    const float4 x4 = *reinterpret_cast<const float4*>(slot_lane + 0 * SEG + 128 * r);
                    const float4 d4 = *reinterpret_cast<const float4*>(slot_lane + 1 * SEG + 128 * r);
                    const float4 a4 = *reinterpret_cast<const float4*>(slot_lane + 2 * SEG + 128 * r);
                    if constexpr (NOISE == GRAD_GIVEN) {
                        if constexpr (EC) worker_step4_given(d4, a4, &v[4 * r]);
                        else local_step4_given(x4, d4, a4, p.neg_gamma, &h[4 * r], &v[4 * r]);
                    } else {
                        const float4 c4 = *reinterpret_cast<const float4*>(slot_lane + 3 * SEG + 128 * r);
                        float4 z4;
                        if constexpr (kNoiseAhead) z4 = make_float4(zn[4 * r + 0], zn[4 * r + 1], zn[4 * r + 2], zn[4 * r + 3]);
                        else z4 = noise4<NOISE>(p.rs, (uint32_t)node, (uint32_t)(k0 + seg0 + e0));
                        if constexpr (EC) worker_step4(x4, d4, a4, c4, z4, p.sigma, &v[4 * r]);
                        else local_step4(x4, d4, a4, c4, z4, p.sigma, p.neg_gamma, &h[4 * r], &v[4 * r]);
                    }
                    if constexpr (EC) { h[4 * r + 0] = x4.x; h[4 * r + 1] = x4.y; h[4 * r + 2] = x4.z; h[4 * r + 3] = x4.w; }
    #pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if (!FULL && j >= nv) { h[4 * r + j] = 0.0f; v[4 * r + j] = 0.0f; }
                        if constexpr (T::kSign) sum += (double)fabsf(v[4 * r + j]);
                        else if constexpr (!T::kIdentity) mx = fmaxf(mx, fabsf(v[4 * r + j]));
                    }
                } else {
    #pragma unroll
                    for (int j = 0; j < 4; ++j) { h[4 * r + j] = 0.0f; v[4 * r + j] = 0.0f; }
                }
            }
            // the slot is in registers: refill it with the segment of the next tile
            __syncwarp();
            {
                const int64_t next = col + gridDim.x;
                pending = (next < p.tile_end) ? issue(next) : false;
            }

            // ---- scale of the (node, tile) -----------------------------------
            float s;
            if constexpr (T::kIdentity) {
                s = 1.0f;                       // C[v] = v: nothing to scale
            } else if (p.prescaled) {
                if constexpr (T::kNorm) s = p.gmax[node];          // the maximum that spans the grid
                else s = p.scales[(size_t)node * (size_t)p.scales_pitch];
            } else {
                double part;
                if constexpr (T::kSign) part = warp_sum(sum);
                else part = (double)__uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(mx)));
                if (G > 1) {
                    double* red = reinterpret_cast<double*>(smem + L.red_off);
                    if (lane == 0) red[warp] = part;
                    __syncthreads();
                    part = 0.0;
                    for (int w = 0; w < G; ++w) {
                        const double t = red[node * G + w];
                        if constexpr (T::kSign) part += t;
                        else part = fmax(part, t);
                    }
                }
                if constexpr (T::kSign) {
                    s = (float)(part / (double)m_len);
                } else {
                    s = (float)part;
                    if (s == 0.0f || !(fabsf(s) <= 3.402823466e+38f)) s = 0.0f;
                }
            }
            const bool degenerate = (!T::kSign && s == 0.0f);
            const bool fast = T::kLut && s >= 0x1p-60f && s <= 0x1p+60f;
            const float inv_s = fast ? __fdiv_rn(1.0f, s) : 0.0f;
            const size_t code_row = (size_t)node * (size_t)p.code_pitch + (size_t)(((k0 + seg0) * T::kBits) >> 5);
            float* cval_mine = cval + (size_t)node * p.tile + seg0;
            // per-lane bases: element 4*(32*r + lane) of the segment is base + 128*r
            float* const cval_lane = cval_mine + 4 * lane;
            float* const delta_lane = p.delta + row + 4 * lane;
            float* const x_lane = p.x + row + 4 * lane;
            uint32_t* const codes_lane = p.codes + code_row + lane / T::kLanesPerWord;
            // norm-matched codes: the whole chunk is coded first (two more warp
            // reductions), s becomes the norm that is sent, dscale the decode factor
            uint32_t qn[T::kNorm ? E : 1];
            float cvn[T::kNorm ? E : 1];
            float dscale = s;
            if constexpr (T::kNorm) {
                auto valid = [&](int t) { return 4 * (32 * (t >> 2) + lane) + (t & 3) < live_len; };
                double sv2, sl2;
                norm_codes<CODE, E, FULL>(v, valid, s, lut, qn, cvn, sv2, sl2);
                float nrm;
                if (p.prescaled) {
                    // one norm per node, computed by the earlier launches
                    nrm = p.scales[(size_t)node * (size_t)p.scales_pitch];
                    dscale = p.dscales[(size_t)node * (size_t)p.scales_pitch];
                } else {
                    if (G > 1) {
                        // the sums of the chunk's warps, added in warp order
                        double* red2 = reinterpret_cast<double*>(smem + L.red_off) + nwarps;
                        double* red3 = red2 + nwarps;
                        if (lane == 0) { red2[warp] = sv2; red3[warp] = sl2; }
                        __syncthreads();
                        sv2 = 0.0; sl2 = 0.0;
                        for (int w = 0; w < G; ++w) { sv2 += red2[node * G + w]; sl2 += red3[node * G + w]; }
                    }
                    norm_finish(s, sv2, sl2, nrm, dscale);
                }
    #pragma unroll
                for (int t = 0; t < E; ++t) cvn[t] = __fmul_rn(dscale, cvn[t]);
                s = nrm;
            }

            // ---- phase B: compress, residual, pack -----------------------------
    #pragma unroll
            for (int r = 0; r < V; ++r) {
                const int f = 32 * r + lane;                     // float4 index inside the segment
                const int e0 = 4 * f;
                const int nv = FULL ? 4 : min(max(live_len - e0, 0), 4);
                uint32_t piece = 0u;
                if (nv > 0) {
                    float dn[4], cv[4];
                    if constexpr (T::kIdentity) {
                        // D-PSGD: what is sent is v itself (32 bits per element)
    #pragma unroll
                        for (int j = 0; j < 4; ++j) cv[j] = v[4 * r + j];
                        st_partial(reinterpret_cast<float*>(p.codes + code_row) + e0,
                                   make_float4(cv[0], cv[1], cv[2], cv[3]), nv);
                    } else if constexpr (T::kNorm) {
    #pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            cv[j] = cvn[4 * r + j];
                            if (FULL || j < nv) piece |= qn[4 * r + j] << (T::kBits * j);
                        }
                    } else if constexpr (T::kSign) {
    #pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint32_t bit = (v[4 * r + j] >= 0.0f) ? 1u : 0u;
                            cv[j] = bit ? s : -s;
                            if (FULL || j < nv) piece |= bit << j;
                        }
                    } else if (fast) {
                        const float4 rr = make_float4(mn[4 * r + 0], mn[4 * r + 1], mn[4 * r + 2], mn[4 * r + 3]);
                        uint32_t q[4];
                        quantise_recip2(v[4 * r + 0], v[4 * r + 1], s, inv_s, rr.x, rr.y, kHalfL, (int)kL, q[0], q[1]);
                        quantise_recip2(v[4 * r + 2], v[4 * r + 3], s, inv_s, rr.z, rr.w, kHalfL, (int)kL, q[2], q[3]);
                        const float2 ca = __fmul2_rn(splat(s), make_float2(lut[q[0]], lut[q[1]]));
                        const float2 cb = __fmul2_rn(splat(s), make_float2(lut[q[2]], lut[q[3]]));
                        cv[0] = ca.x; cv[1] = ca.y; cv[2] = cb.x; cv[3] = cb.y;
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            if (FULL || j < nv) piece |= q[j] << (T::kBits * j);
                    } else {
                        const float rv[4] = {__fmul_rn(mn[4 * r + 0], 0x1p-24f), __fmul_rn(mn[4 * r + 1], 0x1p-24f),
                                             __fmul_rn(mn[4 * r + 2], 0x1p-24f), __fmul_rn(mn[4 * r + 3], 0x1p-24f)};
    #pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint32_t q = degenerate ? 0u : quantise(v[4 * r + j], s, rv[j], kHalfL, (int)kL);
                            cv[j] = __fmul_rn(s, lut[q]);
                            if (FULL || j < nv) piece |= q << (T::kBits * j);
                        }
                    }
                        {
                        const float2 da = __fadd2_rn(make_float2(v[4 * r + 0], v[4 * r + 1]), make_float2(-cv[0], -cv[1]));
                        const float2 db = __fadd2_rn(make_float2(v[4 * r + 2], v[4 * r + 3]), make_float2(-cv[2], -cv[3]));
                        dn[0] = da.x; dn[1] = da.y; dn[2] = db.x; dn[3] = db.y;
                    }
                    st_partial(delta_lane + 128 * r, make_float4(dn[0], dn[1], dn[2], dn[3]), nv);
                    *reinterpret_cast<float4*>(cval_lane + 128 * r) = make_float4(cv[0], cv[1], cv[2], cv[3]);
                }
                uint32_t word = piece << ((4 * T::kBits * (lane % T::kLanesPerWord)) & 31);
    #pragma unroll
                for (int o = 1; o < T::kLanesPerWord; o <<= 1) word |= __shfl_xor_sync(0xffffffffu, word, o);
                if constexpr (!T::kIdentity) {
                    if ((lane % T::kLanesPerWord) == 0 && (FULL || e0 < live_len))
                        codes_lane[(32 / T::kLanesPerWord) * r] = word;
                }
            }
            if (!T::kIdentity && !p.prescaled && alive && wg == 0 && lane == 0)
            {
                p.scales[(size_t)node * (size_t)p.scales_pitch + (size_t)col] = s;
                if constexpr (T::kNorm) p.dscales[(size_t)node * (size_t)p.scales_pitch + (size_t)col] = dscale;
            }

            // C[v] of this node is in shared memory: say so, then wait for the neighbours' only.
            // (W is symmetric, so the nodes waited for are exactly the ones that read this node's
            // C[v]: their arrival at the NEXT tile also tells that they are done reading this buffer
            // before it is written again two tiles later.)
            __syncwarp();
            if (lane == 0) mbar_arrive(nbar0 + 8u * (uint32_t)(buf * p.n + node));
            {
                const uint32_t nphase = (iter >> 1) & 1u;
                bool ok = true;
                for (int e = rp[node]; e < rp[node + 1]; ++e) {
                    if (G == 1 && cj[e] == node) continue;      // this warp wrote its own C[v]: __syncwarp() above orders it
                    ok = mbar_wait_bounded(nbar0 + 8u * (uint32_t)(buf * p.n + cj[e]), nphase, 2000000000ull, abort_sm) && ok;
                }
                if (!ok) {
                    abort_sm[buf] = 1;
                    if (lane == 0) *p.error_flag = 1;
                }
            }
            if (abort_sm[0] | abort_sm[1]) return true;

            // ---- phase C: local update from the neighbours' C[v] ---------------
            float acc[E];
    #pragma unroll
            for (int t = 0; t < E; ++t) acc[t] = 0.0f;
            const int e_beg = rp[node], e_end = rp[node + 1];
            for (int e = e_beg; e < e_end; ++e) {
                const float w = wp[e];
                const float* cn = cval + (size_t)cj[e] * p.tile + seg0;
    #pragma unroll
                for (int r = 0; r < V; ++r) {
                    const int e0 = 4 * (32 * r + lane);
                    if (!FULL && e0 >= live_len) continue;
                    const float4 c4 = *reinterpret_cast<const float4*>(cn + 4 * lane + 128 * r);
                    {
                        const float2 w2 = splat(w);
                        const float2 aa = __ffma2_rn(w2, make_float2(c4.x, c4.y), make_float2(acc[4 * r + 0], acc[4 * r + 1]));
                        const float2 ab = __ffma2_rn(w2, make_float2(c4.z, c4.w), make_float2(acc[4 * r + 2], acc[4 * r + 3]));
                        acc[4 * r + 0] = aa.x; acc[4 * r + 1] = aa.y; acc[4 * r + 2] = ab.x; acc[4 * r + 3] = ab.y;
                    }
                }
            }
    #pragma unroll
            for (int r = 0; r < V; ++r) {
                const int e0 = 4 * (32 * r + lane);
                const int nv = FULL ? 4 : min(max(live_len - e0, 0), 4);
                if (nv > 0) {
                    const float2 et = splat(p.eta);
                    const float2 xa = __ffma2_rn(et, make_float2(acc[4 * r + 0], acc[4 * r + 1]), make_float2(h[4 * r + 0], h[4 * r + 1]));
                    const float2 xb = __ffma2_rn(et, make_float2(acc[4 * r + 2], acc[4 * r + 3]), make_float2(h[4 * r + 2], h[4 * r + 3]));
                    st_partial(x_lane + 128 * r, make_float4(xa.x, xa.y, xb.x, xb.y), nv);
                }
            }
            if (col + gridDim.x < p.tile_end) draw_noise(col + gridDim.x);
            return false;
        };
        const bool aborted = full ? tile_body(std::true_type{}) : tile_body(std::false_type{});
        if (aborted) drain = true;
        buf ^= 1;
    }
    // Leaving early (error path): let the copy that is still in flight land
    // before the block's shared memory is given away.
    if (pending) (void)mbar_wait_bounded(bar, parity);
}

template <int CODE, int NOISE, int E>
cudaError_t launch_tma_one(const LaunchShape& sh, const StepParams& p, cudaStream_t stream) {
    if (sh.block.x <= 512) {
        auto kern = ds_fused_tma_kernel<CODE, NOISE, E, 512>;
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh.smem);
        if (e != cudaSuccess) return e;
        kern<<<sh.grid, sh.block, sh.smem, stream>>>(p);
    } else {
        auto kern = ds_fused_tma_kernel<CODE, NOISE, E, 1024>;
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh.smem);
        if (e != cudaSuccess) return e;
        kern<<<sh.grid, sh.block, sh.smem, stream>>>(p);
    }
    return cudaGetLastError();
}

// Centralized error-compensated SGD: 16 elements per lane, blocks of up to 512 threads.
template <int CODE>
cudaError_t launch_tma_ecsgd_code(const LaunchShape& sh, const StepParams& p, cudaStream_t stream) {
    if (sh.elems_per_lane != 16 || sh.block.x > 512) return cudaErrorInvalidValue;
#define DS_TMA_EC_CASE(NZ) \
    if (sh.noise == NZ) { \
        auto kern = ds_fused_tma_kernel<CODE, NZ, 16, 512, true>; \
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh.smem); \
        if (e != cudaSuccess) return e; \
        kern<<<sh.grid, sh.block, sh.smem, stream>>>(p); \
        return cudaGetLastError(); \
    }
    DS_TMA_EC_CASE(NOISE_NONE) DS_TMA_EC_CASE(NOISE_GAUSS) DS_TMA_EC_CASE(NOISE_T3) DS_TMA_EC_CASE(NOISE_T3I) DS_TMA_EC_CASE(GRAD_GIVEN)
#undef DS_TMA_EC_CASE
    return cudaErrorInvalidValue;
}

template <int CODE>
cudaError_t launch_tma_code(const LaunchShape& sh, const StepParams& p, cudaStream_t stream) {
#define DS_TMA_CASE(NZ, EE) \
    if (sh.noise == NZ && sh.elems_per_lane == EE) return launch_tma_one<CODE, NZ, EE>(sh, p, stream);
    DS_TMA_CASE(NOISE_NONE, 4) DS_TMA_CASE(NOISE_NONE, 8) DS_TMA_CASE(NOISE_NONE, 16)
    DS_TMA_CASE(NOISE_GAUSS, 4) DS_TMA_CASE(NOISE_GAUSS, 8) DS_TMA_CASE(NOISE_GAUSS, 16)
    DS_TMA_CASE(NOISE_T3, 4) DS_TMA_CASE(NOISE_T3, 8) DS_TMA_CASE(NOISE_T3, 16)
    DS_TMA_CASE(NOISE_T3I, 4) DS_TMA_CASE(NOISE_T3I, 8) DS_TMA_CASE(NOISE_T3I, 16)
    DS_TMA_CASE(GRAD_GIVEN, 4) DS_TMA_CASE(GRAD_GIVEN, 8) DS_TMA_CASE(GRAD_GIVEN, 16)
#undef DS_TMA_CASE
    return cudaErrorInvalidValue;
}

}  // namespace ds
