// Persistent TMA-staged fused kernel for 17..32 nodes and chunks of 256
// elements: ds_fused_tma_kernel with TWO nodes per warp.
//
// A column tile of 32 nodes needs 32 (node, tile) owners.  As 32 warps they
// form a 1024-thread block, which leaves 64 registers per thread -- too few to
// keep x - gamma g, v and the random numbers of a tile in registers.  Here a
// block has n/2 warps (512 threads at most, 128 registers each) and warp w
// owns the tile's 256 elements of node w AND of node w + n/2: the lane's 16
// elements are 8 of each node (float4 groups 0,1 -> first node, 2,3 -> second).
// Staging (four bulk copies per node into the warp's slot, counted on the
// warp's mbarrier), the one-tile-ahead drawing of noise and rounding uniforms
// with all Philox blocks in lockstep, C[v] of the tile in shared memory and the
// bounded waits are those of ds_fused_tma_kernel; scale, codes and local update
// are taken per node.
#pragma once

#include <type_traits>

#include "ds_fused_tma_kernel.cuh"

namespace ds {

// rng_blocks() with a node of its own for every block.
template <int NB>
__device__ __forceinline__ void rng_blocks_of_nodes(const RngStep& rs, const uint32_t (&node)[NB],
                                                    const uint32_t (&stream)[NB], const uint32_t (&block)[NB],
                                                    uint4 (&out)[NB]) {
    uint32_t c0[NB], c1[NB], c2[NB], c3[NB];
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        c0[b] = block[b]; c1[b] = node[b]; c2[b] = rs.step_lo; c3[b] = rs.step_hi8 | stream[b];
    }
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t ka = rs.k0[r], kb = rs.k1[r];
#pragma unroll
        for (int b = 0; b < NB; ++b) {
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
    for (int b = 0; b < NB; ++b) out[b] = make_uint4(c0[b], c1[b], c2[b], c3[b]);
}

constexpr int kPairTile = 256;

template <int CODE, int NOISE>
__global__ void __launch_bounds__(512, 1) ds_fused_tma_pair_kernel(const __grid_constant__ StepParams p) {
    using T = CodeTraits<CODE>;
    static_assert(!T::kIdentity && !T::kNorm, "sign and stochastic b-bit codes only");
    constexpr int E = 16, V = 4, NPW = 2;
    constexpr int VS = V / NPW;                       // float4 groups per lane and node
    constexpr int SUB = kPairTile;                    // elements per (node, tile)
    constexpr int SEG = E * 32;                       // floats per staged array of a warp (both nodes)
    extern __shared__ __align__(128) unsigned char smem[];
    const int nwarps = blockDim.x >> 5;               // = n / 2
    const TmaSmemLayout L = tma_smem_layout(T::kLut, E, nwarps, 1, kPairTile, p.n, p.nnz);
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int node_of[NPW] = {warp, warp + nwarps};

    float* lut = reinterpret_cast<float*>(smem + L.lut_off);
    int32_t* rp = reinterpret_cast<int32_t*>(smem + L.rowptr_off);
    int32_t* cj = reinterpret_cast<int32_t*>(smem + L.col_off);
    float* wp = reinterpret_cast<float*>(smem + L.w_off);
    volatile int* abort_sm = reinterpret_cast<volatile int*>(smem + L.abort_off);
    const float* slot = reinterpret_cast<const float*>(smem + L.slots_off + (size_t)warp * 4u * L.seg_bytes);
    const uint32_t slot_addr = smem_u32(slot);
    const float* const slot_lane = slot + 4 * lane;
    const uint32_t bar = smem_u32(smem + L.mbar_off + warp * 8);

    if constexpr (T::kLut)
        for (int t = threadIdx.x; t < (1 << T::kBits); t += blockDim.x) lut[t] = p.lut[t];
    for (int t = threadIdx.x; t <= p.n; t += blockDim.x) rp[t] = p.row_ptr[t];
    for (int t = threadIdx.x; t < p.nnz; t += blockDim.x) { cj[t] = p.col_idx[t]; wp[t] = p.wprime[t]; }
    if (threadIdx.x < 2) abort_sm[threadIdx.x] = 0;
    if (lane == 0) mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();

    // bulk copies of both nodes' segments of tile `col` into the warp's slot
    auto issue = [&](int64_t col) {
        if (lane == 0) {
            const int64_t remain = p.N - col * SUB;
            const int len = (int)(remain < SUB ? remain : SUB);
            const uint32_t bytes = (uint32_t)((len + 3) & ~3) * 4u;
            fence_proxy_async();      // earlier generic reads of the slot are ordered before the refill
            mbar_expect_tx(bar, 4u * NPW * bytes);
#pragma unroll
            for (int s = 0; s < NPW; ++s) {
                const size_t at = (size_t)node_of[s] * (size_t)p.ld + (size_t)(col * SUB);
                const uint32_t dst = slot_addr + (uint32_t)s * SUB * 4u;
                bulk_g2s(dst + 0u * L.seg_bytes, p.x + at, bytes, bar);
                bulk_g2s(dst + 1u * L.seg_bytes, p.delta + at, bytes, bar);
                bulk_g2s(dst + 2u * L.seg_bytes, p.a + at, bytes, bar);
                bulk_g2s(dst + 3u * L.seg_bytes, p.c + at, bytes, bar);
            }
        }
    };

    constexpr bool kNoiseAhead = (NOISE == NOISE_GAUSS || NOISE == NOISE_T3);
    constexpr bool kRndAhead = T::kLut;
    float zn[kNoiseAhead ? E : 1];
    float mn[kRndAhead ? E : 1];
    auto draw_noise = [&](int64_t c) {
        if constexpr (kNoiseAhead || kRndAhead) {
            const uint32_t kbase = (uint32_t)(c * SUB) + 4u * (uint32_t)lane;
            constexpr int kNz = kNoiseAhead ? V : 0;
            constexpr int kRn = kRndAhead ? V : 0;
            uint32_t nodes[kNz + kRn], stream[kNz + kRn], block[kNz + kRn];
            uint4 w[kNz + kRn];
#pragma unroll
            for (int r = 0; r < V; ++r) {
                const uint32_t blk = (kbase + 128u * (uint32_t)(r % VS)) >> 2;
                if constexpr (kNz > 0) { nodes[r] = (uint32_t)node_of[r / VS]; stream[r] = STREAM_NOISE; block[r] = blk; }
                if constexpr (kRn > 0) { nodes[kNz + r] = (uint32_t)node_of[r / VS]; stream[kNz + r] = STREAM_ROUND; block[kNz + r] = blk; }
            }
            rng_blocks_of_nodes<kNz + kRn>(p.rs, nodes, stream, block, w);
#pragma unroll
            for (int r = 0; r < V; ++r) {
                if constexpr (kNz > 0) {
                    const float4 z4 = noise_of_block<NOISE>(w[r]);
                    zn[4 * r + 0] = z4.x; zn[4 * r + 1] = z4.y; zn[4 * r + 2] = z4.z; zn[4 * r + 3] = z4.w;
                }
                if constexpr (kRn > 0) {
                    const uint4 u = w[kNz + r];
                    mn[4 * r + 0] = __uint2float_rn(u.x >> 8); mn[4 * r + 1] = __uint2float_rn(u.y >> 8);
                    mn[4 * r + 2] = __uint2float_rn(u.z >> 8); mn[4 * r + 3] = __uint2float_rn(u.w >> 8);
                }
            }
        }
    };

    int64_t col = p.tile_begin + blockIdx.x;
    bool pending = false;
    if (col < p.tile_end) { issue(col); pending = true; draw_noise(col); }
    uint32_t parity = 0;
    int buf = 0;
    constexpr float kL = (float)((1u << (T::kBits & 15)) - 1u);
    constexpr float kHalfL = 0.5f * kL;

    for (; col < p.tile_end; col += gridDim.x) {
        const int64_t k0 = col * SUB;
        const int64_t remain = p.N - k0;
        const int m_len = (int)(remain < SUB ? remain : SUB);
        float* cval = reinterpret_cast<float*>(smem + L.cval_off) + (size_t)buf * p.n * SUB;

        bool alive = true;
        if (pending) {
            alive = mbar_wait_bounded(bar, parity);
            parity ^= 1u;
            if (!alive) {
                abort_sm[buf] = 1;
                if (lane == 0) *p.error_flag = 1;
            }
        }
        if (DS_CHECKED_BUILD &&
            !(ds_part_ok(p, node_of[0], k0, m_len, T::kBits, col) && ds_part_ok(p, node_of[NPW - 1], k0, m_len, T::kBits, col))) {
            alive = false;              // refused: the warp stores nothing and the block winds down
            abort_sm[buf] = 1;
        }
        const int live_len = alive ? m_len : 0;
        const bool full = (live_len == SUB);

        auto tile_body = [&](auto full_tag) -> bool {
            constexpr bool FULL = decltype(full_tag)::value;
            // ---- phase A: slot -> registers, local step, scale partials ----
            float h[E], v[E];
            double sum[NPW] = {0.0, 0.0};
            float mx[NPW] = {0.0f, 0.0f};
#pragma unroll
            for (int r = 0; r < V; ++r) {
                const int s = r / VS;
                const int e0 = 4 * (32 * (r % VS) + lane);           // offset inside the node's 256 elements
                const int nv = FULL ? 4 : min(max(live_len - e0, 0), 4);
                if (nv > 0) {
                    const float4 x4 = *reinterpret_cast<const float4*>(slot_lane + 0 * SEG + 128 * r);
                    const float4 d4 = *reinterpret_cast<const float4*>(slot_lane + 1 * SEG + 128 * r);
                    const float4 a4 = *reinterpret_cast<const float4*>(slot_lane + 2 * SEG + 128 * r);
                    const float4 c4 = *reinterpret_cast<const float4*>(slot_lane + 3 * SEG + 128 * r);
                    float4 z4 = make_float4(0.f, 0.f, 0.f, 0.f);
                    if constexpr (kNoiseAhead) z4 = make_float4(zn[4 * r + 0], zn[4 * r + 1], zn[4 * r + 2], zn[4 * r + 3]);
                    local_step4(x4, d4, a4, c4, z4, p.sigma, p.neg_gamma, &h[4 * r], &v[4 * r]);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if (!FULL && j >= nv) { h[4 * r + j] = 0.0f; v[4 * r + j] = 0.0f; }
                        if constexpr (T::kSign) sum[s] += (double)fabsf(v[4 * r + j]);
                        else mx[s] = fmaxf(mx[s], fabsf(v[4 * r + j]));
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j) { h[4 * r + j] = 0.0f; v[4 * r + j] = 0.0f; }
                }
            }
            // the slot is in registers: refill it with the segments of the next tile
            __syncwarp();
            {
                const int64_t next = col + gridDim.x;
                pending = next < p.tile_end;
                if (pending) issue(next);
            }

            // ---- scales of the two (node, tile) ----
            float sc[NPW], inv_s[NPW];
            bool fast[NPW], degenerate[NPW];
#pragma unroll
            for (int s = 0; s < NPW; ++s) {
                if constexpr (T::kSign) {
                    sc[s] = (float)(warp_sum(sum[s]) / (double)m_len);
                } else {
                    sc[s] = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(mx[s])));
                    if (sc[s] == 0.0f || !(fabsf(sc[s]) <= 3.402823466e+38f)) sc[s] = 0.0f;
                }
                degenerate[s] = (!T::kSign && sc[s] == 0.0f);
                fast[s] = T::kLut && sc[s] >= 0x1p-60f && sc[s] <= 0x1p+60f;
                inv_s[s] = fast[s] ? __fdiv_rn(1.0f, sc[s]) : 0.0f;
            }
            float* cval_lane[NPW];
            float* delta_lane[NPW];
            float* x_lane[NPW];
            uint32_t* codes_lane[NPW];
#pragma unroll
            for (int s = 0; s < NPW; ++s) {
                const size_t row = (size_t)node_of[s] * (size_t)p.ld + (size_t)k0;
                cval_lane[s] = cval + (size_t)node_of[s] * SUB + 4 * lane;
                delta_lane[s] = p.delta + row + 4 * lane;
                x_lane[s] = p.x + row + 4 * lane;
                codes_lane[s] = p.codes + (size_t)node_of[s] * (size_t)p.code_pitch + (size_t)((k0 * T::kBits) >> 5) +
                                lane / T::kLanesPerWord;
            }

            // ---- phase B: compress, residual, pack ----
#pragma unroll
            for (int r = 0; r < V; ++r) {
                const int s = r / VS, rr = r % VS;
                const int e0 = 4 * (32 * rr + lane);
                const int nv = FULL ? 4 : min(max(live_len - e0, 0), 4);
                uint32_t piece = 0u;
                if (nv > 0) {
                    float cv[4];
                    if constexpr (T::kSign) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint32_t bit = (v[4 * r + j] >= 0.0f) ? 1u : 0u;
                            cv[j] = bit ? sc[s] : -sc[s];
                            if (FULL || j < nv) piece |= bit << j;
                        }
                    } else if (fast[s]) {
                        uint32_t q[4];
                        quantise_recip2(v[4 * r + 0], v[4 * r + 1], sc[s], inv_s[s], mn[4 * r + 0], mn[4 * r + 1], kHalfL, (int)kL, q[0], q[1]);
                        quantise_recip2(v[4 * r + 2], v[4 * r + 3], sc[s], inv_s[s], mn[4 * r + 2], mn[4 * r + 3], kHalfL, (int)kL, q[2], q[3]);
                        const float2 ca = __fmul2_rn(splat(sc[s]), make_float2(lut[q[0]], lut[q[1]]));
                        const float2 cb = __fmul2_rn(splat(sc[s]), make_float2(lut[q[2]], lut[q[3]]));
                        cv[0] = ca.x; cv[1] = ca.y; cv[2] = cb.x; cv[3] = cb.y;
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            if (FULL || j < nv) piece |= q[j] << (T::kBits * j);
                    } else {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const float rj = __fmul_rn(mn[kRndAhead ? 4 * r + j : 0], 0x1p-24f);
                            const uint32_t q = degenerate[s] ? 0u : quantise(v[4 * r + j], sc[s], rj, kHalfL, (int)kL);
                            cv[j] = __fmul_rn(sc[s], lut[q]);
                            if (FULL || j < nv) piece |= q << (T::kBits * j);
                        }
                    }
                    const float2 da = __fadd2_rn(make_float2(v[4 * r + 0], v[4 * r + 1]), make_float2(-cv[0], -cv[1]));
                    const float2 db = __fadd2_rn(make_float2(v[4 * r + 2], v[4 * r + 3]), make_float2(-cv[2], -cv[3]));
                    st_partial(delta_lane[s] + 128 * rr, make_float4(da.x, da.y, db.x, db.y), nv);
                    *reinterpret_cast<float4*>(cval_lane[s] + 128 * rr) = make_float4(cv[0], cv[1], cv[2], cv[3]);
                }
                uint32_t word = piece << ((4 * T::kBits * (lane % T::kLanesPerWord)) & 31);
#pragma unroll
                for (int o = 1; o < T::kLanesPerWord; o <<= 1) word |= __shfl_xor_sync(0xffffffffu, word, o);
                if ((lane % T::kLanesPerWord) == 0 && (FULL || e0 < live_len))
                    codes_lane[s][(32 / T::kLanesPerWord) * rr] = word;
            }
            if (alive && lane == 0) {
#pragma unroll
                for (int s = 0; s < NPW; ++s)
                    p.scales[(size_t)node_of[s] * (size_t)p.scales_pitch + (size_t)col] = sc[s];
            }

            __syncthreads();       // C[v] of every node of this tile is in shared memory
            if (abort_sm[buf]) return true;

            // ---- phase C: local update from the neighbours' C[v] ----
#pragma unroll
            for (int s = 0; s < NPW; ++s) {
                float acc[E / NPW];
#pragma unroll
                for (int t = 0; t < E / NPW; ++t) acc[t] = 0.0f;
                const int e_beg = rp[node_of[s]], e_end = rp[node_of[s] + 1];
                for (int e = e_beg; e < e_end; ++e) {
                    const float2 w2 = splat(wp[e]);
                    const float* cn = cval + (size_t)cj[e] * SUB + 4 * lane;
#pragma unroll
                    for (int rr = 0; rr < VS; ++rr) {
                        if (!FULL && 4 * (32 * rr + lane) >= live_len) continue;
                        const float4 c4 = *reinterpret_cast<const float4*>(cn + 128 * rr);
                        const float2 aa = __ffma2_rn(w2, make_float2(c4.x, c4.y), make_float2(acc[4 * rr + 0], acc[4 * rr + 1]));
                        const float2 ab = __ffma2_rn(w2, make_float2(c4.z, c4.w), make_float2(acc[4 * rr + 2], acc[4 * rr + 3]));
                        acc[4 * rr + 0] = aa.x; acc[4 * rr + 1] = aa.y; acc[4 * rr + 2] = ab.x; acc[4 * rr + 3] = ab.y;
                    }
                }
#pragma unroll
                for (int rr = 0; rr < VS; ++rr) {
                    const int r = s * VS + rr;
                    const int e0 = 4 * (32 * rr + lane);
                    const int nv = FULL ? 4 : min(max(live_len - e0, 0), 4);
                    if (nv > 0) {
                        const float2 et = splat(p.eta);
                        const float2 xa = __ffma2_rn(et, make_float2(acc[4 * rr + 0], acc[4 * rr + 1]), make_float2(h[4 * r + 0], h[4 * r + 1]));
                        const float2 xb = __ffma2_rn(et, make_float2(acc[4 * rr + 2], acc[4 * rr + 3]), make_float2(h[4 * r + 2], h[4 * r + 3]));
                        st_partial(x_lane[s] + 128 * rr, make_float4(xa.x, xa.y, xb.x, xb.y), nv);
                    }
                }
            }
            if (col + gridDim.x < p.tile_end) draw_noise(col + gridDim.x);
            return false;
        };
        const bool aborted = full ? tile_body(std::true_type{}) : tile_body(std::false_type{});
        if (aborted) break;
        buf ^= 1;
    }
    // Leaving early (error path): let the copy that is still in flight land
    // before the block's shared memory is given away.
    if (pending) (void)mbar_wait_bounded(bar, parity);
}

// Launcher (defined in ds_kernels_tma_pair.cu): n even, 17..32 nodes, tile = 256.
cudaError_t launch_fused_tma_pair(const LaunchShape& shape, const StepParams& p, cudaStream_t stream);

}  // namespace ds
