// Persistent, TMA-staged fused kernel for columns too wide for one pass
// (many nodes or long chunks): the node-batch sweeps of ds_wide_fused_kernel
// on the staging machinery of ds_fused_tma_kernel.
//
// One 512-thread block per SM walks over the column tiles.  It holds
// `nodes_per_block` nodes at a time (a group of G warps per node, a contiguous
// segment of E*32 elements and a private shared-memory slot per warp) and
// treats the tile as a sequence of ITEMS, one per batch of nodes:
//   sweep 1, per item: wait for the slot (bulk copies x, delta, a, c -> shared,
//     counted on the warp's mbarrier), move it to registers and take the local
//     step, issue the copies of the NEXT item (next batch, or the first batch of
//     the next tile), reduce the scale, compress: delta' and the packed codes go
//     to global memory, x - gamma g is parked in x, the codes and the decode
//     scale of the node also stay in shared memory;
//   one block barrier;
//   sweep 2, per batch: re-read the parked x - gamma g (an L2 hit), decode the
//     neighbours' codes from shared memory in registers, write x'.
// The gradient noise (and the rounding uniforms) of an item are drawn while the
// previous item is being finished, with their Philox blocks in lockstep.
// Waits on mbarriers are bounded as in ds_fused_tma_kernel.
#pragma once

#include <type_traits>

#include "ds_fused_tma_kernel.cuh"

namespace ds {

struct WideTmaSmemLayout {
    uint32_t slots_off, codes_off, scale_off, table_off, red_off, mbar_off, lut_off, rowptr_off, col_off,
        w_off, abort_off, total;
    uint32_t seg_bytes, cw;
};

__host__ __device__ inline WideTmaSmemLayout wide_tma_smem_layout(int code_bits, bool has_lut, int E,
                                                                  int nwarps, int64_t tile, int n, int nnz) {
    WideTmaSmemLayout L;
    uint32_t off = 0;
    L.seg_bytes = (uint32_t)E * 32u * 4u;
    L.cw = (uint32_t)((tile * code_bits + 31) / 32);
    L.slots_off = off;   off += (uint32_t)nwarps * 4u * L.seg_bytes;
    L.codes_off = off;   off += 2u * (uint32_t)n * L.cw * 4u;
    L.scale_off = off;   off += 2u * (uint32_t)n * 4u;
    L.table_off = off;   off += (has_lut && code_bits <= 4) ? 2u * (uint32_t)n * 16u * 4u : 0u;
    off = (off + 7u) & ~7u;
    L.red_off = off;     off += 2u * 3u * (uint32_t)nwarps * 8u;     // two alternating sets of (scale partial, two norm sums)
    L.mbar_off = off;    off += (uint32_t)nwarps * 8u;
    L.lut_off = off;     off += has_lut ? 256u * 4u : 0u;
    L.rowptr_off = off;  off += (uint32_t)(n + 1) * 4u;
    L.col_off = off;     off += (uint32_t)nnz * 4u;
    L.w_off = off;       off += (uint32_t)nnz * 4u;
    L.abort_off = off;   off += 8u;
    L.total = (off + 127u) & ~127u;
    return L;
}

template <int CODE, int NOISE, int E>
__global__ void __launch_bounds__(512, 1) ds_wide_tma_kernel(const __grid_constant__ StepParams p) {
    using T = CodeTraits<CODE>;
    static_assert(!T::kIdentity, "the identity compressor runs on other kernels");
    constexpr int V = E / 4;
    constexpr int SEG = E * 32;
    extern __shared__ __align__(128) unsigned char smem[];
    const int G = p.warps_per_group;
    const int npb = p.nodes_per_block;
    const int nwarps = blockDim.x >> 5;
    const int batches = (p.n + npb - 1) / npb;
    const WideTmaSmemLayout L = wide_tma_smem_layout(T::kBits, T::kLut, E, nwarps, p.tile, p.n, p.nnz);
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int grp = warp / G;
    const int wg = warp - grp * G;
    const int seg0 = wg * SEG;

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
    // norm-matched codes: squares of the levels in binary64 (exact), in the unused part of the table
    if constexpr (T::kNorm)
        for (int t = threadIdx.x; t < (1 << T::kBits); t += blockDim.x)
            reinterpret_cast<double*>(lut + 32)[t] = (double)p.lut[t] * (double)p.lut[t];
    for (int t = threadIdx.x; t <= p.n; t += blockDim.x) rp[t] = p.row_ptr[t];
    for (int t = threadIdx.x; t < p.nnz; t += blockDim.x) { cj[t] = p.col_idx[t]; wp[t] = p.wprime[t]; }
    if (threadIdx.x < 2) abort_sm[threadIdx.x] = 0;
    if (lane == 0) mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();

    // L2 eviction hints, chosen by the host from the shape (StepParams::l2_hints):
    //   bit 0  the staged inputs are fetched "evict first" (read once; with many nodes per column
    //          they would otherwise push the parked x - gamma g out of L2 before the second sweep)
    //   bit 1  x - gamma g is parked "evict last" and re-read "evict first"
    const uint64_t pol_first = l2_policy_evict_first();
    const uint64_t pol_last = l2_policy_evict_last();
    const bool hint_inputs = (p.l2_hints & 1) != 0;
    const bool hint_parked = (p.l2_hints & 2) != 0;
    auto seg_len_of = [&](int64_t col) -> int {
        const int64_t remain = p.N - col * p.tile;
        const int m_len = (int)(remain < p.tile ? remain : p.tile);
        return min(max(m_len - seg0, 0), SEG);
    };
    // bulk copies of this warp's segment of item (col, batch b); false if the item has nothing for this warp
    auto issue = [&](int64_t col, int b) -> bool {
        const int node = b * npb + grp;
        const int len = seg_len_of(col);
        if (node >= p.n || len <= 0) return false;
        if (DS_CHECKED_BUILD && !ds_part_ok(p, node, col * p.tile + seg0, len, T::kBits, -1)) return false;
        if (lane == 0) {
            const uint32_t bytes = (uint32_t)((len + 3) & ~3) * 4u;
            const size_t at = (size_t)node * (size_t)p.ld + (size_t)(col * p.tile) + (size_t)seg0;
            fence_proxy_async();
            constexpr uint32_t kArrays = (NOISE == GRAD_GIVEN) ? 3u : 4u;
            mbar_expect_tx(bar, kArrays * bytes);
            if (hint_inputs) {
                bulk_g2s_hint(slot_addr + 0u * L.seg_bytes, p.x + at, bytes, bar, pol_first);
                bulk_g2s_hint(slot_addr + 1u * L.seg_bytes, p.delta + at, bytes, bar, pol_first);
                bulk_g2s_hint(slot_addr + 2u * L.seg_bytes, p.a + at, bytes, bar, pol_first);
                if constexpr (NOISE != GRAD_GIVEN) bulk_g2s_hint(slot_addr + 3u * L.seg_bytes, p.c + at, bytes, bar, pol_first);
            } else {
                bulk_g2s(slot_addr + 0u * L.seg_bytes, p.x + at, bytes, bar);
                bulk_g2s(slot_addr + 1u * L.seg_bytes, p.delta + at, bytes, bar);
                bulk_g2s(slot_addr + 2u * L.seg_bytes, p.a + at, bytes, bar);
                if constexpr (NOISE != GRAD_GIVEN) bulk_g2s(slot_addr + 3u * L.seg_bytes, p.c + at, bytes, bar);
            }
        }
        return true;
    };
    // noise and rounding uniforms of item (col, b), Philox blocks in lockstep
    constexpr bool kGaussAhead = (NOISE == NOISE_GAUSS || NOISE == NOISE_T3);
    constexpr bool kRndAhead = T::kLut && !T::kNorm;
    float zn[kGaussAhead ? E : 1];
    float mn[kRndAhead ? E : 1];
    auto draw = [&](int64_t col, int b) {
        const int node = b * npb + grp;
        const uint32_t kbase = (uint32_t)(col * p.tile + seg0) + 4u * (uint32_t)lane;
        if constexpr (kGaussAhead || kRndAhead) {
            constexpr int kGa = kGaussAhead ? V : 0;
            constexpr int kRn = kRndAhead ? V : 0;
            uint32_t stream[kGa + kRn], block[kGa + kRn];
            uint4 w[kGa + kRn];
#pragma unroll
            for (int r = 0; r < V; ++r) {
                if constexpr (kGa > 0) { stream[r] = STREAM_NOISE; block[r] = (kbase + 128u * (uint32_t)r) >> 2; }
                if constexpr (kRn > 0) { stream[kGa + r] = STREAM_ROUND; block[kGa + r] = (kbase + 128u * (uint32_t)r) >> 2; }
            }
            rng_blocks<kGa + kRn>(p.rs, (uint32_t)node, stream, block, w);
#pragma unroll
            for (int r = 0; r < V; ++r) {
                if constexpr (kGa > 0) {
                    const float4 z4 = noise_of_block<NOISE>(w[r]);
                    zn[4 * r + 0] = z4.x; zn[4 * r + 1] = z4.y; zn[4 * r + 2] = z4.z; zn[4 * r + 3] = z4.w;
                }
                if constexpr (kRn > 0) {
                    const uint4 u = w[kGa + r];
                    mn[4 * r + 0] = __uint2float_rn(u.x >> 8); mn[4 * r + 1] = __uint2float_rn(u.y >> 8);
                    mn[4 * r + 2] = __uint2float_rn(u.z >> 8); mn[4 * r + 3] = __uint2float_rn(u.w >> 8);
                }
            }
        }
    };

    constexpr float kL = (float)((1u << (T::kBits & 15)) - 1u);
    constexpr float kHalfL = 0.5f * kL;
    int64_t col = p.tile_begin + blockIdx.x;
    bool pending = (col < p.tile_end) ? issue(col, 0) : false;
    if (col < p.tile_end) draw(col, 0);
    uint32_t parity = 0;
    int buf = 0, red_parity = 0;

    for (; col < p.tile_end; col += gridDim.x) {
        const int64_t k0 = col * p.tile;
        const int64_t remain = p.N - k0;
        const int m_len = (int)(remain < p.tile ? remain : p.tile);
        const int seg_len = min(max(m_len - seg0, 0), SEG);
        uint32_t* codes_sm = reinterpret_cast<uint32_t*>(smem + L.codes_off) + (size_t)buf * p.n * L.cw;
        float* scale_sm = reinterpret_cast<float*>(smem + L.scale_off) + buf * p.n;
        float* table_sm = reinterpret_cast<float*>(smem + L.table_off) + buf * p.n * 16;
        const int word0 = (seg0 * T::kBits) >> 5;         // first code word of this warp's segment in the tile

        // ================= sweep 1: one item per batch of nodes =================
        for (int b = 0; b < batches; ++b) {
            const int node = b * npb + grp;
            const bool node_ok = node < p.n;
            bool alive = true;
            if (pending) {
                alive = mbar_wait_bounded(bar, parity);
                parity ^= 1u;
                if (!alive) {
                    abort_sm[buf] = 1;
                    if (lane == 0) *p.error_flag = 1;
                }
            }
            if (DS_CHECKED_BUILD && node_ok && seg_len > 0 &&
                !ds_part_ok(p, node, k0 + seg0, seg_len, T::kBits, p.prescaled ? -1 : col)) {
                alive = false;          // refused: the warp stores nothing and the block stops after this sweep
                abort_sm[buf] = 1;
            }
            const int live_len = (alive && node_ok) ? seg_len : 0;
            const bool full = (live_len == SEG);
            const int nb = (b + 1 < batches) ? b + 1 : 0;
            const int64_t ncol = (b + 1 < batches) ? col : col + gridDim.x;
            const bool has_next = ncol < p.tile_end;
            const size_t row = (size_t)(node_ok ? node : 0) * (size_t)p.ld + (size_t)k0 + (size_t)seg0;

            auto item_body = [&](auto full_tag) {
                constexpr bool FULL = decltype(full_tag)::value;
                float* const x_lane = p.x + row + 4 * lane;
                float* const delta_lane = p.delta + row + 4 * lane;
                // ---- phase A: slot -> registers, local step, park x - gamma g ----
                float v[E];
                double sum = 0.0;
                float mx = 0.0f;
#pragma unroll
                for (int r = 0; r < V; ++r) {
                    const int e0 = 4 * (32 * r + lane);
                    const int nv = FULL ? 4 : min(max(live_len - e0, 0), 4);
                    if (nv > 0) {
                        const float4 x4 = *reinterpret_cast<const float4*>(slot_lane + 0 * SEG + 128 * r);
                        const float4 d4 = *reinterpret_cast<const float4*>(slot_lane + 1 * SEG + 128 * r);
                        const float4 a4 = *reinterpret_cast<const float4*>(slot_lane + 2 * SEG + 128 * r);
                        float h[4];
                        if constexpr (NOISE == GRAD_GIVEN) {
                            local_step4_given(x4, d4, a4, p.neg_gamma, h, &v[4 * r]);
                        } else {
                            const float4 c4 = *reinterpret_cast<const float4*>(slot_lane + 3 * SEG + 128 * r);
                            float4 z4;
                            if constexpr (kGaussAhead) z4 = make_float4(zn[4 * r + 0], zn[4 * r + 1], zn[4 * r + 2], zn[4 * r + 3]);
                            else z4 = noise4<NOISE>(p.rs, (uint32_t)node, (uint32_t)(k0 + seg0 + e0));
                            local_step4(x4, d4, a4, c4, z4, p.sigma, p.neg_gamma, h, &v[4 * r]);
                        }
                        if (FULL || nv == 4) {
                            // parked for the second sweep
                            if (hint_parked) st4_hint(x_lane + 128 * r, make_float4(h[0], h[1], h[2], h[3]), pol_last);
                            else *reinterpret_cast<float4*>(x_lane + 128 * r) = make_float4(h[0], h[1], h[2], h[3]);
                        } else {
                            for (int j = 0; j < nv; ++j) x_lane[128 * r + j] = h[j];
                        }
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            if (!FULL && j >= nv) v[4 * r + j] = 0.0f;
                            if constexpr (T::kSign) sum += (double)fabsf(v[4 * r + j]);
                            else mx = fmaxf(mx, fabsf(v[4 * r + j]));
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 4; ++j) v[4 * r + j] = 0.0f;
                    }
                }
                // the slot is in registers: refill it with this warp's segment of the next item
                __syncwarp();
                pending = has_next ? issue(ncol, nb) : false;

                // ---- scale ----
                float s;
                double* const red = reinterpret_cast<double*>(smem + L.red_off) + red_parity * (3 * nwarps);
                if (G > 1 && !p.prescaled) red_parity ^= 1;
                if (p.prescaled) {
                    if constexpr (T::kNorm) s = node_ok ? p.gmax[node] : 0.0f;       // the maximum that spans the grid
                    else s = node_ok ? p.scales[(size_t)node * (size_t)p.scales_pitch] : 0.0f;
                } else {
                    double part;
                    if constexpr (T::kSign) part = warp_sum(sum);
                    else part = (double)__uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(mx)));
                    if (G > 1) {
                        if (lane == 0) red[warp] = part;
                        // only the G warps of this node meet (named barrier 1 + group): the other
                        // groups of the block are not held back
                        asm volatile("bar.sync %0, %1;" ::"r"(1 + grp), "r"(32 * G) : "memory");
                        part = 0.0;
                        for (int w = 0; w < G; ++w) {
                            const double t = red[grp * G + w];
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
                uint32_t* const codes_lane = p.codes + (size_t)(node_ok ? node : 0) * (size_t)p.code_pitch +
                                             (size_t)(((k0 + seg0) * T::kBits) >> 5) + lane / T::kLanesPerWord;
                uint32_t* const codes_sm_lane = codes_sm + (size_t)(node_ok ? node : 0) * L.cw + word0 + lane / T::kLanesPerWord;
                // norm-matched codes: the whole chunk is coded first; s becomes the norm that is
                // sent, dscale the factor the receiver applies to the levels
                uint32_t qn[T::kNorm ? E : 1];
                float cvn[T::kNorm ? E : 1];
                float dscale = s;
                if constexpr (T::kNorm) {
                    auto valid = [&](int t) { return 4 * (32 * (t >> 2) + lane) + (t & 3) < live_len; };
                    double sv2, sl2;
                    norm_codes<CODE, E, FULL>(v, valid, s, lut, qn, cvn, sv2, sl2);
                    float nrm;
                    if (p.prescaled) {
                        nrm = node_ok ? p.scales[(size_t)node * (size_t)p.scales_pitch] : 0.0f;
                        dscale = node_ok ? p.dscales[(size_t)node * (size_t)p.scales_pitch] : 0.0f;
                    } else {
                        if (G > 1) {
                            double* red2 = red + nwarps;
                            double* red3 = red2 + nwarps;
                            if (lane == 0) { red2[warp] = sv2; red3[warp] = sl2; }
                            asm volatile("bar.sync %0, %1;" ::"r"(1 + grp), "r"(32 * G) : "memory");
                            sv2 = 0.0; sl2 = 0.0;
                            for (int w = 0; w < G; ++w) { sv2 += red2[grp * G + w]; sl2 += red3[grp * G + w]; }
                        }
                        norm_finish(s, sv2, sl2, nrm, dscale);
                    }
#pragma unroll
                    for (int t = 0; t < E; ++t) cvn[t] = __fmul_rn(dscale, cvn[t]);
                    s = nrm;
                }

                // ---- phase B: compress, residual, pack ----
#pragma unroll
                for (int r = 0; r < V; ++r) {
                    const int e0 = 4 * (32 * r + lane);
                    const int nv = FULL ? 4 : min(max(live_len - e0, 0), 4);
                    uint32_t piece = 0u;
                    if (nv > 0) {
                        float cv[4];
                        if constexpr (T::kNorm) {
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
                            uint32_t q[4];
                            quantise_recip2(v[4 * r + 0], v[4 * r + 1], s, inv_s, mn[4 * r + 0], mn[4 * r + 1], kHalfL, (int)kL, q[0], q[1]);
                            quantise_recip2(v[4 * r + 2], v[4 * r + 3], s, inv_s, mn[4 * r + 2], mn[4 * r + 3], kHalfL, (int)kL, q[2], q[3]);
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                cv[j] = __fmul_rn(s, lut[q[j]]);
                                if (FULL || j < nv) piece |= q[j] << (T::kBits * j);
                            }
                        } else {
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const float rj = __fmul_rn(mn[(kRndAhead ? 4 * r + j : 0)], 0x1p-24f);
                                const uint32_t q = degenerate ? 0u : quantise(v[4 * r + j], s, rj, kHalfL, (int)kL);
                                cv[j] = __fmul_rn(s, lut[q]);
                                if (FULL || j < nv) piece |= q << (T::kBits * j);
                            }
                        }
                        const float2 da = __fadd2_rn(make_float2(v[4 * r + 0], v[4 * r + 1]), make_float2(-cv[0], -cv[1]));
                        const float2 db = __fadd2_rn(make_float2(v[4 * r + 2], v[4 * r + 3]), make_float2(-cv[2], -cv[3]));
                        st_partial(delta_lane + 128 * r, make_float4(da.x, da.y, db.x, db.y), nv);
                    }
                    uint32_t word = piece << ((4 * T::kBits * (lane % T::kLanesPerWord)) & 31);
#pragma unroll
                    for (int o = 1; o < T::kLanesPerWord; o <<= 1) word |= __shfl_xor_sync(0xffffffffu, word, o);
                    if ((lane % T::kLanesPerWord) == 0 && (FULL || e0 < live_len)) {
                        codes_sm_lane[(32 / T::kLanesPerWord) * r] = word;
                        codes_lane[(32 / T::kLanesPerWord) * r] = word;
                    }
                }
                if (node_ok && alive && wg == 0) {
                    if (lane == 0) {
                        scale_sm[node] = dscale_of<T::kNorm>(s, dscale);
                        if (!p.prescaled) {
                            p.scales[(size_t)node * (size_t)p.scales_pitch + (size_t)col] = s;
                            if constexpr (T::kNorm) p.dscales[(size_t)node * (size_t)p.scales_pitch + (size_t)col] = dscale;
                        }
                    }
                    if constexpr (T::kTable) {
                        if (lane < (1 << T::kBits)) table_sm[node * 16 + lane] = __fmul_rn(dscale_of<T::kNorm>(s, dscale), lut[lane]);
                    }
                }
                // the randomness of the next item, while its copies are in flight
                if (has_next) draw(ncol, nb);
            };
            if (full) item_body(std::true_type{});
            else item_body(std::false_type{});
        }
        __syncthreads();          // codes and scales of all n nodes of the tile are in shared memory
        if (abort_sm[buf]) break;

        // ================= sweep 2: mix, one batch of nodes at a time =================
        for (int b = 0; b < batches; ++b) {
            const int node = b * npb + grp;
            if (node >= p.n || seg_len <= 0) continue;
            if (DS_CHECKED_BUILD && !ds_part_ok(p, node, k0 + seg0, seg_len, T::kBits, -1)) continue;
            float* const x_lane = p.x + (size_t)node * (size_t)p.ld + (size_t)k0 + (size_t)seg0 + 4 * lane;
            auto mix_body = [&](auto full_tag) {
                constexpr bool FULL = decltype(full_tag)::value;
                // the parked x - gamma g (this block's own earlier stores, ordered by the barrier)
                float4 hv[V];
#pragma unroll
                for (int r = 0; r < V; ++r) {
                    const int e0 = 4 * (32 * r + lane);
                    const int nv = FULL ? 4 : min(max(seg_len - e0, 0), 4);
                    hv[r] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (nv == 4) {
                        if (hint_parked) hv[r] = ld4_hint(x_lane + 128 * r, pol_first);      // last use of the parked line
                        else hv[r] = *reinterpret_cast<const float4*>(x_lane + 128 * r);
                    } else if (nv > 0) {
                        float* hp = reinterpret_cast<float*>(&hv[r]);
                        for (int j = 0; j < nv; ++j) hp[j] = x_lane[128 * r + j];
                    }
                }
                float acc[E];
#pragma unroll
                for (int t = 0; t < E; ++t) acc[t] = 0.0f;
                const int e_beg = rp[node], e_end = rp[node + 1];
                for (int e = e_beg; e < e_end; ++e) {
                    const int j = cj[e];
                    const float w = wp[e];
                    const float sj = scale_sm[j];
                    const float* table_j = table_sm + j * 16;
                    const uint32_t* row_j = codes_sm + (size_t)j * L.cw + word0 + lane / T::kLanesPerWord;
#pragma unroll
                    for (int r = 0; r < V; ++r) {
                        if (!FULL && 4 * (32 * r + lane) >= seg_len) continue;
                        const uint32_t word = row_j[(32 / T::kLanesPerWord) * r];
                        const uint32_t piece = (word >> ((4 * T::kBits * (lane % T::kLanesPerWord)) & 31)) & T::kPieceMask;
                        float cv[4];
#pragma unroll
                        for (int t = 0; t < 4; ++t) {
                            if constexpr (T::kSign) {
                                const uint32_t neg = (~piece << (31 - t)) & 0x80000000u;
                                cv[t] = __uint_as_float(__float_as_uint(sj) ^ neg);
                            } else {
                                const uint32_t q = (piece >> (T::kBits * t)) & ((1u << T::kBits) - 1u);
                                if constexpr (T::kTable) cv[t] = table_j[q];
                                else cv[t] = __fmul_rn(sj, lut[q]);
                            }
                        }
                        const float2 w2 = splat(w);
                        const float2 aa = __ffma2_rn(w2, make_float2(cv[0], cv[1]), make_float2(acc[4 * r + 0], acc[4 * r + 1]));
                        const float2 ab = __ffma2_rn(w2, make_float2(cv[2], cv[3]), make_float2(acc[4 * r + 2], acc[4 * r + 3]));
                        acc[4 * r + 0] = aa.x; acc[4 * r + 1] = aa.y; acc[4 * r + 2] = ab.x; acc[4 * r + 3] = ab.y;
                    }
                }
#pragma unroll
                for (int r = 0; r < V; ++r) {
                    const int e0 = 4 * (32 * r + lane);
                    const int nv = FULL ? 4 : min(max(seg_len - e0, 0), 4);
                    if (nv > 0) {
                        const float2 et = splat(p.eta);
                        const float2 xa = __ffma2_rn(et, make_float2(acc[4 * r + 0], acc[4 * r + 1]), make_float2(hv[r].x, hv[r].y));
                        const float2 xb = __ffma2_rn(et, make_float2(acc[4 * r + 2], acc[4 * r + 3]), make_float2(hv[r].z, hv[r].w));
                        st_partial(x_lane + 128 * r, make_float4(xa.x, xa.y, xb.x, xb.y), nv);
                    }
                }
            };
            if (seg_len == SEG) mix_body(std::true_type{});
            else mix_body(std::false_type{});
        }
        buf ^= 1;
    }
    // error path: let a copy that is still in flight land before shared memory is given away
    if (pending) (void)mbar_wait_bounded(bar, parity);
}

template <int CODE, int NOISE, int E>
cudaError_t launch_wide_tma_one(const LaunchShape& sh, const StepParams& p, cudaStream_t stream) {
    auto kern = ds_wide_tma_kernel<CODE, NOISE, E>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh.smem);
    if (e != cudaSuccess) return e;
    kern<<<sh.grid, sh.block, sh.smem, stream>>>(p);
    return cudaGetLastError();
}

template <int CODE>
cudaError_t launch_wide_tma_code(const LaunchShape& sh, const StepParams& p, cudaStream_t stream) {
#define DS_WT_CASE(NZ, EE) \
    if (sh.noise == NZ && sh.elems_per_lane == EE) return launch_wide_tma_one<CODE, NZ, EE>(sh, p, stream);
    DS_WT_CASE(NOISE_NONE, 8) DS_WT_CASE(NOISE_NONE, 16)
    DS_WT_CASE(NOISE_GAUSS, 8) DS_WT_CASE(NOISE_GAUSS, 16)
    DS_WT_CASE(NOISE_T3, 8) DS_WT_CASE(NOISE_T3, 16)
    DS_WT_CASE(NOISE_T3I, 8) DS_WT_CASE(NOISE_T3I, 16)
    DS_WT_CASE(GRAD_GIVEN, 8) DS_WT_CASE(GRAD_GIVEN, 16)
#undef DS_WT_CASE
    return cudaErrorInvalidValue;
}
}  // namespace ds
