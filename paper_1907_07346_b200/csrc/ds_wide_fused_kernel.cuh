// Fused kernel for columns too wide for one pass (many nodes or long chunks).
//
// A block still owns one column tile of ALL n nodes, but holds only
// `nodes_per_block` of them at a time: it sweeps the nodes in batches, first
// compressing every batch (x - gamma g is parked in x itself, delta', codes and
// scales are final), then -- after one block barrier -- sweeping the batches
// again to mix: each thread re-reads the x - gamma g it parked (its own earlier
// store, still in L2: the block touches the same few hundred KB in both sweeps),
// decodes its neighbours' packed codes from shared memory in registers and
// writes x'.  DRAM traffic stays at the algorithmic bytes as long as the parked
// lines survive in L2 between the two sweeps; the price is one extra L2 round
// trip of 8 bytes per element.
//
// Steps of Algorithm 1: gradient and error-compensated variable (sweep 1, phase
// A), compression and residual (sweep 1, phase B), local update (sweep 2).
#pragma once

#include "ds_column_kernel.cuh"

namespace ds {

struct WideSmemLayout {
    uint32_t codes_off, scale_off, table_off, red_off, lut_off, rowptr_off, col_off, w_off, total;
    uint32_t cw;
};

__host__ __device__ inline WideSmemLayout wide_smem_layout(int code_bits, bool has_lut, int npb, int G,
                                                           int64_t tile, int n, int nnz) {
    WideSmemLayout L;
    uint32_t off = 0;
    L.cw = (uint32_t)((tile * code_bits + 31) / 32);
    L.red_off = off;     off += 2u * 3u * (uint32_t)(npb * G) * 8u;   // two alternating sets of (scale partial, two norm sums)
    L.codes_off = off;   off += 2u * (uint32_t)n * L.cw * 4u;
    L.scale_off = off;   off += 2u * (uint32_t)n * 4u;
    L.table_off = off;   off += (has_lut && code_bits <= 4) ? 2u * (uint32_t)n * 16u * 4u : 0u;
    L.lut_off = off;     off += has_lut ? 256u * 4u : 0u;
    L.rowptr_off = off;  off += (uint32_t)(n + 1) * 4u;
    L.col_off = off;     off += (uint32_t)nnz * 4u;
    L.w_off = off;       off += (uint32_t)nnz * 4u;
    L.total = (off + 15u) & ~15u;
    return L;
}

template <int CODE, int NOISE, int E, bool FULL>
__device__ __forceinline__ void wide_column(const StepParams& p, const WideSmemLayout& L,
                                            unsigned char* smem, int64_t col, int buf, int& red_parity,
                                            int lane, int grp, int wg) {
    using T = CodeTraits<CODE>;
    constexpr int V = E / 4;
    const int G = p.warps_per_group;
    const int npb = p.nodes_per_block;
    const int batches = (p.n + npb - 1) / npb;
    const int64_t k0 = col * p.tile;
    const int64_t remain = p.N - k0;
    const int m_len = (int)(remain < p.tile ? remain : p.tile);
    const int fstride = 32 * G;
    const int f0 = wg * 32 + lane;
    constexpr float kL = (float)((1u << (T::kBits & 15)) - 1u);
    constexpr float kHalfL = 0.5f * kL;

    const float* lut = reinterpret_cast<const float*>(smem + L.lut_off);
    uint32_t* codes_sm = reinterpret_cast<uint32_t*>(smem + L.codes_off) + (size_t)buf * p.n * L.cw;
    float* scale_sm = reinterpret_cast<float*>(smem + L.scale_off) + buf * p.n;
    float* table_sm = reinterpret_cast<float*>(smem + L.table_off) + buf * p.n * 16;

    // ---------------- sweep 1: compress every batch of nodes ----------------
    for (int b = 0; b < batches; ++b) {
        const int node = b * npb + grp;
        bool node_ok = node < p.n;
        // checked build: a refused (node, tile) is treated like a node beyond the last one
        if (DS_CHECKED_BUILD && node_ok && !ds_part_ok(p, node, k0, m_len, T::kBits, p.prescaled ? -1 : col)) node_ok = false;
        const size_t row = (size_t)node * (size_t)p.ld + (size_t)k0;
        float v[E];
        double sum = 0.0;
        float mx = 0.0f;
#pragma unroll
        for (int r = 0; r < V; ++r) {
            const int e0 = 4 * (f0 + fstride * r);
            const int nv = !node_ok ? 0 : (FULL ? 4 : min(max(m_len - e0, 0), 4));
            if (nv > 0) {
                const float4 x4 = ld4(p.x + row + e0);
                const float4 d4 = ld4(p.delta + row + e0);
                const float4 a4 = ld4(p.a + row + e0);      // the gradient itself when it is given
                float h[4];
                if constexpr (NOISE == GRAD_GIVEN) {
                    local_step4_given(x4, d4, a4, p.neg_gamma, h, &v[4 * r]);
                } else {
                    const float4 c4 = ld4(p.c + row + e0);
                    const float4 z4 = noise4<NOISE>(p.rs, (uint32_t)node, (uint32_t)(k0 + e0));
                    local_step4(x4, d4, a4, c4, z4, p.sigma, p.neg_gamma, h, &v[4 * r]);
                }
                // park x - gamma g in x (read back by this same thread in sweep 2)
                if (FULL || nv == 4) {
                    *reinterpret_cast<float4*>(p.x + row + e0) = make_float4(h[0], h[1], h[2], h[3]);
                } else {
                    for (int j = 0; j < nv; ++j) p.x[row + e0 + j] = h[j];
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
        float s;
        // two sets of partials, alternating: a fast warp may already write the
        // next batch's partial while a slow one still reads this batch's
        double* const red = reinterpret_cast<double*>(smem + L.red_off) + red_parity * (3 * npb * G);
        if (G > 1 && !p.prescaled) red_parity ^= 1;
        if (p.prescaled) {
            if constexpr (T::kNorm) s = node_ok ? p.gmax[node] : 0.0f;       // the maximum that spans the grid
            else s = node_ok ? p.scales[(size_t)node * (size_t)p.scales_pitch] : 0.0f;
        } else {
            double part;
            if constexpr (T::kSign) part = warp_sum(sum);
            else part = (double)__uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(mx)));
            if (G > 1) {
                if (lane == 0) red[grp * G + wg] = part;
                __syncthreads();
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
        const size_t code_row = (size_t)node * (size_t)p.code_pitch + (size_t)((k0 * T::kBits) >> 5);
        // norm-matched codes: the whole chunk is coded first; s becomes the norm that is sent,
        // dscale the factor the receiver applies to the levels
        uint32_t qn[T::kNorm ? E : 1];
        float cvn[T::kNorm ? E : 1];
        float dscale = s;
        if constexpr (T::kNorm) {
            auto valid = [&](int t) { return node_ok && 4 * (f0 + fstride * (t >> 2)) + (t & 3) < m_len; };
            double sv2, sl2;
            norm_codes<CODE, E, FULL>(v, valid, s, lut, qn, cvn, sv2, sl2);
            float nrm;
            if (p.prescaled) {
                nrm = node_ok ? p.scales[(size_t)node * (size_t)p.scales_pitch] : 0.0f;
                dscale = node_ok ? p.dscales[(size_t)node * (size_t)p.scales_pitch] : 0.0f;
            } else {
                if (G > 1) {
                    double* red2 = red + npb * G;
                    double* red3 = red2 + npb * G;
                    if (lane == 0) { red2[grp * G + wg] = sv2; red3[grp * G + wg] = sl2; }
                    __syncthreads();
                    sv2 = 0.0; sl2 = 0.0;
                    for (int w = 0; w < G; ++w) { sv2 += red2[grp * G + w]; sl2 += red3[grp * G + w]; }
                }
                norm_finish(s, sv2, sl2, nrm, dscale);
            }
#pragma unroll
            for (int t = 0; t < E; ++t) cvn[t] = __fmul_rn(dscale, cvn[t]);
            s = nrm;
        }
#pragma unroll
        for (int r = 0; r < V; ++r) {
            const int f = f0 + fstride * r;
            const int e0 = 4 * f;
            const int nv = !node_ok ? 0 : (FULL ? 4 : min(max(m_len - e0, 0), 4));
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
                    const float4 rr = rnd24x4_unscaled(p.rs, (uint32_t)node, (uint32_t)(k0 + e0));
                    uint32_t q[4];
                    quantise_recip2(v[4 * r + 0], v[4 * r + 1], s, inv_s, rr.x, rr.y, kHalfL, (int)kL, q[0], q[1]);
                    quantise_recip2(v[4 * r + 2], v[4 * r + 3], s, inv_s, rr.z, rr.w, kHalfL, (int)kL, q[2], q[3]);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        cv[j] = __fmul_rn(s, lut[q[j]]);
                        if (FULL || j < nv) piece |= q[j] << (T::kBits * j);
                    }
                } else {
                    const float4 rr = rnd24x4(p.rs, (uint32_t)node, (uint32_t)(k0 + e0));
                    const float rv[4] = {rr.x, rr.y, rr.z, rr.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint32_t q = degenerate ? 0u : quantise(v[4 * r + j], s, rv[j], kHalfL, (int)kL);
                        cv[j] = __fmul_rn(s, lut[q]);
                        if (FULL || j < nv) piece |= q << (T::kBits * j);
                    }
                }
                const float2 da = __fadd2_rn(make_float2(v[4 * r + 0], v[4 * r + 1]), make_float2(-cv[0], -cv[1]));
                const float2 db = __fadd2_rn(make_float2(v[4 * r + 2], v[4 * r + 3]), make_float2(-cv[2], -cv[3]));
                st_partial(p.delta + row + e0, make_float4(da.x, da.y, db.x, db.y), nv);
            }
            uint32_t word = piece << ((4 * T::kBits * (lane % T::kLanesPerWord)) & 31);
#pragma unroll
            for (int o = 1; o < T::kLanesPerWord; o <<= 1) word |= __shfl_xor_sync(0xffffffffu, word, o);
            if ((lane % T::kLanesPerWord) == 0 && node_ok && e0 < m_len) {
                codes_sm[(size_t)node * L.cw + f / T::kLanesPerWord] = word;
                p.codes[code_row + f / T::kLanesPerWord] = word;
            }
        }
        if (node_ok && wg == 0) {
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
    }
    __syncthreads();        // codes and scales of all n nodes of this tile are in shared memory

    // ---------------- sweep 2: mix every batch of nodes ---------------------
    const int32_t* rp = reinterpret_cast<const int32_t*>(smem + L.rowptr_off);
    const int32_t* cj = reinterpret_cast<const int32_t*>(smem + L.col_off);
    const float* wp = reinterpret_cast<const float*>(smem + L.w_off);
    for (int b = 0; b < batches; ++b) {
        const int node = b * npb + grp;
        if (node >= p.n) continue;
        if (DS_CHECKED_BUILD && !ds_part_ok(p, node, k0, m_len, T::kBits, -1)) continue;
        const size_t row = (size_t)node * (size_t)p.ld + (size_t)k0;
        float acc[E];
#pragma unroll
        for (int t = 0; t < E; ++t) acc[t] = 0.0f;
        const int e_beg = rp[node], e_end = rp[node + 1];
        for (int e = e_beg; e < e_end; ++e) {
            const int j = cj[e];
            const float w = wp[e];
            const float sj = scale_sm[j];
            const float* table_j = table_sm + j * 16;
            const uint32_t* row_j = codes_sm + (size_t)j * L.cw;
#pragma unroll
            for (int r = 0; r < V; ++r) {
                const int f = f0 + fstride * r;
                if (!FULL && 4 * f >= m_len) continue;
                const uint32_t word = row_j[f / T::kLanesPerWord];
                const uint32_t piece = (word >> ((4 * T::kBits * (f % T::kLanesPerWord)) & 31)) & T::kPieceMask;
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
            const int e0 = 4 * (f0 + fstride * r);
            const int nv = FULL ? 4 : min(max(m_len - e0, 0), 4);
            if (nv == 4) {
                const float4 h4 = *reinterpret_cast<const float4*>(p.x + row + e0);
                const float2 et = splat(p.eta);
                const float2 xa = __ffma2_rn(et, make_float2(acc[4 * r + 0], acc[4 * r + 1]), make_float2(h4.x, h4.y));
                const float2 xb = __ffma2_rn(et, make_float2(acc[4 * r + 2], acc[4 * r + 3]), make_float2(h4.z, h4.w));
                st4(p.x + row + e0, make_float4(xa.x, xa.y, xb.x, xb.y));
            } else {
                for (int j = 0; j < nv; ++j)
                    p.x[row + e0 + j] = __fmaf_rn(p.eta, acc[4 * r + j], p.x[row + e0 + j]);
            }
        }
    }
}

template <int CODE, int NOISE, int E>
__global__ void __launch_bounds__(512, 2) ds_wide_fused_kernel(const __grid_constant__ StepParams p) {
    using T = CodeTraits<CODE>;
    static_assert(!T::kIdentity, "the identity compressor runs on the two-kernel path");
    extern __shared__ __align__(16) unsigned char smem[];
    const int G = p.warps_per_group;
    const WideSmemLayout L = wide_smem_layout(T::kBits, T::kLut, p.nodes_per_block, G, p.tile, p.n, p.nnz);
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int grp = warp / G;
    const int wg = warp - grp * G;

    if constexpr (T::kLut) {
        float* lut = reinterpret_cast<float*>(smem + L.lut_off);
        for (int t = threadIdx.x; t < (1 << T::kBits); t += blockDim.x) lut[t] = p.lut[t];
        // norm-matched codes: squares of the levels in binary64 (exact), in the unused part of the table
        if constexpr (T::kNorm)
            for (int t = threadIdx.x; t < (1 << T::kBits); t += blockDim.x)
                reinterpret_cast<double*>(lut + 32)[t] = (double)p.lut[t] * (double)p.lut[t];
    }
    int32_t* rp = reinterpret_cast<int32_t*>(smem + L.rowptr_off);
    int32_t* cj = reinterpret_cast<int32_t*>(smem + L.col_off);
    float* wp = reinterpret_cast<float*>(smem + L.w_off);
    for (int t = threadIdx.x; t <= p.n; t += blockDim.x) rp[t] = p.row_ptr[t];
    for (int t = threadIdx.x; t < p.nnz; t += blockDim.x) { cj[t] = p.col_idx[t]; wp[t] = p.wprime[t]; }
    __syncthreads();

    const int64_t full_len = (int64_t)E * 32 * G;
    int buf = 0, red_parity = 0;
    for (int64_t col = p.tile_begin + blockIdx.x; col < p.tile_end; col += gridDim.x) {
        const int64_t remain = p.N - col * p.tile;
        const bool full = (p.tile == full_len) && (remain >= p.tile);
        if (full) wide_column<CODE, NOISE, E, true>(p, L, smem, col, buf, red_parity, lane, grp, wg);
        else wide_column<CODE, NOISE, E, false>(p, L, smem, col, buf, red_parity, lane, grp, wg);
        buf ^= 1;
    }
}

template <int CODE, int NOISE, int E>
cudaError_t launch_wide_one(const LaunchShape& sh, const StepParams& p, cudaStream_t stream) {
    auto kern = ds_wide_fused_kernel<CODE, NOISE, E>;
    if (sh.smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh.smem);
        if (e != cudaSuccess) return e;
    }
    kern<<<sh.grid, sh.block, sh.smem, stream>>>(p);
    return cudaGetLastError();
}

template <int CODE>
cudaError_t launch_wide_code(const LaunchShape& sh, const StepParams& p, cudaStream_t stream) {
#define DS_WIDE_CASE(NZ, EE) \
    if (sh.noise == NZ && sh.elems_per_lane == EE) return launch_wide_one<CODE, NZ, EE>(sh, p, stream);
    DS_WIDE_CASE(NOISE_NONE, 4) DS_WIDE_CASE(NOISE_NONE, 8) DS_WIDE_CASE(NOISE_NONE, 16)
    DS_WIDE_CASE(NOISE_GAUSS, 4) DS_WIDE_CASE(NOISE_GAUSS, 8) DS_WIDE_CASE(NOISE_GAUSS, 16)
    DS_WIDE_CASE(NOISE_T3, 4) DS_WIDE_CASE(NOISE_T3, 8) DS_WIDE_CASE(NOISE_T3, 16)
    DS_WIDE_CASE(NOISE_T3I, 4) DS_WIDE_CASE(NOISE_T3I, 8) DS_WIDE_CASE(NOISE_T3I, 16)
    DS_WIDE_CASE(GRAD_GIVEN, 4) DS_WIDE_CASE(GRAD_GIVEN, 8) DS_WIDE_CASE(GRAD_GIVEN, 16)
#undef DS_WIDE_CASE
    return cudaErrorInvalidValue;
}

}  // namespace ds
