// The column kernel: gradient + error-compensated compress (+ gossip mix).
//
// Work decomposition.  A row (node) is cut into column tiles of `tile`
// elements (one compressor chunk, or a free tile width when the scale is per
// node).  A group of G warps owns one (node, tile): each lane holds E
// consecutive-by-four elements in registers from the first load until the last
// store.  A thread block holds the groups of `nodes_per_block` nodes for the
// same tile.
//
//   MODE_FUSED     the block holds ALL n nodes of the tile.  After the codes of
//                  the tile are in shared memory (one block barrier), every
//                  group decodes its neighbours' codes from shared memory and
//                  writes x' -- x - gamma g never leaves the registers and
//                  nothing is re-read from global memory.
//   MODE_COMPRESS  first half of the two-kernel path: writes x - gamma g into
//                  x, delta', codes and scales; the mix kernel finishes.
//                  With StepParams::ecsgd set it is the worker half of
//                  centralized error-compensated SGD (Section 1): v = g + delta
//                  is compressed, delta' and the codes are written, x is not.
//   MODE_REDUCE    only the per-(node, tile) partial of the scale reduction
//                  (used when one scale covers a whole node).
//
// Steps of Algorithm 1 per element: gradient and error-compensated variable
// (local_step), compression and residual (phase B), local update (phase C).
#pragma once

#include "ds_internal.h"

namespace ds {

struct SmemLayout {
    uint32_t codes_off, scale_off, table_off, red_off, lut_off, rowptr_off, col_off, w_off, total;
    uint32_t cw;   // code words per (node, tile)
};

__host__ __device__ inline SmemLayout smem_layout(int mode, int code_bits, bool has_lut,
                                                  int npb, int G, int64_t tile, int n, int nnz) {
    SmemLayout L;
    uint32_t off = 0;
    L.cw = (uint32_t)((tile * code_bits + 31) / 32);
    L.red_off = off;                      // three binary64 slots per warp: scale partial, two norm sums
    off += (G > 1) ? 3u * (uint32_t)(npb * G) * 8u : 0u;
    L.codes_off = off;
    off += (mode == MODE_FUSED) ? 2u * (uint32_t)npb * L.cw * 4u : 0u;
    L.scale_off = off;
    off += (mode == MODE_FUSED) ? 2u * (uint32_t)npb * 4u : 0u;
    // decode tables s_j * level[q] of the tile, for codes of up to 4 bits
    L.table_off = off;
    off += (mode == MODE_FUSED && has_lut && code_bits <= 4) ? 2u * (uint32_t)npb * 16u * 4u : 0u;
    L.lut_off = off;
    off += has_lut ? 256u * 4u : 0u;
    L.rowptr_off = off;
    off += (mode == MODE_FUSED) ? (uint32_t)(n + 1) * 4u : 0u;
    L.col_off = off;
    off += (mode == MODE_FUSED) ? (uint32_t)nnz * 4u : 0u;
    L.w_off = off;
    off += (mode == MODE_FUSED) ? (uint32_t)nnz * 4u : 0u;
    L.total = (off + 15u) & ~15u;
    return L;
}

template <int CODE>
struct CodeTraits {
    static constexpr bool kSign = (CODE == CODE_SIGN);
    static constexpr bool kIdentity = (CODE == CODE_ID32);
    static constexpr bool kNorm = (CODE == CODE_N2 || CODE == CODE_N4);
    static constexpr int kBits = (CODE == CODE_SIGN || CODE == CODE_U1) ? 1
                               : (CODE == CODE_U2 || CODE == CODE_N2) ? 2
                               : (CODE == CODE_U4 || CODE == CODE_N4) ? 4
                               : (CODE == CODE_U8) ? 8 : 32;
    static constexpr bool kLut = !(kSign || kIdentity);
    static constexpr bool kTable = kLut && kBits <= 4;   // per-node decode table in shared memory
    // lanes whose four-element pieces share one 32-bit code word
    static constexpr int kLanesPerWord = (kBits >= 8) ? 1 : 8 / kBits;
    static constexpr uint32_t kPieceMask = (kBits >= 8) ? 0xffffffffu : ((1u << (4 * kBits)) - 1u);
};

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Norm-matched b-bit compression (Section 5, "Compression": b bits per element
// plus the Euclidean norm of the tensor; the receiver rescales what it decodes
// to that norm), in two halves so that a chunk may be spread over several warps
// or, with one norm per node, over several launches:
//   m = max |v| spans the grid; code = clamp(floor(fma(v/m, L/2, L/2) + 1/2), 0, L)
//   (round to nearest level); l_k = level[code];
//   nrm = sqrt(sum v_k^2), lnorm = sqrt(sum l_k^2) (binary64 sums, rounded to binary32);
//   r = nrm / lnorm;  C_k = r * l_k.
// norm_codes(): codes and levels of the E elements a lane holds, and the two
// binary64 sums over the WARP's valid elements (lane order, then a butterfly);
// valid(t) tells whether the lane's element t counts.  m = 0 or not finite:
// codes 0.  The caller adds up the sums of the chunk's warps in warp order.
template <int CODE, int E, bool FULL, class ValidFn>
__device__ __forceinline__ void norm_codes(const float* v, ValidFn valid, float m, const float* lut,
                                           uint32_t* q, float* lv, double& sv2_out, double& sl2_out) {
    constexpr int kBits = (CODE == CODE_N2) ? 2 : 4;
    constexpr int kLi = (1 << kBits) - 1;
    constexpr float kHalfL = 0.5f * (float)kLi;
    const bool dead = (m == 0.0f) || !(m <= 3.402823466e+38f);
    const bool fast = !dead && m >= 0x1p-60f && m <= 0x1p+60f;
    const float inv = fast ? __fdiv_rn(1.0f, m) : 0.0f;
    double sv2 = 0.0, sl2 = 0.0;
    // level[q]^2 in binary64, stored behind the 16 levels of the table: a product of two binary32
    // numbers is exact in binary64, so adding the stored square rounds exactly like the fused form
    const double* lut_sq = reinterpret_cast<const double*>(lut + 32);
    // u + 1/2 for all elements: on the packed binary32x2 pipe when the reciprocal form of the
    // quotient applies (each half rounds like the scalar operation), else element by element
    float up[E];
    if (fast) {
        const float2 iv = splat(inv), hl = splat(kHalfL);
#pragma unroll
        for (int t = 0; t < E; t += 2) {
            const float2 vv = make_float2(v[t], v[t + 1]);
            const float2 q0 = __fmul2_rn(vv, iv);
            const float2 rem = __ffma2_rn(make_float2(-q0.x, -q0.y), splat(m), vv);
            const float2 y = __ffma2_rn(rem, iv, q0);
            const float2 u = __ffma2_rn(y, hl, hl);
            const float2 h = __fadd2_rn(u, splat(0.5f));
            up[t] = h.x; up[t + 1] = h.y;
        }
    } else {
#pragma unroll
        for (int t = 0; t < E; ++t) {
            const float y = dead ? 0.0f : __fdiv_rn(v[t], m);
            up[t] = __fadd_rn(__fmaf_rn(y, kHalfL, kHalfL), 0.5f);
        }
    }
#pragma unroll
    for (int t = 0; t < E; ++t) {
        const bool ok = FULL || valid(t);
        const uint32_t code = dead ? 0u : (uint32_t)min(max(__float2int_rd(up[t]), 0), kLi);
        q[t] = code;
        lv[t] = lut[code];
        if (ok) {
            // products of two binary32 numbers are exact in binary64, so the fused
            // form rounds exactly like "sum += product"
            sv2 = __fma_rn((double)v[t], (double)v[t], sv2);
            sl2 = __dadd_rn(sl2, lut_sq[code]);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        sv2 += __shfl_xor_sync(0xffffffffu, sv2, o);
        sl2 += __shfl_xor_sync(0xffffffffu, sl2, o);
    }
    sv2_out = sv2;
    sl2_out = sl2;
}

// norm_finish(): from the two sums of the whole chunk the scalar that is sent
// (nrm) and the factor the receiver applies to the levels (r).  m = 0 or not
// finite, or a norm that is not finite: nrm = r = 0.
__device__ __forceinline__ void norm_finish(float m, double sv2, double sl2, float& nrm, float& r) {
    const bool dead = (m == 0.0f) || !(m <= 3.402823466e+38f);
    nrm = dead ? 0.0f : (float)sqrt(sv2);
    const float lnorm = (float)sqrt(sl2);
    r = (dead || lnorm == 0.0f || !(nrm <= 3.402823466e+38f)) ? 0.0f : __fdiv_rn(nrm, lnorm);
    if (!(nrm <= 3.402823466e+38f)) nrm = 0.0f;
}

// The factor a receiver multiplies the levels by: the scale that is sent, except for
// norm-matched codes, where the sent scalar is the norm and the factor norm / ||levels||.
template <bool NORM>
__device__ __forceinline__ float dscale_of(float sent, float factor) { return NORM ? factor : sent; }

__device__ __forceinline__ float4 ld4(const float* p) {
    return __ldcs(reinterpret_cast<const float4*>(p));
}
__device__ __forceinline__ void st4(float* p, float4 v) {
    __stcs(reinterpret_cast<float4*>(p), v);
}

// Store the first nv (1..4) elements of v at p.
__device__ __forceinline__ void st_partial(float* p, float4 v, int nv) {
    if (nv >= 4) { st4(p, v); return; }
    p[0] = v.x;
    if (nv > 1) p[1] = v.y;
    if (nv > 2) p[2] = v.z;
}

template <int CODE, int NOISE, int E, int MODE, bool FULL>
__device__ __forceinline__ void column_body(const StepParams& p, const SmemLayout& L,
                                            unsigned char* smem, int64_t col, int buf,
                                            int lane, int grp, int wg, int node, bool node_ok) {   // (node_ok: by value)
    using T = CodeTraits<CODE>;
    constexpr int V = E / 4;
    const int G = p.warps_per_group;
    const int64_t k0 = col * p.tile;
    const int64_t remain = p.N - k0;
    const int m_len = (int)(remain < p.tile ? remain : p.tile);
    const int fstride = 32 * G;
    const int f0 = wg * 32 + lane;
    const size_t row = (size_t)node * (size_t)p.ld + (size_t)k0;
    // checked build: a refused (node, tile) is treated like a node beyond the last one
    // (no loads, no stores; the block's barriers are still met)
    if (DS_CHECKED_BUILD && node_ok &&
        !ds_part_ok(p, node, k0, m_len, MODE == MODE_REDUCE ? 0 : T::kBits,      // (a reduction writes no codes)
                    (T::kIdentity || p.prescaled || MODE == MODE_REDUCE) ? -1 : col))
        node_ok = false;
    if (DS_CHECKED_BUILD && MODE == MODE_REDUCE && node_ok && !ds_partial_ok(p, node, p.n, col)) node_ok = false;

    float h[E], v[E];

    // ---------------- phase A: local step, scale partial -----------------
    double sum = 0.0;
    float mx = 0.0f;
#pragma unroll
    for (int r = 0; r < V; ++r) {
        const int e0 = 4 * (f0 + fstride * r);
        const int nv = FULL ? 4 : (node_ok ? min(max(m_len - e0, 0), 4) : 0);
        if (FULL ? node_ok : (nv > 0)) {
            const float4 x4 = ld4(p.x + row + e0);
            const float4 d4 = ld4(p.delta + row + e0);
            const float4 a4 = ld4(p.a + row + e0);      // the gradient itself when it is given
            if constexpr (NOISE == GRAD_GIVEN) {
                local_step4_given(x4, d4, a4, p.neg_gamma, &h[4 * r], &v[4 * r]);
                if (MODE != MODE_FUSED && p.ecsgd) worker_step4_given(d4, a4, &v[4 * r]);
            } else {
                const float4 c4 = ld4(p.c + row + e0);
                const float4 z4 = noise4<NOISE>(p.rs, (uint32_t)node, (uint32_t)(k0 + e0));
                if (MODE != MODE_FUSED && p.ecsgd) {
                    worker_step4(x4, d4, a4, c4, z4, p.sigma, &v[4 * r]);
#pragma unroll
                    for (int j = 0; j < 4; ++j) h[4 * r + j] = 0.0f;
                } else {
                    local_step4(x4, d4, a4, c4, z4, p.sigma, p.neg_gamma, &h[4 * r], &v[4 * r]);
                }
            }
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

    // ---------------- scale of the (node, tile) --------------------------
    float s = 1.0f;
    // norm-matched codes with one norm per node take two reductions: the maximum that spans
    // the grid (norm_phase 0, like every per-node scale), then, with the maximum known, the two
    // sums of squares (norm_phase 2)
    const bool norm_sums_pass = T::kNorm && MODE == MODE_REDUCE && p.norm_phase == 2;
    if constexpr (!T::kIdentity) {
        if (p.prescaled && (MODE != MODE_REDUCE || norm_sums_pass)) {
            if constexpr (T::kNorm) s = node_ok ? p.gmax[node] : 0.0f;
            else s = node_ok ? p.scales[(size_t)node * (size_t)p.scales_pitch] : 0.0f;
        } else {
            double part;
            if constexpr (T::kSign) part = warp_sum(sum);
            else part = (double)__uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(mx)));
            if (G > 1) {
                double* red = reinterpret_cast<double*>(smem + L.red_off);
                if (lane == 0) red[grp * G + wg] = part;
                __syncthreads();
                part = 0.0;
                for (int w = 0; w < G; ++w) {
                    const double t = red[grp * G + w];
                    if constexpr (T::kSign) part += t;
                    else part = fmax(part, t);
                }
                if (MODE == MODE_REDUCE || MODE == MODE_COMPRESS) __syncthreads();   // red reused next tile
            }
            if constexpr (MODE == MODE_REDUCE) {
                if (node_ok && wg == 0 && lane == 0)
                    p.partials[(size_t)node * (size_t)p.tiles + (size_t)col] = part;
                return;
            }
            if constexpr (T::kSign) {
                s = (float)(part / (double)m_len);
            } else {
                s = (float)part;
                if (s == 0.0f || !(fabsf(s) <= 3.402823466e+38f)) s = 0.0f;
            }
        }
    }
    if constexpr (MODE == MODE_REDUCE && !T::kNorm) return;
    const bool degenerate = (!T::kSign && !T::kIdentity && s == 0.0f);
    // the quotient v/s may use the reciprocal only while s is far from the
    // ends of the exponent range (uniform over the group)
    const bool fast = T::kLut && s >= 0x1p-60f && s <= 0x1p+60f;
    const float inv_s = fast ? __fdiv_rn(1.0f, s) : 0.0f;

    const float* lut = reinterpret_cast<const float*>(smem + L.lut_off);
    uint32_t* codes_sm = reinterpret_cast<uint32_t*>(smem + L.codes_off) + (size_t)buf * p.nodes_per_block * L.cw;
    float* scale_sm = reinterpret_cast<float*>(smem + L.scale_off) + buf * p.nodes_per_block;
    const size_t code_row = (size_t)node * (size_t)p.code_pitch
                          + (size_t)((k0 * T::kBits) >> 5);

    // norm-matched codes: code the whole chunk first; s becomes the norm that is sent,
    // dscale the factor the receiver applies
    uint32_t qn[T::kNorm ? E : 1];
    float cvn[T::kNorm ? E : 1];
    float dscale = s;
    if constexpr (T::kNorm) {
        auto valid = [&](int t) { return node_ok && 4 * (f0 + fstride * (t >> 2)) + (t & 3) < m_len; };
        double sv2, sl2;
        norm_codes<CODE, E, FULL>(v, valid, s, lut, qn, cvn, sv2, sl2);
        float nrm;
        if (p.prescaled && MODE != MODE_REDUCE) {
            // one norm per node, computed by the earlier launches
            nrm = node_ok ? p.scales[(size_t)node * (size_t)p.scales_pitch] : 0.0f;
            dscale = node_ok ? p.dscales[(size_t)node * (size_t)p.scales_pitch] : 0.0f;
        } else {
            if (G > 1) {
                // the sums of the chunk's warps, added in warp order
                double* red2 = reinterpret_cast<double*>(smem + L.red_off) + (size_t)p.nodes_per_block * G;
                double* red3 = red2 + (size_t)p.nodes_per_block * G;
                if (lane == 0) { red2[grp * G + wg] = sv2; red3[grp * G + wg] = sl2; }
                __syncthreads();
                sv2 = 0.0; sl2 = 0.0;
                for (int w = 0; w < G; ++w) { sv2 += red2[grp * G + w]; sl2 += red3[grp * G + w]; }
                if (MODE == MODE_REDUCE) __syncthreads();      // the slots are written again for the next tile
            }
            if constexpr (MODE == MODE_REDUCE) {
                if (node_ok && wg == 0 && lane == 0) {
                    p.partials[(size_t)node * (size_t)p.tiles + (size_t)col] = sv2;
                    p.partials[((size_t)p.n + (size_t)node) * (size_t)p.tiles + (size_t)col] = sl2;
                }
                return;
            }
            norm_finish(s, sv2, sl2, nrm, dscale);
        }
#pragma unroll
        for (int t = 0; t < E; ++t) cvn[t] = __fmul_rn(dscale, cvn[t]);
        s = nrm;
    }
    if constexpr (MODE == MODE_REDUCE) return;

    // ---------------- phase B: compress, residual, pack ------------------
    constexpr float kL = (float)((1u << (T::kBits & 15)) - 1u);
    constexpr float kHalfL = 0.5f * kL;
#pragma unroll
    for (int r = 0; r < V; ++r) {
        const int f = f0 + fstride * r;
        const int e0 = 4 * f;
        const int nv = FULL ? (node_ok ? 4 : 0) : (node_ok ? min(max(m_len - e0, 0), 4) : 0);
        uint32_t piece = 0u;
        if constexpr (T::kIdentity) {
            if (nv > 0) {
                // C = v: the codes are v itself, the residual is zero.
                st_partial(reinterpret_cast<float*>(p.codes + code_row) + e0,
                           make_float4(v[4 * r], v[4 * r + 1], v[4 * r + 2], v[4 * r + 3]), nv);
                st_partial(p.delta + row + e0,
                           make_float4(__fadd_rn(v[4 * r], -v[4 * r]), __fadd_rn(v[4 * r + 1], -v[4 * r + 1]),
                                       __fadd_rn(v[4 * r + 2], -v[4 * r + 2]), __fadd_rn(v[4 * r + 3], -v[4 * r + 3])), nv);
            }
        } else {
            if (nv > 0) {
                float dn[4];
                if constexpr (T::kNorm) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        dn[j] = __fadd_rn(v[4 * r + j], -cvn[4 * r + j]);
                        if (FULL || j < nv) piece |= qn[4 * r + j] << (T::kBits * j);
                    }
                } else if constexpr (T::kSign) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint32_t bit = (v[4 * r + j] >= 0.0f) ? 1u : 0u;
                        const float cv = bit ? s : -s;
                        dn[j] = __fadd_rn(v[4 * r + j], -cv);
                        if (FULL || j < nv) piece |= bit << j;
                    }
                } else if (fast) {
                    const float4 rr = rnd24x4_unscaled(p.rs, (uint32_t)node, (uint32_t)(k0 + e0));
                    const float rv[4] = {rr.x, rr.y, rr.z, rr.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint32_t q = quantise_recip(v[4 * r + j], s, inv_s, rv[j], kHalfL, (int)kL);
                        const float cv = __fmul_rn(s, lut[q]);
                        dn[j] = __fadd_rn(v[4 * r + j], -cv);
                        if (FULL || j < nv) piece |= q << (T::kBits * j);
                    }
                } else {
                    const float4 rr = rnd24x4(p.rs, (uint32_t)node, (uint32_t)(k0 + e0));
                    const float rv[4] = {rr.x, rr.y, rr.z, rr.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint32_t q = degenerate ? 0u : quantise(v[4 * r + j], s, rv[j], kHalfL, (int)kL);
                        const float cv = __fmul_rn(s, lut[q]);
                        dn[j] = __fadd_rn(v[4 * r + j], -cv);
                        if (FULL || j < nv) piece |= q << (T::kBits * j);
                    }
                }
                st_partial(p.delta + row + e0, make_float4(dn[0], dn[1], dn[2], dn[3]), nv);
                if constexpr (MODE == MODE_COMPRESS) {
                    if (!p.ecsgd)
                        st_partial(p.x + row + e0, make_float4(h[4 * r], h[4 * r + 1], h[4 * r + 2], h[4 * r + 3]), nv);
                }
            }
            // gather the pieces of kLanesPerWord neighbouring lanes into one word
            uint32_t word = piece << ((4 * T::kBits * (lane % T::kLanesPerWord)) & 31);
#pragma unroll
            for (int o = 1; o < T::kLanesPerWord; o <<= 1) word |= __shfl_xor_sync(0xffffffffu, word, o);
            if ((lane % T::kLanesPerWord) == 0 && node_ok && e0 < m_len) {
                if constexpr (MODE == MODE_FUSED) codes_sm[(size_t)grp * L.cw + f / T::kLanesPerWord] = word;
                else p.codes[code_row + f / T::kLanesPerWord] = word;
            }
        }
        if constexpr (T::kIdentity && MODE == MODE_COMPRESS) {
            if (nv > 0 && !p.ecsgd)
                st_partial(p.x + row + e0, make_float4(h[4 * r], h[4 * r + 1], h[4 * r + 2], h[4 * r + 3]), nv);
        }
    }
    if constexpr (!T::kIdentity) {
        if (!p.prescaled && node_ok && wg == 0 && lane == 0) {
            p.scales[(size_t)node * (size_t)p.scales_pitch + (size_t)col] = s;
            if constexpr (T::kNorm) p.dscales[(size_t)node * (size_t)p.scales_pitch + (size_t)col] = dscale;
        }
    }

    if constexpr (MODE == MODE_FUSED) {
        if (wg == 0 && lane == 0) scale_sm[grp] = dscale;
        float* table_sm = reinterpret_cast<float*>(smem + L.table_off) + buf * p.nodes_per_block * 16;
        if constexpr (T::kTable) {
            if (wg == 0 && lane < (1 << T::kBits)) table_sm[grp * 16 + lane] = __fmul_rn(dscale, lut[lane]);
        }
        __syncthreads();    // codes and scales of all nodes of this tile are in shared memory
        if (!node_ok) return;

        // the tile's packed codes leave for global memory ("send")
        const int cw_valid = (m_len * T::kBits + 31) >> 5;
        for (int w = wg * 32 + lane; w < cw_valid; w += fstride)
            p.codes[code_row + w] = codes_sm[(size_t)grp * L.cw + w];

        // ---------------- phase C: decode neighbours, mix ----------------
        const int32_t* rp = reinterpret_cast<const int32_t*>(smem + L.rowptr_off);
        const int32_t* cj = reinterpret_cast<const int32_t*>(smem + L.col_off);
        const float* wp = reinterpret_cast<const float*>(smem + L.w_off);
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
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    float cv;
                    if constexpr (T::kSign) {
                        const uint32_t neg = ((~piece >> t) & 1u) << 31;
                        cv = __uint_as_float(__float_as_uint(sj) ^ neg);
                    } else {
                        const uint32_t q = (piece >> (T::kBits * t)) & ((1u << T::kBits) - 1u);
                        if constexpr (T::kTable) cv = table_j[q];
                        else cv = __fmul_rn(sj, lut[q]);
                    }
                    acc[4 * r + t] = __fmaf_rn(w, cv, acc[4 * r + t]);
                }
            }
        }
#pragma unroll
        for (int r = 0; r < V; ++r) {
            const int e0 = 4 * (f0 + fstride * r);
            const int nv = FULL ? 4 : min(max(m_len - e0, 0), 4);
            if (nv > 0)
                st_partial(p.x + row + e0,
                           make_float4(__fmaf_rn(p.eta, acc[4 * r + 0], h[4 * r + 0]),
                                       __fmaf_rn(p.eta, acc[4 * r + 1], h[4 * r + 1]),
                                       __fmaf_rn(p.eta, acc[4 * r + 2], h[4 * r + 2]),
                                       __fmaf_rn(p.eta, acc[4 * r + 3], h[4 * r + 3])), nv);
        }
    }
}

template <int CODE, int NOISE, int E, int MODE>
__global__ void __launch_bounds__(1024, 1) ds_column_kernel(const __grid_constant__ StepParams p) {
    using T = CodeTraits<CODE>;
    extern __shared__ __align__(16) unsigned char smem[];
    const int G = p.warps_per_group;
    const SmemLayout L = smem_layout(MODE, T::kBits, T::kLut, p.nodes_per_block, G, p.tile, p.n, p.nnz);
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int grp = warp / G;
    const int wg = warp - grp * G;
    const int node = blockIdx.y * p.nodes_per_block + grp;
    const bool node_ok = node < p.n;

    if constexpr (T::kLut) {
        float* lut = reinterpret_cast<float*>(smem + L.lut_off);
        for (int t = threadIdx.x; t < (1 << T::kBits); t += blockDim.x) lut[t] = p.lut[t];
        // norm-matched codes: squares of the levels in binary64 (exact), in the unused part of the table
        if constexpr (T::kNorm)
            for (int t = threadIdx.x; t < (1 << T::kBits); t += blockDim.x)
                reinterpret_cast<double*>(lut + 32)[t] = (double)p.lut[t] * (double)p.lut[t];
    }
    if constexpr (MODE == MODE_FUSED) {
        int32_t* rp = reinterpret_cast<int32_t*>(smem + L.rowptr_off);
        int32_t* cj = reinterpret_cast<int32_t*>(smem + L.col_off);
        float* wp = reinterpret_cast<float*>(smem + L.w_off);
        for (int t = threadIdx.x; t <= p.n; t += blockDim.x) rp[t] = p.row_ptr[t];
        for (int t = threadIdx.x; t < p.nnz; t += blockDim.x) { cj[t] = p.col_idx[t]; wp[t] = p.wprime[t]; }
    }
    __syncthreads();

    const int64_t full_len = (int64_t)E * 32 * G;
    int buf = 0;
    for (int64_t col = p.tile_begin + blockIdx.x; col < p.tile_end; col += gridDim.x) {
        const int64_t remain = p.N - col * p.tile;
        const bool full = (p.tile == full_len) && (remain >= p.tile);
        if (full) column_body<CODE, NOISE, E, MODE, true>(p, L, smem, col, buf, lane, grp, wg, node, node_ok);
        else column_body<CODE, NOISE, E, MODE, false>(p, L, smem, col, buf, lane, grp, wg, node, node_ok);
        buf ^= 1;
    }
}

template <int CODE, int NOISE, int E, int MODE>
cudaError_t launch_one(const LaunchShape& sh, const StepParams& p, cudaStream_t stream) {
    auto kern = ds_column_kernel<CODE, NOISE, E, MODE>;
    if (sh.smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh.smem);
        if (e != cudaSuccess) return e;
    }
    kern<<<sh.grid, sh.block, sh.smem, stream>>>(p);
    return cudaGetLastError();
}

template <int CODE, int MODE>
cudaError_t launch_code(const LaunchShape& sh, const StepParams& p, cudaStream_t stream) {
#define DS_CASE(NZ, EE) \
    if (sh.noise == NZ && sh.elems_per_lane == EE) return launch_one<CODE, NZ, EE, MODE>(sh, p, stream);
    DS_CASE(NOISE_NONE, 4) DS_CASE(NOISE_NONE, 8) DS_CASE(NOISE_NONE, 16)
    DS_CASE(NOISE_GAUSS, 4) DS_CASE(NOISE_GAUSS, 8) DS_CASE(NOISE_GAUSS, 16)
    DS_CASE(NOISE_T3, 4) DS_CASE(NOISE_T3, 8) DS_CASE(NOISE_T3, 16)
    DS_CASE(NOISE_T3I, 4) DS_CASE(NOISE_T3I, 8) DS_CASE(NOISE_T3I, 16)
    DS_CASE(GRAD_GIVEN, 4) DS_CASE(GRAD_GIVEN, 8) DS_CASE(GRAD_GIVEN, 16)
#undef DS_CASE
    return cudaErrorInvalidValue;
}

}  // namespace ds
