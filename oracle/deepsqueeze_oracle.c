/*
 * DeepSqueeze CPU oracle -- TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, element-by-element statement of one iteration of
 * Algorithm 1 (DeepSqueeze) for n simulated nodes, with the synthetic
 * quadratic objective used as the stochastic-gradient stand-in.  Only the
 * tests, the smoke check and the benchmark's CPU-baseline leg may call it.
 * It shares no code, header, table or generator with the CUDA library.
 *
 * What follows the paper:
 *   Algorithm 1, "compute local stochastic gradient"      -> phase 1 of oracle_step()
 *   Algorithm 1, "error-compensated variable" v = x-γg+δ  -> phase 1
 *   Algorithm 1, "compress v ... update the error"        -> oracle_compress_chunk()
 *   Algorithm 1, "send / receive" (i is in N(i))          -> the C array all nodes read
 *   Algorithm 1, "update local model"
 *        x <- x - γg + η Σ_{j in N(i)} (W_ij - I_ij) C[v_j] -> phase 2
 *   Section 3 (matrix form X_{t+1} = X - γG + η C[.](W - I)) is the same rule.
 *
 * Where the paper is silent (quantiser grid, scale, rounding, chunking,
 * random streams) the conventions are the ones documented beside each
 * function; every one of them is a reading, not a quotation.
 *
 * Every floating-point line below is ONE IEEE-754 binary32 operation with
 * round-to-nearest-even (or one fused multiply-add where fmaf is written);
 * build with -ffp-contract=off so the compiler adds no fusion of its own.
 * Scale sums are accumulated in binary64.
 *
 * oracle_ecsgd_step() is the centralized error-compensated SGD of Section 1
 * (a baseline that shares the compressors), stated the same way.
 *
 * Parity pins: see tests/test_oracle_*.py (compression identity, mean
 * preservation, dense float64 matrix form, D-PSGD closed form, gradient
 * descent closed form, hand-worked golden cases, exhaustive accuracy of the
 * elementary functions, independent Philox restatement).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------ */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11): the published    */
/* round function and key schedule.                                    */
/* ------------------------------------------------------------------ */
void oracle_philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2],
                          uint32_t out[4])
{
    uint32_t c0 = ctr_in[0], c1 = ctr_in[1], c2 = ctr_in[2], c3 = ctr_in[3];
    uint32_t k0 = key_in[0], k1 = key_in[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/*
 * Stream addressing (a convention of this library; the workload description
 * only says "keyed (seed, node, step, index)"):
 *   key     = (seed low 32 bits, seed high 32 bits)
 *   counter = (block, node, step low 32 bits, (step >> 32) << 8 | stream)
 * stream 0 = gradient noise, stream 1 = stochastic rounding.
 * block < 2^32 and step < 2^56 are required.
 */
enum { STREAM_NOISE = 0, STREAM_ROUND = 1 };

static void philox_block(uint64_t seed, uint32_t node, uint64_t step,
                         uint32_t stream, uint32_t block, uint32_t out[4])
{
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t ctr[4] = { block, node, (uint32_t)step,
                        (uint32_t)((step >> 32) << 8) | stream };
    oracle_philox4x32_10(ctr, key, out);
}

/* ------------------------------------------------------------------ */
/* Deterministic elementary functions.  They are part of the DEFINITION */
/* of the synthetic noise: fixed polynomials evaluated in binary32 in a */
/* fixed order, so that any IEEE machine reproduces them bit for bit.   */
/* ------------------------------------------------------------------ */

/* ln(j * 2^-24) for an integer 1 <= j <= 2^24.
 * Split u = 2^e * m with m in [sqrt(1/2), sqrt(2)), f = m - 1, and
 * ln(1+f) = f - f^2/2 + f^3 * P(f), P a degree-7 polynomial. */
float oracle_log_u24(uint32_t j)
{
    float u = (float)j * 0x1p-24f;               /* exact */
    uint32_t bits; memcpy(&bits, &u, 4);
    int e = (int)((bits >> 23) & 0xffu) - 127;
    uint32_t mbits = (bits & 0x007fffffu) | 0x3f800000u;
    float m; memcpy(&m, &mbits, 4);              /* m in [1, 2) */
    if (m > 0x1.6a09e6p+0f) { m = m * 0.5f; e = e + 1; }
    float f = m - 1.0f;
    float p = -0x1.38b4ccp-4f;
    p = fmaf(p, f, 0x1.055b46p-3f);
    p = fmaf(p, f, -0x1.0d8552p-3f);
    p = fmaf(p, f, 0x1.22da22p-3f);
    p = fmaf(p, f, -0x1.547244p-3f);
    p = fmaf(p, f, 0x1.99a008p-3f);
    p = fmaf(p, f, -0x1.000228p-2f);
    p = fmaf(p, f, 0x1.555554p-2f);
    float f2 = f * f;
    float f3 = f2 * f;
    float fe = (float)e;
    float y = f3 * p;
    y = fmaf(fe, -0x1.bd0106p-13f, y);           /* e * (ln2 - 0.693359375) */
    y = fmaf(-0.5f, f2, y);
    float r = f + y;
    r = fmaf(fe, 0.693359375f, r);
    return r;
}

/* cos and sin of 2*pi*k/2^24 for an integer 0 <= k < 2^24.
 * The angle is reduced exactly on the integer: n = nearest quarter turn,
 * r in [-1/2, 1/2) the remainder in quarter turns; then
 * sin(pi/2 r) = r S(r^2), cos(pi/2 r) = 1 + r^2 Q(r^2). */
void oracle_sincos_u24(uint32_t k, float *cos_out, float *sin_out)
{
    uint32_t n = (k + (1u << 21)) >> 22;
    int32_t ri = (int32_t)k - (int32_t)(n << 22);
    float r = (float)ri * 0x1p-22f;              /* exact */
    float z = r * r;
    float sp = -0x1.2d9332p-8f;
    sp = fmaf(sp, z, 0x1.465e94p-4f);
    sp = fmaf(sp, z, -0x1.4abbbap-1f);
    sp = fmaf(sp, z, 0x1.921fb6p+0f);
    float s = r * sp;
    float cq = 0x1.d9d58p-11f;
    cq = fmaf(cq, z, -0x1.55c5ep-6f);
    cq = fmaf(cq, z, 0x1.03c1dep-2f);
    cq = fmaf(cq, z, -0x1.3bd3ccp+0f);
    float c = fmaf(z, cq, 1.0f);
    switch (n & 3u) {
    case 0: *cos_out = c;  *sin_out = s;  break;
    case 1: *cos_out = -s; *sin_out = c;  break;
    case 2: *cos_out = -c; *sin_out = -s; break;
    default: *cos_out = s; *sin_out = -c; break;
    }
}

/* Box-Muller: two 32-bit words -> two standard normals.
 * u1 = ((wa >> 8) + 1) 2^-24 in (0, 1], u2 = (wb >> 8) 2^-24 in [0, 1). */
static void box_muller(uint32_t wa, uint32_t wb, float *z0, float *z1)
{
    float lg = oracle_log_u24((wa >> 8) + 1u);
    float rho = sqrtf(-2.0f * lg);
    float c, s;
    oracle_sincos_u24(wb >> 8, &c, &s);
    *z0 = rho * c;
    *z1 = rho * s;
}

/* Radius of a Student-t(3) pair: sqrt(3 (u^(-2/3) - 1)) for u = j 2^-24,
 * 1 <= j <= 2^24.  With theta uniform, (rho cos theta, rho sin theta) is then a
 * spherical bivariate Student-t vector with 3 degrees of freedom (Bailey's
 * polar method, Math. Comp. 62, 1994): both components are t(3) variates.
 *   w = -(2/3) ln u >= 0;  k = nearest integer to w / ln 2;  r = w - k ln 2
 *   (two-constant reduction, ln 2 = 0.693359375 - 2.1219444e-4);
 *   expm1(r) = r + r^2 P(r), P of degree 5;
 *   E = u^(-2/3) - 1 = 2^k expm1(r) + (2^k - 1)  (one fma: 2^k - 1 is exact);
 *   rho = sqrt(3 E).
 * The nearest integer is taken by adding and subtracting 1.5 * 2^23, which
 * rounds to nearest-even in binary32 on every IEEE machine. */
float oracle_t3_radius_u24(uint32_t j)
{
    float lg = oracle_log_u24(j);                       /* <= 0 */
    float w = lg * -0x1.555556p-1f;
    float t = fmaf(w, 0x1.715476p+0f, 12582912.0f);
    float kf = t - 12582912.0f;
    float r = fmaf(kf, -0.693359375f, w);
    r = fmaf(kf, 0x1.bd0106p-13f, r);
    float p = 0x1.9d1158p-13f;
    p = fmaf(p, r, 0x1.6d7cc8p-10f);
    p = fmaf(p, r, 0x1.111394p-7f);
    p = fmaf(p, r, 0x1.5554a6p-5f);
    p = fmaf(p, r, 0x1.555554p-3f);
    p = fmaf(p, r, 0.5f);
    float r2 = r * r;
    float em = fmaf(r2, p, r);
    float scale = ldexpf(1.0f, (int)kf);                /* 2^k, 0 <= k <= 16 */
    float E = fmaf(scale, em, scale - 1.0f);
    return sqrtf(3.0f * E);
}

enum { NOISE_NONE = 0, NOISE_GAUSS = 1, NOISE_STUDENT_T3 = 2, NOISE_STUDENT_T3_IID = 3 };

/* Unit noise z for element k of a node (before the factor sigma).
 * Block k/4 of the noise stream yields the elements 4m..4m+3: words (0,1) ->
 * 4m, 4m+1 and words (2,3) -> 4m+2, 4m+3, each pair as
 * (rho cos 2 pi u2, rho sin 2 pi u2) with u1 = ((wa >> 8) + 1) 2^-24,
 * u2 = (wb >> 8) 2^-24 and
 *   GAUSS:      rho = sqrt(-2 ln u1)              (Box-Muller: two independent normals)
 *   STUDENT_T3: rho = sqrt(3 (u1^(-2/3) - 1))     (a spherical bivariate t(3) pair:
 *               each element is exactly t(3)-distributed; the two elements of a
 *               pair are uncorrelated but share their radius; pairs are independent).
 * STUDENT_T3_IID: independent t(3) coordinates by the textbook construction
 *   t = Z0 / sqrt((Z1^2 + Z2^2 + Z3^2) / 3) from four independent normals: element
 *   k owns block k of the noise stream, (w0, w1) -> Z0, Z1 and (w2, w3) -> Z2, Z3
 *   by Box-Muller as above, q = fma(Z3, Z3, fma(Z2, Z2, Z1 Z1)),
 *   t = Z0 / sqrt(q / 3) (t = 0 if q = 0). */
float oracle_noise_elem(int kind, uint64_t seed, uint32_t node, uint64_t step,
                        int64_t k)
{
    uint32_t w[4];
    float z0, z1;
    if (kind == NOISE_STUDENT_T3_IID) {
        float z2, z3;
        philox_block(seed, node, step, STREAM_NOISE, (uint32_t)k, w);
        box_muller(w[0], w[1], &z0, &z1);
        box_muller(w[2], w[3], &z2, &z3);
        float q = fmaf(z3, z3, fmaf(z2, z2, z1 * z1));
        if (q == 0.0f) return 0.0f;
        float third = q / 3.0f;
        return z0 / sqrtf(third);
    }
    if (kind == NOISE_GAUSS || kind == NOISE_STUDENT_T3) {
        philox_block(seed, node, step, STREAM_NOISE, (uint32_t)(k >> 2), w);
        int pair = (int)((k >> 1) & 1);
        if (kind == NOISE_GAUSS) {
            box_muller(w[2 * pair], w[2 * pair + 1], &z0, &z1);
        } else {
            float rho = oracle_t3_radius_u24((w[2 * pair] >> 8) + 1u);
            float c, s;
            oracle_sincos_u24(w[2 * pair + 1] >> 8, &c, &s);
            z0 = rho * c;
            z1 = rho * s;
        }
        return (k & 1) ? z1 : z0;
    }
    return 0.0f;
}

/* Uniform r in [0,1) with 24 bits for stochastic rounding of element k:
 * word k%4 of block k/4 of the rounding stream. */
float oracle_rnd24_elem(uint64_t seed, uint32_t node, uint64_t step, int64_t k)
{
    uint32_t w[4];
    philox_block(seed, node, step, STREAM_ROUND, (uint32_t)(k >> 2), w);
    return (float)(w[k & 3] >> 8) * 0x1p-24f;
}

/* ------------------------------------------------------------------ */
/* Compressors C_omega (Algorithm 1, compression step; Section 5,       */
/* "Compression": b bits per element plus one scalar per tensor).       */
/* ------------------------------------------------------------------ */
enum { COMP_IDENTITY = 0, COMP_SIGN1_L1 = 1, COMP_UNIFORM_STOCH_MAXABS = 2,
       COMP_UNIFORM_NEAREST_L2 = 3 };

/* Reconstruction level q of the b-bit grid: 2^b points evenly spaced on
 * [-1, 1] including both ends. */
float oracle_level(int bits, int q)
{
    int L = (1 << bits) - 1;
    return (float)((double)(2 * q - L) / (double)L);
}

/*
 * Compress one chunk v[0..m) of one node.
 *   SIGN1_L1 : s = (Σ|v_k|)/m (binary64 sum, rounded once to binary32),
 *              code 1 if v_k >= 0 else 0, C_k = +s / -s.
 *   UNIFORM  : s = max|v_k|.  If s is 0 or not finite the stored scale is 0,
 *              every code is 0 and C_k = 0 * level[0].
 *              Otherwise y = v_k/s, u = y*(L/2) + L/2 (one fma),
 *              code = clamp(floor(u + r_k), 0, L), C_k = s * level[code].
 *              NaN elements code to 0.
 *   IDENTITY : C_k = v_k, the "code" is the bit pattern of v_k.
 *   NEAREST_L2 : the paper's "bit compression" (Section 5, "Compression"): b bits
 *              per element and the Euclidean norm of the tensor, the receiver
 *              rescaling what it decodes to that norm.  Grid as above with
 *              g = max|v_k|: code = clamp(floor(fma(v_k/g, L/2, L/2) + 1/2), 0, L)
 *              (nearest level), l_k = level[code]; the scalar sent is
 *              nrm = sqrt(sum v_k^2), the receiver forms lnorm = sqrt(sum l_k^2)
 *              (both sums in binary64, rounded to binary32) and
 *              C_k = (nrm / lnorm) * l_k.  g = 0 or not finite, or a norm that is
 *              not finite: nrm = 0 is sent and C = 0 * l_k.
 * q_out receives one code per element (unpacked); *scale_out is what is sent.
 */
void oracle_compress_chunk(int kind, int bits, const float *v, int64_t m,
                           const float *r, float *scale_out,
                           uint32_t *q_out, float *C_out)
{
    if (kind == COMP_IDENTITY) {
        for (int64_t k = 0; k < m; ++k) {
            C_out[k] = v[k];
            memcpy(&q_out[k], &v[k], 4);
        }
        *scale_out = 1.0f;
        return;
    }
    if (kind == COMP_SIGN1_L1) {
        double sum = 0.0;
        for (int64_t k = 0; k < m; ++k) sum += (double)fabsf(v[k]);
        float s = (float)(sum / (double)m);
        for (int64_t k = 0; k < m; ++k) {
            int bit = (v[k] >= 0.0f) ? 1 : 0;
            q_out[k] = (uint32_t)bit;
            C_out[k] = bit ? s : -s;
        }
        *scale_out = s;
        return;
    }
    if (kind == COMP_UNIFORM_NEAREST_L2) {
        int L = (1 << bits) - 1;
        float g = 0.0f;
        for (int64_t k = 0; k < m; ++k) g = fmaxf(g, fabsf(v[k]));
        int dead = (g == 0.0f || !isfinite(g));
        float hl = 0.5f * (float)L;
        double sv2 = 0.0, sl2 = 0.0;
        for (int64_t k = 0; k < m; ++k) {
            int q = 0;
            if (!dead) {
                float y = v[k] / g;
                float u = fmaf(y, hl, hl);
                float t = floorf(u + 0.5f);
                if (t >= 1.0f) q = (t >= (float)L) ? L : (int)t;
            }
            q_out[k] = (uint32_t)q;
            float l = oracle_level(bits, q);
            C_out[k] = l;                          /* unit reconstruction for now */
            sv2 += (double)v[k] * (double)v[k];
            sl2 += (double)l * (double)l;
        }
        float nrm = dead ? 0.0f : (float)sqrt(sv2);
        float lnorm = (float)sqrt(sl2);
        float ratio = 0.0f;
        if (!dead && lnorm != 0.0f && isfinite(nrm)) ratio = nrm / lnorm;
        if (!isfinite(nrm)) nrm = 0.0f;
        for (int64_t k = 0; k < m; ++k) C_out[k] = ratio * C_out[k];
        *scale_out = nrm;
        return;
    }
    /* COMP_UNIFORM_STOCH_MAXABS */
    int L = (1 << bits) - 1;
    float s = 0.0f;
    for (int64_t k = 0; k < m; ++k) s = fmaxf(s, fabsf(v[k]));
    if (s == 0.0f || !isfinite(s)) {
        float s0 = 0.0f;
        for (int64_t k = 0; k < m; ++k) {
            q_out[k] = 0u;
            C_out[k] = s0 * oracle_level(bits, 0);
        }
        *scale_out = s0;
        return;
    }
    float hl = 0.5f * (float)L;
    for (int64_t k = 0; k < m; ++k) {
        float y = v[k] / s;
        float u = fmaf(y, hl, hl);
        float t = floorf(u + r[k]);
        int q = 0;
        if (t >= 1.0f) q = (t >= (float)L) ? L : (int)t;
        q_out[k] = (uint32_t)q;
        C_out[k] = s * oracle_level(bits, q);
    }
    *scale_out = s;
}

/* Pack m codes of `bits` bits each, element-major, little-endian within
 * each 32-bit word: element k sits at bit (k*bits) % 32 of word (k*bits)/32.
 * `words` must be zero-initialised by the caller over the packed range. */
void oracle_pack_codes(int bits, const uint32_t *q, int64_t first_elem,
                       int64_t m, uint32_t *words)
{
    for (int64_t k = 0; k < m; ++k) {
        int64_t bitpos = (first_elem + k) * (int64_t)bits;
        words[bitpos >> 5] |= q[k] << (bitpos & 31);
    }
}

/* ------------------------------------------------------------------ */
/* One DeepSqueeze iteration for all n nodes.                          */
/* ------------------------------------------------------------------ */
/*
 * Inputs  (row-major, row pitch ld >= N, all binary32 unless said):
 *   x, delta           [n][ld]  node models and compression errors, updated in place
 *   a, c               [n][ld]  objective f_i(x) = 1/2 Σ_k a_ik (x_k - c_ik)^2
 *   row_ptr, col_idx, W         CSR of the mixing matrix, columns ascending,
 *                               the diagonal entry present in every row
 *   chunk                       compressor chunk length; 0 = one chunk per node
 * Outputs:
 *   codes  [n][code_pitch]      packed codes of this step (words per node:
 *                               ceil(N*bits/32); bits = 32 for IDENTITY)
 *   scales [n][scales_pitch]    one scale per (node, chunk)
 *   v_out, C_out (optional, [n][N])  the error-compensated variable and its
 *                               decoded compression, for the tests
 *   g_given (optional, [n][ld])  the stochastic gradient itself (Algorithm 1,
 *                               gradient step, computed by the caller); when not
 *                               NULL, a, c, sigma and the noise are not used
 *   k_first                     global index of column 0 in the random streams:
 *                               0 for a whole problem; a multiple of the chunk
 *                               length when the arrays hold a window of columns
 *                               [k_first, k_first + N) of a longer problem
 * Returns 0, or -1 if memory could not be obtained.
 *
 * Operation order per element (one binary32 operation per line):
 *   d  = x - c
 *   nz = sigma * z
 *   g  = fma(a, d, nz)                 stochastic gradient
 *   h  = fma(-gamma, g, x)             x - γ g
 *   v  = h + delta                     error-compensated variable
 *   (C, code) = compress(v)            per chunk
 *   delta' = v - C
 *   acc = 0; for j in N(i) ascending: acc = fma(w'_ij, C_j, acc),
 *         w'_ij = W_ij - (i == j ? 1 : 0) in binary32
 *   x' = fma(eta, acc, h)
 */
int oracle_step(int32_t n, int64_t N, int64_t ld,
                const int32_t *row_ptr, const int32_t *col_idx, const float *W,
                int comp_kind, int bits, int64_t chunk,
                float *x, float *delta, const float *a, const float *c,
                float sigma, int noise_kind, float gamma, float eta,
                uint64_t seed, uint64_t step,
                uint32_t *codes, int64_t code_pitch,
                float *scales, int64_t scales_pitch,
                float *v_out, float *C_out, int64_t k_first, const float *g_given)
{
    if (chunk <= 0) chunk = N;
    int code_bits = (comp_kind == COMP_IDENTITY) ? 32
                  : (comp_kind == COMP_SIGN1_L1) ? 1 : bits;
    int64_t M = (N + chunk - 1) / chunk;
    int64_t words = (N * (int64_t)code_bits + 31) / 32;

    float *h = (float *)malloc(sizeof(float) * (size_t)n * (size_t)N);
    float *C = (float *)malloc(sizeof(float) * (size_t)n * (size_t)N);
    if (!h || !C) { free(h); free(C); return -1; }

    for (int32_t i = 0; i < n; ++i)
        memset(codes + (size_t)i * code_pitch, 0, sizeof(uint32_t) * (size_t)words);

    int failed = 0;
    /* Phase 1: gradient, error-compensated variable, compression, residual. */
    #pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int32_t i = 0; i < n; ++i) {
        for (int64_t mi = 0; mi < M; ++mi) {
            int64_t k0 = mi * chunk;
            int64_t m = (N - k0 < chunk) ? (N - k0) : chunk;
            float *v = (float *)malloc(sizeof(float) * (size_t)m);
            float *r = (float *)malloc(sizeof(float) * (size_t)m);
            uint32_t *q = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)m);
            if (!v || !r || !q) {
                free(v); free(r); free(q);
                #pragma omp atomic write
                failed = 1;
                continue;
            }
            for (int64_t kk = 0; kk < m; ++kk) {
                int64_t k = k0 + kk;
                size_t at = (size_t)i * (size_t)ld + (size_t)k;
                float g;
                if (g_given) {
                    g = g_given[at];         /* the caller's stochastic gradient */
                } else {
                    float z = oracle_noise_elem(noise_kind, seed, (uint32_t)i, step, k_first + k);
                    float d = x[at] - c[at];
                    float nz = sigma * z;
                    g = fmaf(a[at], d, nz);
                }
                float hh = fmaf(-gamma, g, x[at]);
                h[(size_t)i * (size_t)N + (size_t)k] = hh;
                v[kk] = hh + delta[at];
                r[kk] = (comp_kind == COMP_UNIFORM_STOCH_MAXABS)
                            ? oracle_rnd24_elem(seed, (uint32_t)i, step, k_first + k) : 0.0f;
            }
            float s;
            float *Crow = C + (size_t)i * (size_t)N + (size_t)k0;
            oracle_compress_chunk(comp_kind, bits, v, m, r, &s, q, Crow);
            scales[(size_t)i * (size_t)scales_pitch + (size_t)mi] = s;
            for (int64_t kk = 0; kk < m; ++kk) {
                size_t at = (size_t)i * (size_t)ld + (size_t)(k0 + kk);
                delta[at] = v[kk] - Crow[kk];
                if (v_out) v_out[(size_t)i * (size_t)N + (size_t)(k0 + kk)] = v[kk];
            }
            /* chunk*code_bits is a multiple of 32 for every chunk but the last
             * of a row, so chunks never share a code word. */
            oracle_pack_codes(code_bits, q, k0, m, codes + (size_t)i * code_pitch);
            free(v); free(r); free(q);
        }
    }
    if (failed) { free(h); free(C); return -1; }

    /* Phase 2: every node reads C of its neighbours (itself included). */
    #pragma omp parallel for schedule(static)
    for (int32_t i = 0; i < n; ++i) {
        for (int64_t k = 0; k < N; ++k) {
            float acc = 0.0f;
            for (int32_t e = row_ptr[i]; e < row_ptr[i + 1]; ++e) {
                int32_t j = col_idx[e];
                float wp = W[e] - ((j == i) ? 1.0f : 0.0f);
                acc = fmaf(wp, C[(size_t)j * (size_t)N + (size_t)k], acc);
            }
            x[(size_t)i * (size_t)ld + (size_t)k] =
                fmaf(eta, acc, h[(size_t)i * (size_t)N + (size_t)k]);
        }
    }
    if (C_out) memcpy(C_out, C, sizeof(float) * (size_t)n * (size_t)N);
    free(h); free(C);
    return 0;
}

/*
 * Centralized error-compensated SGD, the scheme the paper starts from
 * (Section 1, the three displayed updates) and one of its baselines:
 *     g'    <- C[g + delta]                 on each worker
 *     delta <- (g + delta) - C[g + delta]   on each worker
 *     x     <- x - gamma g'                 on the server
 * The paper writes it for one worker.  Reading for n workers: row i of x is
 * worker i's copy of the model, worker i evaluates its own objective there, and
 * the server's average is the weighted sum over the rows of W (complete graph
 * with W_ij = 1/n = the parameter server; then all rows stay equal):
 *     g  = fma(a, d, sigma z)  (or the given gradient)
 *     v  = g + delta
 *     (C, code) = compress(v) per chunk ;  delta' = v - C
 *     acc = 0; for j in N(i) ascending: acc = fma(W_ij, C_j, acc)
 *     x'  = fma(-gamma, acc, x)
 * Random streams, compressors, chunking and packing are those of oracle_step.
 */
int oracle_ecsgd_step(int32_t n, int64_t N, int64_t ld,
                      const int32_t *row_ptr, const int32_t *col_idx, const float *W,
                      int comp_kind, int bits, int64_t chunk,
                      float *x, float *delta, const float *a, const float *c,
                      float sigma, int noise_kind, float gamma,
                      uint64_t seed, uint64_t step,
                      uint32_t *codes, int64_t code_pitch,
                      float *scales, int64_t scales_pitch, const float *g_given)
{
    if (chunk <= 0) chunk = N;
    int code_bits = (comp_kind == COMP_IDENTITY) ? 32
                  : (comp_kind == COMP_SIGN1_L1) ? 1 : bits;
    int64_t M = (N + chunk - 1) / chunk;
    int64_t words = (N * (int64_t)code_bits + 31) / 32;
    float *C = (float *)malloc(sizeof(float) * (size_t)n * (size_t)N);
    float *v = (float *)malloc(sizeof(float) * (size_t)chunk);
    float *r = (float *)malloc(sizeof(float) * (size_t)chunk);
    uint32_t *q = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)chunk);
    if (!C || !v || !r || !q) { free(C); free(v); free(r); free(q); return -1; }

    /* workers */
    for (int32_t i = 0; i < n; ++i) {
        memset(codes + (size_t)i * code_pitch, 0, sizeof(uint32_t) * (size_t)words);
        for (int64_t mi = 0; mi < M; ++mi) {
            int64_t k0 = mi * chunk;
            int64_t m = (N - k0 < chunk) ? (N - k0) : chunk;
            for (int64_t kk = 0; kk < m; ++kk) {
                int64_t k = k0 + kk;
                size_t at = (size_t)i * (size_t)ld + (size_t)k;
                float g;
                if (g_given) {
                    g = g_given[at];
                } else {
                    float z = oracle_noise_elem(noise_kind, seed, (uint32_t)i, step, k);
                    float d = x[at] - c[at];
                    float nz = sigma * z;
                    g = fmaf(a[at], d, nz);
                }
                v[kk] = g + delta[at];
                r[kk] = (comp_kind == COMP_UNIFORM_STOCH_MAXABS)
                            ? oracle_rnd24_elem(seed, (uint32_t)i, step, k) : 0.0f;
            }
            float s;
            float *Crow = C + (size_t)i * (size_t)N + (size_t)k0;
            oracle_compress_chunk(comp_kind, bits, v, m, r, &s, q, Crow);
            scales[(size_t)i * (size_t)scales_pitch + (size_t)mi] = s;
            for (int64_t kk = 0; kk < m; ++kk)
                delta[(size_t)i * (size_t)ld + (size_t)(k0 + kk)] = v[kk] - Crow[kk];
            oracle_pack_codes(code_bits, q, k0, m, codes + (size_t)i * code_pitch);
        }
    }
    /* server */
    for (int32_t i = 0; i < n; ++i) {
        for (int64_t k = 0; k < N; ++k) {
            float acc = 0.0f;
            for (int32_t e = row_ptr[i]; e < row_ptr[i + 1]; ++e)
                acc = fmaf(W[e], C[(size_t)col_idx[e] * (size_t)N + (size_t)k], acc);
            size_t at = (size_t)i * (size_t)ld + (size_t)k;
            x[at] = fmaf(-gamma, acc, x[at]);
        }
    }
    free(C); free(v); free(r); free(q);
    return 0;
}

/* ------------------------------------------------------------------ */
/* Array helpers so that the tests can sweep the elementary functions   */
/* and the random streams without a Python loop.                        */
/* ------------------------------------------------------------------ */
void oracle_log_u24_array(uint32_t j0, int64_t count, float *out)
{
    for (int64_t t = 0; t < count; ++t) out[t] = oracle_log_u24(j0 + (uint32_t)t);
}

void oracle_t3_radius_u24_array(uint32_t j0, int64_t count, float *out)
{
    for (int64_t t = 0; t < count; ++t) out[t] = oracle_t3_radius_u24(j0 + (uint32_t)t);
}

void oracle_sincos_u24_array(uint32_t k0, int64_t count, float *cos_out, float *sin_out)
{
    for (int64_t t = 0; t < count; ++t)
        oracle_sincos_u24(k0 + (uint32_t)t, &cos_out[t], &sin_out[t]);
}

void oracle_noise_row(int kind, uint64_t seed, uint32_t node, uint64_t step,
                      int64_t k0, int64_t count, float *out)
{
    for (int64_t t = 0; t < count; ++t)
        out[t] = oracle_noise_elem(kind, seed, node, step, k0 + t);
}

void oracle_rnd24_row(uint64_t seed, uint32_t node, uint64_t step,
                      int64_t k0, int64_t count, float *out)
{
    for (int64_t t = 0; t < count; ++t)
        out[t] = oracle_rnd24_elem(seed, node, step, k0 + t);
}

int oracle_num_threads(void)
{
    int t = 1;
#ifdef _OPENMP
    #pragma omp parallel
    {
        #pragma omp single
        t = omp_get_num_threads();
    }
#endif
    return t;
}

/* Host threads the (node, chunk) work items are spread over from now on
 * (the benchmark times the oracle on one thread and on all cores). */
void oracle_set_num_threads(int t)
{
#ifdef _OPENMP
    if (t >= 1) omp_set_num_threads(t);
#else
    (void)t;
#endif
}
