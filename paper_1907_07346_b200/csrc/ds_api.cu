// Host side of the DeepSqueeze C ABI: argument and graph validation,
// workspace carving, launch planning and dispatch.  See include/deepsqueeze.h.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/deepsqueeze.h"
#include "ds_fused_tma_kernel.cuh"
#include "ds_wide_fused_kernel.cuh"
#include "ds_wide_tma_kernel.cuh"
#include "ds_resident_kernel.cuh"
#include "ds_fused_tma_pair_kernel.cuh"
#include "ds_fused_tma_ecsgd.h"

using namespace ds;

namespace {

// ds_noise_kind -> the kernels' NOISE_* value (GRAD_GIVEN sits between them)
inline int noise_template_of(int32_t noise) { return noise == DS_NOISE_STUDENT_T3_IID ? (int)NOISE_T3I : (int)noise; }

constexpr size_t kAlign = 256;
constexpr int64_t kPerNodeTile = 512;   // tile width when one scale covers a node
constexpr int kMaxSmem = 227 * 1024;
constexpr int kMaxSlabs = 16;            // pipeline depth of the host-buffer entry point

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline int64_t round_up64(int64_t v, int64_t m) { return (v + m - 1) / m * m; }

struct Shape {
    int code;             // CODE_*
    int code_bits;
    int64_t chunk;        // elements per scale (N when one per node)
    int64_t M;            // scales per row
    int64_t tile;         // column tile of the kernels
    int64_t tiles;
    bool per_node;        // scale computed by a separate reduction
    int64_t code_words, code_pitch, scales_pitch;
};

struct WsLayout {
    size_t codes, scales, dscales, partials, gmax, rpartials, row_ptr, col_idx, wprime, wplain, lut, error_flag, barrier, total;
};

bool make_shape(int32_t n, int64_t N, const ds_compressor* comp, Shape* sh) {
    if (!comp || n < 1 || N < 1) return false;
    switch (comp->kind) {
        case DS_COMP_IDENTITY: sh->code = CODE_ID32; break;
        case DS_COMP_SIGN1_L1:
            if (comp->bits != 1) return false;
            sh->code = CODE_SIGN;
            break;
        case DS_COMP_UNIFORM_STOCH_MAXABS:
            if (comp->bits == 1) sh->code = CODE_U1;
            else if (comp->bits == 2) sh->code = CODE_U2;
            else if (comp->bits == 4) sh->code = CODE_U4;
            else if (comp->bits == 8) sh->code = CODE_U8;
            else return false;
            break;
        case DS_COMP_UNIFORM_NEAREST_L2:
            // the paper's own settings (2 and 4 bits); any chunk, or chunk = 0: one norm per node,
            // the paper's "one Euclidean norm per tensor"
            if (comp->bits == 2) sh->code = CODE_N2;
            else if (comp->bits == 4) sh->code = CODE_N4;
            else return false;
            break;
        default: return false;
    }
    if (comp->chunk < 0 || (comp->chunk % 32) != 0) return false;
    sh->code_bits = code_bits_of(sh->code);
    const bool identity = (sh->code == CODE_ID32);
    sh->per_node = (comp->chunk == 0) && !identity;
    sh->chunk = (comp->chunk == 0) ? N : comp->chunk;
    sh->M = identity ? 0 : (N + sh->chunk - 1) / sh->chunk;
    sh->tile = (comp->chunk == 0) ? kPerNodeTile : comp->chunk;
    sh->tiles = (N + sh->tile - 1) / sh->tile;
    sh->code_words = (N * sh->code_bits + 31) / 32;
    sh->code_pitch = round_up64(sh->code_words, 4);
    sh->scales_pitch = round_up64(std::max<int64_t>(sh->M, 1), 4);
    return true;
}

// Shapes the resident multi-step kernel takes: one warp per node and tile of 512
// elements, all tiles resident at once when a per-node scale needs the grid barrier.
bool resident_shape(int32_t n, const Shape& sh) {
    if (n > kResidentMaxNodes || sh.tile != kResidentTile) return false;
    if (sh.code != CODE_SIGN && sh.code != CODE_U2 && sh.code != CODE_U4) return false;
    return !sh.per_node || sh.tiles <= 1024;
}

WsLayout make_ws(int32_t n, int32_t nnz, const Shape& sh) {
    WsLayout w;
    size_t off = 0;
    w.codes = off;    off = align_up(off + (size_t)n * (size_t)sh.code_pitch * 4, kAlign);
    w.scales = off;   off = align_up(off + (size_t)n * (size_t)sh.scales_pitch * 4, kAlign);
    const bool norm = (sh.code == CODE_N2 || sh.code == CODE_N4);
    w.dscales = norm ? off : w.scales;      // decode factors only differ from the sent scalars for norm-matched codes
    if (norm) off = align_up(off + (size_t)n * (size_t)sh.scales_pitch * 4, kAlign);
    // per-node scale: one binary64 partial per (node, tile); a per-node norm needs two sums
    w.partials = off; off = align_up(off + (sh.per_node ? (norm ? 2 : 1) * (size_t)n * (size_t)sh.tiles * 8 : 0), kAlign);
    w.gmax = off;     off = align_up(off + (sh.per_node && norm ? (size_t)n * 4 : 0), kAlign);
    // two buffers of per-tile partials for the resident multi-step kernel (small per-node-scale shapes only)
    w.rpartials = off;
    off = align_up(off + (resident_shape(n, sh) && sh.per_node ? 2 * (size_t)n * (size_t)sh.tiles * 8 : 0), kAlign);
    w.row_ptr = off;  off = align_up(off + (size_t)(n + 1) * 4, kAlign);
    w.col_idx = off;  off = align_up(off + (size_t)nnz * 4, kAlign);
    w.wprime = off;   off = align_up(off + (size_t)nnz * 4, kAlign);
    w.wplain = off;   off = align_up(off + (size_t)nnz * 4, kAlign);
    w.lut = off;      off = align_up(off + 256 * 4, kAlign);
    w.error_flag = off; off = align_up(off + 4, kAlign);
    w.barrier = off;  off = align_up(off + 4, kAlign);
    w.total = off;
    return w;
}

struct Plan {
    bool ok = false;
    int elems_per_lane = 0;
    int warps_per_group = 0;
    int nodes_per_block = 0;
    dim3 grid, block;
    size_t smem = 0;
    int l2_hints = 0;          // batch-sweeping TMA kernel only (see StepParams::l2_hints)
};

void pick_lane_shape(int64_t tile, int force_e, int* E, int* G) {
    *E = (force_e > 0) ? force_e : (tile >= 512) ? 16 : (tile >= 256) ? 8 : 4;
    *G = (int)((tile + 32 * (*E) - 1) / (32 * (*E)));
}

Plan plan_column(int mode, const Shape& sh, int32_t n, int32_t nnz, int force_e = 0) {
    Plan pl;
    int E, G;
    pick_lane_shape(sh.tile, force_e, &E, &G);
    pl.elems_per_lane = E;
    pl.warps_per_group = G;
    if (G > 32) return pl;
    int npb;
    if (mode == MODE_FUSED) {
        if (sh.code == CODE_ID32) return pl;
        if ((int64_t)n * G > 32) return pl;
        npb = n;
    } else {
        npb = std::max(1, std::min<int>(n, 8 / G));
    }
    pl.nodes_per_block = npb;
    pl.block = dim3((unsigned)(npb * G * 32));
    const bool lut = !(sh.code == CODE_SIGN || sh.code == CODE_ID32);
    pl.smem = smem_layout(mode, sh.code_bits, lut, npb, G, sh.tile, n, nnz).total;
    if (pl.smem > (size_t)kMaxSmem) return pl;
    const int64_t gx = std::min<int64_t>(sh.tiles, 0x7fffffff);
    pl.grid = dim3((unsigned)gx, (unsigned)((n + npb - 1) / npb));
    pl.ok = true;
    return pl;
}

Plan plan_tma(const Shape& sh, int32_t n, int32_t nnz, int num_sms, int force_e = 0) {
    Plan pl;
    int E, G;
    pick_lane_shape(sh.tile, force_e, &E, &G);
    pl.elems_per_lane = E;
    pl.warps_per_group = G;
    if ((int64_t)n * G > 32 || num_sms < 1) return pl;
    // every warp of a group owns a whole E*32-element segment
    if ((int64_t)G * E * 32 < sh.tile) return pl;
    pl.nodes_per_block = n;
    pl.block = dim3((unsigned)(n * G * 32));
    const bool lut = (sh.code != CODE_SIGN && sh.code != CODE_ID32);
    pl.smem = tma_smem_layout(lut, E, n * G, G, sh.tile, n, nnz).total;
    if (pl.smem > (size_t)kMaxSmem) return pl;
    pl.grid = dim3((unsigned)std::min<int64_t>(sh.tiles, num_sms));
    pl.ok = true;
    return pl;
}

// Persistent TMA-staged kernel with two nodes per warp: 17..32 nodes, chunks of 256.
Plan plan_tma_pair(const Shape& sh, int32_t n, int32_t nnz, int num_sms, int force_e = 0) {
    Plan pl;
    pl.elems_per_lane = 8;
    pl.warps_per_group = 1;
    if (force_e != 0 && force_e != 8) return pl;
    if (sh.tile != kPairTile || sh.per_node || n <= 16 || n > 32 || (n % 2) != 0 || num_sms < 1) return pl;
    if (sh.code == CODE_ID32 || sh.code == CODE_N2 || sh.code == CODE_N4) return pl;
    pl.nodes_per_block = n;
    pl.block = dim3((unsigned)(n / 2 * 32));
    pl.smem = tma_smem_layout(sh.code != CODE_SIGN, 16, n / 2, 1, kPairTile, n, nnz).total;
    if (pl.smem > (size_t)kMaxSmem) return pl;
    pl.grid = dim3((unsigned)std::min<int64_t>(sh.tiles, num_sms));
    pl.ok = true;
    return pl;
}

// Fused kernel that sweeps the nodes of a column in batches of nodes_per_block.
Plan plan_wide(const Shape& sh, int32_t n, int32_t nnz, int force_e = 0) {
    Plan pl;
    int E, G;
    pick_lane_shape(sh.tile, force_e, &E, &G);
    pl.elems_per_lane = E;
    pl.warps_per_group = G;
    if (sh.code == CODE_ID32 || G > 16) return pl;
    const int npb = std::max(1, std::min<int>(n, 16 / G));
    pl.nodes_per_block = npb;
    pl.block = dim3((unsigned)(npb * G * 32));
    const bool lut = (sh.code != CODE_SIGN);
    pl.smem = wide_smem_layout(sh.code_bits, lut, npb, G, sh.tile, n, nnz).total;
    if (pl.smem > (size_t)kMaxSmem) return pl;
    pl.grid = dim3((unsigned)std::min<int64_t>(sh.tiles, 0x7fffffff));
    pl.ok = true;
    return pl;
}

// Persistent TMA-staged kernel that sweeps the nodes of a column in batches.
Plan plan_wide_tma(const Shape& sh, int32_t n, int32_t nnz, int num_sms, int64_t l2_bytes, int force_e = 0) {
    Plan pl;
    int E, G;
    pick_lane_shape(sh.tile, force_e, &E, &G);
    pl.elems_per_lane = E;
    pl.warps_per_group = G;
    if (sh.code == CODE_ID32 || E < 8 || G > 16 || num_sms < 1) return pl;
    const int npb = std::max(1, std::min<int>(n, 16 / G));
    pl.nodes_per_block = npb;
    pl.block = dim3((unsigned)(npb * G * 32));
    const bool lut = (sh.code != CODE_SIGN);
    pl.smem = wide_tma_smem_layout(sh.code_bits, lut, E, npb * G, sh.tile, n, nnz).total;
    if (pl.smem > (size_t)kMaxSmem) return pl;
    pl.grid = dim3((unsigned)std::min<int64_t>(sh.tiles, num_sms));
    // x - gamma g of a whole column is parked in global memory between the two sweeps and should
    // still be in L2 when it is re-read: park it "evict last"; and once the parked columns of all
    // blocks take a quarter of L2 or more (many nodes), fetch the inputs, which are read once,
    // "evict first" (measured on 64 nodes x 1024: 1.46 -> 1.31 ms; on 8 nodes x 4096 that hint
    // costs 2 %, parking "evict last" alone gains 2.5 %)
    const int64_t parked = (int64_t)pl.grid.x * n * sh.tile * 4;
    pl.l2_hints = 2 | ((l2_bytes > 0 && parked * 4 >= l2_bytes) ? 1 : 0);
    pl.ok = true;
    return pl;
}

}  // namespace

struct ds_ctx {
    int32_t n, nnz;
    int64_t N, ld;
    ds_compressor comp;
    Shape sh;
    WsLayout ws;
    unsigned char* base;
    int path_req;
    Plan tma, tma_pair, wide_tma, fused, wide, compress, reduce;
    int num_sms;
    int64_t l2_bytes;
    bool pipe_ready;                                  // streams / events of ds_step_host
    cudaStream_t pipe_stream[3];
    cudaEvent_t pipe_event[2 * kMaxSlabs + 2];
    cudaStream_t capture_stream;                      // ds_run records its graph here
    cudaGraphExec_t run_exec;                         // executable graph of the last ds_run
    int32_t run_exec_steps;                           // T it was instantiated for (0 = none)
};

extern "C" {

const char* ds_strerror(ds_status status) {
    switch (status) {
        case DS_OK: return "ok";
        case DS_ERR_NULL: return "a required pointer is NULL";
        case DS_ERR_ARG: return "argument out of range";
        case DS_ERR_GRAPH: return "malformed CSR graph";
        case DS_ERR_W_NOT_SYMMETRIC: return "W is not symmetric";
        case DS_ERR_W_NOT_STOCHASTIC: return "W is not (doubly) stochastic";
        case DS_ERR_NO_SELF_LOOP: return "a node is not its own neighbour";
        case DS_ERR_ALIGN: return "pointer or pitch misaligned";
        case DS_ERR_WORKSPACE: return "workspace too small";
        case DS_ERR_UNSUPPORTED: return "unsupported combination";
        case DS_ERR_CUDA: return "CUDA runtime error";
        case DS_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out; the step is incomplete";
        case DS_ERR_BOUNDS: return "checked build: a kernel computed an index outside its arrays and skipped that part";
    }
    return "unknown status";
}

size_t ds_workspace_size(int32_t n, int64_t N, const ds_compressor* comp, int32_t nnz) {
    Shape sh;
    if (nnz < 1 || !make_shape(n, N, comp, &sh)) return 0;
    return make_ws(n, nnz, sh).total;
}

ds_status ds_init(ds_ctx** out, const ds_graph* graph, const float* W, int32_t n, int64_t N,
                  int64_t ld, const ds_compressor* comp, void* workspace, size_t workspace_bytes) {
    if (!out) return DS_ERR_NULL;
    *out = nullptr;
    if (!graph || !graph->row_ptr || !graph->col_idx || !W || !comp || !workspace) return DS_ERR_NULL;
    if (n < 1 || N < 1 || N >= ((int64_t)1 << 31) || graph->n != n || ld < N) return DS_ERR_ARG;
    if ((ld % 4) != 0) return DS_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(workspace) % kAlign) != 0) return DS_ERR_ALIGN;
    if (comp->kind < DS_COMP_IDENTITY || comp->kind > DS_COMP_UNIFORM_NEAREST_L2) return DS_ERR_ARG;
    if (comp->chunk < 0 || (comp->chunk % 32) != 0) return DS_ERR_ARG;
    Shape sh;
    if (!make_shape(n, N, comp, &sh)) return DS_ERR_UNSUPPORTED;

    // ---- graph: CSR well formed, sorted, self loop (Algorithm 1: i in N(i)) ----
    const int32_t* rp = graph->row_ptr;
    const int32_t* ci = graph->col_idx;
    if (rp[0] != 0) return DS_ERR_GRAPH;
    for (int32_t i = 0; i < n; ++i)
        if (rp[i + 1] < rp[i]) return DS_ERR_GRAPH;
    const int32_t nnz = rp[n];
    if (nnz < n) {
        // fewer entries than nodes: some row cannot hold its diagonal
        for (int32_t i = 0; i < n; ++i) {
            bool self = false;
            for (int32_t e = rp[i]; e < rp[i + 1]; ++e) self = self || (ci[e] == i);
            if (!self) return DS_ERR_NO_SELF_LOOP;
        }
        return DS_ERR_GRAPH;
    }
    for (int32_t i = 0; i < n; ++i) {
        bool self = false;
        for (int32_t e = rp[i]; e < rp[i + 1]; ++e) {
            if (ci[e] < 0 || ci[e] >= n) return DS_ERR_GRAPH;
            if (e > rp[i] && ci[e] <= ci[e - 1]) return DS_ERR_GRAPH;
            self = self || (ci[e] == i);
        }
        if (!self) return DS_ERR_NO_SELF_LOOP;
    }
    // ---- W: non-negative, symmetric, rows sum to one (Assumption 1) ----
    for (int32_t i = 0; i < n; ++i) {
        double rs = 0.0;
        for (int32_t e = rp[i]; e < rp[i + 1]; ++e) {
            const float w = W[e];
            if (!(w >= 0.0f) || !std::isfinite(w)) return DS_ERR_W_NOT_STOCHASTIC;
            rs += (double)w;
            const int32_t j = ci[e];
            const int32_t* lo = ci + rp[j];
            const int32_t* hi = ci + rp[j + 1];
            const int32_t* it = std::lower_bound(lo, hi, i);
            if (it == hi || *it != i) return DS_ERR_W_NOT_SYMMETRIC;
            if (std::fabs((double)W[it - ci] - (double)w) > 1e-6) return DS_ERR_W_NOT_SYMMETRIC;
        }
        if (std::fabs(rs - 1.0) > 1e-6) return DS_ERR_W_NOT_STOCHASTIC;
    }
    const WsLayout ws = make_ws(n, nnz, sh);
    if (workspace_bytes < ws.total) return DS_ERR_WORKSPACE;

    ds_ctx* ctx = new (std::nothrow) ds_ctx;
    if (!ctx) return DS_ERR_ARG;
    ctx->n = n; ctx->nnz = nnz; ctx->N = N; ctx->ld = ld;
    ctx->comp = *comp; ctx->sh = sh; ctx->ws = ws;
    ctx->base = static_cast<unsigned char*>(workspace);
    ctx->path_req = DS_PATH_AUTO;
    ctx->pipe_ready = false;
    ctx->capture_stream = nullptr;
    ctx->run_exec = nullptr;
    ctx->run_exec_steps = 0;
    ctx->compress = plan_column(MODE_COMPRESS, sh, n, nnz);
    ctx->reduce = plan_column(MODE_REDUCE, sh, n, nnz);
    if (!ctx->compress.ok) { delete ctx; return DS_ERR_UNSUPPORTED; }
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        (void)cudaGetLastError();
        delete ctx;
        return DS_ERR_CUDA;
    }
    ctx->num_sms = sms;
    int l2 = 0;
    if (cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, dev) != cudaSuccess) { (void)cudaGetLastError(); l2 = 0; }
    ctx->l2_bytes = l2;
    ctx->tma = plan_tma(sh, n, nnz, sms);
    ctx->tma_pair = plan_tma_pair(sh, n, nnz, sms);
    ctx->wide_tma = plan_wide_tma(sh, n, nnz, sms, ctx->l2_bytes);
    ctx->fused = plan_column(MODE_FUSED, sh, n, nnz);
    ctx->wide = plan_wide(sh, n, nnz);

    // w'_ij = W_ij - I_ij in binary32; reconstruction levels (2q - L)/L.
    std::vector<float> wprime((size_t)nnz);
    for (int32_t i = 0; i < n; ++i)
        for (int32_t e = rp[i]; e < rp[i + 1]; ++e)
            wprime[(size_t)e] = W[e] - ((ci[e] == i) ? 1.0f : 0.0f);
    float lut[256];
    std::memset(lut, 0, sizeof(lut));
    if (sh.code != CODE_ID32) {
        const int L = (1 << sh.code_bits) - 1;
        for (int q = 0; q <= L; ++q) lut[q] = (float)((double)(2 * q - L) / (double)L);
    }
    cudaError_t e = cudaMemcpy(ctx->base + ws.row_ptr, rp, (size_t)(n + 1) * 4, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(ctx->base + ws.col_idx, ci, (size_t)nnz * 4, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(ctx->base + ws.wprime, wprime.data(), (size_t)nnz * 4, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(ctx->base + ws.wplain, W, (size_t)nnz * 4, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(ctx->base + ws.lut, lut, sizeof(lut), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemset(ctx->base + ws.codes, 0, ws.scales - ws.codes);
    if (e == cudaSuccess) e = cudaMemset(ctx->base + ws.scales, 0, ws.partials - ws.scales);   // scales and decode factors
    if (e == cudaSuccess) e = cudaMemset(ctx->base + ws.error_flag, 0, 4);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        delete ctx;
        return DS_ERR_CUDA;
    }
    *out = ctx;
    return DS_OK;
}

void ds_destroy(ds_ctx* ctx) {
    if (!ctx) return;
    // an executable graph still in flight is freed by the runtime once it completes
    if (ctx->run_exec) (void)cudaGraphExecDestroy(ctx->run_exec);
    if (ctx->capture_stream) (void)cudaStreamDestroy(ctx->capture_stream);
    if (ctx->pipe_ready) {
        for (int i = 0; i < 3; ++i) (void)cudaStreamDestroy(ctx->pipe_stream[i]);
        for (int i = 0; i < 2 * kMaxSlabs + 2; ++i) (void)cudaEventDestroy(ctx->pipe_event[i]);
    }
    delete ctx;
}

// 2: persistent TMA-staged fused kernel, 5: the same with two nodes per warp (synthetic
// gradient only), 4: the same with the nodes in batches, 1: fused kernel with direct loads,
// 3: the same in node batches, 0: two kernels
static int fused_kind(const ds_ctx* ctx, bool grad_given = false) {
    if (ctx->path_req == DS_PATH_SPLIT) return 0;
    if (ctx->path_req != DS_PATH_FUSED_LDG) {
        if (ctx->tma_pair.ok && !grad_given) return 5;
        if (ctx->tma.ok) return 2;
        if (ctx->wide_tma.ok) return 4;
    }
    if (ctx->fused.ok) return 1;
    return ctx->wide.ok ? 3 : 0;
}

ds_status ds_set_path(ds_ctx* ctx, int32_t path) {
    if (!ctx) return DS_ERR_NULL;
    if (path < DS_PATH_AUTO || path > DS_PATH_FUSED_LDG) return DS_ERR_ARG;
    if (path == DS_PATH_FUSED && !ctx->fused.ok && !ctx->tma.ok && !ctx->tma_pair.ok && !ctx->wide.ok && !ctx->wide_tma.ok)
        return DS_ERR_UNSUPPORTED;
    if (path == DS_PATH_FUSED_LDG && !ctx->fused.ok && !ctx->wide.ok) return DS_ERR_UNSUPPORTED;
    ctx->path_req = path;
    return DS_OK;
}

ds_status ds_tune(ds_ctx* ctx, int32_t elems_per_lane) {
    if (!ctx) return DS_ERR_NULL;
    if (elems_per_lane != 0 && elems_per_lane != 4 && elems_per_lane != 8 && elems_per_lane != 16)
        return DS_ERR_ARG;
    const Plan compress = plan_column(MODE_COMPRESS, ctx->sh, ctx->n, ctx->nnz, elems_per_lane);
    if (!compress.ok) return DS_ERR_UNSUPPORTED;
    ctx->compress = compress;
    ctx->reduce = plan_column(MODE_REDUCE, ctx->sh, ctx->n, ctx->nnz, elems_per_lane);
    ctx->tma = plan_tma(ctx->sh, ctx->n, ctx->nnz, ctx->num_sms, elems_per_lane);
    ctx->tma_pair = plan_tma_pair(ctx->sh, ctx->n, ctx->nnz, ctx->num_sms, elems_per_lane);
    ctx->wide_tma = plan_wide_tma(ctx->sh, ctx->n, ctx->nnz, ctx->num_sms, ctx->l2_bytes, elems_per_lane);
    ctx->fused = plan_column(MODE_FUSED, ctx->sh, ctx->n, ctx->nnz, elems_per_lane);
    ctx->wide = plan_wide(ctx->sh, ctx->n, ctx->nnz, elems_per_lane);
    return DS_OK;
}

ds_status ds_get_info(const ds_ctx* ctx, ds_info* info) {
    if (!ctx || !info) return DS_ERR_NULL;
    const int kind = fused_kind(ctx);
    const bool fused = kind != 0;
    const Plan& pl = (kind == 2) ? ctx->tma : (kind == 5) ? ctx->tma_pair : (kind == 4) ? ctx->wide_tma : (kind == 1) ? ctx->fused
                   : (kind == 3) ? ctx->wide : ctx->compress;
    info->path = (kind == 2 || kind == 4 || kind == 5) ? DS_PATH_FUSED : (kind != 0) ? DS_PATH_FUSED_LDG : DS_PATH_SPLIT;
    info->node_batches = (kind == 3 || kind == 4) ? (ctx->n + pl.nodes_per_block - 1) / pl.nodes_per_block : 1;
    const bool norm = (ctx->sh.code == CODE_N2 || ctx->sh.code == CODE_N4);
    info->launches_per_step = (fused ? 1 : 2) + (ctx->sh.per_node ? (norm ? 4 : 2) : 0);
    info->elems_per_lane = pl.elems_per_lane;
    info->warps_per_chunk = pl.warps_per_group;
    info->block_threads = (int32_t)pl.block.x;
    info->grid_blocks = (int32_t)(pl.grid.x * pl.grid.y);
    info->chunks_per_row = ctx->sh.M;
    info->code_words_per_row = ctx->sh.code_words;
    return DS_OK;
}

ds_status ds_codes(ds_ctx* ctx, const uint32_t** codes, int64_t* code_pitch_words,
                   const float** scales, int64_t* scales_pitch) {
    if (!ctx || !codes || !code_pitch_words || !scales || !scales_pitch) return DS_ERR_NULL;
    *codes = reinterpret_cast<const uint32_t*>(ctx->base + ctx->ws.codes);
    *code_pitch_words = ctx->sh.code_pitch;
    *scales = reinterpret_cast<const float*>(ctx->base + ctx->ws.scales);
    *scales_pitch = ctx->sh.scales_pitch;
    return DS_OK;
}

// One iteration; `grad_kind` is a NOISE_* value for the synthetic gradient
// (a, c given) or GRAD_GIVEN (a is the gradient itself, c unused).
// ecsgd: the iteration of centralized error-compensated SGD (Section 1) instead
// of Algorithm 1 -- always two kernels: the workers' compression of g + delta,
// then the server's x <- x - gamma sum_j W_ij C_j, which is the mix kernel run
// with the weights W themselves and -gamma in the place of eta.
static ds_status run_step(ds_ctx* ctx, float* x, float* delta, const float* a, const float* c,
                          float sigma, int grad_kind, const ds_hparams* hp, uint64_t seed,
                          uint64_t step, void* cuda_stream, int64_t tile_begin = 0, int64_t tile_end = -1,
                          bool ecsgd = false) {
    if (step >= ((uint64_t)1 << 56)) return DS_ERR_ARG;
    if (tile_end < 0) tile_end = ctx->sh.tiles;
    const uintptr_t bits = reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(delta) |
                           reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(c);
    if ((bits % 16) != 0) return DS_ERR_ALIGN;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    StepParams p;
    p.x = x; p.delta = delta; p.a = a; p.c = c;
    p.ld = ctx->ld; p.N = ctx->N; p.n = ctx->n; p.nnz = ctx->nnz;
    p.tile = ctx->sh.tile; p.tiles = ctx->sh.tiles;
    p.tile_begin = tile_begin; p.tile_end = tile_end;
    p.row_ptr = reinterpret_cast<const int32_t*>(ctx->base + ctx->ws.row_ptr);
    p.col_idx = reinterpret_cast<const int32_t*>(ctx->base + ctx->ws.col_idx);
    p.wprime = reinterpret_cast<const float*>(ctx->base + ctx->ws.wprime);
    p.lut = reinterpret_cast<const float*>(ctx->base + ctx->ws.lut);
    p.codes = reinterpret_cast<uint32_t*>(ctx->base + ctx->ws.codes);
    p.code_pitch = ctx->sh.code_pitch;
    p.scales = reinterpret_cast<float*>(ctx->base + ctx->ws.scales);
    p.scales_pitch = ctx->sh.scales_pitch;
    p.dscales = reinterpret_cast<float*>(ctx->base + ctx->ws.dscales);
    p.partials = reinterpret_cast<double*>(ctx->base + ctx->ws.partials);
    p.gmax = reinterpret_cast<float*>(ctx->base + ctx->ws.gmax);
    p.norm_phase = 0;
    p.l2_hints = 0;
    p.error_flag = reinterpret_cast<int*>(ctx->base + ctx->ws.error_flag);
    p.sigma = sigma;
    p.neg_gamma = -hp->gamma;
    p.eta = hp->eta;
    p.rs = make_rng_step(seed, step);
    p.prescaled = ctx->sh.per_node ? 1 : 0;
    p.ecsgd = ecsgd ? 1 : 0;
    if (ecsgd) {
        p.wprime = reinterpret_cast<const float*>(ctx->base + ctx->ws.wplain);
        p.eta = -hp->gamma;
    }

    auto shape_of = [&](const Plan& pl, int mode) {
        LaunchShape s;
        s.code = ctx->sh.code; s.noise = grad_kind; s.elems_per_lane = pl.elems_per_lane;
        s.mode = mode; s.grid = pl.grid; s.block = pl.block; s.smem = pl.smem;
        // a launch over part of the tiles needs no more blocks than tiles
        s.grid.x = (unsigned)std::max<int64_t>(1, std::min<int64_t>(pl.grid.x, tile_end - tile_begin));
        return s;
    };
    cudaError_t e = cudaSuccess;
    if (ctx->sh.per_node) {
        p.warps_per_group = ctx->reduce.warps_per_group;
        p.nodes_per_block = ctx->reduce.nodes_per_block;
        e = launch_column_reduce(shape_of(ctx->reduce, MODE_REDUCE), p, stream);
        if (e == cudaSuccess) e = launch_finalize_scales(p, ctx->sh.code, stream);
        if (ctx->sh.code == CODE_N2 || ctx->sh.code == CODE_N4) {
            // one norm per node (Section 5: one Euclidean norm per tensor): with the maximum
            // known, a second reduction takes the sums of v^2 and of level^2
            p.norm_phase = 2;
            if (e == cudaSuccess) e = launch_column_reduce_norm(shape_of(ctx->reduce, MODE_REDUCE), p, stream);
            if (e == cudaSuccess) e = launch_finalize_norms(p, stream);
            p.norm_phase = 0;
        }
    }
    if (e == cudaSuccess) {
        // centralized error-compensated SGD: the fused kernel where the shape allows
        // (16 elements per lane, at most 512 threads), else two kernels
        const bool ecsgd_fused = ecsgd && ctx->path_req != DS_PATH_SPLIT && ctx->path_req != DS_PATH_FUSED_LDG &&
                                 ctx->tma.ok && ctx->tma.elems_per_lane == 16 && ctx->tma.block.x <= 512;
        const int kind = ecsgd ? 0 : fused_kind(ctx, grad_kind == GRAD_GIVEN || grad_kind == NOISE_T3I);
        if (ecsgd_fused) {
            p.ecsgd = 0;          // the fused kernel is its own instantiation; the flag is for the two-kernel path
            p.warps_per_group = ctx->tma.warps_per_group;
            p.nodes_per_block = ctx->tma.nodes_per_block;
            e = launch_fused_tma_ecsgd(shape_of(ctx->tma, MODE_FUSED), p, stream);
        } else if (kind == 5) {
            p.warps_per_group = 1;
            p.nodes_per_block = ctx->n;
            e = launch_fused_tma_pair(shape_of(ctx->tma_pair, MODE_FUSED), p, stream);
        } else if (kind == 2) {
            p.warps_per_group = ctx->tma.warps_per_group;
            p.nodes_per_block = ctx->tma.nodes_per_block;
            e = launch_fused_tma(shape_of(ctx->tma, MODE_FUSED), p, stream);
        } else if (kind == 4) {
            p.warps_per_group = ctx->wide_tma.warps_per_group;
            p.nodes_per_block = ctx->wide_tma.nodes_per_block;
            p.l2_hints = ctx->wide_tma.l2_hints;
            e = launch_fused_wide_tma(shape_of(ctx->wide_tma, MODE_FUSED), p, stream);
        } else if (kind == 3) {
            p.warps_per_group = ctx->wide.warps_per_group;
            p.nodes_per_block = ctx->wide.nodes_per_block;
            e = launch_fused_wide(shape_of(ctx->wide, MODE_FUSED), p, stream);
        } else if (kind == 1) {
            p.warps_per_group = ctx->fused.warps_per_group;
            p.nodes_per_block = ctx->fused.nodes_per_block;
            e = launch_column_fused(shape_of(ctx->fused, MODE_FUSED), p, stream);
        } else {
            p.warps_per_group = ctx->compress.warps_per_group;
            p.nodes_per_block = ctx->compress.nodes_per_block;
            e = launch_column_compress(shape_of(ctx->compress, MODE_COMPRESS), p, stream);
            if (e == cudaSuccess) e = launch_mix_kernel(p, ctx->sh.code, stream);
        }
    }
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return DS_ERR_CUDA;
    }
    return DS_OK;
}

ds_status ds_step(ds_ctx* ctx, float* x, float* delta, const ds_grad_params* gp, const ds_hparams* hp,
                  uint64_t seed, uint64_t step, void* cuda_stream) {
    if (!ctx || !x || !delta || !gp || !hp || !gp->a || !gp->c) return DS_ERR_NULL;
    if (gp->noise < DS_NOISE_NONE || gp->noise > DS_NOISE_STUDENT_T3_IID) return DS_ERR_ARG;
    return run_step(ctx, x, delta, gp->a, gp->c, gp->sigma, noise_template_of(gp->noise), hp, seed, step, cuda_stream);
}

ds_status ds_step_g(ds_ctx* ctx, float* x, float* delta, const float* g, const ds_hparams* hp,
                    uint64_t seed, uint64_t step, void* cuda_stream) {
    if (!ctx || !x || !delta || !g || !hp) return DS_ERR_NULL;
    return run_step(ctx, x, delta, g, nullptr, 0.0f, GRAD_GIVEN, hp, seed, step, cuda_stream);
}

ds_status ds_ecsgd_step(ds_ctx* ctx, float* x, float* delta, const ds_grad_params* gp, float gamma,
                        uint64_t seed, uint64_t step, void* cuda_stream) {
    if (!ctx || !x || !delta || !gp || !gp->a || !gp->c) return DS_ERR_NULL;
    if (gp->noise < DS_NOISE_NONE || gp->noise > DS_NOISE_STUDENT_T3_IID) return DS_ERR_ARG;
    const ds_hparams hp = {gamma, 0.0f};
    return run_step(ctx, x, delta, gp->a, gp->c, gp->sigma, noise_template_of(gp->noise), &hp, seed, step, cuda_stream, 0, -1, true);
}

ds_status ds_ecsgd_step_g(ds_ctx* ctx, float* x, float* delta, const float* g, float gamma,
                          uint64_t seed, uint64_t step, void* cuda_stream) {
    if (!ctx || !x || !delta || !g) return DS_ERR_NULL;
    const ds_hparams hp = {gamma, 0.0f};
    return run_step(ctx, x, delta, g, nullptr, 0.0f, GRAD_GIVEN, &hp, seed, step, cuda_stream, 0, -1, true);
}

ds_status ds_run(ds_ctx* ctx, float* x, float* delta, const ds_grad_params* gp, const float* gammas,
                 const float* etas, int32_t T, uint64_t seed, uint64_t step0, void* cuda_stream) {
    if (!ctx || !x || !delta || !gp || !gp->a || !gp->c || !gammas || !etas) return DS_ERR_NULL;
    if (gp->noise < DS_NOISE_NONE || gp->noise > DS_NOISE_STUDENT_T3_IID) return DS_ERR_ARG;
    if (T < 1 || T > DS_RUN_MAX_STEPS) return DS_ERR_ARG;
    if (step0 >= ((uint64_t)1 << 56) || step0 + (uint64_t)T > ((uint64_t)1 << 56)) return DS_ERR_ARG;
    const uintptr_t bits = reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(delta) |
                           reinterpret_cast<uintptr_t>(gp->a) | reinterpret_cast<uintptr_t>(gp->c);
    if ((bits % 16) != 0) return DS_ERR_ALIGN;
    if (!ctx->capture_stream &&
        cudaStreamCreateWithFlags(&ctx->capture_stream, cudaStreamNonBlocking) != cudaSuccess) {
        (void)cudaGetLastError();
        ctx->capture_stream = nullptr;
        return DS_ERR_CUDA;
    }
    // Record: the launches go into a graph, none of them runs here.
    if (cudaStreamBeginCapture(ctx->capture_stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
        (void)cudaGetLastError();
        return DS_ERR_CUDA;
    }
    ds_status st = DS_OK;
    for (int32_t t = 0; t < T && st == DS_OK; ++t) {
        const ds_hparams hp = {gammas[t], etas[t]};
        st = run_step(ctx, x, delta, gp->a, gp->c, gp->sigma, noise_template_of(gp->noise), &hp, seed, step0 + (uint64_t)t,
                      ctx->capture_stream);
    }
    cudaGraph_t graph = nullptr;
    cudaError_t e = cudaStreamEndCapture(ctx->capture_stream, &graph);    // always ends the capture
    if (st != DS_OK || e != cudaSuccess || !graph) {
        (void)cudaGetLastError();
        if (graph) (void)cudaGraphDestroy(graph);
        return st != DS_OK ? st : DS_ERR_CUDA;
    }
    // Same T as last time: same topology, only kernel arguments differ.
    if (ctx->run_exec && ctx->run_exec_steps == T) {
        cudaGraphExecUpdateResultInfo info;
        if (cudaGraphExecUpdate(ctx->run_exec, graph, &info) != cudaSuccess) {
            (void)cudaGetLastError();
            (void)cudaGraphExecDestroy(ctx->run_exec);
            ctx->run_exec = nullptr;
        }
    } else if (ctx->run_exec) {
        (void)cudaGraphExecDestroy(ctx->run_exec);
        ctx->run_exec = nullptr;
    }
    if (!ctx->run_exec) {
        ctx->run_exec_steps = 0;
        e = cudaGraphInstantiate(&ctx->run_exec, graph, 0);
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            ctx->run_exec = nullptr;
            (void)cudaGraphDestroy(graph);
            return DS_ERR_CUDA;
        }
        ctx->run_exec_steps = T;
    }
    (void)cudaGraphDestroy(graph);
    e = cudaGraphLaunch(ctx->run_exec, static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return DS_ERR_CUDA;
    }
    return DS_OK;
}

ds_status ds_run_resident(ds_ctx* ctx, float* x, float* delta, const ds_grad_params* gp, const float* gammas,
                          const float* etas, int32_t T, uint64_t seed, uint64_t step0, void* cuda_stream) {
    if (!ctx || !x || !delta || !gp || !gp->a || !gp->c || !gammas || !etas) return DS_ERR_NULL;
    if (gp->noise < DS_NOISE_NONE || gp->noise > DS_NOISE_STUDENT_T3_IID) return DS_ERR_ARG;
    if (T < 1 || T > DS_RESIDENT_MAX_STEPS) return DS_ERR_ARG;
    if (step0 >= ((uint64_t)1 << 56) || step0 + (uint64_t)T > ((uint64_t)1 << 56)) return DS_ERR_ARG;
    const uintptr_t bits = reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(delta) |
                           reinterpret_cast<uintptr_t>(gp->a) | reinterpret_cast<uintptr_t>(gp->c);
    if ((bits % 16) != 0) return DS_ERR_ALIGN;
    if (!resident_shape(ctx->n, ctx->sh) || gp->noise == DS_NOISE_STUDENT_T3_IID) return DS_ERR_UNSUPPORTED;
    if (resident_smem_layout(ctx->n, ctx->nnz).total > (size_t)kMaxSmem) return DS_ERR_UNSUPPORTED;

    static_assert(DS_RESIDENT_MAX_STEPS == kResidentMaxSteps, "header and kernel disagree");
    ResidentParams rp;
    StepParams& p = rp.p;
    p.x = x; p.delta = delta; p.a = gp->a; p.c = gp->c;
    p.ld = ctx->ld; p.N = ctx->N; p.n = ctx->n; p.nnz = ctx->nnz;
    p.tile = ctx->sh.tile; p.tiles = ctx->sh.tiles;
    p.tile_begin = 0; p.tile_end = ctx->sh.tiles;
    p.row_ptr = reinterpret_cast<const int32_t*>(ctx->base + ctx->ws.row_ptr);
    p.col_idx = reinterpret_cast<const int32_t*>(ctx->base + ctx->ws.col_idx);
    p.wprime = reinterpret_cast<const float*>(ctx->base + ctx->ws.wprime);
    p.lut = reinterpret_cast<const float*>(ctx->base + ctx->ws.lut);
    p.codes = reinterpret_cast<uint32_t*>(ctx->base + ctx->ws.codes);
    p.code_pitch = ctx->sh.code_pitch;
    p.scales = reinterpret_cast<float*>(ctx->base + ctx->ws.scales);
    p.scales_pitch = ctx->sh.scales_pitch;
    p.dscales = reinterpret_cast<float*>(ctx->base + ctx->ws.dscales);
    p.partials = reinterpret_cast<double*>(ctx->base + ctx->ws.partials);
    p.gmax = nullptr;
    p.norm_phase = 0;
    p.l2_hints = 0;
    p.error_flag = reinterpret_cast<int*>(ctx->base + ctx->ws.error_flag);
    p.sigma = gp->sigma;
    p.neg_gamma = 0.0f; p.eta = 0.0f;
    p.rs = make_rng_step(seed, step0);
    p.warps_per_group = 1; p.nodes_per_block = ctx->n;
    p.prescaled = ctx->sh.per_node ? 1 : 0;
    p.ecsgd = 0;
    rp.partials2 = reinterpret_cast<double*>(ctx->base + ctx->ws.rpartials);
    rp.barrier = reinterpret_cast<unsigned int*>(ctx->base + ctx->ws.barrier);
    rp.step0 = step0;
    rp.T = T;
    std::memcpy(rp.gammas, gammas, (size_t)T * sizeof(float));
    std::memcpy(rp.etas, etas, (size_t)T * sizeof(float));
    const cudaError_t e = launch_resident(ctx->sh.code, gp->noise, rp, ctx->num_sms, static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return e == cudaErrorCooperativeLaunchTooLarge ? DS_ERR_UNSUPPORTED : DS_ERR_CUDA;
    }
    return DS_OK;
}

// Streams and events of the host-buffer entry point, made on first use.
static bool ensure_pipeline(ds_ctx* ctx) {
    if (ctx->pipe_ready) return true;
    bool ok = true;
    for (int i = 0; i < 3 && ok; ++i)
        ok = cudaStreamCreateWithFlags(&ctx->pipe_stream[i], cudaStreamNonBlocking) == cudaSuccess;
    for (int i = 0; i < 2 * kMaxSlabs + 2 && ok; ++i)
        ok = cudaEventCreateWithFlags(&ctx->pipe_event[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) { (void)cudaGetLastError(); return false; }
    ctx->pipe_ready = true;
    return true;
}

ds_status ds_step_host(ds_ctx* ctx, float* x_host, float* delta_host, const float* a_host,
                       const float* c_host, float sigma, int32_t noise, const ds_hparams* hp,
                       uint64_t seed, uint64_t step, float* dev_x, float* dev_delta, float* dev_a,
                       float* dev_c, void* cuda_stream) {
    if (!ctx || !x_host || !delta_host || !a_host || !c_host || !hp || !dev_x || !dev_delta ||
        !dev_a || !dev_c)
        return DS_ERR_NULL;
    if (noise < DS_NOISE_NONE || noise > DS_NOISE_STUDENT_T3_IID) return DS_ERR_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t pitch = (size_t)ctx->ld * sizeof(float);
    const size_t bytes = (size_t)ctx->n * pitch;

    // Column tiles are independent unless one scale covers a whole node, so the
    // step is cut into slabs of tiles and pipelined: slab s+1 travels to the
    // device while slab s is computed and slab s-1 travels back (PCIe carries
    // both directions at once).
    const int64_t tiles = ctx->sh.tiles;
    int slabs = 1;
    if (!ctx->sh.per_node && bytes >= ((size_t)64 << 20)) slabs = (int)std::min<int64_t>(kMaxSlabs, tiles);
    if (slabs == 1 || !ensure_pipeline(ctx)) {
        cudaError_t e = cudaMemcpyAsync(dev_x, x_host, bytes, cudaMemcpyHostToDevice, stream);
        if (e == cudaSuccess) e = cudaMemcpyAsync(dev_delta, delta_host, bytes, cudaMemcpyHostToDevice, stream);
        if (e == cudaSuccess) e = cudaMemcpyAsync(dev_a, a_host, bytes, cudaMemcpyHostToDevice, stream);
        if (e == cudaSuccess) e = cudaMemcpyAsync(dev_c, c_host, bytes, cudaMemcpyHostToDevice, stream);
        if (e != cudaSuccess) { (void)cudaGetLastError(); return DS_ERR_CUDA; }
        const ds_status st = run_step(ctx, dev_x, dev_delta, dev_a, dev_c, sigma, noise_template_of(noise), hp, seed, step, cuda_stream);
        if (st != DS_OK) return st;
        e = cudaMemcpyAsync(x_host, dev_x, bytes, cudaMemcpyDeviceToHost, stream);
        if (e == cudaSuccess) e = cudaMemcpyAsync(delta_host, dev_delta, bytes, cudaMemcpyDeviceToHost, stream);
        if (e != cudaSuccess) { (void)cudaGetLastError(); return DS_ERR_CUDA; }
        return DS_OK;
    }

    cudaStream_t s_in = ctx->pipe_stream[0], s_run = ctx->pipe_stream[1], s_out = ctx->pipe_stream[2];
    cudaEvent_t ev_start = ctx->pipe_event[2 * kMaxSlabs], ev_done = ctx->pipe_event[2 * kMaxSlabs + 1];
    cudaError_t e = cudaEventRecord(ev_start, stream);
    for (int i = 0; i < 3 && e == cudaSuccess; ++i) e = cudaStreamWaitEvent(ctx->pipe_stream[i], ev_start, 0);
    const int64_t per = (tiles + slabs - 1) / slabs;
    ds_status failed = DS_OK;
    for (int sidx = 0; sidx < slabs && e == cudaSuccess; ++sidx) {
        const int64_t t0 = sidx * per, t1 = std::min<int64_t>(tiles, t0 + per);
        if (t0 >= t1) break;
        const int64_t c0 = t0 * ctx->sh.tile;
        const int64_t c_in = ((t1 == tiles) ? ctx->ld : t1 * ctx->sh.tile) - c0;     // the last slab carries the padding
        const int64_t c_out = std::min<int64_t>(ctx->N, t1 * ctx->sh.tile) - c0;
        const float* src[4] = {x_host, delta_host, a_host, c_host};
        float* dst[4] = {dev_x, dev_delta, dev_a, dev_c};
        for (int k = 0; k < 4 && e == cudaSuccess; ++k)
            e = cudaMemcpy2DAsync(dst[k] + c0, pitch, src[k] + c0, pitch, (size_t)c_in * sizeof(float),
                                  (size_t)ctx->n, cudaMemcpyHostToDevice, s_in);
        if (e == cudaSuccess) e = cudaEventRecord(ctx->pipe_event[2 * sidx], s_in);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(s_run, ctx->pipe_event[2 * sidx], 0);
        if (e != cudaSuccess) break;
        failed = run_step(ctx, dev_x, dev_delta, dev_a, dev_c, sigma, noise_template_of(noise), hp, seed, step, s_run, t0, t1);
        if (failed != DS_OK) break;
        e = cudaEventRecord(ctx->pipe_event[2 * sidx + 1], s_run);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(s_out, ctx->pipe_event[2 * sidx + 1], 0);
        if (e == cudaSuccess)
            e = cudaMemcpy2DAsync(x_host + c0, pitch, dev_x + c0, pitch, (size_t)c_out * sizeof(float),
                                  (size_t)ctx->n, cudaMemcpyDeviceToHost, s_out);
        if (e == cudaSuccess)
            e = cudaMemcpy2DAsync(delta_host + c0, pitch, dev_delta + c0, pitch, (size_t)c_out * sizeof(float),
                                  (size_t)ctx->n, cudaMemcpyDeviceToHost, s_out);
    }
    if (failed != DS_OK || e != cudaSuccess) {
        // Error path: copies and kernels already enqueued on the internal streams may still be
        // touching the caller's buffers.  Whatever was enqueued is joined into the caller's
        // stream before the error is returned, so that the caller's next work on that stream
        // (or its synchronisation) is ordered after all of it.
        (void)cudaGetLastError();
        cudaEvent_t ev_in = ctx->pipe_event[0], ev_run = ctx->pipe_event[1];
        bool joined = cudaEventRecord(ev_in, s_in) == cudaSuccess && cudaStreamWaitEvent(s_out, ev_in, 0) == cudaSuccess &&
                      cudaEventRecord(ev_run, s_run) == cudaSuccess && cudaStreamWaitEvent(s_out, ev_run, 0) == cudaSuccess &&
                      cudaEventRecord(ev_done, s_out) == cudaSuccess && cudaStreamWaitEvent(stream, ev_done, 0) == cudaSuccess;
        if (!joined) {
            (void)cudaGetLastError();
            for (int i = 0; i < 3; ++i) (void)cudaStreamSynchronize(ctx->pipe_stream[i]);   // last resort: wait here
            (void)cudaGetLastError();
        }
        return failed != DS_OK ? failed : DS_ERR_CUDA;
    }
    // the caller's stream continues when the last slab is back (which implies every earlier stage)
    e = cudaEventRecord(ev_done, s_out);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(stream, ev_done, 0);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        for (int i = 0; i < 3; ++i) (void)cudaStreamSynchronize(ctx->pipe_stream[i]);
        (void)cudaGetLastError();
        return DS_ERR_CUDA;
    }
    return DS_OK;
}

ds_status ds_sync(ds_ctx* ctx, void* cuda_stream) {
    if (!ctx) return DS_ERR_NULL;
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream));
    int flag = 0;
    if (e == cudaSuccess) e = cudaMemcpy(&flag, ctx->base + ctx->ws.error_flag, 4, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return DS_ERR_CUDA; }
    if (flag != 0) {
        (void)cudaMemset(ctx->base + ctx->ws.error_flag, 0, 4);
        return (flag & DS_FLAG_BOUNDS) ? DS_ERR_BOUNDS : DS_ERR_TIMEOUT;
    }
    return DS_OK;
}

ds_status ds_selftest_bounds(ds_ctx* ctx, void* cuda_stream) {
    if (!ctx) return DS_ERR_NULL;
#if DS_CHECKED_BUILD
    StepParams p = {};
    p.n = ctx->n; p.N = ctx->N; p.ld = ctx->ld;
    p.code_pitch = ctx->sh.code_pitch; p.scales_pitch = ctx->sh.scales_pitch; p.tiles = ctx->sh.tiles;
    p.error_flag = reinterpret_cast<int*>(ctx->base + ctx->ws.error_flag);
    const cudaError_t e = launch_bounds_selftest(p, static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) { (void)cudaGetLastError(); return DS_ERR_CUDA; }
    return DS_OK;
#else
    (void)cuda_stream;
    return DS_ERR_UNSUPPORTED;        // the normal build has no index checks
#endif
}

ds_status ds_selftest_math(uint64_t* counts, void* cuda_stream) {
    if (!counts) return DS_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(counts) % 8) != 0) return DS_ERR_ALIGN;
    const cudaError_t e = launch_math_selftest(reinterpret_cast<unsigned long long*>(counts),
                                               static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) { (void)cudaGetLastError(); return DS_ERR_CUDA; }
    return DS_OK;
}

ds_status ds_selftest_timeout(ds_ctx* ctx, void* cuda_stream) {
    if (!ctx) return DS_ERR_NULL;
    const cudaError_t e = launch_wait_selftest(reinterpret_cast<int*>(ctx->base + ctx->ws.error_flag),
                                               static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) { (void)cudaGetLastError(); return DS_ERR_CUDA; }
    return DS_OK;
}

ds_status ds_noise(float* out, int32_t n, int64_t N, int64_t ld_out, int32_t which, int32_t noise,
                   uint64_t seed, uint64_t step, void* cuda_stream) {
    if (!out) return DS_ERR_NULL;
    if (n < 1 || N < 1 || N >= ((int64_t)1 << 31) || ld_out < N || which < 0 || which > 1 ||
        noise < DS_NOISE_NONE || noise > DS_NOISE_STUDENT_T3_IID || step >= ((uint64_t)1 << 56))
        return DS_ERR_ARG;
    const cudaError_t e = launch_noise_kernel(out, n, N, ld_out, which, noise_template_of(noise), make_rng_step(seed, step),
                                              static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) { (void)cudaGetLastError(); return DS_ERR_CUDA; }
    return DS_OK;
}

}  // extern "C"
