/*
 * deepsqueeze.h -- C ABI of the DeepSqueeze node-update library for one
 * NVIDIA B200 (sm_100a).
 *
 * The library runs one iteration of Algorithm 1 ("DeepSqueeze", error-
 * compensated compressed decentralized SGD) for n simulated nodes that are
 * stored as the rows of device arrays on ONE GPU:
 *
 *     g_i      = stochastic gradient of f_i at x_i                (Algorithm 1, gradient step)
 *     v_i      = x_i - gamma g_i + delta_i                        (error-compensated variable)
 *     C[v_i], delta_i <- v_i - C[v_i]                             (compression step)
 *     x_i     <- x_i - gamma g_i + eta sum_{j in N(i)} (W_ij - I_ij) C[v_j]   (local update;
 *                i itself belongs to N(i); Section 3 gives the same rule in matrix form)
 *
 * "Send" and "receive" of Algorithm 1 are a read of the packed codes that all
 * nodes of the simulation share on the device.
 *
 * Conventions
 *   - All arrays are row-major [n][ld] binary32 with a common row pitch ld
 *     (elements), ld >= N, ld a multiple of 4, base pointers 16-byte aligned.
 *     Columns N..ld-1 are padding: read, never changed.
 *   - Pointers are DEVICE pointers unless the comment says "host".
 *   - The caller owns every buffer, the workspace included; the library
 *     calls no device-memory allocator (cudaMalloc and friends).  x and delta
 *     are updated in place.  Two entry points create other driver objects
 *     inside the context, on first use, and ds_destroy releases them:
 *     ds_run records and instantiates a CUDA graph (one internal capture
 *     stream, one executable graph), ds_step_host creates three streams and
 *     34 events for its copy/compute pipeline.  Nothing else creates any.
 *   - Every call returns a ds_status; nothing throws.  ds_step only enqueues
 *     work on the given stream and reports argument and launch errors.
 *   - One ds_ctx must not be used from two streams at once (the steps share
 *     the workspace).
 */
#ifndef DEEPSQUEEZE_H
#define DEEPSQUEEZE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ds_ctx ds_ctx;   /* opaque; created by ds_init, freed by ds_destroy */

typedef enum {
    DS_OK = 0,
    DS_ERR_NULL = 1,             /* a required pointer is NULL */
    DS_ERR_ARG = 2,              /* a size or scalar argument is out of range */
    DS_ERR_GRAPH = 3,            /* CSR malformed: row_ptr not monotone, column out of range, unsorted or duplicate */
    DS_ERR_W_NOT_SYMMETRIC = 4,  /* |W_ij - W_ji| > 1e-6, or the pattern itself is not symmetric */
    DS_ERR_W_NOT_STOCHASTIC = 5, /* a row sum differs from 1 by more than 1e-6, or a weight is negative */
    DS_ERR_NO_SELF_LOOP = 6,     /* some node is not its own neighbour */
    DS_ERR_ALIGN = 7,            /* pointer not 16-byte aligned, or pitch not a multiple of 4 */
    DS_ERR_WORKSPACE = 8,        /* workspace smaller than ds_workspace_size() */
    DS_ERR_UNSUPPORTED = 9,      /* combination not implemented (e.g. bits not in {1,2,4,8}) */
    DS_ERR_CUDA = 10,            /* a CUDA runtime call failed (no device, launch error, ...) */
    DS_ERR_TIMEOUT = 11,         /* a bounded wait inside a kernel ran out; x, delta are incomplete */
    DS_ERR_BOUNDS = 12           /* checked build only: a kernel computed an index outside its arrays; that
                                    part of the step was skipped, nothing out of range was touched */
} ds_status;

/* Node graph in CSR form, HOST memory: row i lists N(i) in ascending order
 * and contains i itself (Algorithm 1, receive step: "i in N(i)"). */
typedef struct {
    int32_t n;
    const int32_t *row_ptr;     /* host, n+1 entries, row_ptr[0] = 0 */
    const int32_t *col_idx;     /* host, row_ptr[n] entries */
} ds_graph;

/* Compressor C_omega (Algorithm 1, compression step; Section 5, "Compression":
 * every element is sent with b bits plus one scalar per tensor).
 *   DS_COMP_IDENTITY             C[v] = v: no compression, i.e. D-PSGD (Section 3.2), the
 *                                baseline the paper compares with; the "codes" are the bit
 *                                patterns of v, 32 bits per element; bits is ignored.
 *   DS_COMP_SIGN1_L1             one bit per element: bit = (v >= 0); C = +s / -s with
 *                                s = (sum |v|)/m over the chunk (binary64 sum); bits must be 1.
 *   DS_COMP_UNIFORM_STOCH_MAXABS b in {1,2,4,8} bits: 2^b levels evenly spaced on
 *                                [-s, s], s = max |v| over the chunk, stochastic rounding
 *                                with a Philox4x32-10 stream; unbiased.
 *   DS_COMP_UNIFORM_NEAREST_L2   the paper's own "bit compression" (Section 5): b in {2,4} bits,
 *                                each element rounded to the NEAREST of 2^b levels spanning
 *                                [-max|v|, max|v|]; the scalar sent with the chunk is the
 *                                Euclidean norm ||v||_2, and the receiver rescales what it
 *                                decodes to that norm: C = level[code] * ||v||_2 / ||level[code]||_2.
 *                                Deterministic and biased -- what error compensation is for.
 *                                One chunk = one "tensor"; chunk = 0 is the paper's granularity,
 *                                one norm for the node's whole vector (five launches per step:
 *                                maximum per tile, maximum per node, sums of squares per tile,
 *                                norm per node, then the fused kernel with all three given).
 * chunk: elements per scale, a multiple of 32; 0 = one scale per node. */
typedef enum {
    DS_COMP_IDENTITY = 0,
    DS_COMP_SIGN1_L1 = 1,
    DS_COMP_UNIFORM_STOCH_MAXABS = 2,
    DS_COMP_UNIFORM_NEAREST_L2 = 3
} ds_comp_kind;

typedef struct {
    int32_t kind;               /* ds_comp_kind */
    int32_t bits;
    int64_t chunk;
} ds_compressor;

/* Stochastic gradient of the synthetic objective (Eq. 1 with
 * f_i(x) = 1/2 sum_k a_ik (x_k - c_ik)^2):  g_ik = a_ik (x_ik - c_ik) + sigma z_ik,
 * z drawn inside the kernel from Philox4x32-10 keyed by (seed, node, step, index). */
typedef enum {
    DS_NOISE_NONE = 0,
    DS_NOISE_GAUSS = 1,         /* standard normal (Box-Muller) */
    DS_NOISE_STUDENT_T3 = 2,    /* Student t, 3 degrees of freedom, not re-normalised: consecutive
                                   elements (2m, 2m+1) form a spherical bivariate t(3) pair
                                   (each exactly t(3), uncorrelated, sharing one radius) */
    DS_NOISE_STUDENT_T3_IID = 3 /* the same marginal law with INDEPENDENT coordinates, by the textbook
                                   construction Z0 / sqrt((Z1^2 + Z2^2 + Z3^2) / 3): one Philox block
                                   and four normals per element -- about three times the arithmetic
                                   of the pairs, so steps with it are bound by the instruction
                                   stream, not by memory.  Not taken by ds_run_resident
                                   (DS_ERR_UNSUPPORTED) nor by the two-nodes-per-warp kernel (such
                                   shapes run on the one-node-per-warp kernel) */
} ds_noise_kind;

typedef struct {
    const float *a;             /* device [n][ld] */
    const float *c;             /* device [n][ld] */
    float sigma;
    int32_t noise;              /* ds_noise_kind */
} ds_grad_params;

typedef struct {
    float gamma;                /* learning rate (multiplies g only) */
    float eta;                  /* averaging rate (multiplies the whole neighbour sum) */
} ds_hparams;

/* How a step is executed.
 *   DS_PATH_FUSED      one kernel: a thread block owns one chunk column of ALL nodes, keeps
 *                      x - gamma g in registers and the column's C[v] in shared memory, and
 *                      mixes without re-reading anything from global memory.  Where the
 *                      column fits in shared memory this is the persistent kernel whose
 *                      inputs are staged by bulk asynchronous copies (TMA); for columns of
 *                      many nodes or long chunks the same kernel sweeps the nodes in batches
 *                      (x - gamma g parked in x and re-read from L2, packed codes of the whole
 *                      column in shared memory); otherwise the variant below.
 *   DS_PATH_FUSED_LDG  the fused kernel with direct vector loads and packed codes in shared
 *                      memory (one block per column).  When a block cannot hold all nodes of
 *                      a column at once (many nodes, long chunks) it sweeps them in batches:
 *                      x - gamma g is parked in x, the codes of the whole column stay in shared
 *                      memory, and a second sweep re-reads the parked values (from L2) to mix.
 *   DS_PATH_SPLIT      two kernels: compress (x - gamma g written into x, codes to the
 *                      workspace), then mix (each neighbour's packed codes streamed once and
 *                      decoded in registers).  Works for every shape.
 *   DS_PATH_AUTO       the first of the three that the shape allows. */
typedef enum { DS_PATH_AUTO = 0, DS_PATH_FUSED = 1, DS_PATH_SPLIT = 2, DS_PATH_FUSED_LDG = 3 } ds_path;

typedef struct {
    int32_t path;               /* ds_path actually used by ds_step */
    int32_t launches_per_step;  /* kernels enqueued by one ds_step */
    int32_t elems_per_lane;     /* consecutive elements a lane owns within a chunk */
    int32_t warps_per_chunk;    /* warps that share one (node, chunk) */
    int32_t block_threads;      /* threads per block of the main kernel */
    int32_t grid_blocks;        /* blocks of the main kernel */
    int64_t chunks_per_row;     /* M = ceil(N / chunk) */
    int64_t code_words_per_row; /* ceil(N * code_bits / 32) */
    int32_t node_batches;       /* batches of nodes a block sweeps per column (1 = all at once) */
} ds_info;

/* Bytes of device workspace ds_init needs for this shape (host-only call;
 * returns 0 for invalid arguments).  nnz = row_ptr[n]: the workspace also holds
 * the CSR of W - I and of W (what ds_init validates and copies), so its size
 * depends on the number of edges -- the one argument beyond (n, N, compressor). */
size_t ds_workspace_size(int32_t n, int64_t N, const ds_compressor *comp, int32_t nnz);

/* Validate the graph and W (Assumption 1: W symmetric, doubly stochastic;
 * Algorithm 1: every node its own neighbour), copy them to the workspace and
 * create a context.
 *   graph      host CSR (see ds_graph)
 *   W          host, one binary32 weight per CSR entry, in CSR order
 *   n, N, ld   nodes, parameters per node, row pitch (elements)
 *   comp       compressor
 *   workspace  device memory, 256-byte aligned, at least ds_workspace_size() bytes;
 *              must stay valid until ds_destroy
 * All validation happens before the first CUDA call, so argument errors are
 * reported on machines without a GPU.  On failure *out is NULL. */
ds_status ds_init(ds_ctx **out, const ds_graph *graph, const float *W,
                  int32_t n, int64_t N, int64_t ld, const ds_compressor *comp,
                  void *workspace, size_t workspace_bytes);

/* One iteration of Algorithm 1 for all nodes, enqueued on `cuda_stream`
 * (a cudaStream_t; NULL = default stream).
 *   x, delta   device [n][ld], updated in place
 *   gp         gradient data (a, c device [n][ld]) and noise
 *   hp         gamma, eta of this iteration (the paper decays the learning rate)
 *   seed,step  select the random streams; step < 2^56.  The same
 *              (seed, step) always reproduces the same iteration. */
ds_status ds_step(ds_ctx *ctx, float *x, float *delta, const ds_grad_params *gp,
                  const ds_hparams *hp, uint64_t seed, uint64_t step, void *cuda_stream);

/* The same iteration with the stochastic gradient SUPPLIED by the caller
 * (Algorithm 1, gradient step: g_i = grad F_i(x_i; xi_i) from the caller's own
 * training stack) instead of the synthetic objective:
 *     v_i = x_i - gamma g_i + delta_i, compress, delta_i <- v_i - C[v_i],
 *     x_i <- x_i - gamma g_i + eta sum_j (W_ij - I_ij) C[v_j].
 *   g          device [n][ld], read only, 16-byte aligned, same pitch as x
 *   seed,step  select the rounding stream of the b-bit compressor only
 * Traffic: 20 + b/8 + 4/chunk bytes per node-element (one array less to read,
 * no noise to generate). */
ds_status ds_step_g(ds_ctx *ctx, float *x, float *delta, const float *g, const ds_hparams *hp,
                    uint64_t seed, uint64_t step, void *cuda_stream);

/* One iteration of CENTRALIZED error-compensated SGD (Section 1, the three
 * displayed updates; one of the baselines of Section 5), on the same state
 * layout and with the same compressors, chunking, packing and random streams:
 *     workers:  v_i = g_i + delta_i;  C[v_i];  delta_i <- v_i - C[v_i]
 *     server:   x_i <- x_i - gamma sum_{j in N(i)} W_ij C[v_j]
 * The paper writes it for one worker.  Here row i of x is worker i's copy of
 * the model, and the server's average is the weighted sum over row i of W: a
 * complete graph with W_ij = 1/n is the parameter server (all rows of x then
 * stay equal if they start equal).  Operation order per element:
 *     d = x - c; g = fma(a, d, sigma z); v = g + delta; compress; delta' = v - C;
 *     acc = 0; for j in N(i) ascending: acc = fma(W_ij, C_j, acc); x' = fma(-gamma, acc, x).
 * Where the persistent fused kernel takes the shape with 16 elements per lane
 * and at most 512 threads (chunks of 512 elements or one scale per node, up to
 * 16 nodes; chunks of 1024 up to 8 nodes; ...) the iteration is ONE launch of
 * that kernel's error-compensated-SGD instantiation: 24 + b/8 + 4/chunk bytes
 * per node-element.  Otherwise, and with ds_set_path(DS_PATH_SPLIT), two
 * kernels: the workers' compression, then the server's update, which streams
 * each worker's packed codes once and re-reads x (32 + (deg+2) b/8 bytes).
 * Arguments and errors as ds_step / ds_step_g; ds_codes returns what the
 * workers sent. */
ds_status ds_ecsgd_step(ds_ctx *ctx, float *x, float *delta, const ds_grad_params *gp,
                        float gamma, uint64_t seed, uint64_t step, void *cuda_stream);
ds_status ds_ecsgd_step_g(ds_ctx *ctx, float *x, float *delta, const float *g,
                          float gamma, uint64_t seed, uint64_t step, void *cuda_stream);

/* T consecutive iterations t = step0 .. step0+T-1 of Algorithm 1 with a
 * per-iteration schedule (Section 5 decays the learning rate): iteration t uses
 * gamma = gammas[t-step0] and eta = etas[t-step0].  The launches of all T
 * iterations are recorded once into a CUDA graph (captured on an internal
 * stream, nothing runs during capture) and replayed on `cuda_stream` as one
 * submission, which removes the per-launch host cost that bounds small
 * problems.  The executable graph is kept in the context: a later call with
 * the same T updates its kernel arguments in place instead of instantiating
 * again.  Results are bit-identical to T calls of ds_step.
 *   gammas, etas  host arrays of T binary32 values, read before the call returns
 *   T             1 .. DS_RUN_MAX_STEPS
 * Errors: as ds_step; DS_ERR_ARG if T is out of range or step0 + T > 2^56. */
#define DS_RUN_MAX_STEPS 4096
ds_status ds_run(ds_ctx *ctx, float *x, float *delta, const ds_grad_params *gp,
                 const float *gammas, const float *etas, int32_t T,
                 uint64_t seed, uint64_t step0, void *cuda_stream);

/* T consecutive iterations as ONE kernel launch, for problems small enough to
 * stay on chip between iterations (Algorithm 1 run as a loop; Section 5's
 * learning-rate decay as the schedule).  Column tiles of 512 elements are
 * independent except for the sum or maximum behind a per-node scale, so each
 * thread block keeps one tile of all n nodes -- x and delta in registers, a and
 * c in shared memory -- for all T iterations; global memory is read once at the
 * start and written once at the end, plus the codes and scales every iteration
 * "sends" (ds_codes returns those of the last one).  With one scale per node
 * (chunk = 0) the blocks meet at one grid-wide barrier per iteration (the
 * launch is cooperative, the barrier's wait bounded: DS_ERR_TIMEOUT from
 * ds_sync if it ever runs out, x and delta then unchanged).  Results are
 * bit-identical to T calls of ds_step.
 *   Shapes: n <= 16; chunk = 512 or chunk = 0; DS_COMP_SIGN1_L1 or
 *   DS_COMP_UNIFORM_STOCH_MAXABS with 2 or 4 bits; with chunk = 0 all
 *   ceil(N/512) blocks must be resident at once (N up to a few hundred
 *   thousand).  Anything else: DS_ERR_UNSUPPORTED, nothing runs -- use ds_run.
 *   gammas, etas  host arrays of T values, copied before the call returns
 *   T             1 .. DS_RESIDENT_MAX_STEPS
 * Other arguments and errors as ds_run. */
#define DS_RESIDENT_MAX_STEPS 1024
ds_status ds_run_resident(ds_ctx *ctx, float *x, float *delta, const ds_grad_params *gp,
                          const float *gammas, const float *etas, int32_t T,
                          uint64_t seed, uint64_t step0, void *cuda_stream);

/* Same iteration for HOST buffers: x, delta, a, c (host, [n][ld]) go to the
 * caller's device staging arrays, the step runs, and x and delta come back,
 * all ordered after the work already in `cuda_stream`; that stream continues
 * once the results are back, and the caller synchronises it before reading
 * them.  Host buffers must be page-locked for the copies to overlap.  Unless
 * one scale covers a whole node (chunk = 0), the work is cut into slabs of
 * column tiles and pipelined on three internal streams (created at the first
 * call): while one slab is computed the next is on its way in and the previous
 * on its way out.  Padding columns are copied in, never out.  dev_* are device
 * [n][ld] arrays owned by the caller.  Only the synthetic objective.
 * Not pipelined (four whole-array copies in, one step, two copies out, all on
 * `cuda_stream`): arrays below 64 MiB, one scale per node, and the case that the
 * internal streams or events cannot be created.  If a call fails after work
 * has been enqueued on the internal streams, that work is joined into
 * `cuda_stream` before the error status is returned. */
ds_status ds_step_host(ds_ctx *ctx, float *x_host, float *delta_host,
                       const float *a_host, const float *c_host,
                       float sigma, int32_t noise, const ds_hparams *hp,
                       uint64_t seed, uint64_t step,
                       float *dev_x, float *dev_delta, float *dev_a, float *dev_c,
                       void *cuda_stream);

/* Device pointers to what the nodes "sent" in the last step (Algorithm 1, send
 * step): packed codes [n][*code_pitch_words] (element k of a node occupies
 * bits (k*b)%32 .. of word (k*b)/32, little-endian) and scales
 * [n][*scales_pitch], one per (node, chunk).  Valid until the next ds_step;
 * no copy is made. */
ds_status ds_codes(ds_ctx *ctx, const uint32_t **codes, int64_t *code_pitch_words,
                   const float **scales, int64_t *scales_pitch);

/* Choose the execution path (default DS_PATH_AUTO).  DS_ERR_UNSUPPORTED if
 * DS_PATH_FUSED is asked for a shape it cannot take. */
ds_status ds_set_path(ds_ctx *ctx, int32_t path);

/* Tuning knob: elements a lane keeps in registers per (node, chunk): 4, 8 or 16
 * (0 = the library's choice).  Fewer elements per lane mean more warps per
 * chunk.  Re-plans every path; a path the new shape cannot take falls back as
 * DS_PATH_AUTO describes.  DS_ERR_UNSUPPORTED (nothing changed) if not even the
 * two-kernel path can take it.  Results do not depend on it. */
ds_status ds_tune(ds_ctx *ctx, int32_t elems_per_lane);

/* Launch geometry of the current path (host-only). */
ds_status ds_get_info(const ds_ctx *ctx, ds_info *info);

/* Wait for the stream and report whether any kernel of this context gave up on
 * a bounded wait since the last call (DS_ERR_TIMEOUT; the flag is cleared).
 * The kernels never spin without a limit: a copy that does not arrive ends
 * the step early instead of hanging the device. */
ds_status ds_sync(ds_ctx *ctx, void *cuda_stream);

/* Arithmetic self-test on the device the library runs on.  The noise kernels
 * replace two general routines by shortcuts that are exact only on the
 * arguments that can occur (a branch-free logarithm of j 2^-24 and a
 * one-correction square root, starting from the hardware's reciprocal-square-
 * root estimate, of -2 ln u and of the squared Student-t(3) radius
 * 3 (u^(-2/3) - 1)).  This runs them against the general forms on ALL 2^24
 * possible arguments and ADDS the number of differing results to counts[0]
 * (logarithms), counts[1] (roots of -2 ln u) and counts[2] (roots of the
 * Student-t radii); counts is device memory, three 64-bit integers, zeroed by
 * the caller.  All must stay 0. */
ds_status ds_selftest_math(uint64_t *counts, void *cuda_stream);

/* Failure-reporting self-test: enqueues a one-warp kernel that waits, with a
 * small fixed budget, on a completion that never comes, gives up and raises the
 * context's error flag exactly as the fused kernel does when a staged copy does
 * not arrive.  The next ds_sync must return DS_ERR_TIMEOUT (and clear the flag).
 * Nothing hangs and nothing faults; x and delta are not touched. */
ds_status ds_selftest_timeout(ds_ctx *ctx, void *cuda_stream);

/* Checked build (the library compiled with -DDS_DEBUG, `python -m
 * paper_1907_07346_b200.build --debug`): before a warp touches its part of a row,
 * the kernels validate the indices behind every access of that part -- row,
 * first element, length, code words, scale slot, partial slot -- against the
 * shape; a part that fails is skipped and ds_sync returns DS_ERR_BOUNDS (once;
 * nothing traps, nothing out of range is read or written).  The checked build
 * computes the same results as the normal one.  This self-test asks the checker
 * about a part in the row after the last one: the next ds_sync must return
 * DS_ERR_BOUNDS.  In the normal build it returns DS_ERR_UNSUPPORTED. */
ds_status ds_selftest_bounds(ds_ctx *ctx, void *cuda_stream);

/* Diagnostics: write the random streams the kernels draw from, one value per
 * element, out[node][k] for k < N (device, [n][ld_out]).  which = 0: unit
 * gradient noise z of kind `noise`; which = 1: the rounding uniforms in
 * [0, 1).  Lets a caller check stream reproducibility without running a step. */
ds_status ds_noise(float *out, int32_t n, int64_t N, int64_t ld_out, int32_t which,
                   int32_t noise, uint64_t seed, uint64_t step, void *cuda_stream);

/* Per-node compressor scales with NO device allocation and no workspace.
 * (The paper has no counterpart: this entry point exists for the callers
 * described below, not for a step of Algorithm 1.)
 *
 * Some callers cannot obtain device memory when they call: code running inside
 * a process whose framework has already claimed the whole GPU for its own
 * memory pool, code on a path where an allocation would synchronise the device
 * and stall a latency-critical loop, or code that simply is not allowed to call
 * the allocator (plug-ins, callbacks).  For them this computes, for every node
 * i, the scale of the error-compensated variable v_i = x_i - gamma g_i + delta_i
 * over the WHOLE row -- what ds_step uses when the compressor has chunk = 0:
 *     comp_kind = DS_COMP_SIGN1_L1              s_i = (sum_k |v_ik|) / N
 *     comp_kind = DS_COMP_UNIFORM_STOCH_MAXABS  s_i = max_k |v_ik|  (0 if not finite)
 * and writes it to scales_out[i] (device, n floats).  x, delta, gp->a, gp->c are
 * device [n][ld] arrays as for ds_step and are only read.
 *
 * The reduction's scratch is a fixed array inside the library
 * (DS_NOALLOC_MAX_PARTIALS binary64 partials plus a 1 KiB table, 513 KiB, held on
 * every GPU on which this entry point has been called, until the process exits).
 * Consequences:
 *   - sizes with n * ceil(N / 512) > DS_NOALLOC_MAX_PARTIALS are rejected with
 *     DS_ERR_WORKSPACE;
 *   - all calls on one GPU share the array, so two calls whose kernels can
 *     overlap on the GPU (different streams, no dependency) race; serialise them;
 *   - the array keeps the previous call's contents, which is harmless: each call
 *     overwrites every partial it later reads;
 *   - the first call on each device looks up the array's device address (with
 *     that device current), and that lookup is also the moment the driver gives
 *     the array its storage on that GPU: make the first call at start-up, before
 *     the GPU has been filled (it returns DS_ERR_CUDA if the 513 KiB cannot be
 *     had) and before starting any stream capture.
 * The call allocates nothing: no cudaMalloc, cudaFree or allocating library
 * routine.  It only enqueues two kernels on cuda_stream. */
#define DS_NOALLOC_MAX_PARTIALS 65536
ds_status ds_node_scales_noalloc(float *scales_out, const float *x, const float *delta,
                                 const ds_grad_params *gp, float gamma, int32_t n, int64_t N,
                                 int64_t ld, int32_t comp_kind, uint64_t seed, uint64_t step,
                                 void *cuda_stream);

void ds_destroy(ds_ctx *ctx);

const char *ds_strerror(ds_status status);

#ifdef __cplusplus
}
#endif
#endif /* DEEPSQUEEZE_H */
