/*
 * libgrawa -- the distributed averaging update of GRAWA, MGRAWA and LGRAWA
 * (Dimlioglu & Choromanska, "GRAWA: Gradient-based Weighted Averaging for Distributed
 * Training of Deep Learning Models") for M worker replicas resident on one NVIDIA B200.
 *
 * The update, for workers m = 1..M with flat fp32 parameters x_m and accumulated gradients
 * g_m of n elements cut into K layers, layer k = [layer_offsets[k], layer_offsets[k+1]):
 *
 *   1. S[k][m]  = sum_{j in layer k} g_m[j]^2                      (||G_k||_F^2, Eq. 3 / Eq. 5)
 *   2. score    LGRAWA  A^k_m = sqrt(S[k][m])                      (Eq. 5-6)
 *               MGRAWA  A_m   = sum_k sqrt(S[k][m])                (Eq. 3)
 *               GRAWA   A_m   = sqrt(sum_k S[k][m])                (Eq. 2, flattened gradient)
 *   3. weights  beta_m = (1/A_m) / sum_i (1/A_i), sum_m beta_m = 1 (Eq. 2, Eq. 4); LGRAWA does
 *               this separately in every layer (Eq. 7)
 *   4. centre   x_C[j] = sum_m beta_{m,layer(j)} x_m[j]            (display under Eq. 2; Eq. 7)
 *   5. pull     x_m[j] <- (1-pull) x_m[j] + pull x_C[j]            (same display; the distributed
 *               update of Algorithms 1 and 2), x_C taken from the values before the pull.
 *
 * Conventions common to every entry point
 *   - `params`, `grads`: HOST arrays of M DEVICE pointers, each to n contiguous fp32 values.
 *   - `layer_offsets`: HOST array of n_layers+1 int64, offsets[0] = 0, non-decreasing,
 *     offsets[n_layers] = n.  Empty layers are allowed.
 *   - `center_out`: DEVICE pointer to n fp32 values, fully overwritten; may be NULL.
 *   - The caller owns every buffer.  params[m] are updated in place, grads[m] are only read.
 *     No two of {params[*], center_out} may overlap and grads may not overlap params or
 *     center_out; overlap visible from the pointer ranges is rejected.
 *   - Work is enqueued on `stream` (a cudaStream_t; NULL is the default stream) and the call
 *     returns without synchronising.  The first call with a new (device, stream, n, M, layer
 *     table) builds and caches a plan (device allocations and a small upload); later calls
 *     allocate nothing.
 *   - Arithmetic: fp32 loads; squares accumulated in short fp32 runs, the runs of a work item
 *     combined in fp64 in a fixed order, the items' sums added exactly as fixed-point integers
 *     (so S does not depend on the order in which items finish: bitwise reproducible run to
 *     run); scores and weights in fp64, rounded once to fp32; centre as an fp32
 *     fused-multiply-add chain over m = 0..M-1; pull as fmaf(pull, x_C, (1-pull) * x_m).
 *   - Supported gradient magnitudes: the squares are taken in fp32, so the square of |g| below
 *     about 1e-19 is subnormal (it loses digits) and of |g| below about 3.7e-23 exactly zero (a
 *     layer of only such values scores 0 and takes the zero-score rule below), and |g| above
 *     about 1.8e19 squares to infinity (a non-finite score, rule below).  Between 1e-19 and
 *     1.8e19 the weights meet the 1e-5 relative contract.
 *   - Scores that are exactly zero take the limit of 1/A: inside a normalisation group the Z
 *     workers with zero score get 1/Z each, all others 0.  A non-finite score (NaN/Inf
 *     gradients) gives that worker weight 0, the rest are normalised among themselves (uniform
 *     1/M if none is finite), and the step's status word is set; see grawa_last_step_status.
 *   - Errors detectable on the host return a negative code before anything is enqueued.
 *     Nothing on the device traps.  The only device-side waits are the bulk-copy kernel's waits
 *     for its own copies; each is bounded and reports GRAWA_ERR_TIMEOUT instead of hanging.
 *   - A plan (and its device memory) lives until grawa_clear_plans(); a program that meets many
 *     different shapes or streams should call it now and then.  Steps that share a plan (same
 *     device, stream, shape) must not overlap on the GPU; the stream order guarantees that.
 *   - There is no CPU implementation behind this interface.
 */
#ifndef GRAWA_H
#define GRAWA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GRAWA_MAX_WORKERS 64

typedef struct CUstream_st *grawa_stream_t; /* identical to cudaStream_t */

typedef enum grawa_status {
    GRAWA_OK = 0,
    GRAWA_ERR_INVALID_ARG = -1, /* NULL pointer, bad M/n/offsets/pull, overlapping buffers        */
    GRAWA_ERR_CUDA = -2,        /* a CUDA runtime call failed; text in grawa_last_cuda_error()    */
    GRAWA_ERR_NONFINITE = -3,   /* a gradient score was NaN/Inf (fallback weights were applied)   */
    GRAWA_ERR_WORKSPACE = -4,   /* caller-supplied workspace missing, misaligned or too small     */
    GRAWA_ERR_TIMEOUT = -5,     /* a bounded device-side wait ran out (bulk-copy variant only)    */
    GRAWA_ERR_TOO_LARGE = -6    /* problem larger than the built-in scratch of grawa_sumsq_static */
} grawa_status;

typedef enum grawa_variant { GRAWA_VARIANT_GRAWA = 0, GRAWA_VARIANT_MGRAWA = 1, GRAWA_VARIANT_LGRAWA = 2 } grawa_variant;

/* Optional arguments; a NULL `options` pointer means all defaults.  Zero-initialise before use. */
typedef struct grawa_options {
    float  *weights_out;   /* DEVICE, fp32: beta, [M] for GRAWA/MGRAWA, [n_layers][M] for LGRAWA    */
    double *scores_out;    /* DEVICE, fp64: A, same shape as weights_out                            */
    double *sumsq_out;     /* DEVICE, fp64: S, [n_layers][M] (one row when there is no layer table) */
    void   *workspace;     /* DEVICE scratch, 256-byte aligned; NULL = the cached plan owns one     */
    size_t  workspace_bytes; /* size of `workspace`; at least grawa_workspace_bytes(...)            */
    int    *status_word;   /* DEVICE int, or NULL: receives the step's status bits (0 = clean, bit 0 = a
                              non-finite score met the fallback of step 3) when the weights are
                              finalised, so that a caller who replays a captured step can poll it
                              without the host-synchronising grawa_last_step_status                 */
} grawa_options;

/* Library version, major*10000 + minor*100 + patch. */
int grawa_version(void);

/* Static text for a status code. */
const char *grawa_status_string(grawa_status status);

/* Text of the last CUDA error seen by the calling thread ("" if none). */
const char *grawa_last_cuda_error(void);

/* Bytes of device scratch a step needs for this problem (the exact sums, S, A, beta, status): per
 * (layer, worker) tables only, the same for every storage type and vector length.  layer_offsets
 * may be NULL with n_layers = 0 (one layer).  Returns 0 on invalid arguments.  A caller's
 * workspace needs no particular contents: every step that uses it clears the part that has to
 * start from zero (one small memset in front of the kernels). */
size_t grawa_workspace_bytes(int64_t n, int M, const int64_t *layer_offsets, int n_layers);

/* MGRAWA step (Eq. 3-4, then centre and pull): one weight per worker from the sum of its
 * per-layer gradient norms.  With layer_offsets = NULL / n_layers = 0 the whole vector is one
 * layer and the score is the flat norm, i.e. vanilla GRAWA (Eq. 2).
 * pull must lie in [0, 1].  M in [1, GRAWA_MAX_WORKERS].  n = 0 is a no-op returning GRAWA_OK.
 * M = 1: the single worker is left untouched and copied to center_out. */
grawa_status grawa_mgrawa_step(float *const *params, const float *const *grads, int64_t n, int M,
                               float pull, const int64_t *layer_offsets, int n_layers,
                               float *center_out, const grawa_options *options, grawa_stream_t stream);

/* Vanilla GRAWA step (Eq. 2): one weight per worker from the norm of the flattened gradient.
 * A layer table, if given, only shapes sumsq_out; the weights do not depend on it. */
grawa_status grawa_grawa_step(float *const *params, const float *const *grads, int64_t n, int M,
                              float pull, const int64_t *layer_offsets, int n_layers,
                              float *center_out, const grawa_options *options, grawa_stream_t stream);

/* LGRAWA step (Eq. 5-7, construct, pull): in every layer k separate weights beta^k_m from the
 * layer's gradient norms; the centre is the concatenation of the per-layer weighted averages.
 * Empty layers form no group. */
grawa_status grawa_lgrawa_step(float *const *params, const float *const *grads, int64_t n, int M,
                               float pull, const int64_t *layer_offsets, int n_layers,
                               float *center_out, const grawa_options *options, grawa_stream_t stream);

/* Element type of params / grads / center_out in grawa_step_typed. */
typedef enum grawa_dtype { GRAWA_F32 = 0, GRAWA_BF16 = 1, GRAWA_F16 = 2 } grawa_dtype;

/* The same step (Eq. 2-7, centre, pull) with parameters, gradients and centre STORED in `dtype`:
 * fp32, bfloat16 or IEEE half.  16-bit storage halves the bytes the step moves.  The arithmetic is
 * unchanged: every element is widened exactly to fp32 on load, sums of squares, scores and weights
 * are computed as for fp32, the centre is the fp32 FMA chain, the pull uses the unrounded fp32
 * centre, and each result is rounded to nearest-even once, on its store (pull = 1 still makes
 * every worker bit-equal to center_out, pull = 0 leaves them untouched).
 * params, grads: HOST arrays of M DEVICE pointers to n elements of `dtype`, aligned to the element
 * size (16-byte aligned bases take the vector kernels; fp32 bases aligned to 32 bytes, as every
 * allocator's are, the 32-byte accesses of the centre+pull and proximity kernels); center_out: DEVICE,
 * n elements, or NULL.
 * GRAWA_F32 is exactly the three step entry points above. */
grawa_status grawa_step_typed(grawa_dtype dtype, grawa_variant variant, void *const *params,
                              const void *const *grads, int64_t n, int M, float pull,
                              const int64_t *layer_offsets, int n_layers, void *center_out,
                              const grawa_options *options, grawa_stream_t stream);

/* Same update with HOST buffers: params[m], grads[m] and center_out are HOST pointers (pinned
 * memory gives asynchronous copies; pageable memory works and is slower).  The call uploads the
 * M gradient and parameter vectors to device staging buffers owned by the cached plan, runs the
 * step of `variant`, downloads the updated parameters and the centre, and synchronises `stream`
 * before returning, so the results are in the host buffers on return.  The staging buffers take
 * (2M+1)*n*4 bytes of device memory and are allocated on the first call for a problem shape. */
grawa_status grawa_step_host(grawa_variant variant, float *const *params, const float *const *grads,
                             int64_t n, int M, float pull, const int64_t *layer_offsets, int n_layers,
                             float *center_out, grawa_stream_t stream);

/* Synchronises `stream` and reports the status word of the last step enqueued on it by the
 * calling process: GRAWA_OK, GRAWA_ERR_NONFINITE or GRAWA_ERR_TIMEOUT (GRAWA_ERR_CUDA if the
 * synchronisation itself fails, GRAWA_ERR_INVALID_ARG if no step was enqueued on it). */
grawa_status grawa_last_step_status(grawa_stream_t stream);

/* Proximity-search step of the local phase (the "Prox." update of Algorithms 1 and 2):
 * x_m[j] <- (1 - mu_over_tau) x_m[j] + mu_over_tau * center[j] for all M workers in one pass,
 * with `center` (DEVICE, n fp32, read only) the centre stored by the last averaging step.
 * mu_over_tau must lie in [0, 1]. */
grawa_status grawa_prox_step(float *const *params, const float *center, int64_t n, int M,
                             float mu_over_tau, grawa_stream_t stream);

/* The "Local" variants of the paper's appendix (Local MGRAWA / Local LGRAWA) take the norms from
 * the local optimizer's own gradients instead of a dedicated batch.  Three calls cover them:
 *
 * grawa_layer_norms: norms_out[k] = ||grad[layer k]||_2 for ONE worker's gradient (the vector
 * g_cur of that algorithm).  grad: DEVICE, n fp32, read only.  norms_out: DEVICE, n_layers doubles
 * (1 when there is no layer table); empty layers give 0. */
grawa_status grawa_layer_norms(const float *grad, int64_t n, const int64_t *layer_offsets, int n_layers,
                               double *norms_out, grawa_stream_t stream);

/* grawa_norm_ema: the running estimate, exactly as the appendix algorithm prints it:
 *   g_mvg <- gamma g_mvg + (1 - gamma) g_cur ;  g_est <- gamma g_mvg / (1 - gamma^t)
 * on DEVICE vectors of n_layers doubles (g_mvg in place; g_est may alias g_cur).  t >= 1 is the
 * local iteration count since the last reset, gamma in [0, 1).  (The leading gamma of g_est is
 * the paper's; it cancels in the weights when all workers share t.) */
grawa_status grawa_norm_ema(double *g_mvg, const double *g_cur, int n_layers, double gamma, int64_t t,
                            double *g_est, grawa_stream_t stream);

/* grawa_step_from_layer_norms: the averaging step with the scores taken from given per-layer norms
 * instead of gradients ("form x_C using the running gradient norm estimate"): layer_norms is
 * DEVICE, [n_layers][M] doubles (row k holds the M workers' norm estimates of layer k).
 * LGRAWA: A^k_m = layer_norms[k][m]; MGRAWA: A_m = sum_k layer_norms[k][m]; GRAWA:
 * A_m = sqrt(sum_k layer_norms[k][m]^2).  Everything else as in the step entry points; no
 * gradient is read (the step moves (2M+1)*4n bytes instead of (3M+1)*4n). */
grawa_status grawa_step_from_layer_norms(grawa_variant variant, float *const *params, const double *layer_norms,
                                         int64_t n, int M, float pull, const int64_t *layer_offsets,
                                         int n_layers, float *center_out, const grawa_options *options,
                                         grawa_stream_t stream);

/* Element-range sharding over several GPUs (each GPU holds the same index range of all M
 * replicas; derived from Eq. 3-7: sums of squares add over disjoint index ranges).  Two calls, with
 * one all-gather of a [n_layers][M] table of doubles between them (the caller's, e.g. NCCL):
 *
 * grawa_layer_sumsq: sumsq_out[k][m] = sum over the LOCAL elements of layer k of grads[m][j]^2.
 * grads: HOST array of M DEVICE pointers (n local elements each); layer_offsets: the local layer
 * table (layers without local elements are empty layers); sumsq_out: DEVICE, [n_layers][M]. */
grawa_status grawa_layer_sumsq(const float *const *grads, int64_t n, int M, const int64_t *layer_offsets,
                               int n_layers, double *sumsq_out, grawa_stream_t stream);

/* grawa_step_from_layer_sums: the averaging step on the local elements with S[k][m] = the sum, in
 * part order (so every GPU gets the same bits), of layer_sums[r][k][m], r = 0..parts-1.
 * layer_sums: DEVICE, [parts][n_layers][M] doubles, e.g. the all-gathered tables of all ranks.
 * Scores, weights, centre and pull follow as in the step entry points; no gradient is read. */
grawa_status grawa_step_from_layer_sums(grawa_variant variant, float *const *params, const double *layer_sums,
                                        int parts, int64_t n, int M, float pull, const int64_t *layer_offsets,
                                        int n_layers, float *center_out, const grawa_options *options,
                                        grawa_stream_t stream);

/* The other entry points on 16-bit storage.  Each `_typed` call is the call of the same name above with
 * parameters, gradients and centre stored in `dtype` (GRAWA_F32 gives exactly that call); pointers to
 * them are untyped, aligned to the element size, and every stored result is rounded to nearest-even
 * once, as in grawa_step_typed.  Tables of norms, sums of squares, scores and weights keep their
 * types (fp64 / fp32).  Together they let a caller who keeps bfloat16 or half replicas run
 * Algorithm 1 / 2 end to end: the proximity step of every local iteration, the Local variants of
 * the appendix and the element-range sharded step.
 *
 * grawa_prox_step_typed: the "Prox." update of Algorithms 1 and 2; mu_over_tau = 0 leaves the workers'
 * bits untouched, mu_over_tau = 1 makes them bit-equal to `center`. */
grawa_status grawa_prox_step_typed(grawa_dtype dtype, void *const *params, const void *center, int64_t n, int M,
                                   float mu_over_tau, grawa_stream_t stream);

/* grawa_layer_norms_typed / grawa_layer_sumsq_typed: per-layer norms of one gradient, per-layer sums of
 * squares of M gradients, from 16-bit gradients (widened exactly to fp32 before squaring). */
grawa_status grawa_layer_norms_typed(grawa_dtype dtype, const void *grad, int64_t n, const int64_t *layer_offsets,
                                     int n_layers, double *norms_out, grawa_stream_t stream);
grawa_status grawa_layer_sumsq_typed(grawa_dtype dtype, const void *const *grads, int64_t n, int M,
                                     const int64_t *layer_offsets, int n_layers, double *sumsq_out,
                                     grawa_stream_t stream);

/* grawa_step_from_layer_norms_typed / grawa_step_from_layer_sums_typed: the averaging step from given
 * scores (appendix algorithm of the Local variants; sums of squares added over element-range shards,
 * Eq. 3 / Eq. 5) on parameters and centre of `dtype`. */
grawa_status grawa_step_from_layer_norms_typed(grawa_dtype dtype, grawa_variant variant, void *const *params,
                                               const double *layer_norms, int64_t n, int M, float pull,
                                               const int64_t *layer_offsets, int n_layers, void *center_out,
                                               const grawa_options *options, grawa_stream_t stream);
grawa_status grawa_step_from_layer_sums_typed(grawa_dtype dtype, grawa_variant variant, void *const *params,
                                              const double *layer_sums, int parts, int64_t n, int M, float pull,
                                              const int64_t *layer_offsets, int n_layers, void *center_out,
                                              const grawa_options *options, grawa_stream_t stream);

/* grawa_step_host_typed: grawa_step_host with HOST buffers of `dtype` (Eq. 2-7, centre, pull); the
 * device staging buffers take (2M+1)*n elements of `dtype`. */
grawa_status grawa_step_host_typed(grawa_dtype dtype, grawa_variant variant, void *const *params,
                                   const void *const *grads, int64_t n, int M, float pull,
                                   const int64_t *layer_offsets, int n_layers, void *center_out,
                                   grawa_stream_t stream);

/* Largest number of partial sums grawa_sumsq_static can hold: M * ceil(n / 16384) must not
 * exceed it (for example M = 16 workers of up to 134 million elements each). */
#define GRAWA_STATIC_MAX_PARTIALS 131072

/* Squared gradient norms without any allocation (the paper has no counterpart of this entry
 * point; it exists for the sake of callers, not of the method): sumsq_out[m] = sum_j grads[m][j]^2
 * for m = 0..M-1, the quantity under the square root of Eq. 2.
 *
 * Who needs it: a host program whose device memory is already fully claimed by another
 * allocator (a training framework's caching pool, a fixed partition handed out at start-up),
 * where a raw cudaMalloc inside a library fails or fragments that pool; and a latency-bound
 * loop that cannot afford the device-wide synchronisation cudaMalloc and cudaFree imply.  The
 * step entry points above build a plan on their first call for a shape (device allocations);
 * this one never calls cudaMalloc, cudaFree or any allocating routine, on any call.
 *
 * Its scratch for the per-tile partial sums is a fixed array of GRAWA_STATIC_MAX_PARTIALS
 * doubles (1 MiB) compiled into the library; every GPU that loads the library holds that
 * megabyte until the process exits.  grads: HOST array of M DEVICE pointers to n fp32 values
 * (read only).  sumsq_out: DEVICE, M doubles, overwritten.  Same arithmetic as step 1 of the
 * step entry points with tiles of 16384 elements: fp32 runs combined in fp64 in a fixed order,
 * bitwise reproducible.
 *
 * Errors: GRAWA_ERR_INVALID_ARG for NULL pointers, M outside [1, GRAWA_MAX_WORKERS] or n < 0;
 * GRAWA_ERR_TOO_LARGE when M * ceil(n / 16384) > GRAWA_STATIC_MAX_PARTIALS (nothing is
 * enqueued); GRAWA_ERR_CUDA for a failed launch or address look-up.  n = 0 writes zeros.
 *
 * The first call on each device looks up the device address of the built-in array (the device
 * must be current); make that first call outside any stream capture.  All calls on a device
 * share the one array and it keeps the previous call's contents (every slot a call reads it
 * has first overwritten, so nothing needs clearing): two calls whose kernels can overlap on
 * the GPU, for instance on different streams without an ordering between them, race on it
 * and give wrong sums.  Calls on one stream are safe. */
grawa_status grawa_sumsq_static(const float *const *grads, int64_t n, int M, double *sumsq_out,
                                grawa_stream_t stream);

/* Self-test of the library's bounded device waits: launches one small kernel that waits on a
 * barrier nobody signals.  The wait must give up after limit_ns (1 us .. 1 s) of wall time, the
 * kernel records the timeout and returns, and grawa_last_step_status(stream) then reports
 * GRAWA_ERR_TIMEOUT with the context still usable.  Touches no caller memory. */
grawa_status grawa_selftest_bounded_wait(int64_t limit_ns, grawa_stream_t stream);

/* Debug build only (the library compiled with -DGRAWA_DEBUG_BOUNDS, in which every global access of
 * the streaming kernels is first checked against the work item it belongs to and the vector, and
 * every index into scratch memory against its table; violations are counted and the access
 * skipped): returns the number of violations on the current device since the last call and resets
 * it; synchronises the device.  With selfcheck != 0 it first feeds the checker seven planted
 * violations and two clean probes (arithmetic only, no memory access), so a healthy debug build
 * returns exactly 7 more.  Returns -1 in the normal build, -2 on a CUDA error. */
int64_t grawa_debug_bounds_violations(int selfcheck);

/* Trace build only (the library compiled with -DGRAWA_TRACE): the sum-of-squares, finalisation and
 * register centre+pull kernels stamp the device's nanosecond timer, one row per launch of each kind
 * (64 rows, wrapping): {entry of the first CTA, first CTA past the dependency wait, last CTA past
 * it, exit of the last CTA}.  Copies up to max_rows rows of 3 kinds x 4 uint64 to rows_out (HOST,
 * may be NULL), then resets the rows and the launch counters; synchronises the device.  Call it
 * once before the steps to be traced (reset) and once after.  All traced launches of one kind must
 * have the same grid size.  Returns the number of rows kept (64), -1 in the normal build, -2 on a
 * CUDA error. */
int grawa_trace_read(uint64_t *rows_out, int max_rows);

/* Tuning knobs, process wide; they change speed, never results beyond fp32 summation order
 * of the sums of squares ("sumsq_tile").  Returns GRAWA_ERR_INVALID_ARG for an unknown name
 * or a value out of range.
 *   "sumsq_tile"   elements per sum-of-squares work item (multiple of 1024, 1024..1048576)
 *   "pull_tile"    elements per centre+pull work item (multiple of 1024, 1024..1048576);
 *                  0 (default) = what one CTA of the register kernel covers in a single pass,
 *                  8192 / 4096 / 2048 / 1024 elements for M <= 2 / 4 / 8 / 16; above 16 workers
 *                  what one CTA of the shared-memory kernel covers (4 elements per thread)
 *   "pull_variant" 0 and 1 = register kernel (vector loads) up to 16 workers and, above 16, a
 *                  kernel that stages each thread's 16-byte columns through shared memory by
 *                  asynchronous copies (both storage widths); 2 = bulk-copy kernel (fp32 only:
 *                  shared-memory staging by 1-D bulk asynchronous copies and bulk stores)
 *   "bulk_tile"    elements per slice of a bulk-copy stage (multiple of 256, up to 16384);
 *                  0 = chosen from M so that three stages fit in shared memory
 *   "kernel_timing" 1 = every device-buffer step also records CUDA events around its three
 *                  phases on the step's stream (see grawa_collect_kernel_times); do not use
 *                  while capturing a CUDA graph.  Default 0.
 *   "dependent_launch" 1 (default) = the kernels of a step are launched with programmatic
 *                  stream serialisation, so each one's launch overlaps the tail of the one
 *                  before it on the stream (it still waits for that kernel's results);
 *                  0 = plain stream order.
 *   "pull_preload"  1 (default) = a device-buffer step's centre+pull kernel loads its first
 *                  parameters ahead of its wait for the weights; 0 = after it.
 *   "pull_prefetch_waves", "sumsq_prefetch_waves" (0..8; defaults 3 and 1) on short steps the CTAs
 *                  that are resident when a kernel starts hint the data of the items that many
 *                  grid-fuls further on into L2 while they wait for the kernel in front; 0 = off.
 *   "pull_wide"     1 (default) = when every parameter vector and the centre are 32-byte aligned, the fp32
 *                  centre+pull kernel for up to 16 workers, the 16-bit one for up to 4 workers and the
 *                  fp32 proximity step move their columns by 32-byte loads and stores; 0 = 16-byte
 *                  accesses always.  Same results bit for bit.
 *   "pull16_staged" 1 (default) = on 16-bit storage with 5..16 workers the centre+pull kernel stages
 *                  its columns through shared memory (per-thread asynchronous 16-byte copies);
 *                  0 = the register kernel for every worker count.  Drops the cached plans.
 *   "sumsq_ctas_per_sm", "pull_ctas_per_sm" (0..32) CTAs per SM of the grid that streams
 *                  through the work items of the sum-of-squares / centre+pull kernel;
 *                  0 = one CTA per work item.
 * Changing a tile size or the variant drops the cached plans. */
grawa_status grawa_set_option(const char *name, int64_t value);

/* Current value of a tuning knob, or -1 for an unknown name. */
int64_t grawa_get_option(const char *name);

/* Number of kernels this library has launched in the calling process since it was loaded. */
int64_t grawa_launch_count(void);

/* Sums, in milliseconds, of the device time of the three phases (sum-of-squares kernel; scores +
 * weights kernel; centre+pull kernel) over the steps enqueued while
 * "kernel_timing" was 1 since the previous call, and the number of those steps.  Any output
 * pointer may be NULL.  Synchronises the device. */
grawa_status grawa_collect_kernel_times(double *sumsq_ms, double *finalize_ms, double *center_pull_ms,
                                        int64_t *steps);

/* Frees every cached plan (device allocations included) on every device.  Synchronises. */
void grawa_clear_plans(void);

#ifdef __cplusplus
}
#endif
#endif /* GRAWA_H */
