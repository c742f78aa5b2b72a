/*
 * cdadam.h - C interface of the B200 (sm_100a) CD-Adam library.
 *
 * One context simulates, on ONE GPU, the n workers and the server of the paper's
 * Algorithm 1 (communication-compressed distributed AMSGrad).  The caller owns the n
 * stochastic gradients of the problem statement (Section 3, Eq. 1); the context owns the
 * model x, the moments m, v, vhat and all compression state.  One call of cdadam_step is one
 * iteration t of Algorithm 1:
 *
 *   worker i :  c^(i) = C(g^(i) - ghat^(i));  ghat^(i) += c^(i)
 *   server   :  ghat += (1/n) sum_i c^(i);  c = C(ghat - gtil);  gtil += c
 *   worker   :  gtil += c (the same vector on every worker, kept once);
 *               m = b1 m + (1-b1) gtil;  v = b2 v + (1-b2) gtil^2;
 *               vhat = max(vhat, v);  x -= lr * m / sqrt(vhat + eps)
 *
 * C is the scaled-sign compressor (||u||_1 / |segment| * sign(u), one bit per coordinate plus
 * one float per segment), the top-k compressor (k (index, value) pairs) or the identity
 * (Appendix A).  eps is the paper's nu: it sits INSIDE the square root and there is no bias
 * correction.  All vectors are IEEE binary32; every operation above is rounded once, in the
 * order written, without fused multiply-add.  The l1 norm is accumulated in double-double
 * arithmetic in a fixed order, rounded to binary64, divided by the segment length in
 * binary64 and rounded to binary32, so the scale is the correctly rounded value and does
 * not depend on the launch shape.  The sum over workers runs over i = 0, 1, ..., n-1 in
 * binary32 and is divided once by (float)n.
 *
 * Conventions.  "device" pointers are CUDA global-memory addresses on the context's GPU
 * (the device current at cdadam_create); "host" pointers are ordinary CPU addresses.  All
 * functions returning int return CDADAM_OK (0) or a negative CDADAM_ERR_* code and never
 * abort; cdadam_last_error() gives the message of the calling thread's last failure.
 * Unless stated, work is queued on the given stream (a cudaStream_t passed as void*, NULL =
 * the legacy default stream) and the call returns without waiting.  A context must be used
 * from one host thread at a time and with one stream at a time.  Gradients must be finite;
 * the result for NaN or infinite input is unspecified (no call hangs or faults on them).
 */
#ifndef CDADAM_H
#define CDADAM_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct cdadam_ctx cdadam_ctx;

/* compressor C of Algorithm 1 (Appendix A) */
enum { CDADAM_SIGN = 0, CDADAM_TOPK = 1, CDADAM_IDENTITY = 2, CDADAM_RANDK = 3 };

/* recursion around the compressor */
enum {
    CDADAM_MARKOV = 0,   /* Algorithm 1: Markov compression sequences (Section 5), the default */
    CDADAM_EF = 1,       /* classical error feedback at workers and server (Section 4) */
    CDADAM_NAIVE = 2     /* naive compression (Section 4): no state, C applied both ways */
};

/* status codes */
enum {
    CDADAM_OK = 0,
    CDADAM_ERR_ARG = -1,     /* invalid argument; nothing was queued */
    CDADAM_ERR_ALLOC = -2,   /* device or host allocation failed */
    CDADAM_ERR_CUDA = -3,    /* a CUDA runtime call failed; see cdadam_last_error */
    CDADAM_ERR_STATE = -4,   /* call not allowed in the context's current state */
    CDADAM_ERR_TIMEOUT = -5  /* a kernel's bounded wait on an asynchronous copy ran out */
};

/* names of the state vectors for cdadam_get_state / cdadam_set_state */
enum {
    CDADAM_STATE_GHAT_W = 0, /* worker Markov states ghat^(i), n x d row-major */
    CDADAM_STATE_GHAT_S = 1, /* server aggregate ghat, d */
    CDADAM_STATE_GTIL = 2,   /* second Markov state gtil, d */
    CDADAM_STATE_M = 3,
    CDADAM_STATE_V = 4,
    CDADAM_STATE_VHAT = 5,
    CDADAM_STATE_X = 6
};

#define CDADAM_SERVER (-1)   /* "who" argument of cdadam_last_payload */

/*
 * Create a context (inputs of Algorithm 1: beta1, beta2, nu = eps, step size lr, C).
 *   d          model dimension, 1 <= d < 2^32
 *   n          number of simulated workers, 1 <= n <= 65535
 *   compressor CDADAM_SIGN, CDADAM_TOPK, CDADAM_RANDK or CDADAM_IDENTITY
 *   k          entries kept by top-k / rand-k at the workers and at the server,
 *              1 <= k <= d; ignored for the other compressors
 * All state is allocated here, on the current device, and zero-initialised (Algorithm 1
 * initialisation; x_1 = 0 until cdadam_set_params).  Scaled sign starts with one segment [0, d).
 * Synchronous.  Returns NULL on failure (see cdadam_last_error).  The caller destroys the
 * context with cdadam_destroy.
 */
cdadam_ctx *cdadam_create(int64_t d, int n, int compressor, int64_t k,
                          float beta1, float beta2, float lr, float eps);

/* Free a context and its device memory (waits for the device).  NULL is allowed. */
void cdadam_destroy(cdadam_ctx *ctx);

/*
 * One iteration of Algorithm 1 (its whole loop body) on the n gradients g_t^(i).
 *   grads   device, n x d floats, row i = worker i, row-major, contiguous; borrowed until
 *           the work queued on `stream` has completed; never written.  A base address
 *           that is a multiple of 16 bytes together with d % 4 == 0 selects the
 *           vectorised kernels; any other alignment is accepted and gives the same result.
 *   stream  cudaStream_t; must not be under stream capture (CDADAM_ERR_STATE, nothing
 *           queued): launch arguments alternate between steps, so a step replayed from a
 *           caller's graph would be wrong
 * Allocates no device memory for the method's data: all vectors and scratch were allocated
 * by cdadam_create.  Two kinds of call do create CUDA objects, once each: the second step on a
 * given gradient buffer of a configuration that is replayed from a graph (see below)
 * instantiates that graph (up to four per context; milliseconds, and the driver may allocate
 * for it), and cdadam_step_bf16 / cdadam_step_host allocate their staging buffer at their
 * first call.  Where the step is launch-bound (scaled sign, every pass a
 * single wave of blocks, about n*d <= 2.4e6) the scales are finished inside the passes
 * (3 launches instead of 5) and, from the second step on the same gradient buffer, the
 * launches are replayed from a CUDA graph owned by the context; so are the some thirty
 * launches of every top-k step of Algorithm 1.  After the stream has completed,
 * cdadam_params() holds x_{t+1}.
 */
int cdadam_step(cdadam_ctx *ctx, const float *grads, void *stream);

/*
 * The same iteration with the gradients given in bfloat16 (device, n x d 16-bit values, the
 * upper halves of binary32 numbers).  Widening is exact, so the result is that of
 * cdadam_step on the widened values.  The scaled-sign worker kernels read the 16-bit values
 * directly (2 instead of 4 bytes per gradient; vectorised when the base address is a multiple
 * of 16 bytes and d % 8 == 0); the other compressors first widen into a staging buffer owned
 * by the context (allocated at the first such call).
 */
int cdadam_step_bf16(cdadam_ctx *ctx, const void *grads_bf16, void *stream);

/*
 * The same iteration with the gradients in HOST memory: copies n x d floats host->device
 * into a staging buffer owned by the context (allocated at the first call), runs the step,
 * copies x_{t+1} (d floats) into x_out (host; may be NULL to skip) and waits for `stream`.
 * Pinned host memory makes the copies asynchronous to the host but the call still waits.
 */
int cdadam_step_host(cdadam_ctx *ctx, const float *grads_host, float *x_out_host,
                     void *stream);

/*
 * Distributed deployment of Algorithm 1 (Section 5: the workers send c^(i) to the server, the
 * server sends c to all workers, and every worker keeps gtil, m, v, vhat and x and updates the
 * model itself).  A process creates a context for the workers it holds and runs an iteration
 * in its three stages; between the stages the caller moves the messages (d sign bits and q
 * scales each, the paper's 32 + d bits for q = 1) with whatever transport it has - the
 * library makes no network call.  The result is that of one context holding all n workers,
 * bit for bit, because every stage computes the same binary32 operations in the same order.
 *
 * cdadam_create_shard: as cdadam_create, with CDADAM_SIGN or CDADAM_TOPK, for the workers
 *   [first_worker, first_worker + n_local) of n.  n_local may be 0 (a process that is only
 *   the server).  The worker state ghat^(i) is allocated for the n_local workers only;
 *   CDADAM_STATE_GHAT_W is n_local x d.  The message buffers hold all n worker messages.
 *   cdadam_step, cdadam_step_bf16 and cdadam_step_host are refused (CDADAM_ERR_STATE) when
 *   n_local < n.  Segments, mode, step size, weight decay as for any context, set alike on
 *   every process.
 *
 * cdadam_step_workers: worker stage for the context's own workers (Algorithm 1, the workers'
 *   compression and state update).  grads: device, n_local x d floats, row r is worker
 *   first_worker + r (may be NULL when n_local = 0).  Writes rows [first_worker,
 *   first_worker + n_local) of the worker message buffers.
 * cdadam_step_server: server stage (aggregation, compression, Algorithm 1) from all n worker
 *   messages in the buffers; writes the server message.  Only a process that acts as the
 *   server calls it; calling it on every process, after all n messages have been gathered
 *   everywhere, replaces the server's broadcast by redundant computation.
 * cdadam_step_update: gtil += c and the AMSGrad update from the server message in the
 *   buffers (Algorithm 1, the state update of the server and of every worker).  Completes
 *   the iteration.
 * Order per iteration: workers, [server], update; anything else is CDADAM_ERR_STATE.  All
 * three are asynchronous on `stream`, allocate nothing, and must not be under stream capture.
 * The caller orders its transfers with the stream (the messages are written by the work
 * queued by cdadam_step_workers / cdadam_step_server and read by the next stage).
 *
 * cdadam_exchange_buffers: device pointers, owned by the context, of the message buffers:
 *   worker_bits    n x words uint32, row i = the sign words of worker i (bit layout as in
 *                  cdadam_last_payload)
 *   worker_scales  n x q floats, row i = the scales of worker i.  This buffer ALTERNATES
 *                  between two arrays from one iteration to the next: ask again after every
 *                  cdadam_step_workers
 *   server_bits    words uint32;  server_scales  q floats
 *   words = ceil(d / 32).  Any output pointer may be NULL.  A context that holds all n
 *   workers may use the staged calls too.
 *   With CDADAM_TOPK (Algorithm 1 on the whole vector; not the comparison modes, not per
 *   segment) the same four pointers are the messages' coordinates and values: worker_bits =
 *   n x k uint32 coordinates (increasing in every row), worker_scales = n x k float values,
 *   server_bits / server_scales = the server's k coordinates and values; words = q = k.
 *   A process that skips cdadam_step_server adds the server message it was given to its gtil
 *   in cdadam_step_update.  Messages that arrive from other processes carry no per-tile
 *   offsets, so the server aggregation of such a context searches the sorted coordinates
 *   (slower than the one-context path, same sums in the same order).
 */
cdadam_ctx *cdadam_create_shard(int64_t d, int n, int first_worker, int n_local,
                                int compressor, int64_t k,
                                float beta1, float beta2, float lr, float eps);
int cdadam_step_workers(cdadam_ctx *ctx, const float *grads, void *stream);
int cdadam_step_server(cdadam_ctx *ctx, void *stream);
int cdadam_step_update(cdadam_ctx *ctx, void *stream);
int cdadam_exchange_buffers(cdadam_ctx *ctx, uint32_t **worker_bits, float **worker_scales,
                            uint32_t **server_bits, float **server_scales, int64_t *words,
                            int *q);

/*
 * Coordinate-sharded deployment of Algorithm 1: a context owns the coordinates [lo, hi) of
 * every vector - the n workers' gradients and states ghat^(i), the server's ghat and gtil,
 * and m, v, vhat, x - and several contexts (one per GPU) cover [0, d) between them.  Every
 * assignment of Algorithm 1 acts coordinate by coordinate, except the l1 norms inside the
 * scaled-sign compressor (Appendix A, "Scaled sign": ||x||_1 is a sum over all coordinates of
 * a segment).  So an iteration runs in three stages with two small exchanges in between:
 *
 *   cdadam_range_workers  worker pass on the range: u = g - ghat^(i), its sign words, and this
 *                         range's part of sum |u_j| for every (worker, segment), each part one
 *                         double-double (two binary64 numbers: value and rounding error)
 *   -- exchange 1: every context receives the parts of all ranges: n * q pairs per range --
 *   cdadam_range_server   adds the parts range by range (range 0 first), rounds to binary64,
 *                         divides by the WHOLE segment's length, rounds to binary32: the
 *                         workers' scales, the same on every context.  Then the server pass on
 *                         the range and this range's parts of sum |w_j|, q pairs
 *   -- exchange 2: q pairs per range --
 *   cdadam_range_update   the server's scales likewise; gtil += c and AMSGrad on the range
 *
 * The parts are added in a fixed order and carry about 104 significant bits, so the scales,
 * and with them every bit of the payloads and of the state, are those of one context that
 * holds the whole problem (an all-reduce that adds in an order of the library's choosing
 * would not guarantee that).  The library makes no network call: the caller moves the sums.
 *
 * cdadam_create_range: d, n and the hyper-parameters as in cdadam_create, for the coordinates
 *   lo <= j < hi (0 <= lo < hi <= d), as range number `range` of `ranges` (ranges ordered by
 *   lo; the number only fixes the slot in the exchange buffers and the order of the sums).
 *   CDADAM_SIGN (k is ignored; described here) or CDADAM_TOPK (described below).  All vectors
 *   of this context have hi - lo coordinates:
 *   gradients are n x (hi - lo), cdadam_get_state / cdadam_set_state / cdadam_params move
 *   (hi - lo)-vectors, cdadam_last_payload gives the hi - lo sign bits (bit 0 = coordinate lo)
 *   and one scale per segment that meets the range.  cdadam_set_segments takes the segments
 *   of the WHOLE problem (offsets from 0 to d), the same on every context; cdadam_set_mode
 *   takes CDADAM_MARKOV or CDADAM_EF.  cdadam_step and the cdadam_step_* calls are refused.
 * cdadam_range_workers: grads device, n x (hi - lo) floats, row i = worker i's coordinates
 *   lo..hi-1.  cdadam_range_server, cdadam_range_update: as described above.  Order per
 *   iteration: workers, server, update (anything else: CDADAM_ERR_STATE).  Asynchronous on
 *   `stream`; nothing is allocated; not under stream capture.
 * cdadam_range_buffers: the exchange buffers, device memory owned by the context.
 *   worker_sums: ranges x n x q x 2 doubles; slot [r][i][s] is range r's (value, error) pair for
 *   worker i and segment s of the whole problem (zero where the segment misses the range).
 *   cdadam_range_workers writes slot [range]; before cdadam_range_server the caller fills
 *   the other slots with the other contexts' slot (an in-place all-gather of
 *   *worker_doubles = 2 n q doubles per range).  server_sums: ranges x q x 2 doubles,
 *   written by cdadam_range_server, gathered before cdadam_range_update
 *   (*server_doubles = 2 q per range).  *q_local: segments that meet the range;
 *   *segment_of_local: device, q_local numbers: which segment of the whole problem each
 *   local one is.  The pointers change when cdadam_set_segments or cdadam_set_tile is called.
 *   Any output pointer may be NULL.
 */
/*
 * With CDADAM_TOPK (Appendix A, "Top-k": the k coordinates of largest magnitude of the WHOLE
 * vector) the one thing that crosses the ranges is the threshold: the k-th largest magnitude
 * and, among the coordinates equal to it, which are kept (the lower coordinates first, i.e.
 * the ranges in their order).  The selection is the exact three-level radix select of the
 * one-GPU path without its threshold guess, cut at every point where it needs a sum over the
 * whole vector: the histogram of each level is summed over the ranges (integer sums: order
 * does not matter) before the bucket is picked, and the ties are given out in range order.
 *
 * cdadam_create_range(..., CDADAM_TOPK, k, ...): k = entries kept in the whole vector,
 *   1 <= k <= d, at the workers and at the server (Algorithm 1 only).
 * cdadam_range_topk(ctx, stage, grads, stream): stages 0..9 of one iteration, in order:
 *   0..4 the workers' selection on g^(i) - ghat^(i) restricted to the range and
 *        ghat^(i) += c^(i) (grads: device, n x (hi - lo), needed by all five);
 *   5..9 the server: ghat += mean of the workers' messages (stage 5), the selection on
 *        ghat - gtil, gtil += c, and AMSGrad on the range (stage 9).  grads may be NULL.
 * cdadam_range_topk_buffer(ctx, stage, &buffer, &words): after every stage except 4 and 9
 *   the caller gathers the stage's exchange buffer: `ranges` slots of `words` uint32 each
 *   (n x 2048 after stages 0..3, 2048 after stages 5..8); the stage wrote slot `range`,
 *   the next stage reads all slots (an in-place all-gather, as for the l1 parts).  After
 *   stages 4 and 9 *buffer is NULL and *words 0.
 * cdadam_last_payload on such a context: *count = min(k, hi - lo) entries per message, of
 *   which the range's own kept coordinates come first (increasing, relative to lo) and the
 *   rest carry the coordinate 0xffffffff and the value 0; over all ranges the entries that
 *   are not so marked are the k of the whole vector.
 */
int cdadam_range_topk(cdadam_ctx *ctx, int stage, const float *grads, void *stream);
int cdadam_range_topk_buffer(cdadam_ctx *ctx, int stage, uint32_t **buffer, int64_t *words_per_range);

cdadam_ctx *cdadam_create_range(int64_t d, int n, int64_t lo, int64_t hi, int range, int ranges,
                                int compressor, int64_t k,
                                float beta1, float beta2, float lr, float eps);
int cdadam_range_workers(cdadam_ctx *ctx, const float *grads, void *stream);
int cdadam_range_server(cdadam_ctx *ctx, void *stream);
int cdadam_range_update(cdadam_ctx *ctx, void *stream);
int cdadam_range_buffers(cdadam_ctx *ctx, double **worker_sums, double **server_sums,
                         int64_t *worker_doubles, int64_t *server_doubles, int *q_local,
                         const int32_t **segment_of_local);

/* Device pointer to the model x (d floats), owned by the context, valid until destroy.
 * Its contents are x_{t+1} once the stream of the last step has completed.  NULL if ctx
 * is NULL. */
const float *cdadam_params(cdadam_ctx *ctx);

/* Set the initial point x_1 (Algorithm 1 input) from d device floats. */
int cdadam_set_params(cdadam_ctx *ctx, const float *x0, void *stream);

/*
 * Apply the scaled-sign compressor independently to q contiguous segments ("per tensor"):
 * segment r is [offsets[r], offsets[r+1]), offsets (host, q+1 values) strictly increasing
 * with offsets[0] = 0 and offsets[q] = d; each segment has its own scale
 * ||u_segment||_1 / |segment|, at the workers and at the server; sign bits stay in one
 * d-bit array.  Allowed only before the first step (CDADAM_ERR_STATE afterwards) and only
 * for CDADAM_SIGN.  Synchronous (re-allocates tables).
 */
int cdadam_set_segments(cdadam_ctx *ctx, int q, const int64_t *offsets);

/*
 * Apply the top-k compressor independently to q contiguous segments ("per tensor", as
 * cdadam_set_segments does for the scaled sign; Appendix A defines top-k on a whole vector,
 * here the vector is the segment): segment r = [offsets[r], offsets[r+1]) keeps its
 * k_per_segment[r] coordinates of largest magnitude (ties: lower coordinate), at the workers
 * and at the server.  offsets: host, q+1 values, strictly increasing from 0 to d;
 * k_per_segment: host, q values, 1 <= k_per_segment[r] <= length of segment r.  A message is
 * the concatenation of the segments' lists: sum_r k_per_segment[r] (coordinate, value) pairs,
 * coordinates in the whole vector, increasing; that sum replaces the k given to
 * cdadam_create.  The selection runs segment by segment, so this is meant for a moderate
 * number of large segments.  Only CDADAM_TOPK in the mode CDADAM_MARKOV, only before the
 * first step; synchronous (re-allocates the selection workspaces).
 */
int cdadam_set_topk_segments(cdadam_ctx *ctx, int q, const int64_t *offsets,
                             const int64_t *k_per_segment);

/*
 * Rand-k compressor (Appendix A: C(x) keeps x on k coordinates drawn uniformly at random).
 * The draws are inputs: before each step give the coordinate sets the n workers (device,
 * n x k uint32, row i = worker i) and the server (device, k uint32) use in that step.  Every
 * set must be strictly increasing with all coordinates below d.  The sets are copied; they
 * stay in force until replaced.  A malformed set is never dereferenced out of range; it is
 * reported by cdadam_device_status (CDADAM_ERR_ARG) and invalidates the state.
 */
int cdadam_set_random_sets(cdadam_ctx *ctx, const uint32_t *workers, const uint32_t *server,
                           void *stream);

/*
 * Choose the recursion: CDADAM_MARKOV (Algorithm 1, default) or CDADAM_EF, the error-feedback
 * scheme the paper compares against (Section 4), applied both ways:
 *   worker: p = g + delta^(i), c^(i) = C(p), delta^(i) = p - c^(i);
 *   server: p = (1/n) sum_i c^(i) + delta, c = C(p), delta = p - c; AMSGrad runs on c.
 * In this mode the state named GHAT_W holds the worker errors delta^(i), GTIL the server
 * error delta, and GHAT_S is scratch.
 * CDADAM_NAIVE is AMSGrad with naive compression (first paragraph of Section 4; the third
 * scheme compared in Section 6), compressed both ways like the other two:
 *   worker: c^(i) = C(g^(i));   server: c = C((1/n) sum_i c^(i));   AMSGrad runs on c.
 * GHAT_W and GTIL stay zero; GHAT_S is scratch.
 * Only before the first step.
 */
int cdadam_set_mode(cdadam_ctx *ctx, int mode);

/*
 * Tuning knob: the number of consecutive coordinates one thread block of the scaled-sign
 * kernels owns (a multiple of 4096, at most 262144; 0 = chosen from d and q, separately for
 * the worker pass and for the server side, the default).
 * Results do not depend on it.  Tiles of 16384 coordinates or more select the worker kernel
 * with the asynchronous-copy prefetch ring.  Only before the first step; synchronous.
 * With CDADAM_TOPK the selection always works on 4096-coordinate tiles and the value only
 * picks the kernel of its dense pass: 16384 or more = the prefetch-ring kernel wherever rows
 * are 16-byte aligned, a smaller non-zero value = the plain kernel, 0 = chosen from the size
 * (call it after cdadam_set_topk_segments, if that is used).
 */
int cdadam_set_tile(cdadam_ctx *ctx, int tile);

/* Step size alpha_t for the following steps (Algorithm 1 takes a non-increasing sequence;
 * monotonicity is not enforced).  Ends a schedule set by cdadam_set_lr_milestones. */
int cdadam_set_lr(cdadam_ctx *ctx, float lr);

/*
 * Step-size milestones (Section 6 multiplies the step size by 0.1 at two points of the run):
 * the step with 1-based number t uses alpha_t = base_lr * gamma^(number of after_steps[i]
 * <= t - 1), the product formed by repeated binary32 multiplication.  after_steps: host,
 * `count` (0..64) increasing non-negative numbers of completed steps; gamma in (0, 1].
 * count = 0 sets the constant step size base_lr.  Invalid arguments: CDADAM_ERR_ARG, nothing
 * changed.
 */
int cdadam_set_lr_milestones(cdadam_ctx *ctx, float base_lr, int count, const int64_t *after_steps,
                             float gamma);

/*
 * Decoupled weight decay lambda >= 0 for the following steps (Section 6 trains with a weight
 * decay; the paper does not print the formula, and the decoupled form is used):
 *   x_{t+1} = x_t - alpha_t m_t / sqrt(vhat_t + nu) - (alpha_t lambda) x_t,
 * with alpha_t lambda rounded once to binary32.  0 (the default) is Algorithm 1 as printed.
 */
int cdadam_set_weight_decay(cdadam_ctx *ctx, float lambda);

/*
 * Copy a state vector to / from device memory (dst / src: n*d floats for GHAT_W, else d).
 * get first applies any payload whose application the kernels had deferred, so the values
 * are those of Algorithm 1 after the last completed iteration.  set replaces the vector;
 * used to resume from a checkpoint or to start a step from a given state.
 */
int cdadam_get_state(cdadam_ctx *ctx, int name, float *dst, void *stream);
int cdadam_set_state(cdadam_ctx *ctx, int name, const float *src, void *stream);

/*
 * The message sent in the last iteration by worker `who` (0..n-1) or by the server
 * (CDADAM_SERVER): device pointers owned by the context, valid until the next step.
 *   scaled sign: *a = uint32 words, bit (j % 32) of word j / 32 is 1 iff u_j >= 0 (so a
 *                zero counts as positive), unused high bits of the last word are 0;
 *                *b = q float scales; *count = d.  The message is d + 32 q bits.
 *   top-k, rand-k: *a = k uint32 coordinates in increasing order, *b = their k float values
 *                u_j; *count = k.  Among equal |u_j| the lower j is kept.
 * CDADAM_ERR_STATE before the first step or for the identity compressor.
 */
int cdadam_last_payload(cdadam_ctx *ctx, int who, const void **a, const float **b,
                        int64_t *count);

/* Number of completed calls of cdadam_step on this context. */
int64_t cdadam_step_count(cdadam_ctx *ctx);

/*
 * Resuming from a checkpoint.  The iterate of Algorithm 1 is the seven state vectors plus the
 * iteration counter t (it selects the step size when milestones are set).  To save: read every
 * vector with cdadam_get_state (for scaled sign this first applies the last worker messages to
 * ghat^(i), so the saved vectors are final) and t with cdadam_step_count.  To resume: create a
 * context with the same arguments, segments, mode, step-size schedule and weight decay, load
 * the vectors with cdadam_set_state and t with cdadam_set_step_count; the iterations that
 * follow are those of the uninterrupted run, bit for bit (top-k starts its first selection
 * without a threshold guess, which costs time, not accuracy).  t >= 0; not between the stages
 * of an iteration (CDADAM_ERR_STATE).  Configuration calls that are allowed only before the
 * first step stay allowed while t is 0.
 */
int cdadam_set_step_count(cdadam_ctx *ctx, int64_t t);

/*
 * Waits for `stream` and reports whether any kernel of this context has given up a bounded
 * wait (the large-tile worker kernel waits, with an iteration limit, for its bulk
 * asynchronous copies; it never spins without bound).  CDADAM_ERR_TIMEOUT means the state
 * of the context is no longer valid; the device itself stays usable.
 */
int cdadam_device_status(cdadam_ctx *ctx, void *stream);

/*
 * Polls after which a kernel's wait on one of its bulk asynchronous copies gives up (the
 * prefetch-ring kernels of the scaled-sign worker pass and of the top-k dense pass poll an
 * mbarrier; the default is 2^22 polls, seconds of waiting, never reached by a copy that is
 * merely slow).  polls < 0 restores the default.  0 makes every such wait give up at once:
 * the kernels then report through cdadam_device_status and leave in order, the blocks having
 * first waited, with the default limit, for their copies in flight - which is how the error
 * path can be exercised without anything going wrong on the device.  Applies to the
 * following iterations.  After cdadam_device_status has returned CDADAM_ERR_TIMEOUT the
 * context accepts no further iterations (CDADAM_ERR_STATE): its state is not valid.
 */
int cdadam_set_wait_limit(cdadam_ctx *ctx, int polls);

/* Number of kernels one cdadam_step launches in the context's current configuration. */
int cdadam_launches_per_step(cdadam_ctx *ctx);

/*
 * Optional per-stage timing for benchmarks.  While enabled, cdadam_step records CUDA events
 * on its stream before the first and after every stage (a kernel or, for top-k, a group of
 * kernels).  cdadam_profile_read waits for the recorded events, adds the elapsed
 * milliseconds of every stage over all steps since the last read into ms[0..] (unused slots
 * 0), stores the number of steps in *steps and forgets the events.  cdadam_profile_name
 * gives a stage's name ("" if slot is out of range); the string is static.
 */
#define CDADAM_PROF_SLOTS 8
int cdadam_profile_enable(cdadam_ctx *ctx, int on);
int cdadam_profile_read(cdadam_ctx *ctx, double ms[CDADAM_PROF_SLOTS], int64_t *steps);
const char *cdadam_profile_name(cdadam_ctx *ctx, int slot);

/*
 * Stand-alone compressors of Appendix A on a device vector x of d floats.
 * Scaled sign: writes ceil(d/32) words to bits and q floats to scales (segments as in
 * cdadam_set_segments; offsets == NULL means one segment).  Top-k: writes k increasing
 * coordinates to idx and their values to val.  Both allocate their scratch memory on the
 * current device inside the call and free it before returning, and may wait for `stream`.
 */
int cdadam_compress_sign(const float *x, int64_t d, int q, const int64_t *offsets,
                         uint32_t *bits, float *scales, void *stream);
int cdadam_compress_topk(const float *x, int64_t d, int64_t k, uint32_t *idx, float *val,
                         void *stream);

/*
 * Scaled-sign compressor of one vector (one segment) that allocates nothing.  The paper has
 * no counterpart: this entry point exists for callers that cannot allocate device memory
 * when they call - code that must not risk the implicit device synchronisation of
 * cudaMalloc / cudaFree, processes whose device memory is wholly reserved by a framework's
 * pool, and latency-bound loops where an allocator call is an unbounded delay.
 *   x      device, d floats;  bits  device, ceil(d/32) words;  scale  device, one float
 *   d      1 <= d <= CDADAM_STATIC_MAX_D; larger sizes are rejected with CDADAM_ERR_ARG
 * Same results as cdadam_compress_sign(x, d, 1, NULL, bits, scale, stream).  The partial
 * sums of |x| go to a fixed 256 KiB array inside the library's device image (every GPU
 * that loads the library holds it until the process exits) instead of allocated scratch;
 * no cudaMalloc, cudaFree or other allocating call is made.  The first call on each device
 * looks up the array's device address (cudaGetSymbolAddress); make that first call before
 * any stream capture begins.  All calls on a device share the array and it keeps the last
 * call's contents: every entry a call reads is first overwritten by that call, so nothing
 * needs clearing, but two calls whose kernels overlap on the GPU (different streams, no
 * ordering between them) race on it.  Calls on one stream are safe.
 */
#define CDADAM_STATIC_MAX_D ((int64_t)1 << 28)
int cdadam_compress_sign_static(const float *x, int64_t d, uint32_t *bits, float *scale,
                                void *stream);

/* Message of the calling thread's most recent failure ("" if none).  Never NULL. */
const char *cdadam_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* CDADAM_H */
