/*
 * liec.h - C ABI of the LIEC-SGD compression-step library for NVIDIA B200 (sm_100a).
 *
 * The library runs, on one GPU, the per-iteration bidirectional compression step of
 * LIEC-SGD (Algorithm 1, the branch with compression, i.e. every iteration that is not
 * a model-averaging iteration).  N workers minimise f(x) = 1/N sum_i E f_i(x, xi_i),
 * x in R^d (Eq. 1); they are simulated as the N rows of device tensors:
 *
 *   uplink    p^i = C(g^i)                          worker compress step of Algorithm 1
 *   server    v   = e + (1/N) sum_i p^i             server compensate step
 *   downlink  p   = C(v),  e <- v - p               server compress step, global error update
 *   update    x^i <- x^i - eta (p - p^i + g^i)      local immediate error compensation
 *
 * C is applied per segment (a contiguous block of the flattened model, e.g. one
 * parameter tensor) and is one of: scaled sign  C(x)_j = (||x||_1/n) sign(x_j)
 * (Def. 4; with several segments Def. 5, Blockwise-SignSGD), top-k (Def. 2), identity.
 *
 * Arithmetic contract (the paper does not fix one; results are reproducible bit for bit):
 *   - state and messages are IEEE binary32, every written operation rounded once to
 *     nearest-even, no fused multiply-add; gradients may be binary32 or bfloat16
 *     (bfloat16 is widened exactly before use);
 *   - sign(x) is negative iff x < 0 (zeros decode to +scale);
 *   - ||x||_1 of a segment is accumulated in binary64 over a balanced binary tree on
 *     the segment zero-padded to a power of two, divided by n in binary64 and rounded
 *     once to binary32;
 *   - top-k orders by |x| (binary32 magnitude), ties go to the lower index;
 *   - the server adds the N decoded messages in worker order starting from +0,
 *     divides by (float)N and then adds e;
 *   - the update is evaluated as x - eta*((p - p^i) + g).
 *
 * Message ("wire") layouts, all in the caller's workspace:
 *   sign   : words[W] + scales[T].  Segment t owns ceil(n_t/32) consecutive 32-bit
 *            words starting at sum_{u<t} ceil(n_u/32); bit b (LSB = 0) of its word w is
 *            1 iff element seg_offsets[t]+32w+b is negative; padding bits are 0.
 *   top-k  : idx[K] (uint32 flat index into [0,d)) + val[K] (binary32 copy of the kept
 *            entry), K = sum_t k_t; segment t owns [sum_{u<t} k_u, +k_t), ascending index.
 *   identity: no message buffer; the dense vector itself.
 *
 * Ownership: the caller owns every device buffer (params, error, gradients, workspace).
 * The library owns only the host-side context (for configurations with a scaled-sign downlink, and
 * for top-k / random-k configurations that have segments of at most 8192 elements or segments with
 * 16384 or more selection candidates, also one helper stream and four events, created by liec_init
 * and released by liec_destroy).  The hot calls allocate nothing, never synchronise the device and
 * only enqueue work that is ordered on the given stream: a top-k stage may run part of its kernels
 * on the helper stream, and liec_step runs the error update of a scaled-sign downlink there beside
 * the worker update; the helper stream is forked from and joined back to the given stream by events
 * inside the same call (this also works while the given stream is being captured into a CUDA graph).
 *
 * Errors: every call returns a liec_status; nothing throws, aborts or traps the GPU.
 * liec_last_error() gives a message for the last failing call on that context.
 */
#ifndef LIEC_H
#define LIEC_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct liec_ctx liec_ctx; /* opaque, lives in host memory */

typedef enum {
    LIEC_OK = 0,
    LIEC_ERR_INVALID_ARG = 1,  /* NULL / misaligned pointer, bad sizes, bad segment table, bad k */
    LIEC_ERR_UNSUPPORTED = 2,  /* d >= 2^32, more than 65535 workers or segments (launch grid) */
    LIEC_ERR_WORKSPACE = 3,    /* workspace smaller than liec_workspace_bytes() */
    LIEC_ERR_STATE = 4,        /* staged calls made out of order */
    LIEC_ERR_CUDA = 5,         /* a CUDA runtime call failed; see liec_last_error() */
    LIEC_ERR_DEVICE_CHECK = 6  /* a kernel recorded an internal inconsistency in the status word */
} liec_status;

typedef enum { LIEC_COMP_IDENTITY = 0, LIEC_COMP_SCALED_SIGN = 1, LIEC_COMP_TOPK = 2, LIEC_COMP_RANDK = 3 } liec_comp;
typedef enum { LIEC_F32 = 0, LIEC_BF16 = 1 } liec_dtype;

typedef struct {
    int32_t num_workers;        /* N >= 1 (Eq. 1) */
    int64_t dim;                /* d, 1 <= d < 2^32; N*d may exceed 2^32 */
    int32_t num_segments;       /* T >= 1.  T = 1: whole-vector operator (Def. 4); T > 1: blockwise (Def. 5) */
    const int64_t *seg_offsets; /* host, T+1 entries, [0] = 0, [T] = d, strictly increasing; copied */
    int32_t uplink;             /* liec_comp used by the workers  (C in the worker compress step) */
    int32_t downlink;           /* liec_comp used by the server   (C in the server compress step) */
    const int64_t *topk_k;      /* host, T entries, 1 <= k_t <= n_t; needed iff a side is TOPK or RANDK; copied */
    int32_t grad_dtype;         /* liec_dtype of the gradient rows; params, error, messages are binary32 */
} liec_config;

/* Device pointers into the workspace (NULL for parts the configuration does not use). */
typedef struct {
    const uint32_t *up_words;    /* [N][W]   sign uplink */
    const float *up_scales;      /* [N][T] */
    const uint32_t *up_idx;      /* [N][K]   top-k / random-k uplink */
    const float *up_val;         /* [N][K] */
    const uint32_t *down_words;  /* [W]      sign downlink */
    const float *down_scales;    /* [T] */
    const uint32_t *down_idx;    /* [K]      top-k / random-k downlink */
    const float *down_val;       /* [K] */
    const float *v;              /* [d] v_t; valid between liec_server_aggregate and
                                    liec_downlink_compress (it aliases the error buffer) */
    int64_t num_words;           /* W */
    int64_t num_topk;            /* K (0 when no side is top-k or random-k) */
} liec_messages;

/*
 * Bytes of device workspace needed for this configuration (message buffers, per-tile
 * partial sums, selection scratch).  Pure host arithmetic; returns 0 for an invalid
 * configuration.
 */
size_t liec_workspace_bytes(const liec_config *cfg);

/*
 * Bytes that one compressed iteration puts on the wire per worker: its uplink message, the
 * downlink message it receives, and, for comparison, one full-precision vector (4 d bytes; what
 * P-SGD sends each way and what a model-averaging iteration of Algorithm 1 is charged per
 * direction).  This is the accounting behind the paper's "communication cost per iteration"
 * column (Table of results on CIFAR): total = N * (uplink + downlink).  Pure host arithmetic;
 * any output pointer may be NULL.  Returns LIEC_ERR_INVALID_ARG / LIEC_ERR_UNSUPPORTED for a bad
 * configuration.
 */
liec_status liec_wire_bytes(const liec_config *cfg, int64_t *uplink_bytes, int64_t *downlink_bytes,
                            int64_t *full_precision_bytes);

/* Bytes of the downlink message as copied out by liec_step_host (0 for identity/invalid). */
size_t liec_down_message_bytes(const liec_config *cfg);

/*
 * Creates a context (Algorithm 1, initialisation line: x_0^i = x_0, e_0 = 0 are the
 * caller's job - the buffers are used as they are, which is also how a run is resumed).
 *   params    device, [N][d] binary32, row stride d, 16-byte aligned: the local models x^i.
 *   error     device, [d] binary32, 16-byte aligned: the server's global error e.
 *   workspace device, 256-byte aligned, at least liec_workspace_bytes(cfg) bytes.
 * Copies the segment tables to the workspace with synchronous copies on the current
 * device; the workspace must not be touched by the caller until liec_destroy.
 */
liec_status liec_init(const liec_config *cfg, float *params, float *error,
                      void *workspace, size_t workspace_bytes, liec_ctx **out);

/*
 * The four stages of one iteration.  They must be called in this order (LIEC_ERR_STATE
 * otherwise), all on streams that order them one after another.  `stream` is a
 * cudaStream_t passed as void* (NULL = legacy default stream).
 *   grads  device, [N][d] of cfg.grad_dtype, row stride d, 16-byte aligned; read-only; the
 *          same pointer and contents must be given to liec_worker_update of the same step.
 * Inputs are expected to be finite.  NaN or infinite gradients, parameters or errors do not
 * fault, but what they produce is unspecified: a NaN in a segment makes its scale NaN, top-k
 * orders bit patterns (so NaNs rank above every finite magnitude), and the error entry of a kept
 * top-k / random-k element is stored as +0 rather than computed as v - v.
 */
liec_status liec_uplink_compress(liec_ctx *ctx, const void *grads, void *stream);   /* p^i = C(g^i) */
liec_status liec_server_aggregate(liec_ctx *ctx, void *stream);                      /* v = e + mean_i p^i (into error) */
liec_status liec_downlink_compress(liec_ctx *ctx, void *stream);                     /* p = C(v); error <- v - p */
liec_status liec_worker_update(liec_ctx *ctx, const void *grads, float lr, void *stream); /* x^i -= lr (p - p^i + g^i) */

/*
 * Random-k (Def. 3: keep the entries of a k_t-subset of every segment, the subset drawn uniformly
 * from all k_t-subsets) with subsets brought by the caller: the caller samples them and hands them
 * over before the iteration that uses them (liec_draw_subsets is the alternative that draws them
 * on the GPU from a seed).
 *   up_sets   device, [N][K] uint32, K = sum_t k_t: for worker i and segment t the k_t kept flat
 *             indices (positions in [0, d)), listed segment after segment, strictly ascending
 *             inside a segment.  Needed iff the uplink is RANDK, else may be NULL.
 *   down_set  device, [K] uint32, the server's subset in the same layout.  Needed iff the
 *             downlink is RANDK.
 * The pointers are kept, not copied: the arrays are the caller's and must stay unchanged until
 * the iteration's liec_worker_update has run on the stream.  They may be replaced before every
 * iteration or kept for several.  The message of a RANDK side has the top-k layout (index,
 * value).  An index outside its segment or out of order is not read: the entry is dropped, bit 16
 * of the device status word is set and the iteration's results are unspecified (but no access
 * leaves the buffers).  LIEC_ERR_STATE when called between the stages of an iteration;
 * liec_uplink_compress / liec_downlink_compress return LIEC_ERR_STATE when a RANDK side has no
 * subset.
 */
liec_status liec_set_subsets(liec_ctx *ctx, const uint32_t *up_sets, const uint32_t *down_set);

/*
 * Random-k with a seed instead of index lists (Def. 3: S uniform over the k_t-subsets of a segment;
 * Assumption 4).  Draws the subsets of all N workers and of the server on the GPU and installs them
 * as liec_set_subsets would, without any list crossing the PCIe bus.  Two parties that share
 * (seed, epoch) compute the same subsets, so a message needs to carry the values only
 * (liec_wire_bytes_seeded).  Specification (bit-exact with a plain CPU restatement):
 *   - every element gets a score from the counter-based generator Philox4x32-10 (Salmon, Moraes,
 *     Dror, Shaw, SC 2011): key = (seed mod 2^32, seed div 2^32); counter = (q, t, row, epoch) with
 *     q the block of four consecutive elements of segment t (element j of the segment lies in block
 *     j div 4 and takes output word j mod 4), row = i for worker i and N for the server;
 *     score = word >> 2 (30 bits);
 *   - the subset of (row, t) is the k_t elements of the segment with the highest scores, equal scores
 *     going to the lower index; listed ascending.
 * Ranking by independent uniform scores gives every k_t-subset the same probability; equal scores at
 * the cut (probability about n_t / 2^30 per draw) are the only departure from it.
 * The draw is a top-k selection on a computed vector and runs through the top-k kernels; its cost is
 * about one dense pass of integer arithmetic over N+1 rows.  The lists live in the workspace and stay
 * in use until the next liec_draw_subsets or liec_set_subsets; call it before every iteration with a
 * new epoch (e.g. the iteration number) to redraw, or less often to keep the subsets.
 * LIEC_ERR_STATE between the stages of an iteration; LIEC_ERR_INVALID_ARG when no side is RANDK.
 */
liec_status liec_draw_subsets(liec_ctx *ctx, uint64_t seed, uint32_t epoch, void *stream);

/*
 * As liec_wire_bytes, for parties that share the seed of liec_draw_subsets: a RANDK message then
 * carries its k_t values per segment and no indices (4 K bytes instead of 8 K).  Other operators
 * are charged as in liec_wire_bytes.
 */
liec_status liec_wire_bytes_seeded(const liec_config *cfg, int64_t *uplink_bytes, int64_t *downlink_bytes,
                                   int64_t *full_precision_bytes);

/*
 * The four stages in sequence (one iteration of Algorithm 1's compressed branch); produces the same
 * bytes as calling them one by one.  If a stage fails after an earlier one was enqueued, the context
 * returns to idle (the next iteration may start) and params / error are unspecified, as after
 * liec_abort_step.
 */
liec_status liec_step(liec_ctx *ctx, const void *grads, float lr, void *stream);

/*
 * Gives up the iteration in progress (Algorithm 1 has no such step: this is error recovery for the
 * staged calls).  After a stage has failed, or when the caller decides not to finish an iteration,
 * this returns the context to idle so that liec_uplink_compress / liec_step are accepted again.
 * Enqueues nothing.  The stages already enqueued still run; params and error are then somewhere
 * between two iterations (error may hold v_t): restore them from a copy before going on.
 */
liec_status liec_abort_step(liec_ctx *ctx);

/*
 * The model-averaging iteration of Algorithm 1 (its branch for (t+1) mod floor(1/delta) == 0; the
 * caller decides when, e.g. every 32nd or 100th call): gradients and models travel uncompressed,
 *   v = e + (1/N) sum_i g^i,  p = v,  error <- v - p = 0,
 *   x^i <- (1/N) sum_i x^i - eta (p - g^i + g^i)   for every worker.
 * Worker sums run in worker order in binary32 from +0 and are divided by (float)N.  Must not be
 * called between the stages of a compressed iteration (LIEC_ERR_STATE).  One kernel on `stream`.
 */
liec_status liec_average_step(liec_ctx *ctx, const void *grads, float lr, void *stream);

/*
 * The algorithm's output xbar = (1/N) sum_i x^i (last line of Algorithm 1) into `out`
 * (device, [d] binary32, caller-owned).  One kernel on `stream`.
 */
liec_status liec_mean_params(liec_ctx *ctx, float *out, void *stream);

/*
 * Squared Euclidean norms per segment, for monitoring: out[r][t] = sum of x_j^2 over segment t of
 * row r, accumulated in binary64 over the same balanced tree as the L1 norms (deterministic).
 *   which = LIEC_SUMSQ_ERROR : the global error e (1 row)  -> ||e_t||, the quantity of the paper's
 *                              figure of error norms;
 *           LIEC_SUMSQ_GRADS : `grads` ([N][d] of cfg.grad_dtype, N rows);
 *           LIEC_SUMSQ_PARAMS: the local models (N rows).
 * With these the measured contraction of Def. 1, delta = 1 - ||x - C(x)||^2 / ||x||^2 (the paper's
 * table of measured delta), follows without touching the hot path: scaled sign
 * delta = n s^2 / ||x||^2 per segment (worker side: x = g^i; server side: ||v||^2 = ||e'||^2 + n s^2);
 * top-k delta = ||kept values||^2 / ||x||^2.  One extra read of the chosen array when called.
 *   out  device, [rows][T] binary64, caller-owned.  Two kernels on `stream`.
 */
#define LIEC_SUMSQ_ERROR 0
#define LIEC_SUMSQ_GRADS 1
#define LIEC_SUMSQ_PARAMS 2
liec_status liec_sumsq(liec_ctx *ctx, int32_t which, const void *grads, double *out, void *stream);

/*
 * Telemetry fused into the iteration's own passes: the quantities behind the paper's figure of
 * error norms (||e_t||) and its table of measured delta (Def. 1: delta = 1 - ||x - C(x)||^2 / ||x||^2,
 * worker side x = g^i, server side x = v) at no extra pass over the model-sized arrays.
 *
 * liec_set_telemetry(ctx, 1) makes the following iterations use kernel variants that also leave
 * per-tile partial sums of squares, taken where the values are in registers anyway: e_t^2 and v_t^2
 * in the server pass (which reads e_t and writes v_t), (g^i_t)^2 in the worker update.  With 0 (the
 * state after liec_init) the kernels without any of it run.  Parameters, error and messages are bit
 * for bit the same either way.  LIEC_ERR_STATE between the stages of an iteration.
 *
 * liec_get_telemetry reduces the partial sums of the last completed iteration to per-segment sums,
 * in binary64 over the same balanced tree as liec_sumsq (deterministic, bit-exact with a plain
 * recursive evaluation).  Every output pointer is device memory owned by the caller and may be NULL:
 *   e_sumsq          [T]     ||e_t||^2 per segment: the global error as it ENTERED the iteration
 *                            (Algorithm 1's e_t; the error it left behind, e_{t+1}, is what the next
 *                            iteration reports, or liec_sumsq(LIEC_SUMSQ_ERROR) at any time)
 *   v_sumsq          [T]     ||v_t||^2 per segment
 *   g_sumsq          [N][T]  ||g^i_t||^2 per worker and segment
 *   up_kept_sumsq    [N][T]  top-k / random-k uplink only: sum of squares of the k_t values of the
 *                            worker's message for the segment, over the tree on those k_t values in
 *                            message order (one read of the message values, K floats per row, when called)
 *   down_kept_sumsq  [T]     the same for a top-k / random-k downlink message
 * From these: ||e_t|| = sqrt(sum_t e_sumsq[t]);  scaled sign: ||x - C(x)||^2 = ||x||^2 - 2 s ||x||_1 + n s^2
 * with s the message's scale (delta = n s^2 / ||x||^2 up to the rounding of s);  top-k / random-k:
 * delta = kept / ||x||^2 (the kept entries are copied exactly).
 * A few small kernels on `stream`.  LIEC_ERR_STATE when no iteration has completed since the telemetry
 * was switched on, or between the stages of an iteration; LIEC_ERR_INVALID_ARG when a kept-value norm
 * is asked of a side that sends no (index, value) message.
 */
liec_status liec_set_telemetry(liec_ctx *ctx, int32_t on);
liec_status liec_get_telemetry(liec_ctx *ctx, double *e_sumsq, double *v_sumsq, double *g_sumsq,
                               double *up_kept_sumsq, double *down_kept_sumsq, void *stream);

/*
 * One iteration fed from host memory: copies grads_host ([N][d] of cfg.grad_dtype, pinned
 * memory recommended) into grads_dev (device staging buffer of the same size, caller
 * owned, 16-byte aligned), runs liec_step, copies the downlink message (sign: words then scales;
 * top-k: idx then val; liec_down_message_bytes() bytes) to down_msg_host, all on `stream`.
 * down_msg_host may be NULL to skip the read-back.  Does not synchronise.  LIEC_ERR_STATE, with
 * nothing enqueued, when called between the stages of an iteration.
 */
liec_status liec_step_host(liec_ctx *ctx, const void *grads_host, void *grads_dev, float lr,
                           void *down_msg_host, void *stream);

/* Device pointers of the current messages (valid until the next stage overwrites them). */
liec_status liec_get_messages(const liec_ctx *ctx, liec_messages *out);

/*
 * Synchronises `stream` and reads the device status word: 0 = clean; non-zero bits name an
 * internal check that failed (1 selection rank, 2 candidate buffer, 4 output count, 8 a bulk
 * copy into shared memory that did not complete within its bounded wait; the kernel that saw it
 * returned without touching its outputs; 16 a random-k subset entry outside its segment or out of
 * order).  Returns LIEC_ERR_DEVICE_CHECK when non-zero.
 */
liec_status liec_device_status(liec_ctx *ctx, void *stream, int32_t *out);

/*
 * Clears the device status word (one 4-byte memset on `stream`).  The word is sticky: once a check
 * has failed it stays non-zero until this call, so that a failure anywhere in a run is not lost.
 * The state (params, error) after a flagged iteration is unspecified; restore it before going on.
 */
liec_status liec_clear_status(liec_ctx *ctx, void *stream);

/*
 * Diagnostics for the bounded waits (no counterpart in the paper).  Kernels that stage a tile in
 * shared memory with a bulk copy poll the copy's barrier at most `poll_limit` times (0 = the default,
 * 2^20) before they set bit 8 of the status word and return without touching their outputs.
 * `expect_extra_bytes` (a multiple of 16, at most 1024; 0 in operation) is added to the byte count
 * that each copy's barrier is told to expect: the copy still lands, but its barrier never completes,
 * so every such wait runs out.  That is how a test drives the timeout path without any fault; a
 * flagged kernel waits a further millisecond before it returns, so that nothing is in flight into
 * its shared memory.  Takes effect from the next stage call.
 */
liec_status liec_set_copy_wait(liec_ctx *ctx, uint32_t poll_limit, uint32_t expect_extra_bytes);

/*
 * Diagnostics: which route the top-k selections (Def. 2) of the last iteration took on one side
 * (uplink != 0: the N*T worker problems; 0: the T server problems).  Synchronises `stream`, copies
 * the selection state to the host and counts:
 *   out[0] problems, out[1] uplink problems that finished on the single dense pass seeded by the
 *   previous threshold, out[2] problems that needed the dense second-digit pass (more entries
 *   share the threshold's leading key bits than the candidate buffer holds), out[3] problems that
 *   were finished in the dense source because even then their candidates did not fit (huge groups of
 *   equal magnitudes, e.g. a mostly-zero row whose k exceeds its non-zero count), out[4] problems of a
 *   single-tile segment (at most 8192 elements), which one CTA selects directly in shared memory.
 * per_problem (host, one byte per problem in [row][segment] order, or NULL) receives the same per
 * problem: bit 0 single pass, bit 1 second-digit pass, bit 2 finished in the dense source, bit 3 single tile.
 * The result of the selection never depends on the route.  LIEC_ERR_INVALID_ARG when the side does
 * not use top-k.
 */
liec_status liec_topk_route_counts(liec_ctx *ctx, void *stream, int32_t uplink, int64_t *out /* [5] */,
                                   uint8_t *per_problem);

/* Number of kernel launches enqueued by this context so far (host-side counter). */
int64_t liec_launch_count(const liec_ctx *ctx);

const char *liec_last_error(const liec_ctx *ctx); /* never NULL; ctx may be NULL */

/*
 * Scaled-sign compression of ONE vector with no workspace and no allocation.  (The paper has
 * no counterpart: this is a packaging variant of the uplink compressor, same arithmetic,
 * same words, same scale as liec_uplink_compress with one worker and one segment.)
 *
 * For callers that have no device memory of their own to hand over and must not ask the
 * driver for any: a gradient hook that runs in the middle of a backward pass, where a
 * cudaMalloc/cudaFree would stall every stream of the device, or a process whose framework
 * allocator already owns all of the GPU's memory.  The per-tile partial sums that the
 * regular path keeps in the caller's workspace live here in a fixed 64 KiB array inside the
 * library image (present on every GPU that loads the library, until the process exits), which
 * limits the vector to LIEC_NOALLOC_MAX_ELEMENTS elements; longer vectors are rejected with
 * LIEC_ERR_UNSUPPORTED and a message.
 *   x      device, n elements of `dtype` (liec_dtype), 16-byte aligned
 *   words  device, ceil(n/32) uint32: bit b of word w is 1 iff x[32w+b] < 0, padding bits 0
 *   scale  device, one float: ||x||_1 / n
 * Enqueues two kernels on `stream`; calls no allocation routine and does not synchronise.
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress);
 * make that first call outside of any stream capture.  All calls on a GPU share the one
 * array: calls that may overlap on the GPU (different streams, no ordering between them)
 * race on it and must be serialised by the caller.  Nothing in it needs clearing: a call
 * reads only the entries that it wrote itself.
 */
#define LIEC_NOALLOC_MAX_ELEMENTS (64ll * 1024 * 1024)
liec_status liec_sign_compress_noalloc(const void *x, int32_t dtype, int64_t n, uint32_t *words,
                                       float *scale, void *stream);
const char *liec_noalloc_last_error(void); /* message of the last failing no-alloc call on this thread */
void liec_destroy(liec_ctx *ctx);                  /* frees the host-side context (and its helper stream and events) */

#ifdef __cplusplus
}
#endif
#endif /* LIEC_H */
