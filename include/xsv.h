/*
 * xsv -- compressed-KV streaming attention step (XStreamVGGT hot path), C ABI.
 *
 * One cache object holds, per transformer layer, the pruned and quantised
 * key/value cache of the frame-wise causal global-attention module
 * (paper section 3.1, Eq. 1).  xsv_step() runs one streaming step of one
 * layer: attention of the new frame's queries over [cache ; new frame]
 * (Eq. 2, with the cache dequantised on the fly, Eq. 12), then -- once the
 * total length exceeds the budget L_max -- importance scoring (Eq. 3-7),
 * top-k pruning that always keeps the first and the current frame (Eq. 8),
 * and dimension-adaptive quantisation of the resulting cache (Eq. 9-11:
 * keys per channel over groups of 64 tokens, values per token over 64
 * channels; the quantiser subtracts the group minimum, as the quantiser of
 * KIVI that section 4.1 names does: code = round((x - min) / s),
 * x~ = code * s + min).  Every step of that path runs in CUDA kernels for sm_100a;
 * there is no CPU fallback.
 *
 * Conventions
 *  - Every call returns an xsv_status; nothing throws or aborts.  Argument,
 *    shape and order errors are detected on the host before any launch and
 *    leave the cache unchanged.
 *  - Pointers named "device" are CUDA device pointers, owned by the caller,
 *    and must stay valid until `stream` has passed the call's work.  Pointers
 *    named "host" are ordinary host pointers.
 *  - Q, K, V, out: [heads][n_tokens][head_dim], contiguous, 16-bit elements
 *    (fp16 or bf16 as given by `dtype`), 16-byte aligned.  `out` must not
 *    alias an input.
 *  - Input range: finite values of magnitude at most 65504.  The attention
 *    kernels hold their tensor-core operands as fp16; bf16 inputs convert
 *    without rounding for magnitudes in [2^-14, 65504], smaller ones are
 *    held with an absolute error of at most 2^-25, and a bf16 magnitude of
 *    2^16 or more saturates and sets XSV_ERR_RANGE in the status word (the
 *    default attention kernel reports it; see xsv_cache_status).  One case
 *    differs: a cache kept unquantised (bits = 16) is attended in the inputs'
 *    own type where the copy engine can fetch its tiles (pointers aligned as
 *    required above) -- fp16 as above; bf16 inputs then stay bf16, with no
 *    range limit and the probabilities rounded to bf16 (8-bit significand)
 *    before they multiply V.
 *  - xsv_step only enqueues work on `stream`; it does not synchronise and,
 *    after the call that allocates, creates nothing: all device memory, the
 *    cache's own streams and its events come from xsv_cache_set_options with
 *    max_frame_tokens > 0, else from the first step (or the first import).
 *    Exceptions, each made once and outside the frame loop if wanted so: the
 *    first xsv_step_host call allocates the staging slots and two copy
 *    streams; profiling (off by default) creates events as it needs them.
 *  - All steps of one cache share scratch buffers: issue them on one stream
 *    (or order them yourself).  Each layer is stepped once per frame, frames
 *    in order; layers may be stepped in any order.
 *  - Lengths never need a device read-back: the cache length after a step
 *    follows on the host from the length before it, the sizes of the first
 *    and of the current frame, and the budget (see xsv_cache_len).
 */
#ifndef XSV_H
#define XSV_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct xsv_cache xsv_cache; /* opaque, library-owned */

typedef enum {
    XSV_OK = 0,
    XSV_ERR_ARG = 1,     /* null pointer, value out of range                          */
    XSV_ERR_SHAPE = 2,   /* n_tokens beyond max_frame_tokens, dtype differs, bad alignment */
    XSV_ERR_ORDER = 3,   /* options changed after the first step, layer stepped twice  */
    XSV_ERR_OOM = 4,     /* device or host allocation failed                          */
    XSV_ERR_CUDA = 5,    /* a CUDA runtime call failed                                */
    XSV_ERR_TIMEOUT = 6, /* a bounded device-side wait ran out (status word)          */
    XSV_ERR_RANGE = 7,   /* an input lay beyond the fp16 range (status word)          */
    XSV_ERR_CAPACITY = 8,/* unbounded cache grew past max_cache_tokens                */
    XSV_ERR_LIMIT = 9    /* size beyond the fixed maximum of a no-allocation entry point */
} xsv_status;

typedef enum { XSV_F16 = 0, XSV_BF16 = 1 } xsv_dtype;

/* Which attention kernel xsv_step launches. */
typedef enum {
    XSV_ATTN_AUTO = 0,   /* the tcgen05/TMEM kernel when available for the shape */
    XSV_ATTN_MMA = 1,    /* warp-level mma.sync kernel (portable baseline)       */
    XSV_ATTN_TC5 = 2     /* tcgen05 + TMEM kernel                                */
} xsv_attn_impl;

/* Phases timed by the optional profiling events (xsv_cache_set_profiling). */
enum { XSV_PHASE_ATTN = 0, XSV_PHASE_SCORE = 1, XSV_PHASE_SELECT = 2, XSV_PHASE_QUANT = 3, XSV_PHASE_COUNT = 4 };

/*
 * Create a cache for `layers` independent layers (section 3.1, Eq. 1; the
 * budget and bit width of sections 3.2-3.3).
 *   heads, head_dim : attention geometry; head_dim must be 64.
 *   budget_tokens   : L_max, the cache length bound in tokens; <= 0 means
 *                     unbounded (no pruning; see max_cache_tokens below).
 *   bits            : 2, 4 or 8 -> quantised cache; 16 -> quantisation off
 *                     (the cache keeps the 16-bit inputs).
 * No device memory is allocated until the first step (or set_options with
 * max_frame_tokens > 0).  *out receives the handle.  Uses the current device.
 */
xsv_status xsv_cache_create(xsv_cache** out, int layers, int heads, int head_dim,
                            long long budget_tokens, int bits);

/*
 * Optional settings; must precede the first step (XSV_ERR_ORDER otherwise).
 *   n_special        : camera + register tokens at the head of each frame,
 *                      kept un-pooled by the query pooling (Eq. 3).  Default 5.
 *   pool_group       : g, patch tokens averaged per pooled query (Eq. 3).  Default 16.
 *   quant_group      : G, quantisation group size (section 4.1).  Must be 64.
 *   max_frame_tokens : the most tokens any frame will hold (frames may differ
 *                      in size: inputs resized to a maximum edge, section 4.1);
 *                      allocates now.  0: the first frame's size, i.e. no
 *                      later frame may be larger than the first.
 *   max_cache_tokens : capacity in tokens for an unbounded cache
 *                      (budget_tokens <= 0); ignored otherwise.  Default 16 frames.
 * A negative value leaves a setting unchanged.
 */
xsv_status xsv_cache_set_options(xsv_cache* c, int n_special, int pool_group, int quant_group,
                                 int max_frame_tokens, long long max_cache_tokens);

/* Select the attention kernel (default XSV_ATTN_AUTO); both compute Eq. 2 with Eq. 12 fused. */
xsv_status xsv_cache_set_attn_impl(xsv_cache* c, xsv_attn_impl impl);

/*
 * One streaming step of layer `layer` (Fig. 2; Eq. 2-12).
 *   Q, K, V : device, the new frame's queries / keys / values.
 *   n_tokens: tokens of this frame (T_current of Eq. 8); at most
 *             max_frame_tokens, XSV_ERR_SHAPE beyond.  The first frame's size
 *             is T_first; Eq. 8 keeps k = max(0, L_max - T_first - T_current)
 *             tokens of the middle segment.
 *   out     : device, receives softmax(Q [K~cache ; K]^T / sqrt(head_dim)) [V~cache ; V].
 *   stream  : cudaStream_t (as void*); NULL is the default stream.
 * Afterwards the layer's cache holds [first frame ; kept middle ; this frame],
 * quantised (see xsv_cache_len for its length).
 * Everything is enqueued; nothing synchronises with the host.  A step that
 * prunes runs its selection and re-quantisation kernels (Eq. 8-11, which need
 * the scores but not the attention output) on streams the cache owns, beside
 * the end of the attention kernel, and `stream` waits for them before the step
 * ends: in the order of `stream` the step is complete -- `out` written, the
 * cache updated, Q, K, V free to be reused -- when the call's work has run.
 * All steps of one cache must be ordered with respect to each other (one
 * stream, or streams ordered by events).
 */
xsv_status xsv_step(xsv_cache* c, int layer, const void* Q, const void* K, const void* V,
                    int n_tokens, xsv_dtype dtype, void* out, void* stream);

/*
 * One step for several independent video streams at once (no counterpart in
 * the paper, which streams one video; this is how a server fills the GPU when
 * one stream's step is too small to, e.g. with the paper's own budget of about
 * two frames).  caches[i] is stepped on layer `layer` with the frame
 * Q[i], K[i], V[i] of n_tokens[i] tokens and writes out[i]; each call argument
 * is a HOST array of n entries (device pointers for Q, K, V, out), n at most
 * XSV_MAX_BATCH.  The attention of the n streams is one kernel launch (plus one
 * merge launch) per group of streams, a launch's CTAs dealt to its streams in
 * proportion to their work; the library picks the grouping (all n, or
 * consecutive groups of 4, 2 or 1) that its cost model estimates fastest, since
 * CTAs do not span streams and 148 of them fit e.g. eight long streams badly.
 * Scores, selection and quantisation run per stream, the selection and
 * quantisation on each cache's own streams side by side.  Results and cache
 * states are those of n xsv_step calls.  The caches must be distinct, on one
 * device, with equal heads and bit width (XSV_ERR_SHAPE otherwise) and use the
 * default attention kernel; every cache is checked before anything is launched,
 * so an argument, shape or order error leaves all of them unchanged.
 */
#define XSV_MAX_BATCH 8
xsv_status xsv_step_batch(xsv_cache* const* caches, int n, int layer, const void* const* Q,
                          const void* const* K, const void* const* V, const int* n_tokens,
                          xsv_dtype dtype, void* const* out, void* stream);

/*
 * The cache update of a step without its attention (no counterpart in the
 * paper: a way to fill a cache quickly, e.g. to measure the attention over a
 * long uncompressed cache without paying for every step before it).  Appends
 * the frame's keys and values as xsv_step would, quantised if the cache is.
 * Only for steps that do not prune (the first frame, an unbounded cache, or
 * T_c + n_tokens <= L_max): a pruning step needs the frame's queries and
 * returns XSV_ERR_ORDER here.  Counts as the layer's step for this frame.
 */
xsv_status xsv_cache_append(xsv_cache* c, int layer, const void* K, const void* V, int n_tokens,
                            xsv_dtype dtype, void* stream);

/*
 * Deferred join (off by default).  With on != 0, `stream` does not wait at the
 * end of a pruning step for the selection and re-quantisation kernels on the
 * cache's own streams: they finish under whatever `stream` runs next (the next
 * layer's score kernels and the start of its attention kernel).  The library
 * keeps its own state ordered -- a layer's next step waits for that layer's
 * outstanding work, shared scratch is handed over through events, the host-side
 * queries synchronise every stream -- but two things become the caller's:
 * K and V of a step must stay unchanged until `stream` has passed the next
 * xsv_step on the same layer or an xsv_cache_join, and so must not be freed or
 * overwritten earlier; `out` is complete in `stream` order as always.
 * xsv_cache_join makes `stream` wait for all outstanding side-stream work.
 * (How the launches are ordered is the library's; the paper has no counterpart.)
 */
xsv_status xsv_cache_set_deferred_join(xsv_cache* c, int on);
xsv_status xsv_cache_join(xsv_cache* c, void* stream);

/*
 * Same step with HOST buffers (pinned host memory makes the copies asynchronous).
 * The inputs are copied to device staging owned by the cache on an internal
 * stream, so that the copy of one call overlaps the kernels of the previous
 * one; the step itself runs on `stream`; the call returns without
 * synchronising.  Q_host, K_host, V_host must stay unchanged until `stream` has
 * passed the call.
 *   Default: `out_host` is written on `stream`: it is complete once `stream`
 *   has passed the call.
 *   With xsv_cache_set_host_pipelining(c, 1) the result is copied back on a
 *   second internal stream and the next step does not wait for it: `out_host`
 *   is complete once `stream` has passed a later xsv_cache_host_flush(c, stream)
 *   (at most two results are in flight; a third call waits for the first).
 * The first call allocates the staging slots (sized for max_frame_tokens) and
 * creates the copy streams; later calls allocate nothing.  (Host staging is
 * the library's; the paper has no counterpart.)
 */
xsv_status xsv_step_host(xsv_cache* c, int layer, const void* Q_host, const void* K_host,
                         const void* V_host, int n_tokens, xsv_dtype dtype, void* out_host,
                         void* stream);

/* Deferred copy-back of xsv_step_host results (see there); off by default.
 * XSV_ERR_ORDER while results are in flight (flush first).  (No counterpart in the paper.) */
xsv_status xsv_cache_set_host_pipelining(xsv_cache* c, int defer_output);

/* Makes `stream` wait for every result of xsv_step_host still on its way to the host.
 * (No counterpart in the paper.) */
xsv_status xsv_cache_host_flush(xsv_cache* c, void* stream);

/*
 * Eq. 3-7 on their own: importance scores of `n_keys` keys for one frame's
 * queries, without a cache object.
 *   Q      : device, [heads][n_tokens][64], 16-bit (`dtype`).
 *   keys   : device, [heads][n_keys][64], 16-bit, same dtype (un-quantised keys).
 *   scores : device, float[n_keys]; scores[j] = mean_i (Q_bar K_bar^T)[i][j] with
 *            Q_bar the head-averaged pooled queries (n_special rows kept, patch
 *            rows averaged in groups of pool_group) and K_bar the head-averaged keys.
 * Allocates and frees 32 KB of scratch per call, stream-ordered on `stream`.
 */
xsv_status xsv_importance_scores(const void* Q, const void* keys, int heads, int n_tokens,
                                 long long n_keys, xsv_dtype dtype, int n_special, int pool_group,
                                 float* scores, void* stream);

/*
 * Quantisation error of the two granularities of Eq. 11, the quantity Table 1
 * compares: the tensor x [heads][n_tokens][64] (DEVICE, 16-bit elements) is
 * quantised with Eq. 9-10 -- per channel over groups of 64 consecutive tokens
 * (per_channel != 0: the scheme Eq. 11 gives to keys; a last, partial group
 * holds the remaining tokens) or per token over its 64 channels (per_channel
 * == 0: the scheme for values) -- dequantised with Eq. 12, and the mean of
 * (x - x~)^2 over all elements, accumulated in float64, is written to
 * *mse_host (HOST).  bits: 2, 4 or 8.  Allocates and frees its scratch on
 * `stream` (stream-ordered allocator) and synchronises `stream`.
 */
xsv_status xsv_quantization_mse(const void* x, int heads, long long n_tokens, xsv_dtype dtype, int bits,
                                int per_channel, double* mse_host, void* stream);

/*
 * xsv_importance_scores for callers that must not allocate.  (The paper has no
 * counterpart: this is a property of the library, not of the method.)
 *
 * Some code cannot call cudaMalloc, or anything that may: a frame loop with a
 * latency bound (an allocation can synchronise the whole device), a process
 * whose device memory has all been handed to its own pool, work issued while
 * another thread is capturing a CUDA graph in global capture mode.  This entry point computes
 * the same scores as xsv_importance_scores with the same kernels, but its
 * scratch (the per-head partial sums of the pooled queries) is a fixed array
 * inside the library's device image: 128 KB, present on every GPU that loads
 * the library until the process exits.  It calls no cudaMalloc, cudaFree or
 * other allocating routine; inputs and outputs stay the caller's.
 *
 *   Arguments: as xsv_importance_scores.
 *   Limit    : heads <= 64; more returns XSV_ERR_LIMIT and launches nothing.
 *   Set-up   : the first call on each device (and for each input type) is
 *              set-up: it looks up the array's device address
 *              (cudaGetSymbolAddress, with that device current) and, where the
 *              CUDA runtime loads modules lazily, makes it load the library's
 *              device code, which may allocate and synchronise.  Make that
 *              first call at start-up, outside any stream capture; from the
 *              second call on nothing is allocated.
 *   Sharing  : every call on a device uses the same array.  Contents left by an
 *              earlier call are never read (each call rewrites all it uses), but
 *              two calls that overlap on the GPU -- different streams, no
 *              ordering between them -- race on it.  Order them.
 */
xsv_status xsv_importance_scores_static(const void* Q, const void* keys, int heads, int n_tokens,
                                        long long n_keys, xsv_dtype dtype, int n_special,
                                        int pool_group, float* scores, void* stream);

/* Device bytes held now: codes, scales, offsets, origin ids of all layer
 * buffers plus the spare buffer and scratch (section 4.6's memory figure). */
size_t xsv_cache_bytes(const xsv_cache* c);

/* Bytes of one layer's packed KV at its current length (codes + scales + offsets). */
size_t xsv_cache_layer_kv_bytes(const xsv_cache* c, int layer);

void xsv_cache_destroy(xsv_cache* c);

/* Tokens currently cached in `layer`, kept on the host without a device read
 * (section 3.2's trigger rule and Eq. 8): after a step on a cache of T_c tokens
 * with a frame of F tokens it is T_c + F if this was the layer's first step,
 * the cache is unbounded or T_c + F <= L_max; else
 * T_first + max(0, L_max - T_first - F) + F = max(L_max, T_first + F). */
long long xsv_cache_len(const xsv_cache* c, int layer);

/* Frames stepped so far in `layer` (bookkeeping; the paper has no counterpart). */
long long xsv_cache_frames(const xsv_cache* c, int layer);

/*
 * Copy one layer's logical state to HOST arrays (synchronises `stream`).
 * Any pointer may be NULL to skip it.  With T = xsv_cache_len, H heads, d = head_dim:
 *   k_codes, v_codes : unsigned char [H][T][d], one code per byte (bits < 16);
 *   k_scale / k_zero : float [H][ceil(T/64)][d]  (Eq. 10, per channel per 64-token group: the scale and
 *                      the offset, i.e. the group's minimum; a value is code * scale + offset, Eq. 12);
 *   v_scale / v_zero : float [H][T]              (the same per token);
 *   origin           : long long [T], the running index in the stream of the token in each slot
 *                      (tokens of all earlier frames + its index in its frame);
 *   k_raw, v_raw     : unsigned short [H][T][d], the 16-bit cache when bits == 16.
 */
xsv_status xsv_cache_export_layer(xsv_cache* c, int layer, unsigned char* k_codes, float* k_scale,
                                  float* k_zero, unsigned char* v_codes, float* v_scale, float* v_zero,
                                  long long* origin, unsigned short* k_raw, unsigned short* v_raw,
                                  void* stream);

/*
 * The inverse of xsv_cache_export_layer: load one layer's logical state from
 * HOST arrays (checkpoint restore; also the way to continue a stream on another
 * cache object; the paper has no counterpart).  Synchronises `stream`.
 *   n_cached     : T, tokens in the arrays; at most the cache's capacity
 *                  (max(budget, 2 * max_frame_tokens), or max_cache_tokens when unbounded).
 *   frames_done  : frames this layer has been stepped with (the next step is
 *                  frame frames_done + 1; all layers must agree before stepping on).
 *   frame_tokens : T_first, the tokens of the layer's first frame (they head the arrays);
 *                  also max_frame_tokens if that was not set before.
 *   dtype        : the element type of the stream (fixed per cache).
 *   arrays       : as in xsv_cache_export_layer (codes one per byte, < 2^bits;
 *                  k_raw / v_raw instead when bits == 16); `origin` is required.
 * Every array is validated before anything is written: errors leave the cache
 * unchanged, except XSV_ERR_CUDA.
 */
xsv_status xsv_cache_import_layer(xsv_cache* c, int layer, long long n_cached, long long frames_done,
                                  int frame_tokens, xsv_dtype dtype, const unsigned char* k_codes,
                                  const float* k_scale, const float* k_zero, const unsigned char* v_codes,
                                  const float* v_scale, const float* v_zero, const long long* origin,
                                  const unsigned short* k_raw, const unsigned short* v_raw, void* stream);

/*
 * Importance scores (Eq. 7) of the last pruning step of any layer, copied to
 * a HOST array of capacity `cap` floats; *n receives their count (the length
 * of the prunable middle segment), 0 if the last step did not prune.
 * Synchronises `stream`.
 */
xsv_status xsv_last_scores(xsv_cache* c, float* scores_host, long long cap, long long* n, void* stream);

/* Read (and keep) the sticky device status word; synchronises `stream`.
 * XSV_OK, XSV_ERR_TIMEOUT or XSV_ERR_RANGE. */
xsv_status xsv_cache_status(xsv_cache* c, void* stream);

/* The raw status word behind xsv_cache_status (diagnostic; the paper has no
 * counterpart): bit 0 a bounded wait ran out, bit 1 a value left the supported
 * range, bits 8-14 which wait of the attention kernel gave up (0x100 a
 * producer waiting for a free stage, 0x200 / 0x400 a softmax warp waiting for
 * S / for the completion of P V, 0x800 / 0x1000 / 0x4000 the issuing warp
 * waiting for the query tiles / a filled stage / a sub-tile's probabilities).  Synchronises `stream`; -1 on error. */
int xsv_cache_status_word(xsv_cache* c, void* stream);

/* Per-phase CUDA-event timing.  on = 1: every step records events around each
 * phase on the step's stream; on = 2: around the attention phase only (each
 * pair of events costs the stream a few microseconds, which matters when the
 * whole step is being timed as well); on = 3: around every seventh attention
 * phase (a sample that walks through the layers of a 24-layer stack); on = 4:
 * as 1, and every kernel of the step runs on `stream` in order (the cache's own
 * streams are not used), so that the recorded spans are kernel durations and
 * not spans that include waiting for free multiprocessors; on = 0: none.
 * xsv_cache_profile_read
 * synchronises the recorded events, adds their durations to per-phase totals,
 * and returns the totals (milliseconds) and launch counts accumulated since
 * the last reset.  Events are created when profiling is switched on and, if
 * more phases are recorded between two reads than that pool holds, on demand.
 * (Measurement support; the paper has no counterpart.) */
xsv_status xsv_cache_set_profiling(xsv_cache* c, int on);
xsv_status xsv_cache_profile_read(xsv_cache* c, double ms[XSV_PHASE_COUNT], long long launches[XSV_PHASE_COUNT], int reset);

/*
 * Self-test of the bounded device-side waits (the library's kernels hand work
 * over through barriers; a wait that is never satisfied must not hang the GPU).
 * Launches one tiny kernel whose only wait nothing ends, synchronises `stream`,
 * and returns XSV_ERR_TIMEOUT when the wait gave up after its limit (about two
 * seconds) and reported it -- the expected outcome -- or XSV_OK if it did not.
 * The context stays usable.  (The paper has no counterpart.)
 */
xsv_status xsv_selftest_bounded_wait(void* stream);

/*
 * Host-only self-test of the table in which the library keeps what it has
 * configured per CUDA device (opt-in shared memory of a kernel, occupancy,
 * multiprocessor count): slots of different devices are independent, and
 * device indices beyond the table are never cached.  Needs no GPU; returns 0
 * when the table behaves.  (The paper has no counterpart.)
 */
int xsv_selftest_device_table(void);

/*
 * How xsv_step_batch would group n streams into attention launches: the number
 * of consecutive streams per launch (n, 4, 2 or 1) that the library's cost
 * model estimates fastest for streams with cache_tokens[i] cached tokens and
 * frames of frame_tokens[i] tokens (HOST arrays of n entries), `heads` heads,
 * on a device with `multiprocessors` multiprocessors.  CTAs do not span
 * streams, so e.g. eight long streams on 148 multiprocessors go out as two
 * launches of four (37 CTAs each) rather than one of eight (18 or 19 each).
 * Host arithmetic only: needs no GPU and touches no cache.  Returns -1 for bad
 * arguments (n outside 1..XSV_MAX_BATCH, a null array, a negative length).
 * (The paper has no counterpart.)
 */
int xsv_plan_batch_groups(int n, const int* cache_tokens, const int* frame_tokens, int heads, int multiprocessors);

/* Kernels launched by this library in the calling process since load (the paper has no counterpart). */
long long xsv_kernel_launches(void);

/* Text for a status code (the paper has no counterpart). */
const char* xsv_strerror(xsv_status s);

/* Text of the CUDA runtime error behind the calling thread's most recent
 * XSV_ERR_CUDA from xsv_step / xsv_step_host / xsv_importance_scores
 * ("no error" if there was none).  The pointer is to static storage.  (No counterpart in the paper.) */
const char* xsv_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* XSV_H */
