/*
 * mvla_prune.h -- C ABI of the B200 (sm_100a) prune step for multi-visual-modal
 * VLA inference: tri-stage, modality-salience-aware token pruning
 * ("2D or 3D: Who Governs Salience in VLA Models?", Alg. 1).
 *
 * One prune point inside the LLM prefill does, per sample:
 *   salience  : attention of the instruction (text) queries over every 2D image
 *               token and 3D point token (Sec. 3.2.1), reduced to one score per token;
 *   carry-over: the scores and the four modality indicators are smoothed across
 *               action steps (Alg. 1 step 1; Eqs. 8, 9);
 *   budget    : the keep budget is split between 2D and 3D by the stage rules
 *               (Sec. 4.1 dual threshold, Sec. 4.2 target-object rule, Sec. 4.4 fusion);
 *   select    : the top-k tokens per modality, ties to the lower index (Eq. 10 as an index list);
 *   compact   : surviving hidden / K / V rows are gathered into a dense layout (Sec. 4.4).
 *
 * Conventions
 *   - Every function returns an int32 status (0 = MVLA_OK, negative = error) and never throws.
 *   - "device pointer" = memory of the context's CUDA device; "host pointer" = ordinary memory.
 *   - No function synchronises the stream; work is enqueued on `stream` (a cudaStream_t passed
 *     as void*, NULL = the legacy default stream).  Host arrays (`samples`) are consumed before
 *     the call returns.  The library keeps no caller pointer beyond the enqueued work.
 *   - Input tensors are token-major and packed ragged: Q is [rows, n_heads, head_dim], K and V are
 *     [rows, n_kv_heads, head_dim] (n_kv_heads == n_heads unless the configuration groups them),
 *     hidden is [rows, d_model], rows contiguous, dtype as given at create.  A sample owns the
 *     rows [seq_off, seq_off + n_txt + n_2d + n_3d) split in three contiguous segments.
 *     Base pointers must be 16-byte aligned.
 *   - Visual tokens of a sample are numbered 2D first, then 3D ("visual order").  Arrays
 *     `attn`, `l1`, `ahat` hold sum(n_2d + n_3d) floats, samples back to back in batch order.
 *   - Inputs must be finite.
 *   - A context is not thread-safe; use one per host thread / stream.
 *   - Tracing and logging (the paper has no counterpart; host side only, nothing on the device's path):
 *     every call of the stage and step functions is an NVTX range named after the function, and
 *     mvla_prune_step marks its phases inside it ("mvla: scoring", "mvla: selection + row copy", ...) around
 *     the kernels they enqueue; with MVLA_LOG=1 in the environment (read once per process) each of those
 *     calls also prints one line "[mvla] name(arguments) -> status" to stderr.
 */
#ifndef MVLA_PRUNE_H
#define MVLA_PRUNE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* status codes */
#define MVLA_OK                 0
#define MVLA_ERR_INVALID_ARG   (-1)  /* null / misaligned pointer, bad segment, bad ratio, bad flag */
#define MVLA_ERR_UNSUPPORTED   (-2)  /* shape or dtype outside what was built (see mvla_prune_create) */
#define MVLA_ERR_OOM           (-3)  /* workspace allocation failed */
#define MVLA_ERR_CUDA          (-4)  /* a CUDA call failed (no device, launch error, ...) */
#define MVLA_ERR_CAPACITY      (-5)  /* batch / segment larger than the capacities given at create */
#define MVLA_ERR_TIMEOUT       (-6)  /* a bounded device-side wait gave up in an earlier call (sticky) */
#define MVLA_ERR_STATE         (-7)  /* bad prune point or state slot */

#define MVLA_DTYPE_BF16 0
#define MVLA_DTYPE_FP32 1
#define MVLA_DTYPE_FP8_E4M3 2   /* q, k, v in 8-bit floating point (e4m3, finite: no infinities); hidden stays bf16.
                                   Tensor-core scoring only; not available together with patch_path */

#define MVLA_SALIENCE_AUTO 0
#define MVLA_SALIENCE_FMA  1

#define MVLA_MODE_FIXED    0   /* per-modality keep ratios keep_2d / keep_3d */
#define MVLA_MODE_ADAPTIVE 1   /* one total keep ratio, split by the stage rules */
#define MVLA_MODE_PATCH    2   /* Alg. 1 taken literally, patch by patch: no budget, the masks decide (mvla_prune_step;
                                  needs patch_path = 1 at create and n_2d == n_3d: patch p owns 2D token p and 3D token p) */

#define MVLA_FLAG_RESET_STATE     1u  /* restart the episode: this call is action step t = 1 */
#define MVLA_FLAG_NO_STATE_UPDATE 2u  /* dry run: decide as usual but leave the smoothed state and t untouched */
#define MVLA_FLAG_INPUTS_STABLE   4u  /* mvla_prune_step only.  The caller promises that none of ITS OWN work enqueued on
                                         `stream` before this call and possibly still running writes q, k, hidden or
                                         touches this call's output buffers.  (Earlier prune steps of this context
                                         need no promise: where one of them writes a buffer that this call reads or
                                         writes, the library orders this call after everything enqueued so far.)
                                         Scoring and selection then run on one of a small ring of streams owned by the
                                         context, beside the selection and row copy of the steps before; the row copy
                                         stays on `stream` and waits for the step's selection.  Every result of the
                                         call is complete in the order of `stream`, as without the flag, and the
                                         smoothed state is updated in call order.  Without the flag every kernel waits
                                         for all earlier work of `stream`. */

#define MVLA_SET_2D 1   /* candidate sets are bit sets */
#define MVLA_SET_3D 2

typedef struct mvla_ctx mvla_ctx;   /* opaque */

/* Creation-time configuration.  Paper defaults (Sec. 5.4): tau_2d 0.08, tau_3d 0.20, beta 0.85,
 * window_k 7.  eps_3d (default 0.02) quantifies "3D response near zero" of the target-object
 * rule (Sec. 4.2); floor_ratio (default 0.10) is the share of each modality that always
 * survives, the deterministic form of the 90 % background pruning (Sec. 4.2). */
typedef struct mvla_config {
    int32_t device;            /* CUDA device ordinal */
    int32_t dtype;             /* MVLA_DTYPE_*: element type of q, k, v, hidden (FP8_E4M3: of q, k, v; hidden bf16) */
    int32_t n_heads;           /* H: query heads (key / value heads: n_kv_heads below) */
    int32_t head_dim;          /* d: a multiple of 32 from 64 to 256 (64, 96, 128, ... 256) */
    int32_t d_model;           /* D: hidden width, multiple of 8 (bf16) / 4 (fp32) */
    int32_t max_batch;         /* capacity: samples per call */
    int32_t max_text;          /* capacity: text tokens per sample, <= 64 */
    int32_t max_2d;            /* capacity: 2D tokens per sample */
    int32_t max_3d;            /* capacity: 3D tokens per sample; max_2d + max_3d <= 4096 */
    int32_t n_prune_points;    /* independent smoothed states per slot (e.g. layers 2 and 8 -> 2) */
    int32_t n_state_slots;     /* episodes tracked at once; 0 -> max_batch */
    int32_t window_k;          /* Eq. 8 -> Eq. 9 switch */
    int32_t cold_start_full_keep; /* 1: action step t = 1 keeps every token (Alg. 1 cold start) */
    int32_t salience_path;     /* MVLA_SALIENCE_AUTO (0): tensor cores for bf16, FMA kernel for fp32;
                                  MVLA_SALIENCE_FMA (1): the CUDA-core FMA kernel for either dtype */
    double tau_2d, tau_3d;     /* Sec. 4.1 */
    double beta;               /* Eq. 9 */
    double eps_3d;
    double floor_ratio;
    /* patch-by-patch path (MVLA_MODE_PATCH) */
    double obj_2d_min;         /* target-object rule (Sec. 4.2): {2D} only when M^S2_2D,p > obj_2d_min and
                                  M^S2_3D,p < eps_3d; 0 -> 0.5 */
    int32_t patch_path;        /* 1: allocate the per-patch state and the attention scratch
                                  (n_heads x max_text x max_batch x (max_2d + max_3d) floats) */
    int32_t kmeans_max_iter;   /* rounds of the 1-D K-Means (Sec. 4.2); 0 -> 32 */
    int32_t n_kv_heads;        /* grouped-query attention: k and v are [rows, n_kv_heads, head_dim] and query head h
                                  reads key head h / (n_heads / n_kv_heads); 0 -> n_heads.  Must divide n_heads.
                                  Not available together with patch_path */
    int32_t logit_cache;       /* 1: keep the raw logits of the last step of every (prune point, slot), so that a step
                                  which says which rows changed (mvla_tensors.changed_rows) recomputes only those
                                  (Sec. 4.3 / 5.2: consecutive frames share most of their content).
                                  n_prune_points x slots x n_heads x (max_2d + max_3d) x round16(max_text) floats.
                                  bf16 / e4m3 tensor-core path, samples of up to 2048 visual tokens, budgeted modes */
    int32_t reserved0;
} mvla_config;

/* One batch element (host array).  Offsets are rows relative to seq_off; the three segments
 * must be disjoint and lie inside [0, n_txt + n_2d + n_3d).  n_txt >= 1, n_2d + n_3d >= 1. */
typedef struct mvla_sample {
    int32_t seq_off;           /* first row of the sample in the packed tensors */
    int32_t off_txt, n_txt;
    int32_t off_2d, n_2d;      /* multi-view images are one segment of views x patches */
    int32_t off_3d, n_3d;
    int32_t state_slot;        /* which smoothed state this sample continues, < n_state_slots */
    double keep_2d, keep_3d;   /* FIXED: k_m = min(n_m, floor(keep_m * n_m + 0.5)) */
    double keep_total;         /* ADAPTIVE: B = min(n_vis, floor(keep_total * n_vis + 0.5)) */
} mvla_sample;

/* Per-sample record of what the budget stage decided (device array, optional). */
typedef struct mvla_diag {
    int32_t t;                 /* 1-based action step this call was */
    int32_t c_s1, c_s2, c_final; /* candidate sets (Sec. 4.1, 4.2, 4.4) */
    int32_t budget, k_2d, k_3d;
    int32_t reserved;
    float x[4];                /* instantaneous [M^S1_2D, M^S1_3D, M^S2_2D, M^S2_3D] (Eq. 3-1, P2D, P3D) */
    float mhat[4];             /* the same, smoothed (Eqs. 8, 9) */
} mvla_diag;

/* Per-sample record of the patch-by-patch path (device array, optional). */
#define MVLA_LABEL_BG  0       /* K-Means classes by ascending centre (Sec. 4.2) */
#define MVLA_LABEL_ROB 1
#define MVLA_LABEL_OBJ 2
typedef struct mvla_patch_diag {
    int32_t t;                 /* 1-based action step this call was */
    int32_t iters;             /* K-Means rounds run */
    int32_t n_label[3];        /* patches per class */
    int32_t k_2d, k_3d;        /* kept tokens per modality */
    int32_t n_out;             /* kept rows of the sample = n_txt + k_2d + k_3d */
    float centre[3];           /* class centres, ascending */
    float mu_2d, mu_3d;        /* baselines of Sec. 4.2 */
    float reserved[3];
} mvla_patch_diag;

/* Inputs of the fused step (device pointers). hidden may be NULL in FIXED mode when
 * out_hidden is NULL too. */
typedef struct mvla_tensors {
    const void *q, *k, *v;     /* [rows, H, d] */
    const void *hidden;        /* [rows, D] */
    int64_t rows;              /* rows allocated in each tensor (bounds the TMA descriptors) */
    const float *rand_u;       /* MVLA_MODE_PATCH: one uniform number in [0, 1) per patch, samples back to back
                                  (the draws of the background rule); NULL otherwise */
    const uint8_t *changed_rows; /* HOST array, one byte per row of the packed tensors, or NULL.  Non-zero: the caller
                                  rewrote this row of q / k since the previous step on the sample's state.  Read during
                                  the call (not afterwards).  Used only by contexts created with logit_cache: visual
                                  keys are handled in tiles of 128 per modality, and a tile none of whose rows changed
                                  takes its logits from the previous step instead of K (half the bytes, no MMA); a
                                  changed text row, a reset state, a different sample shape, NULL or the first step
                                  recompute everything.  A mask that hides a change silently reuses stale logits. */
} mvla_tensors;

/* Outputs of the fused step (device pointers, caller-owned). */
typedef struct mvla_outputs {
    void *out_hidden;          /* [sum kept rows, D]     nullable (skipped) */
    void *out_k, *out_v;       /* [sum kept rows, H, d]  nullable (skipped) */
    int32_t *kept_idx;         /* [sum kept rows] positions relative to each sample's seq_off, ascending */
    int32_t *out_offsets;      /* [batch + 1] row offsets of each sample in the outputs */
    int32_t *budgets;          /* [batch][2] = (k_2d, k_3d)  nullable */
    float *attn;               /* [sum n_vis] instantaneous scores a_j  nullable */
    float *ahat;               /* [sum n_vis] smoothed scores used for ranking  nullable */
    float *z;                  /* [sum n_vis] smoothed scores normalised to mean 1 per modality  nullable */
    mvla_diag *diag;           /* [batch]  nullable */
    /* MVLA_MODE_PATCH only, all nullable: */
    float *patch_x;            /* [sum P][4] instantaneous [M^S1_2D, M^S1_3D, M^S2_2D, M^S2_3D] of every patch */
    float *patch_xhat;         /* [sum P][4] the same, smoothed */
    int32_t *patch_info;       /* [sum P] label | C_S1 << 2 | C_S2 << 4 | C_final << 6 */
    struct mvla_patch_diag *patch_diag;   /* [batch] */
} mvla_outputs;

/* Kept rows of a sample: n_txt + B where B = n_2d + n_3d on a cold-start step (t = 1 with
 * cold_start_full_keep), else k_2d + k_3d (FIXED) or the total budget (ADAPTIVE); all host
 * computable.  Allocating sum(n_txt + n_2d + n_3d) rows is always enough. */

/*
 * Create a context on cfg->device: workspace, smoothed state for n_prune_points x
 * n_state_slots episodes, a device status word.  Supported: dtype bf16, fp32, or 8-bit e4m3 for q / k / v
 * (MVLA_DTYPE_FP8_E4M3: tensor-core path only, hidden stays bf16, no patch path); head_dim a multiple of 32 in
 * [64, 256] (fp32 with head_dim 256: up to 32 text tokens); max_text <= 64, max_2d + max_3d <= 4096,
 * max_batch <= 64; logit_cache: tensor-core path, budgeted modes.
 * The library owns *out until mvla_prune_destroy.  (Alg. 1 "Input" / "Init".)
 * Errors: INVALID_ARG, UNSUPPORTED, OOM, CUDA (no usable device).
 */
int32_t mvla_prune_create(const mvla_config *cfg, mvla_ctx **out);

/*
 * Salience (Sec. 3.2.1; Eq. 3-3 takes the L1 norm of a token's attention vector):
 *   l[h,i,j] = <q[h,i], k[h,j]> / sqrt(d)  for text queries i and visual keys j,
 *   alpha    = softmax over all visual keys j (2D and 3D jointly),
 *   a_j      = mean over heads h and text queries i of alpha[h,i,j].
 * and, when both `hidden` and `l1_out` are non-null, the L1 feature norm
 *   n_j = sum_c |hidden[j,c]| of each visual token (Sec. 3.1.2).
 * samples: host array [batch].  q, k, hidden: device, packed, `rows` rows each.
 * attn_out, l1_out: device, sum(n_vis) floats in visual order.  Stateless.
 */
int32_t mvla_salience(mvla_ctx *ctx, int32_t batch, const mvla_sample *samples,
                      const void *q, const void *k, const void *hidden, int64_t rows,
                      float *attn_out, float *l1_out, void *stream);

/*
 * Carry-over, budget and selection (Alg. 1 steps 1-4; Eqs. 8, 9, 10):
 * smooths `attn` into the per-token state and the four indicators into the
 * indicator state of (prune_point, state_slot), decides the per-modality budgets
 * and writes, per sample, the kept positions in ascending order merged with all
 * text positions.  Advances the slot's step counter t (host side) unless
 * MVLA_FLAG_NO_STATE_UPDATE.  `l1` is required in ADAPTIVE mode.
 * kept_idx: device, capacity >= sum kept rows; out_offsets: device [batch+1];
 * budgets, ahat_out, z_out, diag: nullable device arrays.  z_out = the smoothed scores
 * normalised to mean 1 inside each modality (ranking inside a modality is the same on either).
 */
int32_t mvla_select(mvla_ctx *ctx, int32_t prune_point, int32_t batch, const mvla_sample *samples,
                    int32_t mode, uint32_t flags, const float *attn, const float *l1,
                    int32_t *kept_idx, int32_t *out_offsets, int32_t *budgets,
                    float *ahat_out, float *z_out, mvla_diag *diag, void *stream);

/*
 * Compaction (Sec. 4.4: tokens with mask 1 proceed, the rest are discarded):
 *   out_X[out_offsets[b] + r, :] = X[seq_off_b + kept_idx[out_offsets[b] + r], :]
 * for X in {hidden, k, v}; a null input/output pair is skipped.  Rows are copied
 * bit-exactly in 16-byte vectors.  `total_kept` is the host-known number of output
 * rows (= out_offsets[batch]).  Outputs must not alias inputs.
 */
int32_t mvla_compact(mvla_ctx *ctx, int32_t batch, const mvla_sample *samples,
                     const int32_t *kept_idx, const int32_t *out_offsets, int32_t total_kept,
                     const void *hidden, const void *k, const void *v,
                     void *out_hidden, void *out_k, void *out_v, void *stream);

/*
 * The whole prune point (Alg. 1) as one submission: salience (+ L1 norms in
 * ADAPTIVE mode), carry-over, budget, select, compact.  Equivalent to the three
 * calls above on the same arguments.  `total_kept_out` (host, nullable) receives
 * the number of output rows.  In MVLA_MODE_PATCH the chain is mvla_patch_indicators, mvla_patch_select,
 * mvla_compact; the row count is then known only on the device (out_offsets[batch]) and
 * `total_kept_out` receives the capacity bound sum(n_txt + n_2d + n_3d); `budgets` receives the kept
 * counts per modality; MVLA_FLAG_INPUTS_STABLE overlaps neighbouring steps as on the budgeted path (when the
 * context could afford one attention copy per step in flight: six copies within 1 GiB).
 */
int32_t mvla_prune_step(mvla_ctx *ctx, int32_t prune_point, int32_t batch,
                        const mvla_sample *samples, int32_t mode, uint32_t flags,
                        const mvla_tensors *in, const mvla_outputs *out,
                        int32_t *total_kept_out, void *stream);

/*
 * Measurement aid (the paper has no counterpart).  While `event` (a cudaEvent_t created with timing, passed
 * as void*; null switches it off) is set, every mvla_prune_step that is not overlapped with its neighbours
 * (no MVLA_FLAG_INPUTS_STABLE) records it on the call's stream between its scoring kernel(s) and its
 * selection + row-copy kernel.  With events of the caller's own around the call this gives the duration of
 * each of the step's kernels as the step runs them.  The record sits between two kernels that otherwise
 * overlap at their edges, so the step is slightly slower while it is on; leave it off otherwise.  For
 * batches of more than 32 samples the event is recorded once per launch of 32.  The library never destroys it.
 */
int32_t mvla_set_stage_event(mvla_ctx *ctx, void *event);

/*
 * Key tiles that mvla_prune_step recomputed and reused so far on this context (cumulative; contexts created
 * with logit_cache; either pointer may be null).  Host-side counters: the decision is taken on the host from
 * the caller's changed_rows.
 */
int32_t mvla_logit_cache_stats(mvla_ctx *ctx, int64_t *tiles_computed, int64_t *tiles_reused);

/*
 * Measurement aid (the paper has no counterpart): time stamps taken by the step's own kernels.  An event
 * between two kernels of a step removes their overlap and costs microseconds inside a CUDA graph, so it
 * cannot time them as the step runs them; a handful of stores of the global nanosecond timer can.  While
 * `device_buffer` (device memory, 2 x 4096 x 2 uint64, zero-filled by the caller; null switches it off) is
 * set, every non-overlapped mvla_prune_step of the budgeted modes (MVLA_MODE_PATCH steps take no stamps) on
 * shapes the fused kernels cover makes CTA c (linear index,
 * c < 4096) of its scoring kernel write buffer[0][c][0] = the time it was free to start its loads (its
 * predecessor complete) and buffer[0][c][1] = the time it ended, and CTA c of its selection + row-copy kernel
 * the same into buffer[1][c][..] (start: past its wait for the scoring kernel; the selecting CTAs, which come
 * first, report the time the kept list was written as both).  Entries of CTAs that do not exist stay as they
 * were.  The pointer is read when the step is enqueued (or captured), so every captured step can have a buffer
 * of its own.  For batches of more than 32 samples the launches of 32 share the buffer.
 */
int32_t mvla_set_kernel_stamps(mvla_ctx *ctx, uint64_t *device_buffer);

/*
 * Failure-detection self-test (the paper has no counterpart).  Every device-side wait of this library is
 * bounded: when it runs out the kernel gives up, returns, and leaves MVLA_ERR_TIMEOUT in the context's status
 * word; from then on every call on the context returns MVLA_ERR_TIMEOUT (sticky) and a new context must be
 * created.  This call makes exactly that happen on purpose and harmlessly: one warp runs the library's
 * wait for a kept-list word on a word that nothing ever sets, with a limit of `limit_us` microseconds
 * (1 .. 1000000) instead of the second used in production.  Nothing hangs and nothing faults: the kernel
 * ends by itself after `limit_us`.  Enqueues on `stream`, does not synchronise; once the stream has run
 * it, the context is in the timed-out state.  Errors: INVALID_ARG, CUDA.
 */
int32_t mvla_selftest_wait_timeout(mvla_ctx *ctx, uint32_t limit_us, void *stream);

/*
 * Salience scores without a context and without any allocation.  (The paper has no counterpart:
 * this is a packaging variant of mvla_salience, same arithmetic, same kernels.)
 *
 * For callers that may not allocate device memory at call time: a server whose memory pool is
 * frozen after start-up, code running inside another framework's allocator-controlled region, a
 * control loop that cannot afford the device-wide stall of a cudaMalloc.  mvla_prune_create uses
 * cudaMalloc; this call uses none (no cudaMalloc / cudaFree / cudaHostAlloc, no heap).  Its scratch
 * (per-head partial scores) is a fixed 512 KiB array inside the library image, so:
 *   - limit: n_heads * sum(n_2d + n_3d) <= 131072 floats and batch <= 64, else MVLA_ERR_CAPACITY;
 *     max_text 64 and 4096 visual tokens per sample as elsewhere;
 *   - every GPU that loads the library holds the array until the process exits;
 *   - all calls on a device share the array and it keeps the previous call's contents (every entry
 *     that is read is rewritten first, and the timeout flag is cleared by each call);
 *   - calls whose GPU work may overlap (two streams without ordering) race on it: serialise them;
 *   - the first call on a device looks up the array's device address (host threads may race to be
 *     first: the look-up is guarded by a mutex); with CUDA's lazy module loading that first call is also
 *     when the driver loads the kernels and places the 512 KiB array on the device, so make one warm-up
 *     call per device before the region in which nothing may be allocated begins, and outside any
 *     stream capture.
 * device: CUDA ordinal; dtype: MVLA_DTYPE_BF16 or MVLA_DTYPE_FP32 (no 8-bit inputs here); head_dim: 64 or
 * 128 (the other head dims of mvla_config need a context); n_heads as in mvla_config, keys ungrouped;
 * samples: host array [batch];
 * q, k: device, [rows, n_heads, head_dim], 16-byte aligned; attn_out: device, sum(n_vis) floats in
 * visual order, caller-owned.  Enqueues on `stream`, does not synchronise.  If a bounded
 * device-side wait gives up, every attn_out entry is NaN (there is no context to hold a status).
 * Errors: INVALID_ARG, UNSUPPORTED, CAPACITY, CUDA.
 */
int32_t mvla_salience_noalloc(int32_t device, int32_t dtype, int32_t n_heads, int32_t head_dim,
                              int32_t batch, const mvla_sample *samples, const void *q, const void *k,
                              int64_t rows, float *attn_out, void *stream);

/*
 * Per-patch indicators X_t of Alg. 1 (needs patch_path = 1; every sample has n_2d == n_3d = P):
 *   M^S1_{2D,3D},p = share of the L1 feature norm of the patch's 2D / 3D token (Eq. 3-1, the term of patch p);
 *   M^S2_2D,p      = ||a2||_1 / (||a2||_1 + ||a3||_1) with a2, a3 the attention vectors (one entry per head and
 *                    text query) of the patch's 2D and 3D token (Eq. P2D);
 *   M^S2_3D,p      = ||a3 - <a3,a2>/<a2,a2> a2||_1 / (||a2||_1 + ||a3||_1), the part of a3 orthogonal to a2
 *                    (Eq. 3-4, Eq. P3D).
 * attn_out: device, sum(2P) floats, the per-token scores a_j as mvla_salience writes them.
 * x_out: device, [sum P][4] floats = [M^S1_2D, M^S1_3D, M^S2_2D, M^S2_3D], samples back to back.  Stateless.
 */
int32_t mvla_patch_indicators(mvla_ctx *ctx, int32_t batch, const mvla_sample *samples, const void *q,
                              const void *k, const void *hidden, int64_t rows, float *attn_out,
                              float *x_out, void *stream);

/*
 * Alg. 1 stages 1-4 patch by patch: temporal predictor of the four indicators of every patch (Eqs. 8, 9),
 * dual threshold (Sec. 4.1), 1-D K-Means with K = 3 on the patches' attention mass attn[p] + attn[P + p] and
 * the rules for background / robot / target-object patches (Sec. 4.2), candidate fusion (Sec. 4.4), masks
 * (Eq. 10) written as kept positions in ascending order merged with all text positions.
 *   K-Means: centres start at (min, mean, max); a round assigns every patch to its nearest centre (ties to
 *   the lower one) and, unless no label changed, moves each non-empty class's centre to its mean; at most
 *   kmeans_max_iter rounds; classes by ascending centre are background, robot, target object.
 *   Background patch: discarded when rand_u[p] < 1 - floor_ratio.  Baselines mu: means over the sample's
 *   patches of the smoothed M^S2 shares.  Action step t = 1 with cold_start_full_keep keeps everything.
 * The number of kept rows is data dependent: out_offsets [batch + 1] and counts [batch][2] = kept 2D / 3D
 * tokens are written on the device; kept_idx needs capacity sum(n_txt + 2P).  keep_* of the samples are
 * ignored.  Advances the slots' step counters like mvla_select.  flags: RESET_STATE, NO_STATE_UPDATE.
 * xhat_out [sum P][4], info_out [sum P] (label | C_S1 << 2 | C_S2 << 4 | C_final << 6), diag [batch]: nullable.
 */
int32_t mvla_patch_select(mvla_ctx *ctx, int32_t prune_point, int32_t batch, const mvla_sample *samples,
                          uint32_t flags, const float *attn, const float *x, const float *rand_u,
                          int32_t *kept_idx, int32_t *out_offsets, int32_t *counts, float *xhat_out,
                          int32_t *info_out, mvla_patch_diag *diag, void *stream);

/* Free everything the context owns.  NULL is accepted.  The caller must have
 * synchronised any stream that still runs work enqueued through the context. */
void mvla_prune_destroy(mvla_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* MVLA_PRUNE_H */
