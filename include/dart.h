/*
 * dart.h - C ABI of the B200 (sm_100a) implementation of DART's duplication-aware
 * vision-token reduction step (arxiv 2502.11494, Sec. 3.3: Def. 1-2, Eq. 7-10).
 *
 * The step is inserted into MLLM prefill after a shallow layer: from the layer's key states it
 * picks a few pivot tokens, scores every vision token by its cosine similarity to each pivot,
 * keeps, per pivot, the least similar tokens under a budget, and packs the kept rows of the
 * hidden states (with their indices and position ids) into a shorter dense sequence.
 *
 * Conventions
 *   - Every function returns an int: DART_OK (0) or a negative DART_ERR_* code.  Nothing throws,
 *     aborts or prints.  Errors found on the host are returned before anything is launched.
 *   - "device" pointers are CUDA device memory of the context's device, "host" pointers are
 *     ordinary (preferably pinned) host memory.  The caller owns every tensor; the library owns only
 *     the context and its workspace.  bf16 tensors are passed as void*.
 *   - Tensors are dense row-major: hidden/keys [B, S, d], out_hidden [B, S_out, d],
 *     out_idx / out_pos [B, S_out], with S_out = S - n_vis + n_keep.  Vision tokens occupy rows
 *     [vis_offset, vis_offset + n_vis) of every sample; all other rows are text and always kept.
 *   - All device work is enqueued on the caller's stream; no call synchronises the host except
 *     dart_create, dart_destroy, dart_status, dart_profile_read and dart_reduce_host.
 *   - One context serves one stream at a time.  Results are bitwise reproducible for identical
 *     inputs (no floating-point atomics anywhere).
 */
#ifndef DART_H
#define DART_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DART_VERSION 100 /* major * 10000 + minor * 100 + patch */

enum {
    DART_OK = 0,
    DART_ERR_NULL = -1,        /* a required pointer is NULL */
    DART_ERR_BAD_SHAPE = -2,   /* sizes violate the rules listed at dart_reduce, or exceed the context's maxima */
    DART_ERR_ALIGN = -3,       /* a tensor pointer is not 16-byte aligned */
    DART_ERR_ALIAS = -4,       /* an output overlaps an input */
    DART_ERR_CUDA = -5,        /* a CUDA call failed; see dart_last_cuda_error */
    DART_ERR_NOMEM = -6,       /* host or device allocation failed */
    DART_ERR_TIMEOUT = -7,     /* a bounded device-side wait gave up (reported by dart_status) */
    DART_ERR_CHECK = -8,       /* a device-side self-check failed (reported by dart_status) */
    DART_ERR_UNSUPPORTED = -9  /* option combination not available */
};

/* dart_desc.flags */
#define DART_FLAG_HOST_STAGING 1u /* also allocate the device staging buffers dart_reduce_host needs */

/* dart_opts.path */
#define DART_PATH_AUTO 0
#define DART_PATH_STAGED 1 /* one kernel per step of the method, every intermediate in the workspace */
#define DART_PATH_FUSED 2  /* persistent sweep kernel (scores, pivots and similarities in one launch; with the caller's
                              pivots: scores and similarities from one pass over the keys); needs d % 64 == 0 and
                              n_pivot <= 256, else UNSUPPORTED.  AUTO picks it when it applies. */
#define DART_PATH_TWO_PASS 3 /* two launches instead of the persistent sweep: a plain score pass, pivot selection, then
                              scores' sums of squares and similarities from one tensor-core pass; same limits as FUSED.
                              Reads the keys twice like FUSED but has no waits between CTAs: faster for small batches. */

#define DART_PATH_RESIDENT 4 /* steps 1-3 from ONE read of the keys: every sample is spread over all SMs and stays in their
                              shared and tensor memory until its pivots are known.  Needs n_pivot <= 8, d % 64 == 0,
                              d <= 4096, n_vis <= 32 rows per SM (and the pivots chosen by score, one tensor for
                              steps 1-3), else UNSUPPORTED.  The fastest path for a few samples (AUTO takes it up to
                              four); at half the speed of FUSED on the large batched workloads, where the wait for a
                              sample's pivots is longer than the samples that fit the chip can cover. */

#define DART_PATH_SPLIT 5    /* RESIDENT for a share of every sample's 128-row tiles, one tensor-core pass (as in TWO_PASS)
                              for the others once the pivots are known: the rows that stay on the chip are read once, the
                              others twice.  dart_opts.resident_split sets the share.  Same limits as RESIDENT. */

#define DART_PATH_PAIRED 6   /* persistent kernel in which the same SM reads a block of 16 key rows twice, a few microseconds
                              apart (scores first; similarities as soon as every SM has merged the SMs' short candidate
                              lists into the sample's pivots), so that the second read comes from the L2.  Needs
                              n_pivot <= 16, d % 64 == 0, pivots chosen by score, else UNSUPPORTED. */

/* dart_opts.pivot_source: where step 2 takes the pivots from when the caller does not name them (pivots_in == NULL) */
#define DART_PIVOTS_BY_SCORE 0 /* the n_pivot vision tokens of best score (dart_reduce) */
#define DART_PIVOTS_MIXED 1    /* both modalities (Sec. 5.4; the pivot-selection table uses 4 visual and 4 text tokens):
                                  the n_pivot - n_text_pivots vision tokens and the n_text_pivots text tokens of best score
                                  (same score and direction as BY_SCORE, equal scores to the earlier token); the vision
                                  pivots take their turns first, in rank order, then the text pivots in rank order.  Text
                                  pivots behave as described at text_pivots.  Needs n_text_pivots <= the text tokens of a
                                  sample and n_pivot - n_text_pivots <= n_vis, else BAD_SHAPE. */
#define DART_PIVOTS_RANDOM 2   /* n_pivot distinct vision tokens drawn uniformly at random (Sec. 5.2): token j of sample b
                                  gets the upper 32 bits of output number (sample_base + b) * 2^32 + j of a SplitMix64
                                  generator seeded with `seed`; the smallest n_pivot tickets win, smallest first, equal
                                  tickets to the lower index.  The same seed gives the same pivots on every run. */

/* dart_opts.retention */
#define DART_RETAIN_AUTO 0   /* more samples than SMs: candidate bands; else the bands in one launch for up to 8 pivots
                                and sorted lists for more; where the chosen form's workspace or shared memory does not
                                fit: another one, else one kernel */
#define DART_RETAIN_SERIAL 1 /* one kernel, one CTA per sample: the pivots' selections one after the other */
#define DART_RETAIN_LISTS 2  /* two phases: sorted candidate lists for all (sample, pivot) pairs at once, then the pivots'
                                turns as walks over the lists; needs n_keep - n_pivot <= 4096, else the one-kernel form runs */
#define DART_RETAIN_BANDS 3  /* two phases: per (sample, pivot) pair one warp stores, unsorted, the lowest band of the
                                pivot's dups that holds at least the tokens the pivot could need; then the pivots' turns,
                                each taking its quota's smallest free entries of its band.  Needs n_keep - n_pivot <= 6144,
                                else as without it. */

#define DART_RETAIN_FUSED 4  /* the bands' two phases in one launch, one CTA per sample (a few warps build the sample's
                                bands, then the CTA takes the turns): for batches that cannot fill the GPU.  Same limits as
                                DART_RETAIN_BANDS, else as without it. */

/* dart_opts.rule */
#define DART_RULE_QUOTAS 0 /* one threshold per pivot: pivot i keeps its q_i not-yet-kept tokens of lowest dup (dart_reduce) */
#define DART_RULE_GLOBAL 1 /* one threshold for all pivots (Def. 2 / Eq. 8-9 with a common eps): a token's duplication is
                              its highest dup to any pivot; the n_keep - n_pivot non-pivot tokens of lowest duplication
                              are kept, ties to the lower index.  dbg->eps holds the threshold n_pivot times, dbg->owner the
                              pivot a kept token is most similar to (the first of equals). */

#define DART_RULE_UNION 2  /* independent pivots (Eq. 9-10 read literally: R = P u U_i R_i): pivot i keeps its q_i non-pivot
                              tokens of lowest dup whatever the other pivots keep; a token two pivots keep counts once, so
                              a sample keeps between n_pivot and n_keep vision tokens.  The outputs are then packed WITHOUT
                              padding, as variable-length attention kernels take them: out_hidden, out_idx and out_pos
                              are flat arrays with room for B * S_out rows, sample b's rows are
                              cu_seqlens[b] .. cu_seqlens[b + 1] - 1, and rows from cu_seqlens[B] on are not written.
                              Needs dart_opts.cu_seqlens.  dbg->owner names the first pivot in rank order that kept a
                              token. */

typedef struct dart_ctx dart_ctx; /* opaque: workspace, device status word, profiling events */

/* Maxima a context is sized for.  d is fixed per context (a multiple of 8). */
typedef struct {
    int32_t B_max;  /* samples per call */
    int32_t S_max;  /* sequence length (text + vision) */
    int32_t d;      /* row width of hidden and keys, in elements */
    int32_t P_max;  /* pivots */
    int32_t Kp_max; /* retained vision tokens */
    int32_t device; /* CUDA device ordinal */
    uint32_t flags; /* DART_FLAG_* */
} dart_desc;

/* Options of dart_reduce_ex.  A zeroed struct means the defaults of dart_reduce. */
typedef struct {
    int32_t norm_kind;     /* 0 or 1: L1 row norm (the paper's "K-norm", Sec. 3.3 footnote); 2: Euclidean norm */
    int32_t pivot_smallest; /* 0: pivots = largest scores (Table 1 caption); 1: smallest (ablation variant) */
    int32_t path;          /* DART_PATH_* */
    int32_t wait_limit;    /* 0: default (2 s); > 0: time limit in microseconds of every bounded device-side wait */
    int32_t sweep_lag;     /* 0: default; > 0: fused path, extra tasks between a row's two sweeps (tuning) */
    int32_t test_withhold_pivots; /* testing only: nonzero withholds one hand-over inside the kernel that waits (the persistent
                                     sweep never publishes a sample's pivots; the resident sweep's CTAs never count themselves in;
                                     the one-pass kernel's first pivot-norm warp never hands its norms over; the paired sweeps:
                                     1 = the lists are never counted in, 2 = the pivots' norms never reach the epilogue), so that
                                     the bounded waits expire and the call ends with DART_ERR_TIMEOUT in dart_status */
    int32_t retention;     /* DART_RETAIN_*: how step 4 is scheduled (same result either way) */
    int32_t rule;          /* DART_RULE_*: which tokens step 4 retains */
    int32_t cosine_on_hidden; /* 0: Eq. 7 on the key rows that are scored (one tensor for steps 1-3).  1: the pivots are still
                              ranked by the key rows' L1 scores, but dup(p_i, x_j) is the cosine of the HIDDEN rows (Def. 2
                              speaks of "tokens" without naming the tensor): the keys are read once for the scores, the
                              hidden states once for the similarities.  Needs norm_kind 0/1 (else UNSUPPORTED); no effect
                              when keys is NULL.  dbg->l1 then holds the key rows' scores, dbg->ssq the hidden rows' sums
                              of squares. */
    int32_t text_pivots;   /* with pivots_in: 1 lets an entry name ANY token of the sample (the paper also draws pivots from
                              the text tokens, Sec. 5.4).  Entries stay relative to the vision block, so a text token
                              before it has a negative index and one after it an index >= n_vis; the range is
                              [-vis_offset, S - vis_offset), entries distinct.  A text pivot takes its turn in step 4 like
                              any other but is no vision token: with Pv the pivots inside the vision block, step 4 uses
                              q = (n_keep - Pv) / P and r = (n_keep - Pv) % P (DART_RULE_GLOBAL: n_keep - Pv tokens beside
                              the pivots), and n_keep vision tokens are kept as always (DART_RULE_UNION: at most).
                              dbg->owner marks only the vision pivots.  Needs pivots_in (else UNSUPPORTED). */
    const int32_t *pivots_in; /* NULL: pivots by score (steps 1-2).  Else [B, n_pivot] int32, device: the caller's pivots
                              as vision-relative indices, distinct and in [0, n_vis); their order is the order of the
                              pivots' turns in step 4.  This covers the paper's other ways to choose pivots (Sec. 5.2:
                              random, attention score, value norm): the caller ranks, the library does steps 3-5.
                              Repeated or out-of-range indices end the call with DART_ERR_CHECK in dart_status. */
    int32_t *cu_seqlens;   /* DART_RULE_UNION only: [B + 1] int32, device, written by the call: cu_seqlens[0] = 0,
                              cu_seqlens[b + 1] = cu_seqlens[b] + packed length of sample b. */
    int32_t resident_split; /* DART_PATH_SPLIT: 0 = default (every second tile stays on the chip); k >= 2: the tiles with
                              index % k == 0 stay (a share of 1/k); -k: all other tiles stay (a share of 1 - 1/k) */
    int32_t pivot_source;  /* DART_PIVOTS_*: BY_SCORE (0) unless pivots_in is NULL and another source is wanted.  The other
                              sources run on the paths that take the caller's pivots (AUTO, STAGED, FUSED, TWO_PASS). */
    int32_t n_text_pivots; /* DART_PIVOTS_MIXED: how many of the n_pivot pivots are text tokens */
    uint64_t seed;         /* DART_PIVOTS_RANDOM */
    int32_t sample_base;   /* DART_PIVOTS_RANDOM: number of the call's first sample in the ticket stream (>= 0), so that a batch
                              split over several calls or GPUs draws what the whole batch would */
    int32_t tune;          /* 0 = defaults.  DART_PATH_PAIRED: 256 * n1 + 16 * n2 + n3 = depths of the three shared-memory rings.
                              DART_PATH_FUSED: >= 2 cuts the second pass of a row tile into eight column chunks (one task each)
                              and keeps the first pass within `tune` steps of the second (low 12 bits).  One-pass kernel:
                              bit 0x1000 = one row tile per task, bit 0x2000 = two where they fit (default: two when every
                              CTA gets at least two tasks).  All of them tuning options: same results. */
} dart_opts;

/* Optional per-step outputs of dart_reduce_ex; every member is a device pointer or NULL. */
typedef struct {
    float *l1;          /* [B, n_vis] sum_c |K[j,c]|                       (K-norm footnote)  */
    float *ssq;         /* [B, n_vis] sum_c K[j,c]^2                       (Eq. 7 denominators) */
    int32_t *pivot_idx; /* [B, n_pivot] vision-relative indices in rank order (Def. 1)        */
    float *sim;         /* [B, n_pivot, n_vis] dup(p_i, x_j)               (Eq. 7)             */
    float *eps;         /* [B, n_pivot] per-pivot threshold eps_i, NaN if the pivot's quota is 0 (Eq. 9) */
    uint8_t *keep;      /* [B, n_vis] 1 = retained                         (Eq. 10)            */
    int32_t *owner;     /* [B, n_vis] -1 dropped; i retained by pivot i; n_pivot + i pivot of rank i */
} dart_debug;

/*
 * Create a context for shapes up to the maxima in *desc on desc->device and allocate its
 * workspace with cudaMalloc (the only device allocations the library ever makes).
 * Errors: NULL, BAD_SHAPE (non-positive sizes, d % 8 != 0, P_max > Kp_max, Kp_max > S_max), CUDA, NOMEM.
 */
int dart_create(dart_ctx **out, const dart_desc *desc);

/* Free the workspace and the context.  Synchronises the device.  NULL is accepted. */
int dart_destroy(dart_ctx *ctx);

/* Batch size and sequence length of the following calls (1 <= B <= B_max, 1 <= S <= S_max). */
int dart_set_shape(dart_ctx *ctx, int B, int S);

/*
 * The reduction step (Sec. 3.3), for every sample b independently:
 *   1. score_j = L1 norm of keys[b, vis_offset + j, :]                       (K-norm footnote)
 *   2. pivots p_0..p_{P-1} = the n_pivot vision tokens of largest score, in rank order; equal
 *      scores rank the lower index first                                     (Def. 1, Table 1 caption)
 *   3. dup[i][j] = cosine of key rows p_i and j, fp32 accumulation           (Def. 2, Eq. 7)
 *   4. kept = pivots; with q = (n_keep - P) / P and r = (n_keep - P) % P, pivot i in rank order keeps
 *      its q (+1 if i < r) not-yet-kept tokens of lowest dup[i][.], ties to the lower index; eps_i
 *      is the largest dup it kept                                            (Eq. 9-10)
 *   5. out_idx[b] = ascending sequence indices of all text rows and the kept vision rows;
 *      out_hidden[b, t, :] = hidden[b, out_idx[b, t], :]; out_pos[b, t] = out_idx[b, t].
 *
 *   hidden     [B, S, d] bf16, device, 16-byte aligned, read-only
 *   keys       [B, S, d] bf16, device, or NULL to score and compare the hidden states themselves
 *   out_hidden [B, S_out, d] bf16, device, 16-byte aligned, must not overlap hidden or keys
 *   out_idx    [B, S_out] int32, device
 *   out_pos    [B, S_out] int64, device
 *   stream     a cudaStream_t (NULL = the legacy default stream)
 * Shape rules: 1 <= n_pivot <= n_keep <= n_vis, 0 <= vis_offset, vis_offset + n_vis <= S,
 * n_pivot <= P_max, n_keep <= Kp_max.  n_keep == n_vis is the identity.  Inputs must be finite.
 * Errors: NULL, BAD_SHAPE, ALIGN, ALIAS, CUDA (launch failure).  Asynchronous: dart_status.
 */
int dart_reduce(dart_ctx *ctx, const void *hidden, const void *keys, int vis_offset, int n_vis,
                int n_pivot, int n_keep, void *out_hidden, int32_t *out_idx, int64_t *out_pos,
                void *stream);

/*
 * dart_reduce with caller position ids, options and per-step outputs.
 *   pos_in [B, S] int64 device, or NULL for pos_in[b, s] = s; out_pos[b, t] = pos_in[b, out_idx[b, t]]
 *   opts   NULL = defaults;  dbg NULL = no per-step outputs.
 * Asking for dbg->sim makes every path materialise the whole similarity matrix.
 */
int dart_reduce_ex(dart_ctx *ctx, const void *hidden, const void *keys, const int64_t *pos_in,
                   int vis_offset, int n_vis, int n_pivot, int n_keep, void *out_hidden,
                   int32_t *out_idx, int64_t *out_pos, const dart_opts *opts, const dart_debug *dbg,
                   void *stream);

/*
 * The same step for HOST buffers: copies hidden and keys to the device in chunks of samples,
 * reduces each chunk while the next one is in flight, copies the packed outputs back and returns
 * after everything has completed.  All pointers are host memory (pinned memory makes the copies
 * asynchronous); keys may be NULL.  Needs a context created with DART_FLAG_HOST_STAGING
 * (else UNSUPPORTED).  The shape of the call is the one set by dart_set_shape; B may exceed the
 * chunk size but not B_max.  Since the call waits for its own work it also reads (and clears) the
 * device status word: a bounded wait that gave up or a failed self-check is returned as
 * DART_ERR_TIMEOUT / DART_ERR_CHECK and the host outputs are then not valid.
 */
int dart_reduce_host(dart_ctx *ctx, const void *hidden, const void *keys, int vis_offset, int n_vis,
                     int n_pivot, int n_keep, void *out_hidden, int32_t *out_idx, int64_t *out_pos);

/*
 * Row gather by a packed index list, without a context: out[b, t, :] = src[b, idx[b, t], :].  With idx = the
 * out_idx of a reduction this packs any other per-token tensor the same way as out_hidden: the key and value
 * rows of the layers already run (the paper counts the KV cache of the retained tokens only, Table 2), or the
 * hidden states of a second stream.
 *   src  [B, S, row_bytes] device, 16-byte aligned;  idx [B, S_out] int32 device, every entry in [0, S)
 *   out  [B, S_out, row_bytes] device, 16-byte aligned, must not overlap src
 *   row_bytes a multiple of 16;  device: CUDA device ordinal of the pointers;  stream: a cudaStream_t
 * Allocates nothing and does not synchronise.  Errors: NULL, BAD_SHAPE, ALIGN, ALIAS, CUDA.  Entries of idx are
 * not checked on the device.
 */
int dart_gather_rows(const void *src, const int32_t *idx, int B, int S, int S_out, int row_bytes, void *out,
                     int device, void *stream);

/*
 * Read the device status word (synchronises the context's device): DART_OK, DART_ERR_TIMEOUT if a
 * bounded wait inside a kernel gave up, DART_ERR_CHECK if a self-check failed.  Reading clears it.
 */
int dart_status(dart_ctx *ctx);

/*
 * Where the last non-zero status came from (as read by the last dart_status call that returned an error):
 * detail[0] = which bounded wait of the fused kernel expired (1 pivots not published, 2 ring stage not freed,
 * 3 drain, 4 accumulator not freed, 5/6 tile not loaded (MMA / row sums), 7 accumulator not filled, 8/9 mailbox,
 * 10 sweep-1 tasks not all counted, 11/12 selection queue, 13 first pass held back; 40-55 the paired sweeps' waits (44 a
 * sample's lists not all counted in, 50 its pivots not published, 51 their norms not handed over, ...); 64-70 the one-pass
 * kernel's waits (stage not freed, tile not loaded (MMA / norms), accumulator not freed / not filled, norms not taken /
 * not ready); 80-86 the resident sweep's waits (83 = a sample's candidates not all published); 100 = a failed check of
 * opts->pivots_in),
 * detail[1] = index of the step in the kernel's schedule (or the sample), detail[2] = CTA; for wait 1 also
 * detail[3] = sample.  For bug reports.
 */
int dart_status_detail(const dart_ctx *ctx, int32_t detail[11]);

/* The cudaError_t of the last failed CUDA call made on behalf of this context (0 if none). */
int dart_last_cuda_error(const dart_ctx *ctx);

/* Bytes of device memory the context holds. */
size_t dart_workspace_bytes(const dart_ctx *ctx);

/* Kernels launched on behalf of this context since it was created. */
int64_t dart_launch_count(const dart_ctx *ctx);

/*
 * Per-kernel timing.  While enabled, every kernel launch of dart_reduce* is bracketed by CUDA events
 * on the caller's stream.  dart_profile_read synchronises those events and returns, for each kernel
 * slot k < *n_slots, the accumulated milliseconds and launch count since the last read; names[k]
 * (if names != NULL) points to a static string.  On entry *n_slots is the capacity of the arrays.
 */
int dart_profile_enable(dart_ctx *ctx, int on);
int dart_profile_read(dart_ctx *ctx, float *ms, int32_t *launches, const char **names, int *n_slots);

/*
 * Pivot selection without any allocation (the paper has no counterpart of this entry point; it
 * exists for deployment, not for the method).
 *
 * Some hosts of this library cannot call cudaMalloc when the step runs: serving engines that hand
 * the whole HBM to their own pool at start-up (a later cudaMalloc simply fails), and latency-bound
 * loops that cannot afford cudaMalloc's device-wide synchronisation.  dart_create allocates, so a
 * context is out of reach for them.  This call needs no context: it computes steps 1-2 of
 * dart_reduce (row scores, then the n_pivot best vision tokens per sample in rank order, L1 score,
 * largest first, ties to the lower index) and keeps the per-row scores, its only scratch, in a
 * fixed array that is part of the library image: DART_STATIC_MAX_ROWS rows, 2 MiB, resident on
 * every GPU that loads the library until the process exits.
 *
 *   keys       [B, S, d] bf16, device, 16-byte aligned, read-only
 *   pivot_idx  [B, n_pivot] int32, device: vision-relative indices, rank 0 first (the output)
 *   device     CUDA device ordinal the pointers belong to;  stream: a cudaStream_t on that device
 * Limits: B * n_vis <= DART_STATIC_MAX_ROWS and n_pivot <= 1024, else DART_ERR_BAD_SHAPE; d % 8 == 0;
 * 1 <= n_pivot <= n_vis; vis_offset + n_vis <= S.
 * The first call on a device looks up the array's device address; make that call before any stream
 * capture begins.  The look-up itself allocates nothing, but the CUDA runtime loads a library's
 * image into device memory lazily (the default since CUDA 12.2): the kernels and the 2 MiB array
 * are placed on the device by that first call, or when the library is loaded if
 * CUDA_MODULE_LOADING=EAGER is set.  A host that gives all free memory to its own pool must
 * therefore make one call (any valid small call will do) BEFORE it sizes the pool; a first call
 * that finds no memory left returns DART_ERR_NOMEM.  Every call on a device uses the same array and leaves its
 * scores there: nothing in it has to start at zero (each call overwrites the rows it reads), but
 * two calls whose kernels overlap on the GPU, from different streams or threads, race on it.
 * Calls cudaMalloc, cudaFree or an allocating routine never.  Errors: NULL, BAD_SHAPE, ALIGN, NOMEM, CUDA.
 */
#define DART_STATIC_MAX_ROWS 262144
int dart_pivots_static(const void *keys, int B, int S, int d, int vis_offset, int n_vis, int n_pivot,
                       int32_t *pivot_idx, int device, void *stream);

const char *dart_strerror(int code);
int dart_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DART_H */
