/*
 * libams — the periodic Adaptive Mass-Segmented (AMS) KV-compression step on a
 * paged bf16 KV cache, for NVIDIA B200 (sm_100a).  C ABI: plain pointers and
 * sizes only.  Every pointer marked DEVICE is device memory owned by the caller;
 * the library allocates and frees no device memory.  `stream` arguments are
 * `cudaStream_t` values passed as `void*`.
 *
 * One call of ams_compress performs, for every layer, sequence and KV head,
 * Algorithm 1 of the paper followed by the paged head-wise compaction of its
 * serving appendix:
 *   1. score every cached token (TOVA-style observation-window softmax averaged
 *      over the GQA group — Section 3.2 and Algorithm 1 step 1 — a key-only
 *      KeyDiff-style score, or the expected-attention score of ams_set_query_stats);
 *   2. turn usage into the normalised quality mass (Eq. 1), mix it with the EMA
 *      credit carried across events (Section 3.3, "EMA credit"; Algorithm 1 step 2);
 *   3. prefix-sum the mass, cut at multiples of the segment mass, merge short and
 *      split long segments (Section 3.3, "Mass-based adaptive segmentation";
 *      Algorithm 1 step 3);
 *   4. give each segment its quota of the budget (Section 3.3, "Segment-wise quota
 *      allocation"; Algorithm 1 step 4);
 *   5. keep the top-q_i tokens of each segment, the must-keep prefix/suffix, and
 *      backfill to exactly `budget` positions (Algorithm 1 step 5);
 *   6. move the kept K/V rows of every head into replacement pages and rewrite the
 *      block-table row and the sequence length (the two display equations and the
 *      runtime routine of the paged-KV appendix).
 *
 * Layouts (all contiguous, row-major):
 *   k_pages, v_pages : bf16  [n_layers][num_pages][16][n_kv_heads][128]
 *   block_table      : int32 [batch][block_table_stride]  page ids shared by all layers and heads
 *   seq_lens         : int32 [batch]
 *   obs_queries      : bf16  [n_layers][batch][n_q_heads][window][128]; window query j is the
 *                      decode query at position seq_len - window + j
 *   ema_state        : fp32  [n_layers][max_batch][n_kv_heads][max_seq_len]  credit per cached row
 *   dst_pages        : int32 [batch][ceil(budget/16)]  free pages that receive the kept rows
 *   per-unit views   : [n_layers][batch][n_kv_heads][...]
 *
 * Decisions (cut positions, quotas, kept indices) are taken in integer arithmetic
 * on fixed-point images of the mass, so they do not depend on summation order.
 *
 * Scorer selection is automatic (query rows per KV head >= 64: tensor-core path, otherwise the
 * mma.sync path) and depends on the arguments only: no environment variable changes what runs.
 *
 * Errors: every function returns AMS_OK (0) or a negative code.  Calls are
 * asynchronous on `stream`; conditions found on the device are reported by
 * ams_get_status.  The first kernel of an event checks every sequence: one longer
 * than max_seq_len (AMS_ERR_CAPACITY), one shorter than the observation window, or
 * one whose block-table row or replacement pages name a page outside [0, num_pages)
 * (AMS_ERR_INVALID_ARG, detail = sequence, index in the row, page id) is skipped
 * entirely: its pages, table row, length and credit stay as they were.  A bounded
 * wait that ran out is AMS_ERR_TIMEOUT.  The library serves any number of devices
 * per process (launch state is kept per device); a handle belongs to the device that
 * was current when it was created.
 */
#ifndef AMS_H_
#define AMS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    AMS_OK = 0,
    AMS_ERR_INVALID_ARG = -1, /* null pointer, size out of range, budget < 1, ...            */
    AMS_ERR_UNSUPPORTED = -2, /* head_dim != 128, page_size != 16, n_q_heads % n_kv_heads    */
    AMS_ERR_CAPACITY = -3,    /* workspace too small, or a device-side capacity was exceeded  */
    AMS_ERR_CUDA = -4,        /* a CUDA runtime call or launch failed                         */
    AMS_ERR_TIMEOUT = -5,     /* a bounded device-side wait expired                           */
    AMS_ERR_INTERNAL = -6     /* a device-side consistency check failed                       */
};

enum { AMS_SCORER_TOVA = 0, AMS_SCORER_KEYDIFF = 1, AMS_SCORER_EXTERNAL = 2, AMS_SCORER_EXPECTED = 3 };

typedef struct ams_state ams_state; /* opaque host handle */

typedef struct {
    int32_t n_layers, n_q_heads, n_kv_heads; /* GQA group = n_q_heads / n_kv_heads           */
    int32_t head_dim;                        /* must be 128                                   */
    int32_t page_size;                       /* must be 16                                    */
    int32_t max_batch;                       /* capacity: sequences per call                  */
    int32_t max_seq_len;                     /* capacity: tokens per sequence, <= 131072      */
    int32_t max_window;                      /* capacity: observation queries                 */
    int32_t max_budget;                      /* capacity: tokens kept per head                */
    int32_t max_segments;                    /* capacity: n_segments                          */
    int32_t l_min, l_max;                    /* segment length bounds; l_max = 0: no split    */
    int32_t q_min;                           /* guaranteed quota per segment                  */
    int32_t n_sink, n_last;                  /* must-keep prefix / suffix                     */
    float ema_lambda;                        /* credit decay, in [0, 1)                       */
    float ema_beta;                          /* weight of the current mass; 1 = credit unused */
    float eps;                               /* Eq. 1 epsilon, > 0                            */
    int32_t causal_window;                   /* 1: window query j sees tokens <= T - W + j    */
    int32_t pool_kernel;                     /* odd, 1..63: width of the average pooling applied
                                                to the usage scores before Eq. 1 (Algorithm 1
                                                step 1, optional smoothing); 1 = none         */
    int32_t decoupled;                       /* 1: reserve room for a mass signal that differs
                                                from the base scores (see ams_compress)       */
    int32_t fixed_segments;                  /* 1: component ablation "fixed-length segments":
                                                cut k at floor(k seq_len / S) instead of at the
                                                mass quantile; merge and split as usual       */
    int32_t uniform_quotas;                  /* 1: component ablation "w/o mass-weighted quotas":
                                                the budget is shared by segment length        */
    int32_t expected_scorer;                 /* 1: reserve room for AMS_SCORER_EXPECTED (one fp32
                                                logit per query head and cached token)        */
} ams_config;

/* Optional device outputs for inspection and tests; any member may be NULL.
 * T = max_seq_len, C = ams_segment_capacity(cfg).  Units that were skipped
 * (seq_len <= budget) are left untouched. */
typedef struct {
    float *scores;       /* [L][batch][H][T]   base scores g                                */
    float *usage;        /* [L][batch][H][T]   usage u the mass is built from (after smoothing;
                                               equals g unless smoothed or decoupled)       */
    float *mass;         /* [L][batch][H][T]   Eq. 1 mass of the current event              */
    int32_t *n_segments; /* [L][batch][H]      segments after merge and split               */
    int32_t *seg_bounds; /* [L][batch][H][C+1] boundaries a_0 = 0 < ... < a_n = seq_len     */
    int32_t *quotas;     /* [L][batch][H][C]                                                 */
    int32_t *keep_idx;   /* [L][batch][H][budget] kept positions, ascending                 */
    /* Diagnostic of the paper's mechanistic-diagnostics appendix: retained-set IoU between the previous
     * event and this one.  prev_kept (input, DEVICE int32 [batch], may be NULL) gives, per sequence, how
     * many tokens at the front of the cache are the retained set of the previous event (the previous
     * budget; 0 for a sequence never compressed).  With both pointers set, retained_iou receives
     * |R_prev & R_now| / |R_prev | R_now| per unit, R_now being this event's kept tokens. */
    const int32_t *prev_kept;
    float *retained_iou; /* [L][batch][H] */
} ams_debug_views;

/* Paper defaults: segment mass 0.1 (n_segments = 10 is passed per call), lengths
 * 16 / 256, q_min 1, lambda = beta = 0.9, 4 sinks; n_last 16, eps 1e-8; pool_kernel 1 (no
 * smoothing), decoupled 0, both ablation switches 0.  Geometry and capacities are zeroed and must be filled by the caller. */
void ams_config_default(ams_config *cfg);

/* Sizes of the caller-allocated device buffers; 0 if the configuration is invalid. */
size_t ams_ema_state_bytes(const ams_config *cfg);
size_t ams_workspace_bytes(const ams_config *cfg);
/* Per-unit capacity C of the segment views: max_segments + 2*floor(max_seq_len/l_max) + 4. */
int32_t ams_segment_capacity(const ams_config *cfg);

/* Creates the host handle, zero-fills ema_state (DEVICE, ams_ema_state_bytes) on
 * `stream`, and adopts `workspace` (DEVICE, >= ams_workspace_bytes, 256-byte
 * aligned) as scratch for later calls.  Both buffers must outlive the handle. */
int ams_init_state(const ams_config *cfg, void *ema_state, void *workspace, size_t workspace_bytes,
                   void *stream, ams_state **out);

/* One compression event (see the file header).  All pointers DEVICE.
 *  k_pages, v_pages : read at the pages named by block_table, written at the pages named by
 *                     dst_pages (which must not overlap the live pages); nothing else is touched.
 *  num_pages        : pages per layer of the pool.
 *  block_table, seq_lens : updated in place for every sequence with seq_len > budget:
 *                     row <- dst_pages row followed by -1, length <- budget.  Sequences with
 *                     seq_len <= budget are left as they are (nothing to evict).
 *  obs_queries, window : may be NULL / 0 for AMS_SCORER_KEYDIFF, AMS_SCORER_EXPECTED and AMS_SCORER_EXTERNAL.
 *  ema_state        : the buffer given to ams_init_state (or a restored copy of it).
 *  n_segments       : S, the number of mass quantiles (segment mass 1/S), 1..max_segments.
 *  ext_scores       : AMS_SCORER_EXTERNAL only: fp32 [L][batch][H][max_seq_len] (16-byte aligned) base
 *                     scores g; also the usage u unless ext_usage is given.
 *  ext_usage        : AMS_SCORER_EXTERNAL only, optional (NULL: u = g): fp32, same shape and alignment,
 *                     the usage u.
 * Mass signal (Algorithm 1 step 1; the runtime section's "decoupled mass and selection scores"):
 * the mass is built from the usage u, tokens inside a segment are ranked by the base score g.
 * By default u = g = the scorer's output.  With cfg.decoupled = 1, AMS_SCORER_KEYDIFF or
 * AMS_SCORER_EXPECTED and observation queries given (obs_queries != NULL, window >= 1), u is the
 * window attention of AMS_SCORER_TOVA and g the scorer's own score.  cfg.pool_kernel = k > 1 replaces u (never g) by its
 * zero-padded average over k neighbouring positions: u'_t = (sum of u_j, |j - t| <= k/2, j inside
 * the sequence, added left to right in fp32) / k.
 *  dbg              : optional views, or NULL.
 * Calls on the same handle share the workspace and must not overlap on the GPU.  The call allocates
 * nothing and never synchronises; after one direct call (which sets kernel attributes) it can be captured
 * into a CUDA graph.  Its kernels follow one another on `stream` as dependent launches (a kernel may start
 * while its predecessor's last blocks run and waits before touching that kernel's output); work enqueued
 * on `stream` before or after the call is ordered as usual. */
int ams_compress(ams_state *st, void *k_pages, void *v_pages, int64_t num_pages, int32_t *block_table,
                 int32_t block_table_stride, int32_t *seq_lens, int32_t batch, const void *obs_queries,
                 int32_t window, void *ema_state, int32_t budget, int32_t n_segments, int32_t scorer_id,
                 const int32_t *dst_pages, const float *ext_scores, const float *ext_usage,
                 const ams_debug_views *dbg, void *stream);

/* Query statistics for AMS_SCORER_EXPECTED, the expected-attention scorer behind the paper's
 * "AMS-Expected" rows (experimental-setup section and the baseline table of the appendix name it and
 * its regularisation coefficient 1e-2; the formula is the closed form of the work they cite, for
 * queries modelled as Gaussian).  For query head r of a KV head's group and cached token t:
 *     l_{r,t} = mu_r . k_t / sqrt(128) + k_t^T Sigma_r k_t / (2 * 128)
 *     score_t = (mean over r of softmax_t(l_{r,.}) + score_eps) * |v_t|_2
 *   q_mean : DEVICE fp32 [n_layers][batch][n_q_heads][128], 16-byte aligned
 *   q_cov  : DEVICE bf16 [n_layers][batch][n_q_heads][128][128] (row-major; only the symmetric part matters),
 *            16-byte aligned
 * `batch` is that of the ams_compress calls that follow.  The pointers are kept in the handle and read by
 * every later ams_compress with AMS_SCORER_EXPECTED (the buffers stay the caller's and must stay valid);
 * estimating them from the model's recent queries is the caller's job.  cfg.expected_scorer must be 1.
 * With cfg.decoupled = 1 and observation queries given, the mass comes from the window attention and
 * this score ranks the tokens inside the segments (the runtime section's "decoupled mass and selection
 * scores, including TOVA-style and expected-attention selection"). */
int ams_set_query_stats(ams_state *st, const float *q_mean, const void *q_cov, float score_eps);

/* Synchronises `stream`, then returns and clears the device status: AMS_OK or the
 * first device-side error.  detail[0..3] (host, may be NULL) receive the code, the
 * unit index and two values describing it. */
int ams_get_status(ams_state *st, void *stream, int32_t *detail);

/* Failure-handling check without a failure: enqueues a one-thread kernel that waits on a barrier
 * nobody arrives at, gives up after `polls` polls (1 .. 2^20) and records AMS_ERR_TIMEOUT in the
 * handle's status word, the way the bounded waits inside the tensor-core scorer do when they run
 * out.  The next ams_get_status returns that code; nothing else is touched. */
int ams_debug_expire_wait(ams_state *st, uint32_t polls, void *stream);

/* Number of kernels the last ams_compress on this handle launched. */
int32_t ams_last_launch_count(const ams_state *st);

/* Optional per-kernel timing.  With profiling enabled, ams_compress records a CUDA
 * event on its stream after every kernel it launches (events are host objects; no
 * device memory is allocated).  ams_get_kernel_times waits for the last call's final
 * event and writes AMS_KERNEL_SLOTS durations in milliseconds, one per kernel slot
 * named by ams_kernel_name (a slot launched more than once holds the sum). */
#define AMS_KERNEL_SLOTS 10
int ams_set_profiling(ams_state *st, int enable);
int ams_get_kernel_times(ams_state *st, float *ms);
const char *ams_kernel_name(int32_t idx);

/* Selection without any allocation (the paper has no counterpart: this is an interface
 * convenience, not a step of the method).  For callers that cannot obtain device memory:
 * code that runs while a stream is being captured, plug-ins inside a process whose device
 * memory pool belongs to the host framework, paths that must not touch the allocator.
 * Runs steps 1-5 of Algorithm 1 (mass, cuts, merge/split, quotas, per-segment top-k,
 * must-keep, backfill) on caller-supplied scores and writes the kept positions; there is
 * no EMA credit (the mass is that of the given scores alone), no K/V movement, no handle
 * and no workspace argument.  The scratch is a fixed device array inside the library
 * (about 2.4 MB, held by every GPU that loads the library until the process exits).
 *   scores   : DEVICE fp32 [n_units][score_stride], score_stride a multiple of 16, >= seq_len
 *   keep_idx : DEVICE int32 [n_units][budget], ascending positions
 *   cfg      : only l_min, l_max, q_min, n_sink, n_last and eps are read
 * Limits: n_units <= 8, seq_len <= 32768, n_segments + 2*floor(seq_len/l_max) + 4 <= 1024;
 * beyond them AMS_ERR_CAPACITY is returned and nothing is launched.  1 <= budget < seq_len.
 * The first call on a device looks up the array's address on that device (with that device
 * current); make that first call before starting a stream capture.  All calls share the one
 * array, which keeps the previous call's contents: the entry point re-initialises what must
 * start at zero, but two calls that overlap on the GPU (different streams, or a captured
 * graph replayed concurrently) race on it.  Asynchronous on `stream`. */
int ams_select_static(const ams_config *cfg, const float *scores, int32_t score_stride, int32_t n_units,
                      int32_t seq_len, int32_t budget, int32_t n_segments, int32_t *keep_idx, void *stream);

/* Status of the ams_select_static calls on the current device: synchronises `stream`, returns and
 * clears the first condition their kernels found on the device (AMS_ERR_CAPACITY: more segments
 * than the fixed array holds; AMS_ERR_INTERNAL: a kept-count check failed), AMS_OK otherwise.  A unit
 * that reported leaves its keep_idx row as the caller passed it.  detail[0..3] (host, may be NULL)
 * as in ams_get_status.  Allocates nothing (the paper has no counterpart). */
int ams_select_static_status(int32_t *detail, void *stream);

/* Releases the host handle only. */
int ams_free(ams_state *st);

const char *ams_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* AMS_H_ */
