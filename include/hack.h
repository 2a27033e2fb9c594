/*
 * hack.h - C ABI of the B200 (sm_100a) library for the per-scale decoding step of head-aware
 * KV-cache compression in next-scale visual autoregressive transformers.
 *
 * One "step" serves one (layer, scale): the new scale's keys/values join the cache (Eq. 3), every
 * candidate key of a head whose cache would exceed its budget is scored with a small query subset
 * (Eq. 9), a budgeted subset is selected per head with the contextual rule (Eq. 10) or the
 * structural rule (Eq. 11) under asymmetric budgets (Eq. 7-8), the survivors are compacted into a
 * ragged per-head cache, and the scale's queries attend over it (Eq. 4 on the compressed cache,
 * compression preceding attention, section "Asymmetric Head Budget Allocation").
 *
 * Conventions for every entry point
 *  - Q, K, V, O are CALLER-OWNED DEVICE buffers, dense row-major [batch, n_heads, N_k, head_dim]
 *    in the cache's dtype, 16-byte aligned, N_k = side_k^2 of the scale being decoded.  Only the
 *    *_host entry point takes host pointers.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls only
 *    enqueue work and return; nothing synchronises unless stated.
 *  - Layers and scales are 0-based.  Each layer walks its scales in order 0,1,2,...; a call for
 *    any other scale returns HACK_ERR_STATE.  Within a scale a layer is served either by
 *    hack_scale_step, or by [hack_score, hack_select,] hack_compact, hack_attend in that order.
 *  - Stored lengths are a function of the schedule, the budgets and the head type only (the
 *    selection decides WHICH entries survive, never HOW MANY), so the library keeps them on the
 *    host and never reads anything back from the device to plan a launch.
 *  - Candidate index j of a head in a step: j < L addresses the L entries stored before the step
 *    (ascending original position), j >= L the new scale's token j - L.
 *  - Argument errors are detected on the host before anything is launched and leave the cache
 *    unchanged.  Nothing traps on the device.  There is no CPU fallback.
 *  - The cache (K/V planes, position plane, scratch) is owned by the library and released by
 *    hack_free_cache.  A cache is not thread safe; use one cache per stream of work.
 */
#ifndef HACK_H_
#define HACK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define HACK_API __attribute__((visibility("default")))
#else
#define HACK_API
#endif

typedef struct hack_cache hack_cache_t; /* opaque, library-owned */

typedef enum {
  HACK_OK = 0,
  HACK_ERR_INVALID_ARG = 1, /* NULL pointer, size or index out of range, misaligned buffer */
  HACK_ERR_UNSUPPORTED = 2, /* head_dim / dtype / n_obs outside what the kernels implement */
  HACK_ERR_OOM = 3,         /* device or host allocation failed */
  HACK_ERR_CUDA = 4,        /* a CUDA call failed; hack_last_error() has the text */
  HACK_ERR_STATE = 5,       /* call out of order for this layer (wrong scale or phase) */
  HACK_ERR_TIMEOUT = 6      /* a bounded device-side wait expired (reported by hack_poll_status) */
} hack_status_t;

typedef enum { HACK_F32 = 0, HACK_BF16 = 1 } hack_dtype_t;

/* Overflow rule for structural heads when B_S < N_init + N_k (the paper is silent): */
enum { HACK_OVERFLOW_KEEP_PROTECTED = 0, /* keep every protected entry, exceed B_S */
       HACK_OVERFLOW_COMPETE = 1 };      /* protect only the initial scales; keep exactly B_S */

/* Which n = min(N_obs, N_k) queries of the current scale form the subset Q~ of Eq. 9.  The method
 * uses uniform spacing; the others are the alternatives of the paper's query-subset ablation. */
enum { HACK_OBS_UNIFORM = 0, /* floor(m * N_k / n), m = 0..n-1 */
       HACK_OBS_INIT = 1,    /* the first n tokens of the scale */
       HACK_OBS_RECENT = 2,  /* the last n tokens of the scale */
       HACK_OBS_CALLER = 3,  /* rows given per scale with hack_set_obs_rows (random sampling: the
                                caller draws them) */
       HACK_OBS_FULL = 4 };  /* every query of the scale, whatever n_obs: the ablation's full-attention
                                reference; costs ceil(N_k / 32) scoring rounds per step */

typedef struct {
  int32_t n_layers, n_heads, head_dim, batch; /* head_dim in {64, 128} */
  int32_t n_scales;
  const int32_t* scale_sides;        /* host, [n_scales], copied at init; N_k = side^2 */
  int32_t dtype;                     /* hack_dtype_t of Q/K/V/O and of the cache */
  const uint8_t* head_is_contextual; /* host, [n_layers*n_heads], 1 = contextual, 0 = structural
                                        (offline classification, Eq. 6); copied at init */
  int32_t budget_c, budget_s;        /* B_C, B_S: entries per head, >= 1 (Eq. 7-8) */
  int32_t n_obs;                     /* query subset size N_obs, 1..32 (Eq. 9; paper uses 32) */
  int32_t n_init_scales;             /* leading scales always kept in structural heads (paper: 2) */
  float sm_scale;                    /* softmax scale; 0 selects 1/sqrt(head_dim) */
  int32_t overflow_policy;           /* HACK_OVERFLOW_* */
  int32_t device;                    /* CUDA device ordinal */
  int32_t obs_sampler;               /* HACK_OBS_*; 0 = the method's uniform rule */
  int32_t merge_last;                /* 1: at the last scale, contextual heads fold the entries that step
                                        discards into their nearest retained counterparts (the merge
                                        described after Eq. 10; see hack_compact).  bf16 caches only. */
} hack_config_t;

/* Host-side plan of one step of one layer (all lengths in entries per head). */
typedef struct {
  int32_t n_new;                 /* N_k */
  int32_t stored_c, stored_s;    /* L before the step, contextual / structural heads */
  int32_t cand_c, cand_s;        /* T' = L + N_k */
  int32_t kept_c, kept_s;        /* length after the step */
  int32_t triggered_c, triggered_s; /* 1 if T' exceeds the type's budget (strictly) */
  int32_t n_obs_rows;            /* min(N_obs, N_k) */
} hack_step_info_t;

/* Buffer strides a caller of the separate stage calls must use. */
typedef struct {
  int32_t cand_stride; /* floats per (batch, head) row of `scores`: max T' over all steps */
  int32_t kept_stride; /* int32 per (batch, head) row of `idx`: max kept length over all steps */
  int32_t max_new;     /* largest N_k */
} hack_limits_t;

/* Eq. 7, B = alpha*B_C + (1-alpha)*B_S, solved under one of the paper's two allocation rules
 * (appendix, "Model-Specific Configurations").  Host only, no device work.
 *   rule 0 ("fraction"): B_C = floor(param*T_K); B_S = floor((B - alpha*B_C)/(1-alpha)).
 *   rule 1 ("ratio"):    B_C : B_S = 1 : param; B_C = floor(B/(alpha+param*(1-alpha))), B_S = param*B_C.
 * B_S is clamped to T_K and both results are at least 1.  INVALID_ARG unless 0 < alpha < 1. */
HACK_API hack_status_t hack_split_budget(int32_t budget, double alpha, int32_t rule, double param,
                                int32_t total_tokens, int32_t* budget_c, int32_t* budget_s);

/* Allocate the ragged per-head cache for the whole stack (Eq. 5, 8: per head at most its type's
 * budget, or the protected set if that is larger) and all scratch.  *out is set only on
 * success.  Capacity per head = the largest stored length its type reaches over the schedule. */
HACK_API hack_status_t hack_init_cache(const hack_config_t* cfg, hack_cache_t** out);
/* Release everything; synchronises the device first.  NULL is accepted. */
HACK_API hack_status_t hack_free_cache(hack_cache_t* cache);
/* HACK_OBS_CALLER only: the query rows that form Q~ (Eq. 9) at `scale`, for every layer, batch
 * element and head.  rows: host, n = min(N_obs, N_k) distinct indices in [0, N_k), used in the
 * order given (the scores do not depend on the order).  Copied to the device synchronously: a
 * set-up call, made before the steps of that scale are enqueued; the rows stay in force across
 * hack_reset.  A step that has to score while its scale has no rows fails with HACK_ERR_STATE.
 * INVALID_ARG for a wrong n, an index out of range or a repeated index; STATE if the cache was
 * not created with HACK_OBS_CALLER. */
HACK_API hack_status_t hack_set_obs_rows(hack_cache_t* cache, int32_t scale, const int32_t* rows, int32_t n);
/* New image: all layers back to scale 0 with empty caches.  Enqueues nothing. */
HACK_API hack_status_t hack_reset(hack_cache_t* cache);

HACK_API hack_status_t hack_get_limits(const hack_cache_t* cache, hack_limits_t* out);
/* Plan of step (layer, scale) given the layer's current state; scale must be the layer's next. */
HACK_API hack_status_t hack_step_info(const hack_cache_t* cache, int32_t layer, int32_t scale,
                             hack_step_info_t* out);

/* Subset-attention importance (Eq. 9 and the TOPK argument of Eq. 10-11).  For every (b,h) whose
 * type is triggered in this step: scores[(b*H+h)*cand_stride + j] = sum over the
 * min(N_obs, N_k) uniformly spaced query rows i = floor(m*N_k/n) of
 * Softmax_j(sm_scale * <Q[i], K_cand[j]>) over all T' candidates (stored ++ k_new).  Rows of
 * heads that are not triggered are left untouched.  Does not change the cache. */
HACK_API hack_status_t hack_score(hack_cache_t* cache, int32_t layer, int32_t scale, const void* q,
                         const void* k_new, float* scores, void* stream);

/* Budgeted selection per head from fp32 `scores` (layout as above).  Contextual heads keep the
 * B_C best candidates (Eq. 10).  Structural heads keep every entry of the first n_init_scales
 * scales and of the scale being decoded and fill the remaining M = B_S - |protected| slots with
 * the best of the rest (Eq. 11).  Order: score descending on the fp32 bit pattern, ties to the
 * lower candidate index.  Heads that are not triggered keep everything.  Output
 * idx[(b*H+h)*kept_stride + r], r < kept, ascending candidate indices; kept_out[b*H+h] their
 * count (may be NULL).  Does not change the cache. */
HACK_API hack_status_t hack_select(hack_cache_t* cache, int32_t layer, int32_t scale, const float* scores,
                          int32_t* idx, int32_t* kept_out, void* stream);

/* Gather the surviving K/V rows (Eq. 10-11) into the layer's ragged cache in ascending original
 * position; evicted entries are gone for good.  `idx` as written by hack_select for this step;
 * each head's row must hold exactly hack_step_info's kept_c / kept_s entries.  In place.
 * With merge_last, at the last scale, a contextual head that evicts then folds every discarded
 * entry e into the retained entry c whose key has the largest cosine similarity to k_e (lowest
 * index among equals) with weight w_e = max(similarity, 0):
 *   k_c <- (k_c + sum w_e k_e) / (1 + sum w_e), v_c likewise, rounded to bf16
 * (the paper states the operation in one sentence; measure, weights and the treatment of V are this
 * library's reading).  hack_scale_step does the same. */
HACK_API hack_status_t hack_compact(hack_cache_t* cache, int32_t layer, int32_t scale, const int32_t* idx,
                           const void* k_new, const void* v_new, void* stream);

/* O = Softmax(sm_scale * Q K^T) V over the head's compacted cache, all N_k queries, no mask
 * inside the scale (Eq. 4 on the compressed cache).  Requires hack_compact for this scale;
 * completes the step (the layer then expects scale + 1). */
HACK_API hack_status_t hack_attend(hack_cache_t* cache, int32_t layer, int32_t scale, const void* q,
                          void* out, void* stream);

/* hack_attend that also returns the attention variance of every head (Eq. 6, offline head
 * classification): sigma[b*H + h] = sum_j Var_i A[i, j], A = Softmax(sm_scale * Q K^T) the attention
 * matrix of this step's queries (rows) over the head's cache as it stands (columns), Var the
 * population variance over the queries.  For Eq. 6 proper, create the cache with budgets >= T_K, so
 * that nothing is evicted, and call this at the last scale: A is then the N_K x T_K matrix of the
 * final generation step.  sigma: device, [batch*n_heads] floats, written on `stream`.  State rules
 * of hack_attend.  UNSUPPORTED unless the cache is bf16 and the scale has at least 32 tokens (and
 * batch*n_heads*N_k >= 128): the statistics come from the tensor-core attention kernel. */
HACK_API hack_status_t hack_attend_variance(hack_cache_t* cache, int32_t layer, int32_t scale, const void* q,
                                   void* out, float* sigma, void* stream);

/* Head types from the variance matrix (Eq. 6 and the paragraph after it): all n_layers*n_heads heads
 * are ranked by sigma (host, row-major [n_layers][n_heads], already averaged over the samples) and
 * the round(alpha * n_layers * n_heads) lowest are marked contextual (1), the others structural (0);
 * equal values rank by (layer, head).  head_is_contextual: host, [n_layers*n_heads], the mask
 * hack_config_t takes.  Host only.  INVALID_ARG unless 0 <= alpha <= 1 and sigma is finite. */
HACK_API hack_status_t hack_classify_heads(const double* sigma, int32_t n_layers, int32_t n_heads, double alpha,
                                  uint8_t* head_is_contextual);

/* The whole step for one (layer, scale): score -> select -> compact -> attend; heads whose
 * candidate count does not exceed their budget skip scoring and selection and keep everything
 * (section "KV Cache Compression for VAR": compress whenever the length exceeds the budget).
 * bf16 caches: at most two launches (one cluster launch that scores, selects and compacts, one
 * attention launch that also appends the rows of heads which keep the whole new scale).  When one
 * head type compresses and the other only appends, the appending heads' attention is enqueued on a
 * stream of the cache's own, forked from `stream` at the start of the call and joined to it before
 * the call returns, so `stream` still orders everything (also inside a stream capture). */
HACK_API hack_status_t hack_scale_step(hack_cache_t* cache, int32_t layer, int32_t scale, const void* q,
                              const void* k, const void* v, void* out, void* stream);

/* Scores without any allocation (the paper has no counterpart: this exists for deployment).
 * For callers that cannot allocate device memory when they need scores - a server whose pool
 * already owns all of HBM, so cudaMalloc would fail, or a decode loop that cannot afford the
 * device-wide synchronisation cudaMalloc/cudaFree imply - and therefore cannot create a cache.
 * Computes what hack_score computes, on dense caller-owned device tensors:
 *   q       [n_rows, n_queries, head_dim]   (n_rows = batch*heads, dtype as given)
 *   k_cand  [n_rows, n_cand, head_dim]      all candidate keys of each row, in candidate order
 *   scores  [n_rows, score_stride] fp32, score_stride >= n_cand; columns j < n_cand are written.
 * sm_scale 0 selects 1/sqrt(head_dim).  Runs on the calling thread's current device.
 * Intermediates live in a fixed array inside the library's device image (about 8.3 MiB, held
 * by every GPU that loads the library until the process exits), hence the limits
 * n_rows <= 512 and n_rows*n_cand <= 65536; larger sizes return HACK_ERR_UNSUPPORTED.
 * No cudaMalloc, cudaFree or other allocating call is made.  The first call on a device is a
 * set-up call: it resolves the array's address (cudaGetSymbolAddress) and, because CUDA loads a
 * module's device image lazily, it is also the moment the driver reserves those 8.3 MiB on that
 * device.  Make it at start-up, before the caller's own pool claims the rest of the memory and
 * before any stream capture; every later call on that device leaves the device's memory as it is.
 * All calls share the array: calls that overlap on the GPU race, so keep them on one stream or
 * order them yourself.  Only enqueues; does not synchronise. */
HACK_API hack_status_t hack_score_noalloc(const void* q, const void* k_cand, float* scores,
                                          int32_t n_rows, int32_t n_queries, int32_t n_cand,
                                          int32_t score_stride, int32_t head_dim, int32_t dtype,
                                          int32_t n_obs, float sm_scale, void* stream);

/* Same step with HOST buffers (pinned memory, or the copies are not asynchronous): Q/K/V go to
 * library-owned device staging, the step runs on `stream`, O comes back; the call returns without
 * synchronising, and once `stream` has been synchronised out_host is complete.  The uploads and
 * the download run on two private streams with three staging sets, so the upload of the next
 * call overlaps this call's kernels; the host buffers of a call must stay valid until `stream`
 * has passed that call.  The staging sets and streams are created by the first such call on a
 * cache (make it outside any stream capture). */
HACK_API hack_status_t hack_scale_step_host(hack_cache_t* cache, int32_t layer, int32_t scale,
                                   const void* q_host, const void* k_host, const void* v_host,
                                   void* out_host, void* stream);

/* Stored length of every (batch, head) of a layer, host_out[b*H+h].  Host bookkeeping only. */
HACK_API hack_status_t hack_get_lengths(const hack_cache_t* cache, int32_t layer, int32_t* host_out);
/* Test inspection (synchronises the device): copy one head's stored rows to host memory.
 * which = 0: K rows, 1: V rows (dtype of the cache, [len, head_dim]); 2: original global token
 * positions (int32 [len]).  `bytes` is the size of host_out and must cover the stored length. */
HACK_API hack_status_t hack_read_head(hack_cache_t* cache, int32_t layer, int32_t b, int32_t h,
                             int32_t which, void* host_out, size_t bytes);

/* KV bytes (K and V rows only): currently stored, the peak since init/reset, and reserved. */
HACK_API hack_status_t hack_kv_bytes(const hack_cache_t* cache, size_t* live, size_t* peak, size_t* reserved);
/* Number of the library's own kernel launches enqueued through this cache since init. */
HACK_API hack_status_t hack_launch_count(const hack_cache_t* cache, uint64_t* launches);
/* Per-stage device timing for benchmarks.  enable != 0: from now on every stage's launches are
 * bracketed by two CUDA events on the caller's stream (a few microseconds of overhead per
 * stage); accumulators are cleared.  Synchronises the device. */
HACK_API hack_status_t hack_stage_timing(hack_cache_t* cache, int32_t enable);
/* Synchronises the device and returns the accumulated device time in ms and the number of kernel
 * launches per stage since timing was enabled: [0] score, [1] select, [2] compact, [3] attend.  In
 * hack_scale_step on a bf16 cache scoring, selection and compaction are one launch, counted under
 * [0]; while timing is on, the step does not run the two head types' work side by side. */
HACK_API hack_status_t hack_stage_times(hack_cache_t* cache, double* ms, uint64_t* launches);
/* Synchronises `stream`, then reports the device status word: HACK_OK, or HACK_ERR_TIMEOUT if a
 * bounded device-side wait gave up (the word is cleared by the call). */
HACK_API hack_status_t hack_poll_status(hack_cache_t* cache, void* stream);
/* Limit, in SM clock cycles, of every bounded device-side wait (mbarrier waits of the tensor-core
 * kernels) in launches made through this cache from now on; 0 restores the default of about one
 * second.  A wait that outlasts the limit raises the status word (hack_poll_status then returns
 * HACK_ERR_TIMEOUT), the CTA drains what it has in flight, frees its tensor memory and returns; the
 * results of that launch are undefined and the cache should be reset.  Meant for tests of that path
 * (a limit of a few cycles makes the first wait that is not already satisfied give up) and for
 * callers that want a tighter bound than a second.  INVALID_ARG for a negative limit. */
HACK_API hack_status_t hack_set_wait_limit(hack_cache_t* cache, int64_t cycles);
/* 1 if this library is the checked build (compiled with HACK_DEBUG_CHECKS), else 0.  The checked
 * build stands in for a memory checker: its kernels compare every ragged index they form with its
 * bound, skip the access on a violation and put the site's code into the status word
 * (hack_poll_status then returns HACK_ERR_STATE), and its planes carry one guard row behind the
 * rows of every (layer, batch, head). */
HACK_API int32_t hack_debug_build(void);
/* Checked build only: synchronises the device and counts the guard rows (K, V and position planes)
 * that no longer hold their pattern; hack_last_error() names the first.  UNSUPPORTED in the normal
 * build. */
HACK_API hack_status_t hack_debug_check(hack_cache_t* cache, int32_t* violations);
/* Text of the calling thread's last error; never NULL. */
HACK_API const char* hack_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* HACK_H_ */
