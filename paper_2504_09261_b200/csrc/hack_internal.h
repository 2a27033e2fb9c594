// Internal declarations shared by the host API and the kernel translation units.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "hack.h"

namespace hack {

constexpr int kMaxObs = 32;        // rows of the observation window the kernels are built for
constexpr int kScoreChunk = 128;   // candidate keys per CTA in the SIMT scoring pass

// Everything a kernel needs to know about one (layer, scale) step.  Passed by value.
// Per-type arrays are indexed by the head's mask byte: [0] structural, [1] contextual.
struct StepArgs {
  int n_heads, batch, head_dim;
  int n_new;            // N_k
  int stored[2];        // L before the step
  int cand[2];          // T' = L + N_k
  int kept[2];          // length after the step
  int cap[2];           // rows a head of this type owns in the planes (checked builds compare against it)
  int trig[2];          // compression triggered for this type
  int seg_new[2];       // tensor-core attention reads this type's new rows from the caller's K/V and
                        // appends them itself (the type keeps the whole new scale in this step)
  long long wait_cycles;   // limit of every bounded device-side wait of the step's kernels
  int n_obs_rows;       // min(N_obs, N_k)
  int obs_first, obs_span;      // observation row i = obs_first + floor(i * obs_span / n_obs_rows) ...
  const int32_t* obs_rows;      // ... unless the caller supplied the rows (device, [n_obs_rows])
  int obs_full;                 // every query observes: the scoring kernels run once per group of 32 rows
  int score_accumulate;         // the scores of this round are added to those already there
  float sm_scale;
  int t_init;           // tokens in the always-kept leading scales (structural heads)
  int protect_new;      // structural heads: the new scale's tokens are protected
  int pos_base;         // global position of the new scale's first token (T_{k-1})
  int cand_stride, kept_stride;
  const uint8_t* is_ctx;   // device, [n_heads] of this layer
  const int32_t* row_off;  // device, [batch*n_heads] first row of each head in the planes
  void* k_plane;           // device, [rows, head_dim] of this layer
  void* v_plane;
  int32_t* pos_plane;      // device, [rows]
  int* status;             // device status word
  int32_t* n_old;          // device, [batch*n_heads]: survivors that were already stored (compaction)
  // tensor-core attention only (host pointers to 128-byte tensor maps of this layer's planes)
  const void* k_map;
  const void* v_map;
  const int32_t* head_order;   // device, [batch*n_heads], heads with the longer cache first
};

struct Scratch {
  float* logits;    // [batch*n_heads, kMaxObs, cand_stride]
  float* partials;  // [batch*n_heads, max_chunks, kMaxObs, 2]  (row max, row sum per chunk)
  int max_chunks;
};

// Scratch of the final-scale merge of contextual heads (bf16 caches): the rows the last step
// discards, their list, inverse key norms, and the counterpart and weight of every discarded row.
struct MergeScratch {
  int stride;                  // rows per (batch, head) in the arrays below
  __nv_bfloat16* ev_k;         // [b*H, stride, D] discarded key rows
  __nv_bfloat16* ev_v;         // [b*H, stride, D] discarded value rows
  int32_t* ev_idx;             // [b*H, stride] their candidate indices, ascending
  float* ev_inv_norm;          // [b*H, stride] 1 / |k_e|
  float* kept_inv_norm;        // [b*H, kept_stride] 1 / |k_c|
  int32_t* assign;             // [b*H, stride] retained row each discarded row is folded into
  float* weight;               // [b*H, stride] max(cosine similarity, 0)
  const void* ev_map;          // host pointer to the 128-byte tensor map over ev_k
};
// Before the compaction of the step (idx = the kept lists of launch_select) and after it.
int launch_merge_prepare(const StepArgs& a, const MergeScratch& ms, const int32_t* idx, const void* k_new,
                         const void* v_new, cudaStream_t st);
int launch_merge_finish(const StepArgs& a, const MergeScratch& ms, cudaStream_t st);

// Kernel launchers (each returns the number of kernels it enqueued, or -1 on a launch error).
int launch_score(const StepArgs& a, int dtype, const void* q, const void* k_new, float* scores,
                 const Scratch& s, cudaStream_t st);
// bf16 caches: the same scores with the logits formed on the tensor cores (two launches).
int launch_score_tc(const StepArgs& a, const void* q, const void* k_new, float* scores, const Scratch& s,
                    cudaStream_t st);
int launch_select(const StepArgs& a, const float* scores, int32_t* idx, int32_t* kept_out,
                  cudaStream_t st);
// bf16 caches: scores only (idx == nullptr) or scoring, selection and in-place compaction of the step
// in one launch of one thread-block cluster per head.  1: launched; 0: the step is outside what the
// kernel holds, take the separate launches; -1: launch error.
int launch_compress_cluster(const StepArgs& a, const void* q, const void* k_new, const void* v_new, float* scores,
                            int32_t* idx, cudaStream_t st, int reserved_sms = 0);
// idx == nullptr: every head appends (keeps all candidates).  idx_all != 0: idx rows are valid for
// heads that are not triggered as well (identity lists written by launch_select).
int launch_compact(const StepArgs& a, int dtype, const int32_t* idx, int idx_all, const void* k_new,
                   const void* v_new, cudaStream_t st);
int launch_attend(const StepArgs& a, int dtype, const void* q, void* out, cudaStream_t st);

int launch_attend_simt(const StepArgs& a, int dtype, const void* q, void* out, cudaStream_t st);
// row_stats (optional, device [b*H, N_k, 2]): per query row the reference maximum m (raw logit
// units; within the lazy-rescaling margin of the true maximum) and l = sum_j exp2(c (z_j - m)).
// k_new / v_new (optional): the caller's K/V of this scale; head types with a.seg_new set then attend
// over [kept - N_k cache rows ; the N_k new rows read from k_new / v_new] and the kernel appends
// those rows to the cache, so no append or copy launch precedes it for them.  n_heads_served: 0 for
// every head, else only the first n_heads_served heads of head_order are served (the heads of one type);
// shares_gpu: another kernel of the step runs beside this launch.  follows_compression: the launch ahead
// of this one in the stream is the step's compression launch (the queries, which no kernel of the step
// writes, may then be read before the dependency wait).
int launch_attend_tc(const StepArgs& a, const void* k_map, const void* v_map, const int32_t* head_order,
                     const void* q, void* out, float* row_stats, const void* k_new, const void* v_new,
                     int n_heads_served, bool shares_gpu, cudaStream_t st, bool follows_compression = false);
constexpr long long kDefaultWaitCycles = 2000000000ll;   // about one second: no wait is legitimately longer
// Attention variance per (batch, head) over the compacted cache (Eq. 6) from the row statistics of
// launch_attend_tc; block_var: device scratch [b*H, max_blocks]; sigma: device [b*H].  bf16 only.
int launch_attention_variance(const StepArgs& a, const void* q, const float* row_stats, float* block_var,
                              int max_blocks, float* sigma, cudaStream_t st);
bool attend_tc_serves(const StepArgs& a, int dtype);   // the tensor-core kernel takes this step's attention
// 2-D bf16 tensor map (128 x 64 boxes, 128-byte swizzle) over rows x head_dim; false on failure.
bool make_rows_map(void* out_map, const void* base, uint64_t rows, int head_dim);

// Untriggered step with at most kSmallQueries new tokens: append and attention in one SIMT launch.
int launch_append_attend_small(const StepArgs& a, int dtype, const void* q, const void* k_new,
                               const void* v_new, void* out, cudaStream_t st);
constexpr int kSmallQueries = 31;

constexpr int kTcMinQueries = 32;   // below this the SIMT kernel serves bf16 as well

void set_error(const std::string& msg);
// Number of SMs of the current device (asked once per device); the grid heuristics size to it.
int sm_count();

// Every kernel of the step is launched with programmatic stream serialisation: its CTAs may start
// while the previous kernel of the stream drains, and stop at pdl_wait() until that kernel has
// completed and its writes are visible.  Nothing that another kernel produces or still reads is
// touched before pdl_wait().
template <typename... KArgs, typename... Args>
inline void launch_k(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}
// Checked build (-DHACK_DEBUG_CHECKS), the stand-in for a memory checker: every ragged index a
// kernel forms (a list entry, a row of a head, a candidate, a slot of the index list) is compared
// with its bound before it is used; on a violation the access is skipped and the code of the site
// goes to the status word (nothing traps), which hack_poll_status reports.  The planes of a checked
// build also carry a canary row behind every head, verified on the host by hack_debug_check.  In
// the normal build the test is constant-true and costs nothing.
constexpr int kDebugCodeBase = 100;     // status codes of the bounds checks start here
constexpr unsigned char kCanaryByte = 0x5A;
#if defined(__CUDACC__)
#if defined(HACK_DEBUG_CHECKS)
__device__ __forceinline__ bool dbg_ok(bool cond, int* status, int code) {
  if (!cond) atomicExch(status, kDebugCodeBase + code);
  return cond;
}
#else
__device__ __forceinline__ bool dbg_ok(bool, int*, int) { return true; }
#endif
// Query row that serves as observation row i (Eq. 9's subset Q~).
__device__ __forceinline__ int obs_row(const StepArgs& a, int i) {
  return a.obs_rows ? a.obs_rows[i] : a.obs_first + (int)(((long long)i * a.obs_span) / a.n_obs_rows);
}
__device__ __forceinline__ void pdl_wait() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
#endif

// Opt-in to more than 48 KB of dynamic shared memory.  The attribute belongs to the (function,
// device) pair, so it is set once per pair, on the device that is current (thread safe).
// False (with the error text recorded) if the driver refuses; the pair is then asked again next time.
bool allow_dynamic_smem_impl(const void* kern, size_t bytes);
template <typename F>
inline bool allow_dynamic_smem(F* kern, size_t bytes) {
  return allow_dynamic_smem_impl(reinterpret_cast<const void*>(kern), bytes);
}

// After a kernel launch: n if it was accepted, else -1 with the CUDA error text recorded.
inline int launched(int n) {
  const cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) return n;
  set_error(std::string("kernel launch: ") + cudaGetErrorString(e));
  return -1;
}

}  // namespace hack
