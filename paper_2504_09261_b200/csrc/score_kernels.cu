// Subset-attention importance scores (Eq. 9 and the TOPK argument of Eq. 10-11).
//
// Two launches per step.  Pass 1 walks the candidate keys once: each CTA takes 128 candidates of
// one head, stages them in shared memory with 16-byte coalesced loads, forms the logits against
// the (at most 32) observation rows, stores them to scratch and publishes per-row (max, sum-exp)
// partials for its chunk.  Pass 2 merges the partials into the row statistics of the full
// softmax over all T' candidates and reduces every column: s_j = sum_i exp(z_ij - m_i) / l_i.
#include <algorithm>

#include "hack_internal.h"
#include "score_simt.cuh"

namespace hack {
namespace {

using simt::Elem;
static_assert(simt::kObs == kMaxObs && simt::kChunk == kScoreChunk, "the shared SIMT body is built for these sizes");

// Row pointer of candidate j of head bh: stored entries first, then the new scale's tokens.
template <typename T>
__device__ __forceinline__ const T* cand_row(const StepArgs& a, const T* plane, const T* fresh,
                                             int bh, int stored, int j) {
  if (j < stored) return plane + (size_t)(a.row_off[bh] + j) * a.head_dim;
  return fresh + ((size_t)bh * a.n_new + (j - stored)) * a.head_dim;
}

template <typename T, int D>
__global__ void __launch_bounds__(kScoreChunk)
score_logits_kernel(const StepArgs a, const T* __restrict__ q, const T* __restrict__ k_new,
                    float* __restrict__ logits, float* __restrict__ partials, int max_chunks) {
  pdl_wait();
  const int bh = blockIdx.y;
  const int ctx = a.is_ctx[bh % a.n_heads];
  if (!a.trig[ctx]) return;
  const int cand = a.cand[ctx], stored = a.stored[ctx];
  const int j0 = blockIdx.x * kScoreChunk;
  if (j0 >= cand) return;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const T* kp = static_cast<const T*>(a.k_plane);
  const int chunk = blockIdx.x;
  simt::chunk_logits<T, D>(
      smem_raw, j0, cand, a.n_obs_rows, a.sm_scale,
      [&](int i) { return q + ((size_t)bh * a.n_new + obs_row(a, i)) * D; },     // floor(m * N_k / n) under the uniform rule
      [&](int j) { return cand_row(a, kp, k_new, bh, stored, j); },
      [&](int i, int j) -> float& { return logits[((size_t)bh * kMaxObs + i) * a.cand_stride + j]; },
      [&](int i) { return partials + (((size_t)bh * max_chunks + chunk) * kMaxObs + i) * 2; });
}

__global__ void __launch_bounds__(256)
score_reduce_kernel(const StepArgs a, const float* __restrict__ logits,
                    const float* __restrict__ partials, int max_chunks, float* __restrict__ scores) {
  pdl_wait();
  const int bh = blockIdx.y;
  const int ctx = a.is_ctx[bh % a.n_heads];
  if (!a.trig[ctx]) return;
  const int cand = a.cand[ctx];
  const int j0 = blockIdx.x * 256;
  if (j0 >= cand) return;
  __shared__ float row_m[kMaxObs], row_inv_l[kMaxObs];
  const int n_chunks = (cand + kScoreChunk - 1) / kScoreChunk;
  float s;
  if (!simt::column_scores(
          row_m, row_inv_l, j0, cand, a.n_obs_rows, n_chunks,
          [&](int c, int i) { return partials + (((size_t)bh * max_chunks + c) * kMaxObs + i) * 2; },
          [&](int i, int j) { return logits[((size_t)bh * kMaxObs + i) * a.cand_stride + j]; }, s))
    return;
  float* dst = scores + (size_t)bh * a.cand_stride + j0 + threadIdx.x;
  *dst = a.score_accumulate ? *dst + s : s;
}

template <typename T, int D>
int launch_score_t(const StepArgs& a, const void* q, const void* k_new, float* scores,
                   const Scratch& s, cudaStream_t st) {
  const int max_cand = a.cand[0] * a.trig[0] > a.cand[1] * a.trig[1] ? a.cand[0] : a.cand[1];
  const int bh = a.batch * a.n_heads;
  const size_t smem = simt::logits_smem_bytes<T, D>();
  if (!allow_dynamic_smem(score_logits_kernel<T, D>, smem)) return -1;
  dim3 g1((max_cand + kScoreChunk - 1) / kScoreChunk, bh);
  launch_k(score_logits_kernel<T, D>, g1, kScoreChunk, smem, st, 
      a, static_cast<const T*>(q), static_cast<const T*>(k_new), s.logits, s.partials, s.max_chunks);
  dim3 g2((max_cand + 255) / 256, bh);
  launch_k(score_reduce_kernel, g2, 256, 0, st, a, s.logits, s.partials, s.max_chunks, scores);
  return launched(2);
}

}  // namespace

static int launch_score_round(const StepArgs& a, int dtype, const void* q, const void* k_new, float* scores,
                              const Scratch& s, cudaStream_t st) {
  // bf16: tensor-core kernel, unless the new K tensor has fewer rows than one TMA box
  if (dtype == HACK_BF16 && a.k_map && (long long)a.batch * a.n_heads * a.n_new >= 128)
    return launch_score_tc(a, q, k_new, scores, s, st);
  if (dtype == HACK_F32) {
    return a.head_dim == 64 ? launch_score_t<float, 64>(a, q, k_new, scores, s, st)
                            : launch_score_t<float, 128>(a, q, k_new, scores, s, st);
  }
  return a.head_dim == 64 ? launch_score_t<__nv_bfloat16, 64>(a, q, k_new, scores, s, st)
                          : launch_score_t<__nv_bfloat16, 128>(a, q, k_new, scores, s, st);
}

int launch_score(const StepArgs& a, int dtype, const void* q, const void* k_new, float* scores,
                 const Scratch& s, cudaStream_t st) {
  if (!a.trig[0] && !a.trig[1]) return 0;
  if (!a.obs_full) return launch_score_round(a, dtype, q, k_new, scores, s, st);
  // every query observes: one scoring round per group of kMaxObs consecutive query rows; every
  // row's softmax is normalised over all candidates inside its round, so the rounds simply add up
  int n = 0;
  for (int first = 0; first < a.n_new; first += kMaxObs) {
    StepArgs g = a;
    g.n_obs_rows = std::min(kMaxObs, a.n_new - first);
    g.obs_first = first;
    g.obs_span = g.n_obs_rows;
    g.obs_rows = nullptr;
    g.score_accumulate = first > 0;
    const int r = launch_score_round(g, dtype, q, k_new, scores, s, st);
    if (r < 0) return r;
    n += r;
  }
  return n;
}

}  // namespace hack
