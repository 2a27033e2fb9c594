// Subset-attention importance scores (Eq. 9 and the TOPK argument of Eq. 10-11).
//
// Two launches per step.  Pass 1 walks the candidate keys once: each CTA takes 128 candidates of
// one head, stages them in shared memory with 16-byte coalesced loads, forms the logits against
// the (at most 32) observation rows, stores them to scratch and publishes per-row (max, sum-exp)
// partials for its chunk.  Pass 2 merges the partials into the row statistics of the full
// softmax over all T' candidates and reduces every column: s_j = sum_i exp(z_ij - m_i) / l_i.
#include <algorithm>

#include "hack_internal.h"

namespace hack {
namespace {

template <typename T> struct Elem;
template <> struct Elem<float> {
  static constexpr int kPerVec = 4;  // elements per 16 bytes
  __device__ static void unpack(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
    f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
  }
};
template <> struct Elem<__nv_bfloat16> {
  static constexpr int kPerVec = 8;
  __device__ static void unpack(const uint4& v, float* f) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
};

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
  constexpr int VEC = Elem<T>::kPerVec;
  constexpr int ROWV = D / VEC;                 // 16-byte vectors per row
  constexpr int KROW = ROWV + 1;                // padded row stride (in vectors) of the key tile
  const int bh = blockIdx.y;
  const int ctx = a.is_ctx[bh % a.n_heads];
  if (!a.trig[ctx]) return;
  const int cand = a.cand[ctx], stored = a.stored[ctx];
  const int j0 = blockIdx.x * kScoreChunk;
  if (j0 >= cand) return;
  const int tid = threadIdx.x;

  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* qs = reinterpret_cast<float*>(smem_raw);                       // [32][D]
  uint4* ks = reinterpret_cast<uint4*>(smem_raw + kMaxObs * D * 4);     // [128][KROW]
  float* zt = reinterpret_cast<float*>(ks);                             // reused: [32][128]

  const T* kp = static_cast<const T*>(a.k_plane);
  // observation rows: floor(m * N_k / n) under the uniform rule
  for (int v = tid; v < kMaxObs * ROWV; v += kScoreChunk) {
    const int i = v / ROWV, c = v % ROWV;
    float f[VEC];
    if (i < a.n_obs_rows) {
      const int row = obs_row(a, i);
      const uint4 raw = *reinterpret_cast<const uint4*>(q + ((size_t)bh * a.n_new + row) * D + c * VEC);
      Elem<T>::unpack(raw, f);
    } else {
#pragma unroll
      for (int e = 0; e < VEC; ++e) f[e] = 0.f;
    }
#pragma unroll
    for (int e = 0; e < VEC; ++e) qs[i * D + c * VEC + e] = f[e];
  }
  for (int v = tid; v < kScoreChunk * ROWV; v += kScoreChunk) {
    const int r = v / ROWV, c = v % ROWV;
    const int j = j0 + r;
    uint4 raw = make_uint4(0, 0, 0, 0);
    if (j < cand) raw = *reinterpret_cast<const uint4*>(cand_row(a, kp, k_new, bh, stored, j) + c * VEC);
    ks[r * KROW + c] = raw;
  }
  __syncthreads();

  float acc[kMaxObs];
#pragma unroll
  for (int i = 0; i < kMaxObs; ++i) acc[i] = 0.f;
  for (int c = 0; c < ROWV; ++c) {
    float kf[VEC];
    Elem<T>::unpack(ks[tid * KROW + c], kf);
#pragma unroll
    for (int i = 0; i < kMaxObs; ++i) {
      const float4* qv = reinterpret_cast<const float4*>(qs + i * D + c * VEC);
#pragma unroll
      for (int e4 = 0; e4 < VEC / 4; ++e4) {
        const float4 qq = qv[e4];
        acc[i] = fmaf(qq.x, kf[4 * e4 + 0], acc[i]);
        acc[i] = fmaf(qq.y, kf[4 * e4 + 1], acc[i]);
        acc[i] = fmaf(qq.z, kf[4 * e4 + 2], acc[i]);
        acc[i] = fmaf(qq.w, kf[4 * e4 + 3], acc[i]);
      }
    }
  }
  __syncthreads();                     // everyone is done with the key tile; reuse it for logits
  const bool valid = (j0 + tid) < cand;
#pragma unroll
  for (int i = 0; i < kMaxObs; ++i) zt[i * kScoreChunk + tid] = valid ? acc[i] * a.sm_scale : -INFINITY;
  __syncthreads();

  // each warp owns 8 observation rows: store logits (coalesced) and reduce (max, sum-exp)
  const int warp = tid >> 5, lane = tid & 31;
  const int chunk = blockIdx.x;
  for (int i = warp; i < a.n_obs_rows; i += kScoreChunk / 32) {
    float z[4];
    float m = -INFINITY;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      z[u] = zt[i * kScoreChunk + u * 32 + lane];
      m = fmaxf(m, z[u]);
      const int j = j0 + u * 32 + lane;
      if (j < cand) logits[((size_t)bh * kMaxObs + i) * a.cand_stride + j] = z[u];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float l = 0.f;
#pragma unroll
    for (int u = 0; u < 4; ++u) l += expf(z[u] - m);      // exp(-inf) = 0 for padding
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
    if (lane == 0) {
      float* p = partials + (((size_t)bh * max_chunks + chunk) * kMaxObs + i) * 2;
      p[0] = m;
      p[1] = l;
    }
  }
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
  if (threadIdx.x < a.n_obs_rows) {
    const int i = threadIdx.x;
    const float* p = partials + ((size_t)bh * max_chunks * kMaxObs + i) * 2;
    float m = -INFINITY;
    for (int c = 0; c < n_chunks; ++c) m = fmaxf(m, p[(size_t)c * kMaxObs * 2]);
    float l = 0.f;
    for (int c = 0; c < n_chunks; ++c)
      l += p[(size_t)c * kMaxObs * 2 + 1] * expf(p[(size_t)c * kMaxObs * 2] - m);
    row_m[i] = m;
    row_inv_l[i] = 1.f / l;
  }
  __syncthreads();
  const int j = j0 + threadIdx.x;
  if (j >= cand) return;
  float s = 0.f;
  for (int i = 0; i < a.n_obs_rows; ++i) {
    const float z = logits[((size_t)bh * kMaxObs + i) * a.cand_stride + j];
    s += expf(z - row_m[i]) * row_inv_l[i];
  }
  float* dst = scores + (size_t)bh * a.cand_stride + j;
  *dst = a.score_accumulate ? *dst + s : s;
}

template <typename T, int D>
int launch_score_t(const StepArgs& a, const void* q, const void* k_new, float* scores,
                   const Scratch& s, cudaStream_t st) {
  const int max_cand = a.cand[0] * a.trig[0] > a.cand[1] * a.trig[1] ? a.cand[0] : a.cand[1];
  const int bh = a.batch * a.n_heads;
  constexpr int VEC = Elem<T>::kPerVec;
  const size_t smem = (size_t)kMaxObs * D * 4 +
                      (size_t)kScoreChunk * (D / VEC + 1) * 16;   // >= 32*128*4 for the logit tile
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
