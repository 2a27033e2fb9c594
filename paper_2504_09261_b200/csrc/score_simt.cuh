// The SIMT scoring body (Eq. 9 and the TOPK argument of Eq. 10-11) shared by the cache-based fp32
// path (score_kernels.cu) and the entry point without allocation (score_noalloc.cu).
//
// Pass 1: a CTA of 128 threads takes 128 candidate keys of one row-block, stages them and the (at
// most 32) observation rows in shared memory, forms the logits, stores them and publishes the
// (max, sum-exp) of every observation row over the chunk.  Pass 2: the chunk statistics of a
// row-block are merged into the statistics of the full softmax and every column is reduced:
// s_j = sum_i exp(z_ij - m_i) / l_i.  The callers differ only in where a key row, an observation
// row, a logit and a score live; they pass those as small functors.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace hack {
namespace simt {

constexpr int kObs = 32;       // observation rows the kernels are built for
constexpr int kChunk = 128;    // candidate keys per CTA in pass 1 (= threads per CTA)

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

// Dynamic shared memory of pass 1: observation rows as fp32 [32][D], then the key tile
// [128][D/VEC + 1] of 16-byte vectors, which is reused for the logit tile [32][128].
template <typename T, int D>
constexpr size_t logits_smem_bytes() {
  return (size_t)kObs * D * 4 + (size_t)kChunk * (D / Elem<T>::kPerVec + 1) * 16;
}

// Pass 1 for candidates [j0, j0 + 128) of one row-block with n_cand candidates.
//   obs_ptr(i)        -> pointer to observation row i (D elements of T), i < n_obs_rows
//   key_ptr(j)        -> pointer to candidate key j (D elements of T), j < n_cand
//   logit_ref(i, j)   -> reference to where the logit of (observation row i, candidate j) goes
//   part_ptr(i)       -> pointer to the two floats (max, sum-exp) of row i for this chunk
template <typename T, int D, typename ObsPtr, typename KeyPtr, typename LogitRef, typename PartPtr>
__device__ __forceinline__ void chunk_logits(unsigned char* smem_raw, int j0, int n_cand, int n_obs_rows, float sm_scale,
                                             ObsPtr obs_ptr, KeyPtr key_ptr, LogitRef logit_ref, PartPtr part_ptr) {
  constexpr int VEC = Elem<T>::kPerVec;
  constexpr int ROWV = D / VEC;                 // 16-byte vectors per row
  constexpr int KROW = ROWV + 1;                // padded row stride (in vectors) of the key tile
  const int tid = threadIdx.x;
  float* qs = reinterpret_cast<float*>(smem_raw);                       // [32][D]
  uint4* ks = reinterpret_cast<uint4*>(smem_raw + kObs * D * 4);        // [128][KROW]
  float* zt = reinterpret_cast<float*>(ks);                             // reused: [32][128]

  for (int v = tid; v < kObs * ROWV; v += kChunk) {
    const int i = v / ROWV, c = v % ROWV;
    float f[VEC];
    if (i < n_obs_rows) {
      Elem<T>::unpack(*reinterpret_cast<const uint4*>(obs_ptr(i) + c * VEC), f);
    } else {
#pragma unroll
      for (int e = 0; e < VEC; ++e) f[e] = 0.f;
    }
#pragma unroll
    for (int e = 0; e < VEC; ++e) qs[i * D + c * VEC + e] = f[e];
  }
  for (int v = tid; v < kChunk * ROWV; v += kChunk) {
    const int r = v / ROWV, c = v % ROWV;
    const int j = j0 + r;
    uint4 raw = make_uint4(0, 0, 0, 0);
    if (j < n_cand) raw = *reinterpret_cast<const uint4*>(key_ptr(j) + c * VEC);
    ks[r * KROW + c] = raw;
  }
  __syncthreads();

  float acc[kObs];
#pragma unroll
  for (int i = 0; i < kObs; ++i) acc[i] = 0.f;
  for (int c = 0; c < ROWV; ++c) {
    float kf[VEC];
    Elem<T>::unpack(ks[tid * KROW + c], kf);
#pragma unroll
    for (int i = 0; i < kObs; ++i) {
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
  const bool valid = (j0 + tid) < n_cand;
#pragma unroll
  for (int i = 0; i < kObs; ++i) zt[i * kChunk + tid] = valid ? acc[i] * sm_scale : -INFINITY;
  __syncthreads();

  // each warp owns 8 observation rows: store logits (coalesced) and reduce (max, sum-exp)
  const int warp = tid >> 5, lane = tid & 31;
  for (int i = warp; i < n_obs_rows; i += kChunk / 32) {
    float z[4];
    float m = -INFINITY;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      z[u] = zt[i * kChunk + u * 32 + lane];
      m = fmaxf(m, z[u]);
      const int j = j0 + u * 32 + lane;
      if (j < n_cand) logit_ref(i, j) = z[u];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float l = 0.f;
#pragma unroll
    for (int u = 0; u < 4; ++u) l += expf(z[u] - m);      // exp(-inf) = 0 for padding
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
    if (lane == 0) {
      float* p = part_ptr(i);
      p[0] = m;
      p[1] = l;
    }
  }
}

// Pass 2 for a CTA of 256 threads and candidates [j0, j0 + 256): row_m / row_inv_l are two shared
// arrays of 32 floats; part(c, i) points at the (max, sum-exp) of chunk c, row i; returns the score
// of candidate j0 + threadIdx.x through `score` (valid when the function returns true).
template <typename PartPtr, typename LogitVal>
__device__ __forceinline__ bool column_scores(float* row_m, float* row_inv_l, int j0, int n_cand, int n_obs_rows,
                                              int n_chunks, PartPtr part, LogitVal logit, float& score) {
  if ((int)threadIdx.x < n_obs_rows) {
    const int i = threadIdx.x;
    float m = -INFINITY;
    for (int c = 0; c < n_chunks; ++c) m = fmaxf(m, part(c, i)[0]);
    float l = 0.f;
    for (int c = 0; c < n_chunks; ++c) l += part(c, i)[1] * expf(part(c, i)[0] - m);
    row_m[i] = m;
    row_inv_l[i] = 1.f / l;
  }
  __syncthreads();
  const int j = j0 + threadIdx.x;
  if (j >= n_cand) return false;
  float s = 0.f;
  for (int i = 0; i < n_obs_rows; ++i) s += expf(logit(i, j) - row_m[i]) * row_inv_l[i];
  score = s;
  return true;
}

}  // namespace simt
}  // namespace hack
