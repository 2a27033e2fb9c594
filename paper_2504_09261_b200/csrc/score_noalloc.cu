// hack_score_noalloc: subset-attention importance scores for callers that must not allocate.
//
// Some users of this library cannot call cudaMalloc at the point where they need scores: an
// inference server that handed all of HBM to its own pool at start-up (a raw cudaMalloc would
// simply fail), or a latency-critical decode loop where the implicit device-wide synchronisation
// of cudaMalloc / cudaFree is not acceptable.  hack_init_cache allocates, so it is closed to them.
// This entry point needs no cache object: the caller passes dense Q and candidate-key tensors and
// an output buffer, and the two-pass scoring kernels keep their intermediate logits and row
// statistics in a fixed array that lives in the library's own device image.
//
// The array (kScratchFloats floats, about 8.3 MiB) is part of the module: every GPU that loads
// the library holds it until the process exits.  CUDA loads the module's device image lazily, so
// the driver reserves it on a device during the first call made there (the set-up call, to be made
// at start-up); no later call changes the device's memory.  All calls share it and it keeps the previous
// call's contents; nothing in it has to start at zero because pass 1 overwrites every element
// pass 2 reads.  Two calls that overlap on the GPU (different streams, or different host threads
// without ordering) race on it: serialise them.
#include <cmath>
#include <mutex>

#include "hack_internal.h"

namespace hack {
namespace {

constexpr int kChunk = 128;                               // candidate keys per CTA in pass 1
constexpr long long kMaxLogitRows = 65536;                // limit on n_rows * n_cand
constexpr int kMaxRows = 512;                             // limit on n_rows (batch * heads)
constexpr long long kLogitFloats = kMaxLogitRows * kMaxObs;                     // 2 Mi floats
constexpr long long kPartialFloats = (kMaxLogitRows / kChunk + kMaxRows) * kMaxObs * 2;
constexpr long long kScratchFloats = kLogitFloats + kPartialFloats;

// Scratch of the no-allocation entry point.  In host code this name is only a handle for
// cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) float g_noalloc_scratch[kScratchFloats];

template <typename T> struct Ld;
template <> struct Ld<float> {
  static constexpr int kPerVec = 4;
  __device__ static void unpack(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
    f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
  }
};
template <> struct Ld<__nv_bfloat16> {
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

struct DenseArgs {
  int n_queries, n_cand, n_obs_rows, chunks_per_row;
  float sm_scale;
};

// Pass 1: logits of 128 candidates of one row-block against the observation rows, plus the
// (max, sum-exp) of every observation row over this chunk.
template <typename T, int D>
__global__ void __launch_bounds__(kChunk)
noalloc_logits_kernel(const DenseArgs a, const T* __restrict__ q, const T* __restrict__ k_cand,
                      float* __restrict__ logits, float* __restrict__ partials) {
  constexpr int VEC = Ld<T>::kPerVec;
  constexpr int ROWV = D / VEC;
  constexpr int KROW = ROWV + 1;
  const int row = blockIdx.y;
  const int j0 = blockIdx.x * kChunk;
  const int tid = threadIdx.x;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* qs = reinterpret_cast<float*>(smem_raw);
  uint4* ks = reinterpret_cast<uint4*>(smem_raw + kMaxObs * D * 4);
  float* zt = reinterpret_cast<float*>(ks);

  for (int v = tid; v < kMaxObs * ROWV; v += kChunk) {
    const int i = v / ROWV, c = v % ROWV;
    float f[VEC];
    if (i < a.n_obs_rows) {
      const int qrow = (int)(((long long)i * a.n_queries) / a.n_obs_rows);
      Ld<T>::unpack(*reinterpret_cast<const uint4*>(q + ((size_t)row * a.n_queries + qrow) * D + c * VEC), f);
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
    if (j < a.n_cand) raw = *reinterpret_cast<const uint4*>(k_cand + ((size_t)row * a.n_cand + j) * D + c * VEC);
    ks[r * KROW + c] = raw;
  }
  __syncthreads();
  float acc[kMaxObs];
#pragma unroll
  for (int i = 0; i < kMaxObs; ++i) acc[i] = 0.f;
  for (int c = 0; c < ROWV; ++c) {
    float kf[VEC];
    Ld<T>::unpack(ks[tid * KROW + c], kf);
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
  __syncthreads();
  const bool valid = (j0 + tid) < a.n_cand;
#pragma unroll
  for (int i = 0; i < kMaxObs; ++i) zt[i * kChunk + tid] = valid ? acc[i] * a.sm_scale : -INFINITY;
  __syncthreads();
  const int warp = tid >> 5, lane = tid & 31;
  for (int i = warp; i < a.n_obs_rows; i += kChunk / 32) {
    float z[4];
    float m = -INFINITY;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      z[u] = zt[i * kChunk + u * 32 + lane];
      m = fmaxf(m, z[u]);
      const int j = j0 + u * 32 + lane;
      if (j < a.n_cand) logits[((size_t)row * kMaxObs + i) * a.n_cand + j] = z[u];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float l = 0.f;
#pragma unroll
    for (int u = 0; u < 4; ++u) l += expf(z[u] - m);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
    if (lane == 0) {
      float* p = partials + (((size_t)row * a.chunks_per_row + blockIdx.x) * kMaxObs + i) * 2;
      p[0] = m;
      p[1] = l;
    }
  }
}

// Pass 2: merge the chunk statistics into full-softmax row statistics and reduce each column.
__global__ void __launch_bounds__(256)
noalloc_reduce_kernel(const DenseArgs a, const float* __restrict__ logits,
                      const float* __restrict__ partials, float* __restrict__ scores, int score_stride) {
  const int row = blockIdx.y;
  __shared__ float row_m[kMaxObs], row_inv_l[kMaxObs];
  if (threadIdx.x < a.n_obs_rows) {
    const int i = threadIdx.x;
    const float* p = partials + ((size_t)row * a.chunks_per_row * kMaxObs + i) * 2;
    float m = -INFINITY;
    for (int c = 0; c < a.chunks_per_row; ++c) m = fmaxf(m, p[(size_t)c * kMaxObs * 2]);
    float l = 0.f;
    for (int c = 0; c < a.chunks_per_row; ++c)
      l += p[(size_t)c * kMaxObs * 2 + 1] * expf(p[(size_t)c * kMaxObs * 2] - m);
    row_m[i] = m;
    row_inv_l[i] = 1.f / l;
  }
  __syncthreads();
  const int j = blockIdx.x * 256 + threadIdx.x;
  if (j >= a.n_cand) return;
  float s = 0.f;
  for (int i = 0; i < a.n_obs_rows; ++i)
    s += expf(logits[((size_t)row * kMaxObs + i) * a.n_cand + j] - row_m[i]) * row_inv_l[i];
  scores[(size_t)row * score_stride + j] = s;
}

// One scratch address per device, resolved on the first call made with that device current.
std::mutex g_setup_mutex;
float* g_scratch_ptr[64] = {nullptr};

template <typename T, int D>
cudaError_t run(const DenseArgs& a, int n_rows, const void* q, const void* k, float* scratch,
                float* scores, int score_stride, cudaStream_t st) {
  constexpr int VEC = Ld<T>::kPerVec;
  const size_t smem = (size_t)kMaxObs * D * 4 + (size_t)kChunk * (D / VEC + 1) * 16;
  // opt-in to more than 48 KB of dynamic shared memory, once per (kernel, device)
  if (!allow_dynamic_smem(noalloc_logits_kernel<T, D>, smem)) return cudaErrorInvalidValue;
  float* logits = scratch;
  float* partials = scratch + kLogitFloats;
  noalloc_logits_kernel<T, D><<<dim3(a.chunks_per_row, n_rows), kChunk, smem, st>>>(
      a, static_cast<const T*>(q), static_cast<const T*>(k), logits, partials);
  noalloc_reduce_kernel<<<dim3((a.n_cand + 255) / 256, n_rows), 256, 0, st>>>(a, logits, partials, scores,
                                                                               score_stride);
  return cudaGetLastError();
}

}  // namespace
}  // namespace hack

extern "C" hack_status_t hack_score_noalloc(const void* q, const void* k_cand, float* scores,
                                            int32_t n_rows, int32_t n_queries, int32_t n_cand,
                                            int32_t score_stride, int32_t head_dim, int32_t dtype,
                                            int32_t n_obs, float sm_scale, void* stream) {
  using namespace hack;
  if (!q || !k_cand || !scores) { set_error("q, k_cand or scores is NULL"); return HACK_ERR_INVALID_ARG; }
  if (((uintptr_t)q | (uintptr_t)k_cand) & 15u) { set_error("q and k_cand must be 16-byte aligned"); return HACK_ERR_INVALID_ARG; }
  if (n_rows < 1 || n_queries < 1 || n_cand < 1 || score_stride < n_cand) {
    set_error("n_rows, n_queries, n_cand must be positive and score_stride >= n_cand");
    return HACK_ERR_INVALID_ARG;
  }
  if (head_dim != 64 && head_dim != 128) { set_error("head_dim must be 64 or 128"); return HACK_ERR_UNSUPPORTED; }
  if (dtype != HACK_F32 && dtype != HACK_BF16) { set_error("dtype must be HACK_F32 or HACK_BF16"); return HACK_ERR_UNSUPPORTED; }
  if (n_obs < 1 || n_obs > kMaxObs) { set_error("n_obs must be in 1..32"); return HACK_ERR_UNSUPPORTED; }
  if (!(sm_scale >= 0.f) || sm_scale > 3.0e38f) { set_error("sm_scale must be finite and non-negative"); return HACK_ERR_INVALID_ARG; }
  if (n_rows > kMaxRows || (long long)n_rows * n_cand > kMaxLogitRows) {
    set_error("hack_score_noalloc: size beyond the fixed scratch (limits: n_rows <= 512 and "
              "n_rows * n_cand <= 65536); use hack_score with a cache for larger problems");
    return HACK_ERR_UNSUPPORTED;
  }
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= 64) {
    set_error(std::string("cudaGetDevice: ") + cudaGetErrorString(e));
    return HACK_ERR_CUDA;
  }
  float* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_ptr[dev]) {
      // set-up, once per device, with that device current: resolve the array's device address
      float* ptr = nullptr;
      e = cudaGetSymbolAddress((void**)&ptr, g_noalloc_scratch);
      if (e != cudaSuccess || !ptr) {
        set_error(std::string("cudaGetSymbolAddress(scratch): ") + cudaGetErrorString(e));
        return HACK_ERR_CUDA;
      }
      g_scratch_ptr[dev] = ptr;
    }
    scratch = g_scratch_ptr[dev];
  }
  DenseArgs a;
  a.n_queries = n_queries;
  a.n_cand = n_cand;
  a.n_obs_rows = n_obs < n_queries ? n_obs : n_queries;
  a.chunks_per_row = (n_cand + kChunk - 1) / kChunk;
  a.sm_scale = sm_scale > 0.f ? sm_scale : 1.0f / std::sqrt((float)head_dim);
  cudaStream_t st = (cudaStream_t)stream;
  if (dtype == HACK_F32)
    e = head_dim == 64 ? run<float, 64>(a, n_rows, q, k_cand, scratch, scores, score_stride, st)
                       : run<float, 128>(a, n_rows, q, k_cand, scratch, scores, score_stride, st);
  else
    e = head_dim == 64 ? run<__nv_bfloat16, 64>(a, n_rows, q, k_cand, scratch, scores, score_stride, st)
                       : run<__nv_bfloat16, 128>(a, n_rows, q, k_cand, scratch, scores, score_stride, st);
  if (e != cudaSuccess) {
    set_error(std::string("hack_score_noalloc launch: ") + cudaGetErrorString(e));
    return HACK_ERR_CUDA;
  }
  return HACK_OK;
}
