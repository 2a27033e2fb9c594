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
#include "score_simt.cuh"

namespace hack {
namespace {

constexpr int kChunk = simt::kChunk;                      // candidate keys per CTA in pass 1
static_assert(simt::kObs == kMaxObs, "the shared SIMT body is built for 32 observation rows");
constexpr long long kMaxLogitRows = 65536;                // limit on n_rows * n_cand
constexpr int kMaxRows = 512;                             // limit on n_rows (batch * heads)
constexpr long long kLogitFloats = kMaxLogitRows * kMaxObs;                     // 2 Mi floats
constexpr long long kPartialFloats = (kMaxLogitRows / kChunk + kMaxRows) * kMaxObs * 2;
constexpr long long kScratchFloats = kLogitFloats + kPartialFloats;

// Scratch of the no-allocation entry point.  In host code this name is only a handle for
// cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) float g_noalloc_scratch[kScratchFloats];

struct DenseArgs {
  int n_queries, n_cand, n_obs_rows, chunks_per_row;
  float sm_scale;
};

// Pass 1 and pass 2 of the shared SIMT body (score_simt.cuh) on dense tensors: row-block `row` has
// n_queries query rows (observation row i = floor(i * n_queries / n)) and n_cand candidate keys.
template <typename T, int D>
__global__ void __launch_bounds__(kChunk)
noalloc_logits_kernel(const DenseArgs a, const T* __restrict__ q, const T* __restrict__ k_cand,
                      float* __restrict__ logits, float* __restrict__ partials) {
  const int row = blockIdx.y;
  const int chunk = blockIdx.x;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  simt::chunk_logits<T, D>(
      smem_raw, chunk * kChunk, a.n_cand, a.n_obs_rows, a.sm_scale,
      [&](int i) { return q + ((size_t)row * a.n_queries + (int)(((long long)i * a.n_queries) / a.n_obs_rows)) * D; },
      [&](int j) { return k_cand + ((size_t)row * a.n_cand + j) * D; },
      [&](int i, int j) -> float& { return logits[((size_t)row * kMaxObs + i) * a.n_cand + j]; },
      [&](int i) { return partials + (((size_t)row * a.chunks_per_row + chunk) * kMaxObs + i) * 2; });
}

__global__ void __launch_bounds__(256)
noalloc_reduce_kernel(const DenseArgs a, const float* __restrict__ logits,
                      const float* __restrict__ partials, float* __restrict__ scores, int score_stride) {
  const int row = blockIdx.y;
  __shared__ float row_m[kMaxObs], row_inv_l[kMaxObs];
  float s;
  if (simt::column_scores(
          row_m, row_inv_l, blockIdx.x * 256, a.n_cand, a.n_obs_rows, a.chunks_per_row,
          [&](int c, int i) { return partials + (((size_t)row * a.chunks_per_row + c) * kMaxObs + i) * 2; },
          [&](int i, int j) { return logits[((size_t)row * kMaxObs + i) * a.n_cand + j]; }, s))
    scores[(size_t)row * score_stride + blockIdx.x * 256 + threadIdx.x] = s;
}

// One scratch address per device, resolved on the first call made with that device current.
std::mutex g_setup_mutex;
float* g_scratch_ptr[64] = {nullptr};

template <typename T, int D>
cudaError_t run(const DenseArgs& a, int n_rows, const void* q, const void* k, float* scratch,
                float* scores, int score_stride, cudaStream_t st) {
  const size_t smem = simt::logits_smem_bytes<T, D>();
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
