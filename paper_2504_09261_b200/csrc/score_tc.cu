// Subset-attention importance scores (Eq. 9 and the TOPK argument of Eq. 10-11) for bf16 caches
// on the 5th-generation tensor cores.
//
// The logits of 128 candidate keys against the (at most 32) observation rows are one
// tcgen05.mma chain: A = the key tile [128 x D] as TMA wrote it (K-major, 128-byte swizzle),
// B = the observation rows [32 x D] placed in shared memory in the same swizzled layout,
// accumulator [128 lanes x 32 columns] fp32 in tensor memory, so that thread r of the CTA reads
// all 32 logits of key r with one tcgen05.ld.
//
// The full-row softmax needs statistics over all T' candidates, so the kernel runs twice per
// step: MODE 1 publishes per-chunk (max, sum-exp) of every observation row; MODE 2 merges the
// partials of its head, forms the logits again (the keys come from L2 the second time) and
// writes s_j = sum_i exp(z_ij - m_i) / l_i.  Nothing of size T' x N_obs is ever stored.
//
// A chunk never straddles the stored part and the new part of the candidate list: chunks
// 0..ceil(L/128)-1 cover the stored rows of the head in the cache plane, the following ones the
// new scale's rows in the caller's K tensor; lanes past the end of a part are masked.
#include <cuda.h>

#include <algorithm>

#include "hack_internal.h"
#include "tc_ptx.cuh"

namespace hack {
namespace {

using namespace ptx;

constexpr int kChunkTc = 128;
constexpr long long kScoreWaitCycles = 2000000000ll;   // about one second

__device__ __forceinline__ bool wait_bounded(uint64_t* bar, uint32_t parity, int* status, int code) {
  const uint32_t addr = smem_u32(bar);
  const long long t0 = clock64();
  for (uint32_t it = 0;; ++it) {
    if (mbar_try_wait(addr, parity)) return true;
    if ((it & 255u) == 255u && clock64() - t0 > kScoreWaitCycles) break;
  }
  atomicExch(status, code);
  return false;
}

template <int D, int MODE>
__global__ void __launch_bounds__(kChunkTc)
score_tc_kernel(const __grid_constant__ CUtensorMap tm_cache, const __grid_constant__ CUtensorMap tm_new,
                const StepArgs a, const __nv_bfloat16* __restrict__ q, float* __restrict__ partials,
                int max_chunks, float* __restrict__ scores) {
  constexpr int SUB = D / 64;                        // 64-column (128-byte) sub-tiles per row
  constexpr uint32_t K_SUB_BYTES = kChunkTc * 128;   // 128 keys x 128 bytes
  constexpr uint32_t Q_SUB_BYTES = kMaxObs * 128;    // 32 observation rows x 128 bytes
  constexpr uint32_t K_BYTES = SUB * K_SUB_BYTES;

  const int bh = blockIdx.y;
  const int ctx = a.is_ctx[bh % a.n_heads];
  if (!a.trig[ctx]) return;
  const int stored = a.stored[ctx];
  const int n_sc = (stored + kChunkTc - 1) / kChunkTc;
  const int n_nc = (a.n_new + kChunkTc - 1) / kChunkTc;
  const int chunk = blockIdx.x;
  if (chunk >= n_sc + n_nc) return;
  const bool from_cache = chunk < n_sc;
  const int part_row = (from_cache ? chunk : chunk - n_sc) * kChunkTc;
  const int valid = min(kChunkTc, (from_cache ? stored : a.n_new) - part_row);
  const int tma_row = (from_cache ? a.row_off[bh] : bh * a.n_new) + part_row;
  const int j_base = (from_cache ? 0 : stored) + part_row;

  extern __shared__ unsigned char smem_dyn[];
  const uint32_t raw = smem_u32(smem_dyn);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* sm = smem_dyn + (base - raw);
  const uint32_t k_sm = base;
  const uint32_t q_sm = base + K_BYTES;
  float* zt = reinterpret_cast<float*>(sm);          // [32][128] logits, reuses the key tile

  __shared__ uint64_t bar_full, bar_mma;
  __shared__ uint32_t tmem_slot;
  __shared__ float red_m[4][kMaxObs], red_l[4][kMaxObs];
  __shared__ float row_m[kMaxObs], row_inv_l[kMaxObs];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    mbar_init(smem_u32(&bar_full), 1);
    mbar_init(smem_u32(&bar_mma), 1);
    fence_barrier_init();
    fence_proxy_async();
    const CUtensorMap* tm = from_cache ? &tm_cache : &tm_new;
    mbar_expect_tx(smem_u32(&bar_full), K_BYTES);
#pragma unroll
    for (int c = 0; c < SUB; ++c)
      tma_load_2d(k_sm + c * K_SUB_BYTES, tm, c * 64, tma_row, smem_u32(&bar_full));
  }
  // observation rows floor(i * N_k / n) into the swizzled B tile; unused rows are zero
  for (int v = tid; v < kMaxObs * (D / 8); v += kChunkTc) {
    const int i = v / (D / 8), c = v % (D / 8);
    uint4 val = make_uint4(0, 0, 0, 0);
    if (i < a.n_obs_rows) {
      const int row = (int)(((long long)i * a.n_new) / a.n_obs_rows);
      val = *reinterpret_cast<const uint4*>(q + ((size_t)bh * a.n_new + row) * D + c * 8);
    }
    const uint32_t off = (c / 8) * Q_SUB_BYTES + i * 128 + (((c % 8) ^ (i & 7)) << 4);
    *reinterpret_cast<uint4*>(sm + K_BYTES + off) = val;
  }
  fence_proxy_async();
  if (warp == 0) {
    tmem_alloc(smem_u32(&tmem_slot), 32);
    tmem_relinquish();
  }
  if (MODE == 2) {
    // merge the per-chunk partials of this head into the statistics of the full rows
    const int n_chunks = n_sc + n_nc;
    float m = -INFINITY, l = 0.f;
    if (lane < a.n_obs_rows) {
      const float* p = partials + ((size_t)bh * max_chunks * kMaxObs + lane) * 2;
      for (int c = warp; c < n_chunks; c += 4) {
        const float2 ml = *reinterpret_cast<const float2*>(p + (size_t)c * kMaxObs * 2);
        const float mn = fmaxf(m, ml.x);
        l = l * __expf(m - mn) + ml.y * __expf(ml.x - mn);
        m = mn;
      }
    }
    red_m[warp][lane] = m;
    red_l[warp][lane] = l;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);
  if (MODE == 2 && tid < kMaxObs) {
    float m = -INFINITY;
#pragma unroll
    for (int w = 0; w < 4; ++w) m = fmaxf(m, red_m[w][tid]);
    float l = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) l += red_l[w][tid] == 0.f ? 0.f : red_l[w][tid] * __expf(red_m[w][tid] - m);
    row_m[tid] = m;
    row_inv_l[tid] = 1.f / l;
  }

  bool ok = true;
  if (tid == 0) {
    ok = wait_bounded(&bar_full, 0, a.status, 11);
    if (ok) {
      tc_fence_after();
      constexpr uint32_t IDESC = idesc_bf16_f32(kChunkTc, kMaxObs, 0);
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk) {
        const uint32_t ko = (kk / 4) * K_SUB_BYTES + (kk % 4) * 32;
        const uint32_t qo = (kk / 4) * Q_SUB_BYTES + (kk % 4) * 32;
        mma_ss(tmem, smem_desc_sw128(k_sm + ko, 16, 1024), smem_desc_sw128(q_sm + qo, 16, 1024), IDESC, kk > 0);
      }
    }
    mma_commit(smem_u32(&bar_mma));      // arrives at once if nothing was issued
  }
  ok = wait_bounded(&bar_mma, 0, a.status, 12);
  ok = __syncthreads_and(ok);            // also publishes row_m / row_inv_l
  if (ok) {
    tc_fence_after();
    uint32_t acc[kMaxObs];
    tmem_ld32(tmem + (static_cast<uint32_t>(warp * 32) << 16), acc);
    tmem_wait_ld();
    const bool live = tid < valid;
    if (MODE == 1) {
#pragma unroll
      for (int i = 0; i < kMaxObs; ++i)
        zt[i * kChunkTc + tid] = live ? __uint_as_float(acc[i]) * a.sm_scale : -INFINITY;
      __syncthreads();
      for (int i = warp; i < a.n_obs_rows; i += 4) {
        float z[4];
        float m = -INFINITY;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          z[u] = zt[i * kChunkTc + u * 32 + lane];
          m = fmaxf(m, z[u]);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        float l = 0.f;
#pragma unroll
        for (int u = 0; u < 4; ++u) l += __expf(z[u] - m);      // exp(-inf) = 0 for masked lanes
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
        if (lane == 0)
          *reinterpret_cast<float2*>(partials + (((size_t)bh * max_chunks + chunk) * kMaxObs + i) * 2) =
              make_float2(m, l);
      }
    } else {
      float s = 0.f;
#pragma unroll
      for (int i = 0; i < kMaxObs; ++i) {
        if (i < a.n_obs_rows)
          s += __expf(fmaf(__uint_as_float(acc[i]), a.sm_scale, -row_m[i])) * row_inv_l[i];
      }
      if (live) scores[(size_t)bh * a.cand_stride + j_base + tid] = s;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem, 32);
  }
}

template <int D>
int launch_t(const StepArgs& a, const CUtensorMap& tm_cache, const CUtensorMap& tm_new, const void* q,
             float* scores, const Scratch& s, cudaStream_t st) {
  int chunks = 0;
  for (int t = 0; t < 2; ++t)
    if (a.trig[t])
      chunks = std::max(chunks, (a.stored[t] + kChunkTc - 1) / kChunkTc + (a.n_new + kChunkTc - 1) / kChunkTc);
  if (chunks > s.max_chunks) return -1;
  const size_t smem = 1024 + (size_t)(D / 64) * (kChunkTc + kMaxObs) * 128;
  static bool attr_set = false;
  if (!attr_set) {
    cudaFuncSetAttribute(score_tc_kernel<D, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    cudaFuncSetAttribute(score_tc_kernel<D, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    attr_set = true;
  }
  const dim3 grid(chunks, a.batch * a.n_heads);
  const __nv_bfloat16* qp = static_cast<const __nv_bfloat16*>(q);
  score_tc_kernel<D, 1><<<grid, kChunkTc, smem, st>>>(tm_cache, tm_new, a, qp, s.partials, s.max_chunks, scores);
  score_tc_kernel<D, 2><<<grid, kChunkTc, smem, st>>>(tm_cache, tm_new, a, qp, s.partials, s.max_chunks, scores);
  return cudaGetLastError() == cudaSuccess ? 2 : -1;
}

}  // namespace

int launch_score_tc(const StepArgs& a, const void* q, const void* k_new, float* scores, const Scratch& s,
                    cudaStream_t st) {
  CUtensorMap tm_new;
  if (!make_rows_map(&tm_new, k_new, (uint64_t)a.batch * a.n_heads * a.n_new, a.head_dim)) return -1;
  const CUtensorMap& tm_cache = *static_cast<const CUtensorMap*>(a.k_map);
  return a.head_dim == 128 ? launch_t<128>(a, tm_cache, tm_new, q, scores, s, st)
                           : launch_t<64>(a, tm_cache, tm_new, q, scores, s, st);
}

}  // namespace hack
