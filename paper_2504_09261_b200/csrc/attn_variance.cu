// Attention variance of every head (Eq. 6, offline head classification) for bf16 caches:
//   sigma = sum_j Var_i A[i, j],  A = Softmax(sm_scale * Q K^T), rows i = the step's queries,
//   columns j = the head's cached keys, variance over the queries (population variance).
//
// The row statistics of the softmax (reference maximum m_i and sum l_i of every query) come from the
// attention kernel, which has them anyway; this file turns them into the column statistics.  A CTA
// owns one block of 128 keys of one head and walks over all query tiles:
//   warp 0    : TMA producer (the key block once, the query tiles through a ring)
//   warp 1    : tcgen05.mma issuer; S^T = K_blk Q_tile^T, keys on the 128 TMEM lanes, queries on
//               128 columns, two accumulators so that the next MMA runs under the current read-out
//   warps 2-5 : consumers; thread r owns key r: it reads its 128 logits with tcgen05.ld, forms
//               p = exp2(c z - c m_i - log2 l_i) and adds p and p^2 to two registers
// so the sums over the queries stay inside one thread and nothing of size N x T is stored.  At the
// end the thread holds Var_i A[i, j] = sum p^2 / N - (sum p / N)^2 of its key; the CTA adds its 128
// variances and a second, tiny kernel adds the blocks of a head in a fixed order.
// Every mbarrier wait is bounded; on expiry the CTA raises the status word and winds down.
#include <cuda.h>

#include "hack_internal.h"
#include "tc_ptx.cuh"

namespace hack {
namespace {

using namespace ptx;

constexpr int kVarThreads = 192;
constexpr int kVarTile = 128;            // keys per CTA, queries per tile
constexpr int kQStages = 2;             // 96 KB of tiles at head_dim 128: two CTAs per SM
constexpr uint32_t kVarDrainSpins = 1u << 22;

struct VarBars {
  uint64_t k_full;
  uint64_t q_full[kQStages], q_empty[kQStages];
  uint64_t acc_full[2], acc_free[2];
  uint64_t drain;
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ bool var_wait(uint64_t* bar, uint32_t parity, VarBars* b, int* status, int code, long long limit) {
  const uint32_t addr = smem_u32(bar);
  const long long t0 = clock64();
  for (uint32_t it = 0;; ++it) {
    if (mbar_try_wait(addr, parity)) return true;
    if ((it & 63u) == 63u) {
      if (*reinterpret_cast<volatile int*>(&b->abort_flag)) return false;
      if (clock64() - t0 > limit) break;
    }
  }
  *reinterpret_cast<volatile int*>(&b->abort_flag) = 1;
  atomicExch(status, code);
  return false;
}

__device__ __forceinline__ void var_consumer_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

template <int D>
__global__ void __launch_bounds__(kVarThreads)
attn_colstats_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                     const StepArgs a, const float* __restrict__ row_stats, float* __restrict__ block_var,
                     int max_blocks) {
  constexpr int SUB = D / 64;
  constexpr uint32_t SUB_BYTES = kVarTile * 128;
  constexpr uint32_t TILE_BYTES = SUB * SUB_BYTES;

  pdl_wait();
  const int bh = blockIdx.y, kb = blockIdx.x;
  const int len = a.kept[a.is_ctx[bh % a.n_heads]];
  if (kb * kVarTile >= len) return;
  const int n_qt = (a.n_new + kVarTile - 1) / kVarTile;
  const float c = a.sm_scale * 1.4426950408889634f;

  extern __shared__ unsigned char smem_dyn[];
  const uint32_t raw = smem_u32(smem_dyn);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* sm = smem_dyn + (base - raw);
  const uint32_t k_sm = base;
  const uint32_t q_sm = base + TILE_BYTES;
  VarBars* bars = reinterpret_cast<VarBars*>(sm + (1 + kQStages) * TILE_BYTES);
  __shared__ __align__(16) float stat[2][kVarTile];   // -c m_i - log2 l_i of the query tile in accumulator b
  __shared__ float red[4];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    mbar_init(smem_u32(&bars->k_full), 1);
    for (int s = 0; s < kQStages; ++s) { mbar_init(smem_u32(&bars->q_full[s]), 1); mbar_init(smem_u32(&bars->q_empty[s]), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&bars->acc_full[b]), 1); mbar_init(smem_u32(&bars->acc_free[b]), kVarTile); }
    mbar_init(smem_u32(&bars->drain), 1);
    bars->abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&bars->tmem_base), 2 * kVarTile);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&bars->tmem_base);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      prefetch_tensormap(&tm_q);
      prefetch_tensormap(&tm_k);
      {
        const uint32_t bar = smem_u32(&bars->k_full);
        mbar_expect_tx(bar, TILE_BYTES);
        for (int s = 0; s < SUB; ++s) tma_load_2d(k_sm + s * SUB_BYTES, &tm_k, s * 64, a.row_off[bh] + kb * kVarTile, bar);
      }
      int issued = 0;
      bool ok = true;
      for (int t = 0; t < n_qt; ++t) {
        const int s = t % kQStages;
        ok = var_wait(&bars->q_empty[s], ((t / kQStages) & 1) ^ 1, bars, a.status, 31, a.wait_cycles);
        if (!ok) break;
        const uint32_t bar = smem_u32(&bars->q_full[s]);
        mbar_expect_tx(bar, TILE_BYTES);
        for (int x = 0; x < SUB; ++x)
          tma_load_2d(q_sm + s * TILE_BYTES + x * SUB_BYTES, &tm_q, x * 64, bh * a.n_new + t * kVarTile, bar);
        ++issued;
      }
      if (!ok) {
        // give the copies already in flight a bounded chance to land before the CTA leaves
        for (uint32_t it = 0; it < kVarDrainSpins && !mbar_try_wait(smem_u32(&bars->k_full), 0); ++it) {}
        for (int i = max(0, issued - kQStages); i < issued; ++i) {
          const uint32_t bar = smem_u32(&bars->q_full[i % kQStages]);
          for (uint32_t it = 0; it < kVarDrainSpins && !mbar_try_wait(bar, (i / kQStages) & 1); ++it) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t IDESC = idesc_bf16_f32(kVarTile, kVarTile, 0);      // A = keys, B = queries, both K-major
      const uint64_t k_desc = smem_desc_sw128(k_sm, 16, 1024);
      bool ok = var_wait(&bars->k_full, 0, bars, a.status, 32, a.wait_cycles);
      for (int t = 0; t < n_qt && ok; ++t) {
        const int s = t % kQStages, b = t & 1;
        ok = var_wait(&bars->q_full[s], (t / kQStages) & 1, bars, a.status, 33, a.wait_cycles);
        if (ok) ok = var_wait(&bars->acc_free[b], ((t >> 1) & 1) ^ 1, bars, a.status, 34, a.wait_cycles);
        if (!ok) break;
        tc_fence_after();
        const uint64_t q_desc = smem_desc_sw128(q_sm + s * TILE_BYTES, 16, 1024);
        if constexpr (D == 128) mma_ss_chain8(tmem + b * kVarTile, k_desc, q_desc, IDESC, 0);
        else mma_ss_chain4(tmem + b * kVarTile, k_desc, q_desc, IDESC, 0);
        mma_commit(smem_u32(&bars->q_empty[s]));
        mma_commit(smem_u32(&bars->acc_full[b]));
      }
      if (!ok) {
        mma_commit(smem_u32(&bars->drain));
        for (uint32_t it = 0; it < kVarDrainSpins && !mbar_try_wait(smem_u32(&bars->drain), 0); ++it) {}
      }
    }
  } else {
    // ------------------------------------------------------------------ consumers
    const int ct = tid - 64;                                  // 0..127
    const int quad = warp & 3;                                // TMEM lane quadrant this warp may read
    const int key_row = quad * 32 + lane;                     // key of the block this thread owns
    const uint32_t t_lane = tmem + (static_cast<uint32_t>(quad * 32) << 16);
    float sum_p = 0.f, sum_p2 = 0.f;
    bool ok = true;
    for (int t = 0; t < n_qt; ++t) {
      const int b = t & 1;
      {
        // statistics of query ct of this tile; queries past the end of the scale get weight 0
        const int qi = t * kVarTile + ct;
        float st = -INFINITY;                      // exp2(-inf) = 0
        if (qi < a.n_new) {
          const float2 ml = *reinterpret_cast<const float2*>(row_stats + ((size_t)bh * a.n_new + qi) * 2);
          st = -ml.x * c - __log2f(ml.y);          // p = exp2(c z - c m - log2 l): the division is in the exponent
        }
        stat[b][ct] = st;
      }
      var_consumer_sync();
      // a warp whose wait gave up keeps walking the loop, so that it still meets the other consumers
      // on the named barrier above and after the loop; it only stops touching the accumulators
      if (ok) ok = __all_sync(0xffffffffu, var_wait(&bars->acc_full[b], (t >> 1) & 1, bars, a.status, 35, a.wait_cycles));
      if (!ok) continue;
      tc_fence_after();
#pragma unroll
      for (int ch = 0; ch < kVarTile / 32; ++ch) {
        uint32_t acc[32];
        tmem_ld32(t_lane + b * kVarTile + ch * 32, acc);
        tmem_wait_ld();
        if (ch == kVarTile / 32 - 1) {
          tc_fence_before();
          mbar_arrive(smem_u32(&bars->acc_free[b]));
        }
#pragma unroll
        for (int i = 0; i < 32; i += 4) {
          const float4 st = *reinterpret_cast<const float4*>(&stat[b][ch * 32 + i]);
          const float p0 = ex2(fmaf(__uint_as_float(acc[i]), c, st.x));
          const float p1 = ex2(fmaf(__uint_as_float(acc[i + 1]), c, st.y));
          const float p2 = ex2(fmaf(__uint_as_float(acc[i + 2]), c, st.z));
          const float p3 = ex2(fmaf(__uint_as_float(acc[i + 3]), c, st.w));
          sum_p += (p0 + p1) + (p2 + p3);
          sum_p2 = fmaf(p0, p0, fmaf(p1, p1, fmaf(p2, p2, fmaf(p3, p3, sum_p2))));
        }
      }
    }
    // Var_i A[i, j] of this thread's key; keys past the end of the head count nothing (their sums
    // come from rows of another head and may have overflowed)
    const float inv_n = 1.f / (float)a.n_new;
    float var = 0.f;
    if (ok && kb * kVarTile + key_row < len) {
      const float mean = sum_p * inv_n;
      var = fmaxf(fmaf(-mean, mean, sum_p2 * inv_n), 0.f);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) var += __shfl_xor_sync(0xffffffffu, var, o);
    if (lane == 0) red[warp - 2] = ok ? var : NAN;           // a warp that gave up poisons the block's sum
    var_consumer_sync();
    if (ct == 0 && ok) block_var[(size_t)bh * max_blocks + kb] = (red[0] + red[1]) + (red[2] + red[3]);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 2 * kVarTile);
  }
}

// sigma of one head = sum of its key blocks' variances, added in block order by one warp.
__global__ void __launch_bounds__(32)
attn_variance_finish_kernel(const StepArgs a, const float* __restrict__ block_var, int max_blocks,
                            float* __restrict__ sigma) {
  pdl_wait();
  const int bh = blockIdx.x, lane = threadIdx.x;
  const int len = a.kept[a.is_ctx[bh % a.n_heads]];
  const int n_blocks = (len + kVarTile - 1) / kVarTile;
  float s = 0.f;
  for (int kb = lane; kb < n_blocks; kb += 32) s += block_var[(size_t)bh * max_blocks + kb];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if (lane == 0) sigma[bh] = s;
}

template <int D>
size_t var_smem_bytes() {
  return 1024 + (1 + kQStages) * (size_t)(D / 64) * kVarTile * 128 + sizeof(VarBars) + 64;
}

}  // namespace

int launch_attention_variance(const StepArgs& a, const void* q, const float* row_stats, float* block_var,
                              int max_blocks, float* sigma, cudaStream_t st) {
  CUtensorMap tm_q;
  if (!make_rows_map(&tm_q, q, (uint64_t)a.batch * a.n_heads * a.n_new, a.head_dim)) {
    set_error("attention variance: cuTensorMapEncodeTiled failed for the queries");
    return -1;
  }
  const CUtensorMap& tk = *static_cast<const CUtensorMap*>(a.k_map);
  const int bh = a.batch * a.n_heads;
  const int longest = a.kept[0] > a.kept[1] ? a.kept[0] : a.kept[1];
  const int n_blocks = (longest + kVarTile - 1) / kVarTile;
  if (n_blocks > max_blocks) {
    set_error("attention variance: cache longer than the scratch area");
    return -1;
  }
  const dim3 grid(n_blocks, bh);
  if (a.head_dim == 128) {
    if (!allow_dynamic_smem(attn_colstats_kernel<128>, var_smem_bytes<128>())) return -1;
    launch_k(attn_colstats_kernel<128>, grid, kVarThreads, var_smem_bytes<128>(), st, tm_q, tk, a, row_stats, block_var, max_blocks);
  } else {
    if (!allow_dynamic_smem(attn_colstats_kernel<64>, var_smem_bytes<64>())) return -1;
    launch_k(attn_colstats_kernel<64>, grid, kVarThreads, var_smem_bytes<64>(), st, tm_q, tk, a, row_stats, block_var, max_blocks);
  }
  launch_k(attn_variance_finish_kernel, bh, 32, 0, st, a, block_var, max_blocks, sigma);
  return launched(2);
}

}  // namespace hack
