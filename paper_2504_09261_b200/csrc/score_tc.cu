// Subset-attention importance scores (Eq. 9 and the TOPK argument of Eq. 10-11) for bf16 caches
// on the 5th-generation tensor cores.
//
// The logits of 128 candidate keys against the (at most 32) observation rows are one
// tcgen05.mma chain: A = the key tile [128 x D] as TMA wrote it (K-major, 128-byte swizzle),
// B = the observation rows [32 x D] placed in shared memory in the same swizzled layout,
// accumulator [128 lanes x 32 columns] fp32 in tensor memory, so that one thread reads all 32
// logits of one key with a single tcgen05.ld.
//
// A CTA serves a run of consecutive 128-key chunks of one head through a pipeline:
//   warp 0    : TMA producer, key tiles through a ring of shared-memory stages
//   warp 1    : tcgen05.mma issuer (owns the TMEM allocation: four accumulator buffers)
//   warps 2-5 : consumers, thread r <-> key r of the chunk
//
// The full-row softmax needs statistics over all T' candidates, so the kernel runs twice per
// step.  MODE 1: every consumer thread keeps a running (max, sum-exp) per observation row over
// the keys it sees; at the end of the run the CTA folds them into one partial per row.  MODE 2
// merges the partials of its head, forms the logits again (the keys come out of L2 this time)
// and writes s_j = sum_i exp(z_ij - m_i) / l_i.  Nothing of size T' x N_obs is ever stored.
//
// A chunk never straddles the stored part and the new part of the candidate list: chunks
// 0..ceil(L/128)-1 cover the stored rows of the head in the cache plane, the following ones the
// new scale's rows in the caller's K tensor; lanes past the end of a part are masked.
// Every mbarrier wait is bounded; on expiry the CTA raises the status word and winds down.
#include <cuda.h>

#include <algorithm>

#include "hack_internal.h"
#include "tc_ptx.cuh"

namespace hack {
namespace {

using namespace ptx;

constexpr int kChunkTc = 128;
constexpr int kScoreThreads = 192;
constexpr int kAccBufs = 4;
constexpr uint32_t kDrainSpins = 1u << 22;

struct ScoreBars {
  uint64_t full[4], empty[4];
  uint64_t acc_full[kAccBufs], acc_free[kAccBufs];
  uint64_t drain;
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, ScoreBars* b, int* status, int code, long long limit) {
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

__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
// All 128 consumers meet; true when `ok` holds for every one of them.
__device__ __forceinline__ bool consumer_all(bool ok) {
  uint32_t r;
  asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.and.pred p, 1, 128, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(r) : "r"((uint32_t)ok) : "memory");
  return r != 0;
}

template <int D, int MODE>
__global__ void __launch_bounds__(kScoreThreads)
score_tc_kernel(const __grid_constant__ CUtensorMap tm_cache, const __grid_constant__ CUtensorMap tm_new,
                const StepArgs a, const __nv_bfloat16* __restrict__ q, float* __restrict__ partials,
                int max_chunks, int chunks_per_cta, float* __restrict__ scores) {
  constexpr int SUB = D / 64;                        // 64-column (128-byte) sub-tiles per row
  constexpr int STAGES = D == 128 ? 3 : 4;
  constexpr uint32_t K_SUB_BYTES = kChunkTc * 128;   // 128 keys x 128 bytes
  constexpr uint32_t Q_SUB_BYTES = kMaxObs * 128;    // 32 observation rows x 128 bytes
  constexpr uint32_t K_BYTES = SUB * K_SUB_BYTES;
  static_assert(STAGES * K_BYTES >= 2 * kMaxObs * kChunkTc * sizeof(float), "ring is reused for the final fold");

  pdl_wait();      // every CTA waits, so that this grid never completes before its predecessor
  const int bh = blockIdx.y;
  const int ctx = a.is_ctx[bh % a.n_heads];
  if (!a.trig[ctx]) return;
  const int stored = a.stored[ctx];
  const int n_sc = (stored + kChunkTc - 1) / kChunkTc;
  const int n_chunks = n_sc + (a.n_new + kChunkTc - 1) / kChunkTc;
  const int c_begin = blockIdx.x * chunks_per_cta;
  if (c_begin >= n_chunks) return;
  const int n_run = min(chunks_per_cta, n_chunks - c_begin);
  const float zscale = a.sm_scale * 1.4426950408889634f;      // logits in log2 units

  extern __shared__ unsigned char smem_dyn[];
  const uint32_t raw = smem_u32(smem_dyn);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* sm = smem_dyn + (base - raw);
  const uint32_t k_sm = base;
  const uint32_t q_sm = base + STAGES * K_BYTES;
  ScoreBars* bars = reinterpret_cast<ScoreBars*>(sm + STAGES * K_BYTES + SUB * Q_SUB_BYTES);
  float* fold_m = reinterpret_cast<float*>(sm);                 // [32][128], reuses the ring
  float* fold_l = fold_m + kMaxObs * kChunkTc;
  __shared__ float red_m[4][kMaxObs], red_l[4][kMaxObs];
  __shared__ float row_m[kMaxObs], row_inv_l[kMaxObs];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(smem_u32(&bars->full[s]), 1); mbar_init(smem_u32(&bars->empty[s]), 1); }
    for (int b = 0; b < kAccBufs; ++b) { mbar_init(smem_u32(&bars->acc_full[b]), 1); mbar_init(smem_u32(&bars->acc_free[b]), kChunkTc); }
    mbar_init(smem_u32(&bars->drain), 1);
    bars->abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  // observation rows (floor(i * N_k / n) under the uniform rule) into the swizzled B tile; unused rows are zero
  for (int v = tid; v < kMaxObs * (D / 8); v += kScoreThreads) {
    const int i = v / (D / 8), c = v % (D / 8);
    uint4 val = make_uint4(0, 0, 0, 0);
    if (i < a.n_obs_rows) {
      const int row = obs_row(a, i);
      val = *reinterpret_cast<const uint4*>(q + ((size_t)bh * a.n_new + row) * D + c * 8);
    }
    const uint32_t off = (c / 8) * Q_SUB_BYTES + i * 128 + (((c % 8) ^ (i & 7)) << 4);
    *reinterpret_cast<uint4*>(sm + STAGES * K_BYTES + off) = val;
  }
  fence_proxy_async();
  if (warp == 1) {
    tmem_alloc(smem_u32(&bars->tmem_base), kAccBufs * kMaxObs);
    tmem_relinquish();
  }
  if (MODE == 2 && warp >= 2) {
    // merge the partials of this head (one per CTA of pass 1) into the statistics of the full rows
    const int w = warp - 2;
    const int n_parts = (n_chunks + chunks_per_cta - 1) / chunks_per_cta;
    float m = -INFINITY, l = 0.f;
    if (lane < a.n_obs_rows) {
      const float* p = partials + ((size_t)bh * max_chunks * kMaxObs + lane) * 2;
      for (int c = w; c < n_parts; c += 4) {
        const float2 ml = *reinterpret_cast<const float2*>(p + (size_t)c * kMaxObs * 2);
        const float mn = fmaxf(m, ml.x);
        l = l * ex2(m - mn) + ml.y * ex2(ml.x - mn);
        m = mn;
      }
    }
    red_m[w][lane] = m;
    red_l[w][lane] = l;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&bars->tmem_base);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      prefetch_tensormap(&tm_cache);
      prefetch_tensormap(&tm_new);
      int issued = 0;
      bool ok = true;
      for (int i = 0; i < n_run; ++i) {
        const int s = i % STAGES;
        ok = wait_bar(&bars->empty[s], ((i / STAGES) & 1) ^ 1, bars, a.status, 11, a.wait_cycles);
        if (!ok) break;
        const int chunk = c_begin + i;
        const bool from_cache = chunk < n_sc;
        const CUtensorMap* tm = from_cache ? &tm_cache : &tm_new;
        const int row = from_cache ? a.row_off[bh] + chunk * kChunkTc : bh * a.n_new + (chunk - n_sc) * kChunkTc;
        const uint32_t bar = smem_u32(&bars->full[s]);
        mbar_expect_tx(bar, K_BYTES);
#pragma unroll
        for (int c = 0; c < SUB; ++c) tma_load_2d(k_sm + s * K_BYTES + c * K_SUB_BYTES, tm, c * 64, row, bar);
        ++issued;
      }
      if (!ok) {
        // give the copies already in flight a bounded chance to land before the CTA leaves
        for (int i = max(0, issued - STAGES); i < issued; ++i) {
          const uint32_t bar = smem_u32(&bars->full[i % STAGES]);
          for (uint32_t it = 0; it < kDrainSpins && !mbar_try_wait(bar, (i / STAGES) & 1); ++it) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t IDESC = idesc_bf16_f32(kChunkTc, kMaxObs, 0);
      const uint64_t q_desc = smem_desc_sw128(q_sm, 16, 1024);
      bool ok = true;
      for (int i = 0; i < n_run && ok; ++i) {
        const int s = i % STAGES, b = i % kAccBufs;
        ok = wait_bar(&bars->full[s], (i / STAGES) & 1, bars, a.status, 12, a.wait_cycles);
        if (ok) ok = wait_bar(&bars->acc_free[b], ((i / kAccBufs) & 1) ^ 1, bars, a.status, 13, a.wait_cycles);
        if (!ok) break;
        tc_fence_after();
        const uint64_t k_desc = smem_desc_sw128(k_sm + s * K_BYTES, 16, 1024);
        if constexpr (D == 128) mma_ss_chain8_b32rows(tmem + b * kMaxObs, k_desc, q_desc, IDESC, 0);
        else mma_ss_chain4(tmem + b * kMaxObs, k_desc, q_desc, IDESC, 0);
        mma_commit(smem_u32(&bars->empty[s]));
        mma_commit(smem_u32(&bars->acc_full[b]));
      }
      if (!ok) {
        // wait (bounded) for what was issued, so that TMEM can be released safely
        mma_commit(smem_u32(&bars->drain));
        for (uint32_t it = 0; it < kDrainSpins && !mbar_try_wait(smem_u32(&bars->drain), 0); ++it) {}
      }
    }
  } else {
    // ------------------------------------------------------------------ consumers
    const int w = warp - 2;
    const int ct = tid - 64;                                  // 0..127
    const int quad = warp & 3;                                // TMEM lane quadrant this warp may read
    const int key_row = quad * 32 + lane;                     // key of the chunk this thread owns
    const uint32_t t_lane = tmem + (static_cast<uint32_t>(quad * 32) << 16);
    float rm[kMaxObs], rl[kMaxObs];                           // MODE 1: running max / sum; MODE 2: m_i, 1/l_i
    if (MODE == 1) {
#pragma unroll
      for (int i = 0; i < kMaxObs; ++i) { rm[i] = -INFINITY; rl[i] = 0.f; }
    } else {
      if (ct < kMaxObs) {
        float m = -INFINITY;
#pragma unroll
        for (int x = 0; x < 4; ++x) m = fmaxf(m, red_m[x][ct]);
        float l = 0.f;
#pragma unroll
        for (int x = 0; x < 4; ++x) l += red_l[x][ct] == 0.f ? 0.f : red_l[x][ct] * ex2(red_m[x][ct] - m);
        row_m[ct] = m;
        row_inv_l[ct] = 1.f / l;
      }
      consumer_sync();
#pragma unroll
      for (int i = 0; i < kMaxObs; ++i) {        // rows past n_obs_rows are padding: weight 0, finite reference
        rm[i] = i < a.n_obs_rows ? row_m[i] : 0.f;
        rl[i] = i < a.n_obs_rows ? row_inv_l[i] : 0.f;
      }
    }
    bool ok = true;
    for (int i = 0; i < n_run; ++i) {
      const int b = i % kAccBufs;
      ok = __all_sync(0xffffffffu, wait_bar(&bars->acc_full[b], (i / kAccBufs) & 1, bars, a.status, 14, a.wait_cycles));
      if (!ok) break;
      tc_fence_after();
      uint32_t acc[kMaxObs];
      tmem_ld32(t_lane + b * kMaxObs, acc);
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive(smem_u32(&bars->acc_free[b]));
      const int chunk = c_begin + i;
      const bool from_cache = chunk < n_sc;
      const int part_row = (from_cache ? chunk : chunk - n_sc) * kChunkTc;
      const bool live = part_row + key_row < (from_cache ? stored : a.n_new);
      if (MODE == 1) {
        if (live) {
#pragma unroll
          for (int r = 0; r < kMaxObs; ++r) {
            const float z = __uint_as_float(acc[r]) * zscale;
            const float mn = fmaxf(rm[r], z);
            rl[r] = rl[r] * ex2(rm[r] - mn) + ex2(z - mn);
            rm[r] = mn;
          }
        }
      } else {
        float s = 0.f;
#pragma unroll
        for (int r = 0; r < kMaxObs; ++r) s = fmaf(ex2(fmaf(__uint_as_float(acc[r]), zscale, -rm[r])), rl[r], s);
        if (live) {
          float* dst = scores + (size_t)bh * a.cand_stride + (from_cache ? 0 : stored) + part_row + key_row;
          *dst = a.score_accumulate ? *dst + s : s;
        }
      }
    }
    // one warp's wait may have given up while another's completed: the fold below meets on the
    // consumers' named barrier, so all 128 consumers take the same branch
    const bool all_ok = MODE == 1 ? consumer_all(ok) : ok;
    if (MODE == 1 && all_ok) {
      // fold the 128 per-thread statistics of every row into one partial for this CTA; the last
      // accumulator has been read, so every MMA is complete and the ring can be reused
#pragma unroll
      for (int r = 0; r < kMaxObs; ++r) { fold_m[r * kChunkTc + ct] = rm[r]; fold_l[r * kChunkTc + ct] = rl[r]; }
      consumer_sync();
      for (int r = w; r < a.n_obs_rows; r += 4) {
        float m4[4], l4[4];
        float m = -INFINITY;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          m4[u] = fold_m[r * kChunkTc + u * 32 + lane];
          l4[u] = fold_l[r * kChunkTc + u * 32 + lane];
          m = fmaxf(m, m4[u]);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        float l = 0.f;
#pragma unroll
        for (int u = 0; u < 4; ++u) l += l4[u] == 0.f ? 0.f : l4[u] * ex2(m4[u] - m);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
        if (lane == 0)
          *reinterpret_cast<float2*>(partials + (((size_t)bh * max_chunks + blockIdx.x) * kMaxObs + r) * 2) =
              make_float2(m, l);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, kAccBufs * kMaxObs);
  }
}

template <int D>
int launch_t(const StepArgs& a, const CUtensorMap& tm_cache, const CUtensorMap& tm_new, const void* q,
             float* scores, const Scratch& s, cudaStream_t st) {
  constexpr int STAGES = D == 128 ? 3 : 4;
  const int n_new_chunks = (a.n_new + kChunkTc - 1) / kChunkTc;
  int max_chunks = 0;
  long long total = 0;
  const int heads = a.batch * a.n_heads;
  for (int t = 0; t < 2; ++t)
    if (a.trig[t]) {
      const int c = (a.stored[t] + kChunkTc - 1) / kChunkTc + n_new_chunks;
      max_chunks = std::max(max_chunks, c);
      total += (long long)c * heads / 2;             // the split between the types is not known here
    }
  // about two CTAs per SM over the whole grid, each with a run long enough to fill its pipeline
  const int two_per_sm = 2 * sm_count();
  int per_cta = (int)((total + two_per_sm - 1) / two_per_sm);
  per_cta = std::max(per_cta, 2);
  const int splits = (max_chunks + per_cta - 1) / per_cta;
  if (splits > s.max_chunks) {
    set_error("scoring: more CTAs per head than the partial-statistics scratch holds");
    return -1;
  }
  const size_t smem = 1024 + (size_t)STAGES * (D / 64) * kChunkTc * 128 + (size_t)(D / 64) * kMaxObs * 128 +
                      sizeof(ScoreBars) + 16;
  if (!allow_dynamic_smem(score_tc_kernel<D, 1>, smem)) return -1;
  if (!allow_dynamic_smem(score_tc_kernel<D, 2>, smem)) return -1;
  const dim3 grid(splits, heads);
  const __nv_bfloat16* qp = static_cast<const __nv_bfloat16*>(q);
  launch_k(score_tc_kernel<D, 1>, grid, kScoreThreads, smem, st, tm_cache, tm_new, a, qp, s.partials, s.max_chunks, per_cta, scores);
  launch_k(score_tc_kernel<D, 2>, grid, kScoreThreads, smem, st, tm_cache, tm_new, a, qp, s.partials, s.max_chunks, per_cta, scores);
  return launched(2);
}

}  // namespace

int launch_score_tc(const StepArgs& a, const void* q, const void* k_new, float* scores, const Scratch& s,
                    cudaStream_t st) {
  CUtensorMap tm_new;
  if (!make_rows_map(&tm_new, k_new, (uint64_t)a.batch * a.n_heads * a.n_new, a.head_dim)) {
    set_error("scoring: cuTensorMapEncodeTiled failed for the new scale's keys");
    return -1;
  }
  const CUtensorMap& tm_cache = *static_cast<const CUtensorMap*>(a.k_map);
  return a.head_dim == 128 ? launch_t<128>(a, tm_cache, tm_new, q, scores, s, st)
                           : launch_t<64>(a, tm_cache, tm_new, q, scores, s, st);
}

}  // namespace hack
