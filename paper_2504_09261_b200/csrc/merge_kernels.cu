// Final-scale merge of contextual heads (the sentence after Eq. 10): the entries that the last
// step discards are folded into their nearest retained counterparts by similarity-weighted
// averaging.  Reading implemented here (the paper leaves all of it open): nearness = cosine
// similarity between keys, counterpart = the retained key with the largest similarity (lowest index
// among equals), weight w = max(similarity, 0), and for a retained entry c with assigned set E_c
//   k_c <- (k_c + sum_e w_e k_e) / (1 + sum_e w_e),   v_c likewise with the same weights.
// bf16 caches only.  Around the compaction of that step:
//   before it (the discarded rows are still in place):
//     merge_evicted_index_kernel  complement of the ascending kept list, per head
//     merge_prepare_kernel        copies the discarded K, V rows to scratch planes and takes the
//                                 inverse norms of the discarded and of the retained keys
//   after it (the retained rows are contiguous in the cache plane):
//     merge_assign_kernel         S = E K^T on tcgen05, discarded rows on the TMEM lanes: a thread
//                                 owns one discarded key and keeps the running arg-max of
//                                 S[e, c] / |k_c| over the retained tiles
//     merge_apply_kernel          a warp per 8 retained rows walks the assignments once and adds the
//                                 rows assigned to its rows in ascending order (no atomics: the
//                                 result does not depend on scheduling)
// Every mbarrier wait is bounded; on expiry the CTA raises the status word and winds down.
#include <cuda.h>

#include <type_traits>

#include "hack_internal.h"
#include "tc_ptx.cuh"

namespace hack {
namespace {

using namespace ptx;

constexpr int kIdxThreads = 1024;
constexpr int kPrepThreads = 256;
constexpr int kAssignThreads = 192;
constexpr int kTileM = 128;              // discarded rows per CTA, retained rows per tile
constexpr int kRing = 2;
constexpr int kApplyThreads = 256;
constexpr int kApplyRowsPerWarp = 8;     // retained rows per warp (64 per CTA)
constexpr int kApplyChunk = 2048;        // discarded entries staged in shared memory at a time
constexpr int kApplyHits = 256;          // entries a warp lists before it works them off
constexpr uint32_t kMergeDrainSpins = 1u << 22;

// ---------------------------------------------------------------- complement of the kept list
__global__ void __launch_bounds__(kIdxThreads)
merge_evicted_index_kernel(const StepArgs a, const MergeScratch ms, const int32_t* __restrict__ idx) {
  pdl_wait();
  const int bh = blockIdx.x;
  if (!a.is_ctx[bh % a.n_heads]) return;
  const int cand = a.cand[1], kept = a.kept[1];
  const int32_t* list = idx + (size_t)bh * a.kept_stride;
  int32_t* out = ms.ev_idx + (size_t)bh * ms.stride;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int per = (cand + kIdxThreads - 1) / kIdxThreads;
  const int j0 = min(tid * per, cand), j1 = min(j0 + per, cand);
  // first kept entry >= j0 (the list is ascending)
  int lo = 0, hi = kept;
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (list[mid] < j0) lo = mid + 1; else hi = mid;
  }
  int p = lo, gone = 0;
  for (int j = j0; j < j1; ++j) {
    if (p < kept && list[p] == j) ++p; else ++gone;
  }
  // exclusive prefix sum of `gone` over the CTA
  __shared__ int warp_sums[33];
  int incl = gone;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += n;
  }
  if (lane == 31) warp_sums[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const int w = warp_sums[lane];
    int wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += n;
    }
    warp_sums[lane] = wi - w;
  }
  __syncthreads();
  int pos = warp_sums[warp] + incl - gone;
  p = lo;
  for (int j = j0; j < j1; ++j) {
    if (p < kept && list[p] == j) ++p; else out[pos++] = j;
  }
}

// ---------------------------------------------------------------- scratch copies and inverse norms
template <int D>
__global__ void __launch_bounds__(kPrepThreads)
merge_prepare_kernel(const StepArgs a, const MergeScratch ms, const int32_t* __restrict__ idx,
                     const __nv_bfloat16* __restrict__ k_new, const __nv_bfloat16* __restrict__ v_new) {
  pdl_wait();
  const int bh = blockIdx.y;
  if (!a.is_ctx[bh % a.n_heads]) return;
  const int stored = a.stored[1], kept = a.kept[1], n_evict = a.cand[1] - kept;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = blockIdx.x * (kPrepThreads / 32) + warp;
  if (r >= n_evict + kept) return;
  const bool gone = r < n_evict;
  const int j = gone ? ms.ev_idx[(size_t)bh * ms.stride + r] : idx[(size_t)bh * a.kept_stride + (r - n_evict)];
  constexpr int E = D / 32;                                   // bf16 elements per lane
  using Vec = typename std::conditional<E == 4, uint2, uint32_t>::type;
  const size_t src_row = j < stored ? (size_t)a.row_off[bh] + j : (size_t)bh * a.n_new + (j - stored);
  const __nv_bfloat16* ksrc = (j < stored ? static_cast<const __nv_bfloat16*>(a.k_plane) : k_new) + src_row * D;
  const Vec kv = reinterpret_cast<const Vec*>(ksrc)[lane];
  const __nv_bfloat16* ke = reinterpret_cast<const __nv_bfloat16*>(&kv);
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < E; ++i) {
    const float x = __bfloat162float(ke[i]);
    s = fmaf(x, x, s);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  const float inv = s > 0.f ? 1.f / sqrtf(s) : 0.f;
  if (gone) {
    const __nv_bfloat16* vsrc = (j < stored ? static_cast<const __nv_bfloat16*>(a.v_plane) : v_new) + src_row * D;
    const size_t dst = ((size_t)bh * ms.stride + r) * D;
    reinterpret_cast<Vec*>(ms.ev_k + dst)[lane] = kv;
    reinterpret_cast<Vec*>(ms.ev_v + dst)[lane] = reinterpret_cast<const Vec*>(vsrc)[lane];
    if (lane == 0) ms.ev_inv_norm[(size_t)bh * ms.stride + r] = inv;
  } else if (lane == 0) {
    ms.kept_inv_norm[(size_t)bh * a.kept_stride + (r - n_evict)] = inv;
  }
}

// ---------------------------------------------------------------- nearest retained key on the tensor cores
struct AssignBars {
  uint64_t e_full;
  uint64_t k_full[kRing], k_empty[kRing];
  uint64_t acc_full[2], acc_free[2];
  uint64_t drain;
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ bool merge_wait(uint64_t* bar, uint32_t parity, AssignBars* b, int* status, int code, long long limit) {
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

__device__ __forceinline__ void merge_consumer_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

template <int D>
__global__ void __launch_bounds__(kAssignThreads)
merge_assign_kernel(const __grid_constant__ CUtensorMap tm_e, const __grid_constant__ CUtensorMap tm_k,
                    const StepArgs a, const MergeScratch ms) {
  constexpr int SUB = D / 64;
  constexpr uint32_t SUB_BYTES = kTileM * 128;
  constexpr uint32_t TILE_BYTES = SUB * SUB_BYTES;

  pdl_wait();
  const int bh = blockIdx.y, eb = blockIdx.x;
  if (!a.is_ctx[bh % a.n_heads]) return;
  const int kept = a.kept[1], n_evict = a.cand[1] - kept;
  if (eb * kTileM >= n_evict) return;
  const int n_kt = (kept + kTileM - 1) / kTileM;

  extern __shared__ unsigned char smem_dyn[];
  const uint32_t raw = smem_u32(smem_dyn);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* sm = smem_dyn + (base - raw);
  const uint32_t e_sm = base;
  const uint32_t k_sm = base + TILE_BYTES;
  AssignBars* bars = reinterpret_cast<AssignBars*>(sm + (1 + kRing) * TILE_BYTES);
  __shared__ __align__(16) float inv_c[2][kTileM];        // 1 / |k_c| of the retained tile in accumulator b

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    mbar_init(smem_u32(&bars->e_full), 1);
    for (int s = 0; s < kRing; ++s) { mbar_init(smem_u32(&bars->k_full[s]), 1); mbar_init(smem_u32(&bars->k_empty[s]), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&bars->acc_full[b]), 1); mbar_init(smem_u32(&bars->acc_free[b]), kTileM); }
    mbar_init(smem_u32(&bars->drain), 1);
    bars->abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&bars->tmem_base), 2 * kTileM);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&bars->tmem_base);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      prefetch_tensormap(&tm_e);
      prefetch_tensormap(&tm_k);
      {
        const uint32_t bar = smem_u32(&bars->e_full);
        mbar_expect_tx(bar, TILE_BYTES);
        for (int s = 0; s < SUB; ++s) tma_load_2d(e_sm + s * SUB_BYTES, &tm_e, s * 64, bh * ms.stride + eb * kTileM, bar);
      }
      int issued = 0;
      bool ok = true;
      for (int t = 0; t < n_kt; ++t) {
        const int s = t % kRing;
        ok = merge_wait(&bars->k_empty[s], ((t / kRing) & 1) ^ 1, bars, a.status, 41, a.wait_cycles);
        if (!ok) break;
        const uint32_t bar = smem_u32(&bars->k_full[s]);
        mbar_expect_tx(bar, TILE_BYTES);
        for (int x = 0; x < SUB; ++x)
          tma_load_2d(k_sm + s * TILE_BYTES + x * SUB_BYTES, &tm_k, x * 64, a.row_off[bh] + t * kTileM, bar);
        ++issued;
      }
      if (!ok) {
        for (uint32_t it = 0; it < kMergeDrainSpins && !mbar_try_wait(smem_u32(&bars->e_full), 0); ++it) {}
        for (int i = max(0, issued - kRing); i < issued; ++i) {
          const uint32_t bar = smem_u32(&bars->k_full[i % kRing]);
          for (uint32_t it = 0; it < kMergeDrainSpins && !mbar_try_wait(bar, (i / kRing) & 1); ++it) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t IDESC = idesc_bf16_f32(kTileM, kTileM, 0);     // A = discarded keys, B = retained keys, K-major
      const uint64_t e_desc = smem_desc_sw128(e_sm, 16, 1024);
      bool ok = merge_wait(&bars->e_full, 0, bars, a.status, 42, a.wait_cycles);
      for (int t = 0; t < n_kt && ok; ++t) {
        const int s = t % kRing, b = t & 1;
        ok = merge_wait(&bars->k_full[s], (t / kRing) & 1, bars, a.status, 43, a.wait_cycles);
        if (ok) ok = merge_wait(&bars->acc_free[b], ((t >> 1) & 1) ^ 1, bars, a.status, 44, a.wait_cycles);
        if (!ok) break;
        tc_fence_after();
        const uint64_t k_desc = smem_desc_sw128(k_sm + s * TILE_BYTES, 16, 1024);
        if constexpr (D == 128) mma_ss_chain8(tmem + b * kTileM, e_desc, k_desc, IDESC, 0);
        else mma_ss_chain4(tmem + b * kTileM, e_desc, k_desc, IDESC, 0);
        mma_commit(smem_u32(&bars->k_empty[s]));
        mma_commit(smem_u32(&bars->acc_full[b]));
      }
      if (!ok) {
        mma_commit(smem_u32(&bars->drain));
        for (uint32_t it = 0; it < kMergeDrainSpins && !mbar_try_wait(smem_u32(&bars->drain), 0); ++it) {}
      }
    }
  } else {
    // ------------------------------------------------------------------ consumers
    const int ct = tid - 64;                                  // 0..127
    const int quad = warp & 3;                                // TMEM lane quadrant this warp may read
    const int my_row = eb * kTileM + quad * 32 + lane;        // discarded entry this thread owns
    const uint32_t t_lane = tmem + (static_cast<uint32_t>(quad * 32) << 16);
    float best = -INFINITY;
    int arg = 0;
    bool ok = true;
    for (int t = 0; t < n_kt; ++t) {
      const int b = t & 1;
      {
        const int c = t * kTileM + ct;
        inv_c[b][ct] = c < kept ? ms.kept_inv_norm[(size_t)bh * a.kept_stride + c] : 0.f;
      }
      merge_consumer_sync();
      // a warp whose wait gave up keeps walking the loop, so that it still meets the other consumers
      // on the named barrier above; it only stops touching the accumulators
      if (ok) ok = __all_sync(0xffffffffu, merge_wait(&bars->acc_full[b], (t >> 1) & 1, bars, a.status, 45, a.wait_cycles));
      if (!ok) continue;
      tc_fence_after();
      const int n_valid = min(kTileM, kept - t * kTileM);
#pragma unroll
      for (int ch = 0; ch < kTileM / 32; ++ch) {
        uint32_t acc[32];
        tmem_ld32(t_lane + b * kTileM + ch * 32, acc);
        tmem_wait_ld();
        if (ch == kTileM / 32 - 1) {
          tc_fence_before();
          mbar_arrive(smem_u32(&bars->acc_free[b]));
        }
        if (n_valid == kTileM) {
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
            const float4 ic = *reinterpret_cast<const float4*>(&inv_c[b][ch * 32 + i]);
            const float v0 = __uint_as_float(acc[i]) * ic.x, v1 = __uint_as_float(acc[i + 1]) * ic.y;
            const float v2 = __uint_as_float(acc[i + 2]) * ic.z, v3 = __uint_as_float(acc[i + 3]) * ic.w;
            // strict comparisons in ascending column order: the lowest index wins among equals
            if (v0 > best) { best = v0; arg = t * kTileM + ch * 32 + i; }
            if (v1 > best) { best = v1; arg = t * kTileM + ch * 32 + i + 1; }
            if (v2 > best) { best = v2; arg = t * kTileM + ch * 32 + i + 2; }
            if (v3 > best) { best = v3; arg = t * kTileM + ch * 32 + i + 3; }
          }
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const float val = __uint_as_float(acc[i]) * inv_c[b][ch * 32 + i];
            if (ch * 32 + i < n_valid && val > best) {
              best = val;
              arg = t * kTileM + ch * 32 + i;
            }
          }
        }
      }
    }
    if (ok && my_row < n_evict) {
      const size_t o = (size_t)bh * ms.stride + my_row;
      ms.assign[o] = arg;
      ms.weight[o] = fmaxf(best * ms.ev_inv_norm[o], 0.f);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 2 * kTileM);
  }
}

// ---------------------------------------------------------------- weighted average into the retained rows
// A warp owns kApplyRowsPerWarp consecutive retained rows and walks the list of discarded entries
// once, listing those assigned to its rows; the listed rows are then fetched four at a time and
// added to the rows' fp32 accumulators in shared memory.  Entries are taken in ascending order,
// so a row's sum has one fixed order of additions.
template <int D>
__global__ void __launch_bounds__(kApplyThreads, 2)
merge_apply_kernel(const StepArgs a, const MergeScratch ms) {
  pdl_wait();
  const int bh = blockIdx.y;
  if (!a.is_ctx[bh % a.n_heads]) return;
  const int kept = a.kept[1], n_evict = a.cand[1] - kept;
  constexpr int E = D / 32;
  constexpr int R = kApplyRowsPerWarp;
  constexpr int kWarps = kApplyThreads / 32;
  using Vec = typename std::conditional<E == 4, uint2, uint32_t>::type;
  extern __shared__ __align__(16) unsigned char apply_smem[];
  float* acc_all = reinterpret_cast<float*>(apply_smem);                 // [warp][row][K | V][D]
  float* den_all = acc_all + kWarps * R * 2 * D;                          // [warp][row]
  int* s_assign = reinterpret_cast<int*>(den_all + kWarps * R);           // [kApplyChunk]
  float* s_weight = reinterpret_cast<float*>(s_assign + kApplyChunk);     // [kApplyChunk]
  int* s_hits = reinterpret_cast<int*>(s_weight + kApplyChunk);           // [warp][kApplyHits]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int c0 = (blockIdx.x * kWarps + warp) * R;
  float* acc = acc_all + warp * R * 2 * D;
  float* den = den_all + warp * R;
  for (int i = lane; i < R * 2 * D; i += 32) acc[i] = 0.f;
  if (lane < R) den[lane] = 0.f;
  int* hits = s_hits + warp * kApplyHits;                       // entries of this chunk assigned to this warp's rows
  // adds the listed entries, four at a time: their rows are fetched together (the latencies overlap), then added in order
  auto flush = [&](int base, int n_hits) {
    for (int h0 = 0; h0 < n_hits; h0 += 4) {
      Vec kv[4], vv[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (h0 + u < n_hits) {
          const size_t row = ((size_t)bh * ms.stride + base + hits[h0 + u]) * D;
          kv[u] = reinterpret_cast<const Vec*>(ms.ev_k + row)[lane];
          vv[u] = reinterpret_cast<const Vec*>(ms.ev_v + row)[lane];
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (h0 + u < n_hits) {
          const int el = hits[h0 + u];
          const int r = s_assign[el] - c0;
          const float w = s_weight[el];
          const __nv_bfloat16* ke = reinterpret_cast<const __nv_bfloat16*>(&kv[u]);
          const __nv_bfloat16* ve = reinterpret_cast<const __nv_bfloat16*>(&vv[u]);
          float* ak = acc + (r * 2) * D + lane * E;
          float* av = ak + D;
#pragma unroll
          for (int x = 0; x < E; ++x) {
            ak[x] = fmaf(w, __bfloat162float(ke[x]), ak[x]);
            av[x] = fmaf(w, __bfloat162float(ve[x]), av[x]);
          }
          if (lane == 0) den[r] += w;
        }
      }
    }
    __syncwarp();
  };
  for (int base = 0; base < n_evict; base += kApplyChunk) {
    const int n = min(kApplyChunk, n_evict - base);
    const int n_pad = (n + 127) & ~127;
    __syncthreads();
#pragma unroll 4
    for (int i = threadIdx.x; i < n_pad; i += kApplyThreads) {
      s_assign[i] = i < n ? ms.assign[(size_t)bh * ms.stride + base + i] : -1;
      s_weight[i] = i < n ? ms.weight[(size_t)bh * ms.stride + base + i] : 0.f;
    }
    __syncthreads();
    if (c0 >= kept) continue;
    // 128 entries per pass: a lane looks at four consecutive ones (entries past the chunk's end
    // were staged as -1); an entry with weight 0 adds nothing and needs no test here.  Hits go to
    // the warp's list in ascending order; the list is worked off when it fills and at the end.
    int n_hits = 0;
    for (int e4 = 0; e4 < n; e4 += 128) {
      const int4 as = *reinterpret_cast<const int4*>(&s_assign[e4 + lane * 4]);
      const uint32_t mine = ((unsigned)(as.x - c0) < (unsigned)R ? 1u : 0u) | ((unsigned)(as.y - c0) < (unsigned)R ? 2u : 0u) |
                            ((unsigned)(as.z - c0) < (unsigned)R ? 4u : 0u) | ((unsigned)(as.w - c0) < (unsigned)R ? 8u : 0u);
      if (!__any_sync(0xffffffffu, mine != 0u)) continue;
      if (n_hits + 128 > kApplyHits) {
        __syncwarp();
        flush(base, n_hits);
        n_hits = 0;
      }
      // position of this lane's hits = hits of the lower lanes (ascending entry order)
      const int cnt = __popc(mine);
      int incl = cnt;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      int pos = n_hits + incl - cnt;
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (mine & (1u << j)) hits[pos++] = e4 + lane * 4 + j;
      n_hits += __shfl_sync(0xffffffffu, incl, 31);
    }
    __syncwarp();
    flush(base, n_hits);
  }
  __syncwarp();
  // the rows that received something: all of them are fetched before any is written back
  Vec kv[R], vv[R];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    if (c0 + r < kept && den[r] != 0.f) {
      const size_t row = ((size_t)a.row_off[bh] + c0 + r) * D;
      kv[r] = reinterpret_cast<const Vec*>(static_cast<const __nv_bfloat16*>(a.k_plane) + row)[lane];
      vv[r] = reinterpret_cast<const Vec*>(static_cast<const __nv_bfloat16*>(a.v_plane) + row)[lane];
    }
  }
#pragma unroll
  for (int r = 0; r < R; ++r) {
    if (c0 + r < kept && den[r] != 0.f) {                      // else nothing was assigned: the row keeps its bits
      const float inv = 1.f / (1.f + den[r]);
      __nv_bfloat16* ke = reinterpret_cast<__nv_bfloat16*>(&kv[r]);
      __nv_bfloat16* ve = reinterpret_cast<__nv_bfloat16*>(&vv[r]);
      const float* ak = acc + (r * 2) * D + lane * E;
      const float* av = ak + D;
#pragma unroll
      for (int x = 0; x < E; ++x) {
        ke[x] = __float2bfloat16_rn((__bfloat162float(ke[x]) + ak[x]) * inv);
        ve[x] = __float2bfloat16_rn((__bfloat162float(ve[x]) + av[x]) * inv);
      }
      const size_t row = ((size_t)a.row_off[bh] + c0 + r) * D;
      reinterpret_cast<Vec*>(static_cast<__nv_bfloat16*>(a.k_plane) + row)[lane] = kv[r];
      reinterpret_cast<Vec*>(static_cast<__nv_bfloat16*>(a.v_plane) + row)[lane] = vv[r];
    }
  }
}

template <int D>
size_t apply_smem_bytes() {
  return ((size_t)(kApplyThreads / 32) * (kApplyRowsPerWarp * (2 * D + 1) + kApplyHits) + 2 * kApplyChunk) * sizeof(float);
}

template <int D>
size_t assign_smem_bytes() {
  return 1024 + (1 + kRing) * (size_t)(D / 64) * kTileM * 128 + sizeof(AssignBars) + 64;
}

}  // namespace

int launch_merge_prepare(const StepArgs& a, const MergeScratch& ms, const int32_t* idx, const void* k_new,
                         const void* v_new, cudaStream_t st) {
  const int bh = a.batch * a.n_heads;
  const int rows = a.cand[1];                                  // discarded + retained entries of a contextual head
  launch_k(merge_evicted_index_kernel, bh, kIdxThreads, 0, st, a, ms, idx);
  const dim3 grid((rows + kPrepThreads / 32 - 1) / (kPrepThreads / 32), bh);
  const __nv_bfloat16* kn = static_cast<const __nv_bfloat16*>(k_new);
  const __nv_bfloat16* vn = static_cast<const __nv_bfloat16*>(v_new);
  if (a.head_dim == 128) launch_k(merge_prepare_kernel<128>, grid, kPrepThreads, 0, st, a, ms, idx, kn, vn);
  else launch_k(merge_prepare_kernel<64>, grid, kPrepThreads, 0, st, a, ms, idx, kn, vn);
  return launched(2);
}

int launch_merge_finish(const StepArgs& a, const MergeScratch& ms, cudaStream_t st) {
  const int bh = a.batch * a.n_heads;
  const int kept = a.kept[1], n_evict = a.cand[1] - kept;
  const CUtensorMap& te = *static_cast<const CUtensorMap*>(ms.ev_map);
  const CUtensorMap& tk = *static_cast<const CUtensorMap*>(a.k_map);
  const dim3 g_assign((n_evict + kTileM - 1) / kTileM, bh);
  constexpr int kRowsPerCta = (kApplyThreads / 32) * kApplyRowsPerWarp;
  const dim3 g_apply((kept + kRowsPerCta - 1) / kRowsPerCta, bh);
  if (a.head_dim == 128) {
    if (!allow_dynamic_smem(merge_assign_kernel<128>, assign_smem_bytes<128>())) return -1;
    launch_k(merge_assign_kernel<128>, g_assign, kAssignThreads, assign_smem_bytes<128>(), st, te, tk, a, ms);
    if (!allow_dynamic_smem(merge_apply_kernel<128>, apply_smem_bytes<128>())) return -1;
    launch_k(merge_apply_kernel<128>, g_apply, kApplyThreads, apply_smem_bytes<128>(), st, a, ms);
  } else {
    if (!allow_dynamic_smem(merge_assign_kernel<64>, assign_smem_bytes<64>())) return -1;
    launch_k(merge_assign_kernel<64>, g_assign, kAssignThreads, assign_smem_bytes<64>(), st, te, tk, a, ms);
    if (!allow_dynamic_smem(merge_apply_kernel<64>, apply_smem_bytes<64>())) return -1;
    launch_k(merge_apply_kernel<64>, g_apply, kApplyThreads, apply_smem_bytes<64>(), st, a, ms);
  }
  return launched(2);
}

}  // namespace hack
