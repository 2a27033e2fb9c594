// Compression of one step in ONE launch for bf16 caches: subset-attention scores (Eq. 9), budgeted
// selection (Eq. 10 for contextual heads, Eq. 11 for structural heads) and in-place compaction of
// the ragged per-head cache (the gathers of Eq. 10-11).
//
// Every (batch, head) is independent of every other, so a thread-block cluster owns one head
// and nothing leaves the cluster between the first key load and the last row store.  The CTAs of
// the cluster split the head's candidate list into consecutive runs of 128-key chunks (a chunk
// never straddles the stored part and the new part of the list):
//
//   1. scores, pass 1: each CTA streams its chunks through a TMA ring and forms their logits
//      against the (at most 32) observation rows with tcgen05.mma, as score_tc.cu does, but every
//      chunk keeps its own accumulator [128 lanes x 32 columns] in tensor memory (chunks past the
//      15th go through one bounce accumulator into shared memory).  Consumer thread r owns key r
//      of a chunk and keeps the running (max, sum-exp) of the 32 softmax rows.
//   2. the CTAs publish their row statistics in shared memory; after a cluster barrier every CTA
//      merges all of them, in rank order, through distributed shared memory.
//   3. scores, pass 2: the logits are read back from tensor / shared memory (no second key
//      load, no second MMA) and s_j = sum_i exp(z_ij - m_i) / l_i becomes an order-preserving
//      32-bit key in shared memory (protected candidates of structural heads carry the top key).
//   4. exact radix select over the cluster: digits of 12, 12 and 8 bits; every CTA builds the
//      histogram of its own keys (the first one while it forms them), the histograms are added
//      through distributed shared memory after a cluster barrier, and every CTA locates the same
//      digit.  The select stops once all entries left in the located bin survive.  Ties at the
//      threshold go to the lowest candidate indices.
//   5. the CTAs exchange their counts of kept entries, which gives every CTA its offset in the
//      head's ascending index list; every entry goes straight into the shared memory of the CTA
//      that will move it (the list never touches global memory).
//   6. compaction in rounds: entry o of the list becomes row o of the head.  In a round every CTA
//      takes a run of consecutive entries out of memory (a stored survivor comes from the head's
//      own rows, at or behind its destination; a surviving new row from the caller's K/V), most of
//      them into shared memory, the rest into registers, the cluster meets, and the run goes out
//      (bulk stores for the shared-memory part).  The destinations of a round lie at or before
//      its own cache sources and before those of every later round: in place.
//   7. heads that keep the whole new scale stop behind their stored survivors; the attention
//      launch reads their new rows from the caller's tensors and appends them itself.
//
// In score-only mode the kernel stops after step 3 and writes the fp32 scores (hack_score).
// Every mbarrier wait is bounded; a CTA whose wait gives up raises the status word, and the
// cluster agrees at the first exchange to skip the rest, so that every CTA still reaches every
// cluster barrier.  No load in this file uses cluster multicast.
#include <cuda.h>

#include <algorithm>
#include <mutex>
#include <vector>

#include "hack_internal.h"
#include "tc_ptx.cuh"

namespace hack {
namespace {

using namespace ptx;

constexpr int kCkThreads = 256;
constexpr int kCkChunk = 128;
constexpr int kTmemChunks = 16;            // accumulators of 32 columns in 512 columns of tensor memory
constexpr int kMaxOver = 6;                // chunks per CTA whose logits live in shared memory
constexpr int kMaxCpc = kTmemChunks - 1 + kMaxOver;      // 21 chunks = 2688 keys per CTA
constexpr int kMaxCluster = 8;
constexpr uint32_t kCkDrainSpins = 1u << 22;
constexpr int kMaxStages = 4;              // key tiles in flight per CTA (deeper rings measured no faster)
constexpr int kHistBins = 4096;            // bins of a 12-bit digit of the radix select
constexpr int kHistWords = kHistBins / 2;  // 16-bit counters, two per word
constexpr int kMaxStageRows = 512;         // rows (K and V) in a CTA's staging buffers of the compaction
constexpr int kMoveBuffers = 3;            // staging buffers of the compaction: loads run two rounds ahead of the stores
constexpr size_t kSmemBudget = 227 * 1024; // dynamic shared memory a CTA may ask for
static_assert(kHistBins == 16 * kCkThreads, "a thread sums 16 bins of the cluster's histograms");
static_assert(kMaxCpc * kCkChunk < 65536, "16-bit counters per CTA");

struct CkParams {
  int cluster;                // CTAs per head
  int cpc_max;                // most chunks any CTA of this launch holds (sizes shared / tensor memory)
  int n_over;                 // chunks of shared-memory logits reserved per CTA
  int tmem_cols;              // power of two >= 32
  int stages;                 // key tiles in the TMA ring (2 .. kMaxStages)
  int region_bytes;           // front region of shared memory: ring, observation rows, overflow logits; later the row staging
  int stage_rows;             // rows (K and V) a CTA stages in shared memory per round of the compaction
  int score_only;             // stop after the scores
  float* scores;              // [b*H, cand_stride] or nullptr
  int32_t* idx;               // [b*H, kept_stride]
  const uint4* k_new;         // caller's K/V of this scale (compaction of heads whose new rows compete)
  const uint4* v_new;
};

struct CkShared {
  uint64_t full[kMaxStages], empty[kMaxStages];
  uint64_t acc_full[kMaxCpc];
  uint64_t acc_free;
  uint64_t drain;
  uint32_t tmem_base;
  int abort_flag;
  int pub_abort;                         // read by the other CTAs of the cluster
  float pub_stats[kMaxObs][2];           // this CTA's (max, sum-exp) per observation row
  int pub_counts[4];                     // kept above the threshold, equal to it; the same among stored candidates
  int cnt_all[kMaxCluster][4];           // the counts of every CTA of the cluster
  float row_m[kMaxObs], row_inv_l[kMaxObs];
  int warp_sums[kCkThreads / 32 + 1];
  int digit_of[2][2];                    // the located digit, the rank left inside its bin, the bin's count
  int sh_abort;
  int cnt_old[2];
};

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Execution barrier of the cluster without memory ordering: for a point that only has to come after
// every CTA's loads have landed (nothing written before it is read by another CTA after it).
__device__ __forceinline__ void cluster_sync_relaxed() {
  __syncthreads();
  asm volatile("barrier.cluster.arrive.relaxed.aligned;\n\tbarrier.cluster.wait.aligned;" ::: "memory");
}
// Address of the same shared-memory object in the CTA of rank `rank`.
__device__ __forceinline__ uint32_t peer_addr(const void* p, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(p)), "r"(rank));
  return r;
}
__device__ __forceinline__ int ld_peer_i32(uint32_t addr) {
  int v;
  asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ float ld_peer_f32(uint32_t addr) {
  float v;
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ uint4 ld_peer_v4(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared::cluster.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void st_peer_i32(uint32_t addr, int v) {
  asm volatile("st.shared::cluster.s32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void cp_async4(uint32_t dst, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait_group() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ bool ck_wait(uint64_t* bar, uint32_t parity, CkShared* sh, int* status, int code,
                                        long long limit) {
  const uint32_t addr = smem_u32(bar);
  // a limit of a few cycles (a test's way to make a wait run out) is taken literally: the barrier is
  // tested without blocking and the clock is read after every test
  const bool brief = limit < 65536;
  if (brief ? mbar_test_wait(addr, parity) : mbar_try_wait(addr, parity)) return true;
  const long long t0 = clock64();
  for (uint32_t it = 0;; ++it) {
    if (brief ? mbar_test_wait(addr, parity) : mbar_try_wait(addr, parity)) return true;
    if ((it & 63u) == 63u || brief) {
      if (*reinterpret_cast<volatile int*>(&sh->abort_flag)) return false;
      if (clock64() - t0 > limit) break;
    }
  }
  *reinterpret_cast<volatile int*>(&sh->abort_flag) = 1;
  atomicExch(status, code);
  return false;
}

__device__ __forceinline__ void ck_consumer_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// Order-preserving map from fp32 bits to unsigned (larger float -> larger key).
__device__ __forceinline__ uint32_t ck_orderable(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// One more entry in bin `digit` of a histogram of 16-bit counters, two per word (a CTA holds fewer
// than 65 536 keys).  Called by whole warps; lanes that fall into the same bin add once.
__device__ __forceinline__ void hist_add(uint32_t* hist, bool in, uint32_t digit) {
  const uint32_t peers = __match_any_sync(0xffffffffu, in ? digit : 0xffffffffu);
  if (in && (threadIdx.x & 31) == __ffs(peers) - 1)
    atomicAdd(&hist[digit >> 1], (uint32_t)__popc(peers) << (16 * (digit & 1)));
}

// Exclusive prefix sum of one value per thread over the CTA's kCkThreads threads, and the total.
__device__ __forceinline__ int ck_block_scan(int v, int* warp_sums, int& total) {
  constexpr int NW = kCkThreads / 32;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += n;
  }
  if (lane == 31) warp_sums[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const int w = lane < NW ? warp_sums[lane] : 0;
    int wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += n;
    }
    if (lane < NW) warp_sums[lane] = wi - w;
    if (lane == 31) warp_sums[NW] = wi;
  }
  __syncthreads();
  const int res = warp_sums[warp] + incl - v;
  total = warp_sums[NW];
  __syncthreads();
  return res;
}

template <int D>
__global__ void __launch_bounds__(kCkThreads, 1)
compress_cluster_kernel(const __grid_constant__ CUtensorMap tm_cache, const __grid_constant__ CUtensorMap tm_new,
                        const StepArgs a, const __nv_bfloat16* __restrict__ q, const CkParams p) {
  constexpr int SUB = D / 64;
  constexpr uint32_t K_SUB_BYTES = kCkChunk * 128;
  constexpr uint32_t Q_SUB_BYTES = kMaxObs * 128;
  constexpr uint32_t K_BYTES = SUB * K_SUB_BYTES;
  constexpr int PIECES = D * 2 / 16;                      // 16-byte pieces per row
  static_assert(2 * K_BYTES >= 2 * kMaxObs * kCkChunk * sizeof(float), "two ring stages hold the fold");
  const int STAGES = p.stages;
  const uint32_t RING_BYTES = (uint32_t)STAGES * K_BYTES;

  // Nothing that another kernel writes is touched before pdl_wait() below: the head-type table is
  // written when the cache is created, the step's lengths travel in the arguments.
  const int bh = blockIdx.y;
  const int ctx = a.is_ctx[bh % a.n_heads];
  if (!a.trig[ctx]) {                                     // the whole cluster leaves together
    pdl_wait();
    return;
  }
  const int rank = (int)cluster_rank();
  const int CL = p.cluster;
  const int stored = a.stored[ctx], n_new = a.n_new, n_keep = a.kept[ctx];
  const int n_sc = (stored + kCkChunk - 1) / kCkChunk;
  const int n_chunks = n_sc + (n_new + kCkChunk - 1) / kCkChunk;
  const int cpc = (n_chunks + CL - 1) / CL;               // <= p.cpc_max
  const int c_begin = rank * cpc;
  const int n_run = max(0, min(cpc, n_chunks - c_begin));
  const int n_persist = p.cpc_max <= kTmemChunks ? kTmemChunks : kTmemChunks - 1;   // chunks with an accumulator of their own
  const float zscale = a.sm_scale * 1.4426950408889634f;  // logits in log2 units
  const long long wlim = a.wait_cycles;

  extern __shared__ unsigned char smem_dyn[];
  const uint32_t raw = smem_u32(smem_dyn);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* sm = smem_dyn + (base - raw);
  const uint32_t k_sm = base;
  const uint32_t q_sm = base + RING_BYTES;
  float* over = reinterpret_cast<float*>(sm + RING_BYTES + SUB * Q_SUB_BYTES);            // [n_over][32][128]
  const int S_ROWS = p.stage_rows;                          // rows a CTA holds in its staging buffers
  uint32_t* keys = reinterpret_cast<uint32_t*>(sm + p.region_bytes);                            // [cpc_max * 128]
  int32_t* pos_stage = reinterpret_cast<int32_t*>(keys + (size_t)p.cpc_max * kCkChunk);        // [S_ROWS]
  int32_t* src_all = pos_stage + S_ROWS;                    // [cpc_max * 128 + S_ROWS]: this CTA's list entries of every round
  CkShared* sh = reinterpret_cast<CkShared*>(src_all + (size_t)p.cpc_max * kCkChunk + S_ROWS);
  float* fold_m = reinterpret_cast<float*>(sm);           // [32][128], reuses the ring
  float* fold_l = fold_m + kMaxObs * kCkChunk;
  uint32_t* hist32 = reinterpret_cast<uint32_t*>(sm);     // [2][kHistWords], reuses the ring after the fold

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // candidate behind slot (local chunk i, key r): is it a live entry, and its candidate index
  auto slot_info = [&](int slot, int& j) -> bool {
    const int i = slot >> 7, r = slot & 127;
    if (i >= n_run) return false;
    const int chunk = c_begin + i;
    const bool from_cache = chunk < n_sc;
    const int part_row = (from_cache ? chunk : chunk - n_sc) * kCkChunk + r;
    j = (from_cache ? 0 : stored) + part_row;
    return part_row < (from_cache ? stored : n_new);
  };

  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(smem_u32(&sh->full[s]), 1); mbar_init(smem_u32(&sh->empty[s]), 1); }
    for (int i = 0; i < kMaxCpc; ++i) mbar_init(smem_u32(&sh->acc_full[i]), 1);
    mbar_init(smem_u32(&sh->acc_free), kCkChunk);
    mbar_init(smem_u32(&sh->drain), 1);
    sh->abort_flag = 0;
    sh->cnt_old[0] = 0;
    sh->cnt_old[1] = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&sh->tmem_base), p.tmem_cols);
    tmem_relinquish();
  }
  if (warp == 0 && lane == 0) {
    prefetch_tensormap(&tm_cache);
    prefetch_tensormap(&tm_new);
  }
  pdl_wait();     // everything above overlaps the tail of the previous kernel
  // observation rows into the swizzled B tile; unused rows are zero
  for (int v = tid; v < kMaxObs * (D / 8); v += kCkThreads) {
    const int i = v / (D / 8), c = v % (D / 8);
    uint4 val = make_uint4(0, 0, 0, 0);
    if (i < a.n_obs_rows) {
      const int row = obs_row(a, i);
      val = *reinterpret_cast<const uint4*>(q + ((size_t)bh * n_new + row) * D + c * 8);
    }
    const uint32_t off = (c / 8) * Q_SUB_BYTES + i * 128 + (((c % 8) ^ (i & 7)) << 4);
    *reinterpret_cast<uint4*>(sm + RING_BYTES + off) = val;
  }
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&sh->tmem_base);

  // ------------------------------------------------------------------ 1. scores, pass 1
  const int quad = warp & 3;                                // TMEM lane quadrant a consumer warp may read
  const int key_row = quad * 32 + lane;
  const uint32_t t_lane = tmem + (static_cast<uint32_t>(quad * 32) << 16);
  if (warp == 0) {
    if (lane == 0) {
      int issued = 0;
      bool ok = true;
      for (int i = 0; i < n_run; ++i) {
        const int s = i % STAGES;
        ok = ck_wait(&sh->empty[s], ((i / STAGES) & 1) ^ 1, sh, a.status, 51, wlim);
        if (!ok) break;
        const int chunk = c_begin + i;
        const bool from_cache = chunk < n_sc;
        const CUtensorMap* tm = from_cache ? &tm_cache : &tm_new;
        const int row = from_cache ? a.row_off[bh] + chunk * kCkChunk : bh * n_new + (chunk - n_sc) * kCkChunk;
        const uint32_t bar = smem_u32(&sh->full[s]);
        mbar_expect_tx(bar, K_BYTES);
#pragma unroll
        for (int c = 0; c < SUB; ++c) tma_load_2d(k_sm + s * K_BYTES + c * K_SUB_BYTES, tm, c * 64, row, bar);
        ++issued;
      }
      if (!ok) {
        // give the copies already in flight a bounded chance to land before the ring is reused
        for (int i = max(0, issued - STAGES); i < issued; ++i) {
          const uint32_t bar = smem_u32(&sh->full[i % STAGES]);
          for (uint32_t it = 0; it < kCkDrainSpins && !mbar_try_wait(bar, (i / STAGES) & 1); ++it) {}
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t IDESC = idesc_bf16_f32(kCkChunk, kMaxObs, 0);
      const uint64_t q_desc = smem_desc_sw128(q_sm, 16, 1024);
      bool ok = true;
      for (int i = 0; i < n_run && ok; ++i) {
        const int s = i % STAGES;
        const int slot = i < n_persist ? i : kTmemChunks - 1;
        ok = ck_wait(&sh->full[s], (i / STAGES) & 1, sh, a.status, 52, wlim);
        // the bounce accumulator is free again once all 128 consumers have read its previous chunk
        if (ok && i >= n_persist) ok = ck_wait(&sh->acc_free, ((i - n_persist) & 1) ^ 1, sh, a.status, 53, wlim);
        if (!ok) break;
        tc_fence_after();
        const uint64_t k_desc = smem_desc_sw128(k_sm + s * K_BYTES, 16, 1024);
        if constexpr (D == 128) mma_ss_chain8_b32rows(tmem + slot * kMaxObs, k_desc, q_desc, IDESC, 0);
        else mma_ss_chain4(tmem + slot * kMaxObs, k_desc, q_desc, IDESC, 0);
        mma_commit(smem_u32(&sh->empty[s]));
        mma_commit(smem_u32(&sh->acc_full[i]));
      }
      if (!ok) {
        mma_commit(smem_u32(&sh->drain));
        for (uint32_t it = 0; it < kCkDrainSpins && !mbar_try_wait(smem_u32(&sh->drain), 0); ++it) {}
      }
    }
    __syncwarp();
  } else if (warp < 6) {
    const int w = warp - 2;
    const int ct = tid - 64;                                  // 0..127
    float rm[kMaxObs], rl[kMaxObs];
#pragma unroll
    for (int i = 0; i < kMaxObs; ++i) { rm[i] = -INFINITY; rl[i] = 0.f; }
    bool ok = true;
    for (int i = 0; i < n_run; ++i) {
      ok = __all_sync(0xffffffffu, ck_wait(&sh->acc_full[i], 0, sh, a.status, 54, wlim));
      if (!ok) break;
      tc_fence_after();
      uint32_t acc[kMaxObs];
      tmem_ld32(t_lane + (i < n_persist ? i : kTmemChunks - 1) * kMaxObs, acc);
      tmem_wait_ld();
      if (i >= n_persist) {
        float* dst = over + (size_t)(i - n_persist) * kMaxObs * kCkChunk + key_row;
#pragma unroll
        for (int r = 0; r < kMaxObs; ++r) dst[r * kCkChunk] = __uint_as_float(acc[r]);
        tc_fence_before();
        mbar_arrive(smem_u32(&sh->acc_free));
      }
      int j;
      if (slot_info(i * kCkChunk + key_row, j)) {
#pragma unroll
        for (int r = 0; r < kMaxObs; ++r) {
          const float z = __uint_as_float(acc[r]) * zscale;
          const float mn = fmaxf(rm[r], z);
          rl[r] = rl[r] * ex2(rm[r] - mn) + ex2(z - mn);
          rm[r] = mn;
        }
      }
    }
    // the consumers meet on their named barrier below, so they agree first on whether all of them got through
    uint32_t all_ok;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.and.pred p, 1, 128, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(all_ok) : "r"((uint32_t)ok) : "memory");
    if (all_ok) {
      // every accumulator has been read, so every MMA and every key load is complete: the ring is free
#pragma unroll
      for (int r = 0; r < kMaxObs; ++r) { fold_m[r * kCkChunk + ct] = rm[r]; fold_l[r * kCkChunk + ct] = rl[r]; }
      ck_consumer_sync();
      for (int r = w; r < kMaxObs; r += 4) {
        float m4[4], l4[4];
        float m = -INFINITY;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          m4[u] = fold_m[r * kCkChunk + u * 32 + lane];
          l4[u] = fold_l[r * kCkChunk + u * 32 + lane];
          m = fmaxf(m, m4[u]);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        float l = 0.f;
#pragma unroll
        for (int u = 0; u < 4; ++u) l += l4[u] == 0.f ? 0.f : l4[u] * ex2(m4[u] - m);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
        if (lane == 0) { sh->pub_stats[r][0] = m; sh->pub_stats[r][1] = l; }
      }
    }
  }
  __syncthreads();
  if (tid == 0) sh->pub_abort = *reinterpret_cast<volatile int*>(&sh->abort_flag);
  // the ring is idle from here on; its first 16 KB become the two histograms of the radix select
  {
    uint4* z = reinterpret_cast<uint4*>(hist32 + 8 * tid);
    z[0] = z[1] = make_uint4(0, 0, 0, 0);
    z[kHistWords / 4] = z[kHistWords / 4 + 1] = make_uint4(0, 0, 0, 0);
  }

  // ------------------------------------------------------------------ 2. row statistics of the whole head
  cluster_sync();
  if (tid < kMaxObs) {
    float mr[kMaxCluster], lr[kMaxCluster];
#pragma unroll
    for (int r = 0; r < kMaxCluster; ++r) {                 // all loads in flight at once
      mr[r] = lr[r] = 0.f;
      if (r < CL) {
        mr[r] = ld_peer_f32(peer_addr(&sh->pub_stats[tid][0], r));
        lr[r] = ld_peer_f32(peer_addr(&sh->pub_stats[tid][1], r));
      }
    }
    float m = -INFINITY;
#pragma unroll
    for (int r = 0; r < kMaxCluster; ++r)
      if (r < CL) m = fmaxf(m, mr[r]);
    float l = 0.f;
#pragma unroll
    for (int r = 0; r < kMaxCluster; ++r)
      if (r < CL) l += lr[r] == 0.f ? 0.f : lr[r] * ex2(mr[r] - m);
    // rows past n_obs_rows are padding: weight 0, finite reference
    sh->row_m[tid] = tid < a.n_obs_rows ? m : 0.f;
    sh->row_inv_l[tid] = tid < a.n_obs_rows ? 1.f / l : 0.f;
  }
  if (tid == 32) {
    int any = 0;
    for (int r = 0; r < CL; ++r) any |= ld_peer_i32(peer_addr(&sh->pub_abort, r));
    sh->sh_abort = any;
  }
  __syncthreads();
  const bool aborted = sh->sh_abort != 0;                   // the same value in every CTA of the cluster

  // ------------------------------------------------------------------ 3. scores, pass 2
  if (!aborted) {
    // all eight warps: warps 2-5 take the even chunks, warps 6, 7, 0, 1 (the same four lane quadrants)
    // the odd ones; a key's 32 terms are added in the same order by either set
    float rm[kMaxObs], rl[kMaxObs];
#pragma unroll
    for (int i = 0; i < kMaxObs; ++i) { rm[i] = sh->row_m[i]; rl[i] = sh->row_inv_l[i]; }
    const bool structural = ctx == 0;
    for (int i = (warp >= 2 && warp < 6) ? 0 : 1; i < n_run; i += 2) {
      // a chunk of protected candidates only (the new scale of a structural head) is kept whatever
      // its scores are; they are formed only when the caller wants them
      if (!p.scores && structural && a.protect_new && c_begin + i >= n_sc) {
        int j;
        keys[i * kCkChunk + key_row] = 0xffffffffu;
        hist_add(hist32, slot_info(i * kCkChunk + key_row, j), kHistBins - 1);
        continue;
      }
      uint32_t acc[kMaxObs];
      if (i < n_persist) {
        tmem_ld32(t_lane + i * kMaxObs, acc);
        tmem_wait_ld();
      } else {
        const float* src = over + (size_t)(i - n_persist) * kMaxObs * kCkChunk + key_row;
#pragma unroll
        for (int r = 0; r < kMaxObs; ++r) acc[r] = __float_as_uint(src[r * kCkChunk]);
      }
      float s = 0.f;
#pragma unroll
      for (int r = 0; r < kMaxObs; ++r) s = fmaf(ex2(fmaf(__uint_as_float(acc[r]), zscale, -rm[r])), rl[r], s);
      int j = 0;
      const bool live = slot_info(i * kCkChunk + key_row, j);
      uint32_t key = 0;
      if (live) {
        if (p.scores && dbg_ok(j < a.cand_stride, a.status, 8)) p.scores[(size_t)bh * a.cand_stride + j] = s;
        if (structural && (j < a.t_init || (a.protect_new && j >= stored))) {
          key = 0xffffffffu;
        } else {
          key = ck_orderable(s);
          if (key == 0xffffffffu) key = 0xfffffffeu;          // the top key is for protected entries only
        }
      }
      keys[i * kCkChunk + key_row] = key;
      if (!p.score_only) hist_add(hist32, live, key >> 20);   // first digit of the radix select
    }
  }
  tc_fence_before();
  __syncthreads();

  if (!aborted && !p.score_only) {
    // ---------------------------------------------------------------- 4. radix select over the cluster
    // Digits of 12, 12 and 8 bits.  The local histogram of the first digit was filled while the keys
    // were formed; the select stops as soon as every entry left in the located bin survives, which
    // with 24 bits fixed is the usual case.
    const int n_slots = cpc * kCkChunk;
    uint32_t prefix = 0, mask = 0;
    int need = n_keep;
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
      const int shift = pass == 0 ? 20 : (pass == 1 ? 8 : 0);
      const uint32_t dmask = pass == 2 ? 255u : 4095u;
      uint32_t* hist = hist32 + (pass & 1) * kHistWords;
      if (pass > 0) {
        for (int s0 = 0; s0 < n_slots; s0 += kCkThreads) {
          const int slot = s0 + tid;
          int j;
          const bool live = slot < n_slots && slot_info(slot, j);
          const uint32_t k = live ? keys[slot] : 0u;
          const bool in = live && ((k & mask) == prefix);
          hist_add(hist, in, (k >> shift) & dmask);
        }
      }
      cluster_sync();                                         // (orders the CTA's own threads as well)
      // thread t owns bins [16 t, 16 t + 16): two 16-bit counters per word
      int c[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) c[i] = 0;
      {
        uint4 part[kMaxCluster][2];
#pragma unroll
        for (int r = 0; r < kMaxCluster; ++r)                 // all loads in flight at once
          if (r < CL && (pass < 2 || tid < 16)) {               // the 8-bit digit fills 256 bins only
            const uint32_t addr = peer_addr(hist + 8 * tid, r);
            part[r][0] = ld_peer_v4(addr);
            part[r][1] = ld_peer_v4(addr + 16);
          } else {
            part[r][0] = part[r][1] = make_uint4(0, 0, 0, 0);
          }
#pragma unroll
        for (int r = 0; r < kMaxCluster; ++r)
          if (r < CL) {
            const uint32_t w[8] = {part[r][0].x, part[r][0].y, part[r][0].z, part[r][0].w,
                                   part[r][1].x, part[r][1].y, part[r][1].z, part[r][1].w};
#pragma unroll
            for (int i = 0; i < 8; ++i) { c[2 * i] += (int)(w[i] & 0xffffu); c[2 * i + 1] += (int)(w[i] >> 16); }
          }
      }
      // the other buffer is free: every CTA read it before it arrived at the barrier above
      {
        uint4* z = reinterpret_cast<uint4*>(hist32 + ((pass & 1) ^ 1) * kHistWords + 8 * tid);
        z[0] = make_uint4(0, 0, 0, 0);
        z[1] = make_uint4(0, 0, 0, 0);
      }
      int mine = 0;
#pragma unroll
      for (int i = 0; i < 16; ++i) mine += c[i];
      int total;
      const int below = ck_block_scan(mine, sh->warp_sums, total);
      const int above = total - below - mine;                 // entries in the bins of the threads behind this one
      if (above < need && need <= above + mine) {
        int cum = above;
#pragma unroll
        for (int i = 15; i >= 0; --i) {
          if (cum < need && need <= cum + c[i]) {
            sh->digit_of[0][0] = 16 * tid + i;
            sh->digit_of[0][1] = need - cum;
            sh->digit_of[1][0] = c[i];
          }
          cum += c[i];
        }
      }
      __syncthreads();
      prefix |= (uint32_t)sh->digit_of[0][0] << shift;
      need = sh->digit_of[0][1];
      mask |= dmask << shift;
      if (need == sh->digit_of[1][0]) break;                  // the same in every CTA of the cluster
    }
    // ---------------------------------------------------------------- 5. ascending index list
    // prefix = the fixed digits of the n_keep-th largest key; of the entries that agree with it in
    // those digits `need` survive (lowest indices; all of them when the select stopped early)
    const uint32_t thr = prefix;
    const int per = (n_slots + kCkThreads - 1) / kCkThreads;  // thread t owns slots [t*per, t*per + per)
    int gt = 0, eq = 0, gt_old = 0, eq_old = 0;
    for (int e = 0; e < per; ++e) {
      const int slot = tid * per + e;
      int j;
      if (slot < n_slots && slot_info(slot, j)) {
        const uint32_t k = keys[slot] & mask;
        gt += k > thr;
        eq += k == thr;
        if (j < stored) { gt_old += k > thr; eq_old += k == thr; }
      }
    }
    if (gt_old) atomicAdd(&sh->cnt_old[0], gt_old);
    if (eq_old) atomicAdd(&sh->cnt_old[1], eq_old);
    int total;
    const int packed = ck_block_scan(gt | (eq << 16), sh->warp_sums, total);
    if (tid == 0) {
      sh->pub_counts[0] = total & 0xffff;
      sh->pub_counts[1] = total >> 16;
      sh->pub_counts[2] = sh->cnt_old[0];
      sh->pub_counts[3] = sh->cnt_old[1];
    }
    cluster_sync();
    int gt_before = packed & 0xffff, eq_before = packed >> 16;
    int gt_old_all = 0, eq_old_all = 0;
    // one remote load per count, then every thread reads the CTA's own copy
    if (tid < 4 * CL) sh->cnt_all[tid >> 2][tid & 3] = ld_peer_i32(peer_addr(&sh->pub_counts[tid & 3], tid >> 2));
    __syncthreads();
#pragma unroll
    for (int r = 0; r < kMaxCluster; ++r)
      if (r < CL) {
        if (r < rank) { gt_before += sh->cnt_all[r][0]; eq_before += sh->cnt_all[r][1]; }
        gt_old_all += sh->cnt_all[r][2];
        eq_old_all += sh->cnt_all[r][3];
      }
    const int n_old = gt_old_all + min(eq_old_all, need);     // survivors that were already stored
    // Entry o of the head's ascending list is candidate j.  Entry o becomes row o of the head, and
    // rows are compacted in rounds of CL * S consecutive entries, CTA `rk` of the cluster staging S
    // of them: the entry goes straight into that CTA's shared memory.  Heads that keep the whole new
    // scale need only their stored survivors (the attention launch appends the rest).
    const bool attend_appends = a.seg_new[ctx] != 0;
    const int n_rows = attend_appends ? n_old : n_keep;
    // rounds: as few as the staging buffers (a third of the staging rows each) allow, of equal size
    const int s_cap = S_ROWS / kMoveBuffers;
    const int n_rounds = (n_rows + CL * s_cap - 1) / (CL * s_cap);
    const int S = n_rounds > 0 ? (n_rows + CL * n_rounds - 1) / (CL * n_rounds) : 1, RS = CL * S;
    auto deliver = [&](int o, int j) {
      if (o < n_rows && dbg_ok(o >= 0 && o < n_keep, a.status, 9)) {
        const int t = o / RS, w = o - t * RS, rk = w / S, lr = w - rk * S;
        st_peer_i32(peer_addr(&src_all[t * S + lr], rk), j);
      }
    };
    for (int e = 0; e < per; ++e) {
      const int slot = tid * per + e;
      int j;
      if (slot < n_slots && slot_info(slot, j)) {
        const uint32_t k = keys[slot] & mask;
        if (k > thr) {
          deliver(gt_before + min(eq_before, need), j);
          ++gt_before;
        } else if (k == thr) {
          if (eq_before < need) deliver(gt_before + eq_before, j);
          ++eq_before;
        }
      }
    }
    cluster_sync();                                           // every CTA holds its part of the list

    // ---------------------------------------------------------------- 6. and 7. compaction in rounds
    // A stored survivor moves forward (its source is a row of the head at or behind its
    // destination), a surviving new row comes out of the caller's K/V.  In a round every CTA stages
    // its S entries in shared memory, the cluster meets, and the rows go out with bulk stores (the
    // destinations of a CTA are one contiguous run).  The destinations of a round lie at or before
    // its own cache sources and before the cache sources of every later round, so nothing is
    // overwritten before it has been read: in place, no second buffer.
    const size_t off = a.row_off[bh];
    uint4* kp = reinterpret_cast<uint4*>(a.k_plane) + off * PIECES;
    uint4* vp = reinterpret_cast<uint4*>(a.v_plane) + off * PIECES;
    int32_t* pos = a.pos_plane + off;
    const uint4* kn = p.k_new + (size_t)bh * n_new * PIECES;
    const uint4* vn = p.v_new + (size_t)bh * n_new * PIECES;
    constexpr uint32_t ROWB = PIECES * 16;
    // Staging buffer b holds S key rows, then S value rows.  The loads of round t + 2 are issued
    // while round t stores: a later round's sources lie behind every earlier round's destinations.
    const uint32_t buf_bytes = 2u * (uint32_t)s_cap * ROWB;
    auto slice_first = [&](int t) { return t * RS + rank * S; };
    auto slice_rows = [&](int t) { return max(0, min(S, n_rows - slice_first(t))); };
    // ascending entries with source >= destination: if the last stored row of the slice stays
    // where it is, so does every row of the slice
    auto slice_moves = [&](int t) {
      const int rows = slice_rows(t), last = src_all[t * S + max(rows, 1) - 1];
      return rows > 0 && !(last == slice_first(t) + rows - 1 && last < stored);
    };
    auto issue_loads = [&](int t) {
      if (t < n_rounds && slice_moves(t)) {
        const int first = slice_first(t), rows = slice_rows(t);
        const int32_t* srcs = src_all + t * S;
        const uint32_t kb = base + (uint32_t)(t % kMoveBuffers) * buf_bytes, vb = kb + (uint32_t)S * ROWB;
        int32_t* ps = pos_stage + (t % kMoveBuffers) * s_cap;
        for (int v = tid; v < rows * PIECES; v += kCkThreads) {
          const int lr = v / PIECES, piece = v % PIECES;
          int src = srcs[lr];
          // a checked build turns an entry outside [destination, candidates) into "stays where it is"
          if (!dbg_ok(src >= first + lr && src < stored + n_new && first + lr < a.cap[ctx], a.status, 10))
            src = first + lr < stored ? first + lr : stored;
          const uint4* ks = src < stored ? kp + (size_t)src * PIECES : kn + (size_t)(src - stored) * PIECES;
          const uint4* vs = src < stored ? vp + (size_t)src * PIECES : vn + (size_t)(src - stored) * PIECES;
          cp_async16(kb + (uint32_t)lr * ROWB + piece * 16, ks + piece);
          cp_async16(vb + (uint32_t)lr * ROWB + piece * 16, vs + piece);
        }
        for (int lr = tid; lr < rows; lr += kCkThreads) {
          const int src = srcs[lr];
          if (src < stored) cp_async4(smem_u32(&ps[lr]), pos + max(src, 0));
          else ps[lr] = a.pos_base + (src - stored);
        }
      }
      cp_async_commit();                                      // one group per round, empty or not
    };
    issue_loads(0);
    issue_loads(1);
    for (int t = 0; t < n_rounds; ++t) {
      cp_async_wait_group<1>();                               // the loads of round t (all but the latest group) have landed
      fence_proxy_async();                                    // the bulk stores below read what these threads wrote
      cluster_sync_relaxed();                                 // every source of this round has been read
      const bool moving = slice_moves(t);
      if (moving) {
        const int first = slice_first(t), rows = slice_rows(t);
        const uint32_t kb = base + (uint32_t)(t % kMoveBuffers) * buf_bytes, vb = kb + (uint32_t)S * ROWB;
        if (tid == 0) {
          constexpr uint32_t kPiece = 32768;                  // bytes per bulk store
          const uint32_t bytes = (uint32_t)rows * ROWB;
          for (uint32_t o = 0; o < bytes; o += kPiece) {
            const uint32_t n = min(kPiece, bytes - o);
            bulk_store(reinterpret_cast<unsigned char*>(kp + (size_t)first * PIECES) + o, kb + o, n);
            bulk_store(reinterpret_cast<unsigned char*>(vp + (size_t)first * PIECES) + o, vb + o, n);
          }
        }
        const int32_t* ps = pos_stage + (t % kMoveBuffers) * s_cap;
        for (int lr = tid; lr < rows; lr += kCkThreads) pos[first + lr] = ps[lr];
      }
      if (tid == 0) {
        bulk_commit();                                        // one group per round, empty or not
        bulk_wait_read<1>();                                  // round t - 1 has left its buffer, which round t + 2 fills
      }
      __syncthreads();
      issue_loads(t + 2);
    }
    if (tid == 0) bulk_wait_read<0>();                        // shared memory is read out before the CTA leaves
  }
  // no CTA leaves while another may still read its shared memory
  cluster_sync();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, p.tmem_cols);
  }
}

// Shared memory of one CTA: the front region (ring, observation rows and overflow logits; the
// compaction later stages rows over all of it), keys, the two per-row staging arrays, barriers and
// exchange area.
template <int D>
size_t ck_smem_bytes(const CkParams& p) {
  const size_t rows = (size_t)p.stage_rows;
  return 1024 + (size_t)p.region_bytes + (size_t)p.cpc_max * kCkChunk * sizeof(uint32_t) +
         (2 * rows + (size_t)p.cpc_max * kCkChunk) * sizeof(int32_t) + sizeof(CkShared) + 64;
}

// Ring depth and staging rows for this launch: as many key tiles in flight as the CTA has chunks
// (more would never be used) and as shared memory holds; the front region then grows to what is
// left of the budget, so that a round of the compaction stages as many rows as possible.
template <int D>
void ck_size(CkParams& p) {
  const size_t k_bytes = (size_t)(D / 64) * kCkChunk * 128;
  const size_t row_bytes = 2 * (size_t)D * 2;                // a key row and a value row
  const size_t q_over = (size_t)(D / 64) * kMaxObs * 128 + (size_t)p.n_over * kMaxObs * kCkChunk * sizeof(float);
  p.stage_rows = kMaxStageRows;
  p.region_bytes = 0;
  const size_t other = ck_smem_bytes<D>(p);                   // everything but the front region
  const size_t room = kSmemBudget > other ? kSmemBudget - other : 0;
  const int fit = room > q_over ? (int)((room - q_over) / k_bytes) : 0;
  p.stages = std::max(2, std::min({fit, kMaxStages, std::max(p.cpc_max, 2)}));
  const size_t need = p.stages * k_bytes + q_over;
  const size_t region = std::max(need, std::min(room, (size_t)kMaxStageRows * row_bytes)) / 1024 * 1024;
  p.region_bytes = (int)std::max(region, (need + 1023) / 1024 * 1024);
  p.stage_rows = (int)std::min<size_t>(kMaxStageRows, p.region_bytes / row_bytes);
}

template <int D>
cudaLaunchConfig_t ck_config(const StepArgs& a, const CkParams& p, cudaLaunchAttribute* attr, cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p.cluster, a.batch * a.n_heads);
  cfg.blockDim = dim3(kCkThreads);
  cfg.dynamicSmemBytes = ck_smem_bytes<D>(p);
  cfg.stream = st;
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = p.cluster;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cfg;
}

// Clusters of this shape the device runs at the same time (asked once per shape and device).
template <int D>
int ck_active_clusters(const StepArgs& a, const CkParams& p) {
  struct Known { int dev, cluster; size_t smem; int n; };
  static std::mutex mu;
  static std::vector<Known> known;
  int dev = 0;
  cudaGetDevice(&dev);
  const size_t smem = ck_smem_bytes<D>(p);
  std::lock_guard<std::mutex> lock(mu);
  for (const Known& k : known)
    if (k.dev == dev && k.cluster == p.cluster && k.smem == smem) return k.n;
  cudaLaunchAttribute attr[2];
  cudaLaunchConfig_t cfg = ck_config<D>(a, p, attr, nullptr);
  cfg.numAttrs = 2;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, compress_cluster_kernel<D>, &cfg) != cudaSuccess) {
    cudaGetLastError();
    n = 0;
  }
  known.push_back({dev, p.cluster, smem, n});
  return n;
}

template <int D>
int launch_t(const StepArgs& a, const CUtensorMap& tm_cache, const CUtensorMap& tm_new, const void* q, CkParams p,
             int max_chunks, int n_clusters, int reserved_sms, cudaStream_t st) {
  // the opt-in is made once per (kernel, device), so it asks for the most any launch can need
  if (!allow_dynamic_smem(compress_cluster_kernel<D>, kSmemBudget)) return -1;
  // CTAs per head: at least what holds the longest candidate list; more spread the key stream over
  // more SMs, as long as every cluster of the launch still runs at the same time
  auto shape = [&](int cl) {
    p.cluster = cl;
    p.cpc_max = (max_chunks + cl - 1) / cl;
    p.n_over = p.cpc_max > kTmemChunks ? p.cpc_max - (kTmemChunks - 1) : 0;
    int cols = 32;
    while (cols < kMaxObs * std::min(p.cpc_max, kTmemChunks)) cols *= 2;
    p.tmem_cols = cols;
    ck_size<D>(p);
  };
  int cl = p.cluster;
  shape(cl);
  // a launch that runs beside another one leaves that one its SMs, if both fit the device at all
  const int sms = sm_count();
  const bool beside = reserved_sms > 0 && n_clusters * cl + reserved_sms <= sms;
  while (cl < kMaxCluster && (max_chunks + 2 * cl - 1) / (2 * cl) >= 2) {
    if (beside && n_clusters * 2 * cl + reserved_sms > sms) break;
    shape(2 * cl);
    if (ck_active_clusters<D>(a, p) < n_clusters) break;
    cl *= 2;
  }
  // beside another launch the SMs left over need not hold a power of two per head
  while (beside && cl < kMaxCluster && (max_chunks + cl) / (cl + 1) >= 2 && n_clusters * (cl + 1) + reserved_sms <= sms) {
    shape(cl + 1);
    if (ck_active_clusters<D>(a, p) < n_clusters) break;
    ++cl;
  }
  shape(cl);
  if (ck_smem_bytes<D>(p) > kSmemBudget) {
    set_error("compression: shared memory plan beyond the limit");
    return -1;
  }
  cudaLaunchAttribute attr[2];
  cudaLaunchConfig_t cfg = ck_config<D>(a, p, attr, st);
  cudaLaunchKernelEx(&cfg, compress_cluster_kernel<D>, tm_cache, tm_new, a, static_cast<const __nv_bfloat16*>(q), p);
  return launched(1);
}

}  // namespace

// Scores only (scores != nullptr, idx == nullptr) or the whole compression of the step (idx != nullptr).
// Returns 1 (one launch), -1 on a launch error, or 0 when this step is outside what the kernel holds
// (candidate lists beyond 8 x 21 chunks per head, the every-query scoring rounds): the caller then
// takes the separate scoring, selection and compaction launches.  reserved_sms: CTAs of a launch
// that is enqueued to run beside this one (0 if none).
int launch_compress_cluster(const StepArgs& a, const void* q, const void* k_new, const void* v_new, float* scores,
                            int32_t* idx, cudaStream_t st, int reserved_sms) {
  if (!a.k_map || a.obs_full || a.score_accumulate) return 0;
  int max_chunks = 0, types = 0;
  const int n_new_chunks = (a.n_new + kCkChunk - 1) / kCkChunk;
  for (int t = 0; t < 2; ++t)
    if (a.trig[t]) {
      max_chunks = std::max(max_chunks, (a.stored[t] + kCkChunk - 1) / kCkChunk + n_new_chunks);
      ++types;
    }
  if (types == 0) return 0;
  int cl = 1;
  while (cl <= kMaxCluster && (max_chunks + cl - 1) / cl > kMaxCpc) cl *= 2;
  if (cl > kMaxCluster) return 0;
  CkParams p{};
  p.cluster = cl;
  p.score_only = idx == nullptr;
  p.scores = scores;
  p.idx = idx;
  p.k_new = static_cast<const uint4*>(k_new);
  p.v_new = static_cast<const uint4*>(v_new);
  // clusters that do work: the heads of the triggered types (the split between the types is not
  // known here; half of the heads each is the usual case)
  const int n_clusters = std::max(1, a.batch * a.n_heads * types / 2);
  CUtensorMap tm_new;
  if (!make_rows_map(&tm_new, k_new, (uint64_t)a.batch * a.n_heads * a.n_new, a.head_dim)) {
    set_error("compression: cuTensorMapEncodeTiled failed for the new scale's keys");
    return -1;
  }
  const CUtensorMap& tm_cache = *static_cast<const CUtensorMap*>(a.k_map);
  return a.head_dim == 128 ? launch_t<128>(a, tm_cache, tm_new, q, p, max_chunks, n_clusters, reserved_sms, st)
                           : launch_t<64>(a, tm_cache, tm_new, q, p, max_chunks, n_clusters, reserved_sms, st);
}

}  // namespace hack
