// Attention over the compacted per-head cache on the 5th-generation tensor cores (bf16 inputs,
// fp32 accumulation): O = Softmax(sm_scale * Q K^T) V with ragged per-head lengths (Eq. 4 on the
// compressed cache).
//
// One CTA serves one (batch, head) and up to two 128-row query tiles, which take turns on the
// tensor pipe so that the softmax of one tile overlaps the MMAs of the other.
//   warp  0     : issuer of the Q K^T products; also owns the TMEM allocation
//   warp  1     : TMA producer (K and V tiles of 128 cache rows through rings)
//   warp  2     : issuer of the P V products (a single issuing thread for both products was the
//                 bottleneck of the CTA: 0.212 -> 0.174 ms on the largest launch)
//   warp  3     : appends the new scale's rows to the cache with bulk copies (heads that keep it whole)
//   warps 4-7   : softmax of tile 0 (thread r owns query row r: one TMEM lane, no shuffles)
//   warps 8-11  : softmax of tile 1
//   The first warpgroup hands most of its registers to the softmax warpgroups (setmaxnreg) so that
//   a whole 128-column score row lives in registers.
//
// What shapes the kernel (all measured on the device):
//  * The thread that issues the MMAs needs instruction-issue slots of its scheduler; many busy
//    softmax warps starve it (with four always-ready warps per scheduler one tcgen05.mma took
//    over 200 cycles to issue against about 70 to execute).  Hence one thread per query row (two
//    softmax warps per scheduler, normally only one of them active) rather than more, lighter
//    threads, and as few softmax instructions as possible: scale / sum / max work runs on packed
//    or 3-input instructions.
//  * Exponentials are scarce (16 per clock and SM against 8192 tensor flops): kPolyOf8 of every
//    8 pairs can be evaluated with a cubic on the FMA pipe instead.  Two of eight made the loop
//    2.4 % faster, but a probability from the cubic can round to the other bf16 neighbour than
//    the one the row-sum correction below assumes, which cost 5e-3 of output accuracy: off.
// TMEM (512 columns): S [0,128)  P0 [128,192)  P1 [192,256)  O0 [256,256+D)  O1 [256+D,256+2D).
// There is ONE logit buffer, which the two tiles use in turn, and a probability buffer per tile.  A
// softmax thread reads its whole logit row into registers first and hands the buffer back at once
// (s_free), so the next Q K^T product (the other tile's, or with one tile per CTA this tile's next
// block) runs while it computes; the probabilities go to the tile's own buffer, from where the
// second MMA takes them, so that no product waits for another to release columns it writes.  With
// one buffer per tile holding first the logits and then the probabilities (the earlier form), each
// tile was a serial chain softmax -> P V -> Q K^T -> softmax of about 3 400 cycles per 128 keys,
// and the two tiles only interleaved; now the tensor pipe and the exponentials each run at their own
// rate.  K tiles are K-major operands, V tiles MN-major operands, both 128-byte swizzled as TMA
// writes them.  Softmax keeps a running maximum that is only raised (and O rescaled in TMEM) when
// a row's maximum grows by more than 2^32, so rescaling is rare after the first tile.
// (Tried and dropped: logits in two buffers of 64 keys per tile.  The 128 x 64 x 16 MMA re-reads the
// whole Q operand from shared memory for half the keys and takes nearly as long as the
// 128 x 128 x 16 one: the last-scale launch of the 10 521-token workload went from 0.233 to 0.301 ms.)
// The keys and values of a head come in two segments: len_a rows of the head's cache, then len_b
// rows of the new scale taken straight from the caller's K/V tensors (second pair of tensor maps).
// Heads that keep the whole new scale (steps without eviction; structural heads, whose latest scale
// is protected, Eq. 11) are served that way before the new rows are in the cache: the append
// (Eq. 3) is done by warp 3 of the same CTAs with bulk copies through a small staging buffer, each
// CTA of a head taking a slice of the rows; nothing in this launch reads the rows they write.
// A tile's output rows leave through the shared memory of its query tile (free once the last Q K^T
// product has read it) and one tiled store per 64 columns; the store's 3-D tensor map of the output
// clips the rows behind a head's last query.
// Every mbarrier wait is bounded; on expiry the CTA raises the status word, drains what it has in
// flight, frees its TMEM and returns.
#include <cuda.h>

#include "hack_internal.h"
#include "tc_ptx.cuh"

namespace hack {
namespace {

using namespace ptx;

constexpr int kBM = 128;                 // query rows per tile
constexpr int kBN = 128;                 // cache rows per K/V tile
constexpr int kThreadsTc = 384;
constexpr int kMmaWarp = 0, kProducerWarp = 1, kPvWarp = 2, kAppendWarp = 3;   // an issuer is the oldest warp of its scheduler
constexpr int kSoftmaxRegs = 224, kOtherRegs = 56;   // 2*128*224 + 128*56 = 384*168 registers
constexpr int kPolyOf8 = 0;              // pairs out of 8 whose 2^x runs on the FMA pipe
constexpr int kKStages = 2;
constexpr int kVStages = 2;
constexpr uint32_t kSpinLimit = 1u << 22;          // polls while draining after an abort
constexpr uint32_t kCopyChunk = 16384;             // bytes per bulk copy of the append
constexpr float kRescaleThreshold = 32.0f;   // log2 units: p <= 2^32, far inside the bf16 / fp32 range

struct TcParams {
  int n_heads, n_new, n_pairs;           // n_pairs: CTAs per head
  int tiles_per_cta;                     // 2, or 1 when the grid would not fill the GPU otherwise
  int len_a[2], len_b[2];                // per head type: rows read from the cache, then from the caller's K/V
  int append_new;                        // heads with len_b > 0 also store those rows behind their len_a cache rows
  int q_before_wait;                     // the queries may be read ahead of the dependency wait
  int pos_base;                          // global position of the new scale's first token
  int head_dim_pieces;                   // 16-byte pieces per row
  int cap[2];                            // rows a head of each type owns (checked builds)
  long long wait_cycles;                 // limit of every mbarrier wait
  uint4* k_plane;                        // cache planes of this layer (append only)
  uint4* v_plane;
  int32_t* pos_plane;
  const uint4* k_new;                    // the caller's K/V (append only)
  const uint4* v_new;
  float scale_log2;                      // sm_scale * log2(e)
  const uint8_t* is_ctx;
  const int32_t* row_off;
  const int32_t* head_order;             // longest heads first
  __nv_bfloat16* out;
  float* row_stats;                      // optional [b*H, N_k, 2]: reference maximum and sum of every softmax row
  int* status;
};

struct Bars {
  uint64_t q_full[2];
  uint64_t k_full[kKStages], k_empty[kKStages];
  uint64_t v_full[kVStages], v_empty[kVStages];
  uint64_t s_full[2], s_free, p_full[2], p_free[2], o_final[2];
  uint64_t copy_full[2];                            // append: a chunk of new rows has landed in its staging half
  uint64_t drain, drain2;
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, Bars* b, int* status, int code,
                                         long long limit) {
  const uint32_t addr = smem_u32(bar);
  if (mbar_try_wait(addr, parity)) return true;
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

template <int D>
__global__ void __launch_bounds__(kThreadsTc, 1)
attend_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                 const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_kn,
                 const __grid_constant__ CUtensorMap tm_vn, const __grid_constant__ CUtensorMap tm_o,
                 const TcParams p) {
  constexpr int SUB = D / 64;                       // 64-column (128-byte) sub-tiles per row
  constexpr uint32_t SUB_BYTES = kBN * 128;         // one sub-tile: 128 rows x 128 bytes
  constexpr uint32_t TILE_BYTES = SUB * SUB_BYTES;
  constexpr uint32_t S_COL = 0, P_COL = 128, O_COL = 256;

  extern __shared__ unsigned char smem_dyn[];
  const uint32_t raw = smem_u32(smem_dyn);
  const uint32_t base = (raw + 1023u) & ~1023u;     // 128-byte swizzle needs 1024-byte alignment
  unsigned char* sm = smem_dyn + (base - raw);
  const uint32_t q_sm = base;
  const uint32_t k_sm = q_sm + 2 * TILE_BYTES;
  const uint32_t v_sm = k_sm + kKStages * TILE_BYTES;
  const uint32_t copy_sm = v_sm + kVStages * TILE_BYTES;           // 2 x kCopyChunk bytes: staging of the append
  Bars* bars = reinterpret_cast<Bars*>(sm + (2 + kKStages + kVStages) * TILE_BYTES + 2 * kCopyChunk);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int bh = p.head_order[blockIdx.x / p.n_pairs];
  const int pair = blockIdx.x % p.n_pairs;
  const int type = p.is_ctx[bh % p.n_heads];
  const int len_a = p.len_a[type], len_b = p.len_b[type];
  const int nblk_a = (len_a + kBN - 1) / kBN;
  const int nblk = nblk_a + (len_b + kBN - 1) / kBN;      // >= 1: a head never attends over nothing
  const int q0 = pair * p.tiles_per_cta * kBM;
  const int ntile = (p.tiles_per_cta == 2 && q0 + kBM < p.n_new) ? 2 : 1;

  const int qrow = bh * p.n_new + q0;
  const int krow = p.row_off[bh];
  const int nrow = bh * p.n_new;
  const long long wlim = p.wait_cycles;
  // K / V tile j of this head: which tensor it comes from and its first row there
  auto k_src = [&](int j) { return j < nblk_a ? &tm_k : &tm_kn; };
  auto v_src = [&](int j) { return j < nblk_a ? &tm_v : &tm_vn; };
  auto tile_row = [&](int j) { return j < nblk_a ? krow + j * kBN : nrow + (j - nblk_a) * kBN; };
  if (warp == kProducerWarp && lane == 0) {
    for (int t = 0; t < 2; ++t) {
      mbar_init(smem_u32(&bars->q_full[t]), 1);
      mbar_init(smem_u32(&bars->s_full[t]), 1);
      mbar_init(smem_u32(&bars->p_full[t]), 4);     // one arrival per warp of the tile
      mbar_init(smem_u32(&bars->p_free[t]), 1);
      mbar_init(smem_u32(&bars->o_final[t]), 1);
    }
    for (int s = 0; s < kKStages; ++s) { mbar_init(smem_u32(&bars->k_full[s]), 1); mbar_init(smem_u32(&bars->k_empty[s]), 1); }
    for (int s = 0; s < kVStages; ++s) { mbar_init(smem_u32(&bars->v_full[s]), 1); mbar_init(smem_u32(&bars->v_empty[s]), 1); }
    mbar_init(smem_u32(&bars->s_free), 4);          // the four warps of the tile whose logits were in the buffer
    mbar_init(smem_u32(&bars->copy_full[0]), 1);
    mbar_init(smem_u32(&bars->copy_full[1]), 1);
    mbar_init(smem_u32(&bars->drain), 1);
    mbar_init(smem_u32(&bars->drain2), 1);
    bars->abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
    // the producer starts the first loads at once: they run under the TMEM allocation, the
    // block-wide synchronisation and the register reallocation below
    prefetch_tensormap(&tm_q);
    prefetch_tensormap(&tm_k);
    prefetch_tensormap(&tm_v);
    prefetch_tensormap(&tm_o);
    if (len_b > 0) {
      prefetch_tensormap(&tm_kn);
      prefetch_tensormap(&tm_vn);
    }
    // The queries are the caller's input.  When the kernel ahead of this one in the stream is the
    // step's own compression launch, whatever produced them had completed before that launch passed
    // its dependency wait, hence before any CTA of this launch started: they are loaded ahead of the
    // wait, under the compression's last CTAs.
    auto load_queries = [&]() {
      for (int t = 0; t < ntile; ++t) {
        const uint32_t bar = smem_u32(&bars->q_full[t]);
        mbar_expect_tx(bar, TILE_BYTES);
        for (int c = 0; c < SUB; ++c)
          tma_load_2d(q_sm + t * TILE_BYTES + c * SUB_BYTES, &tm_q, c * 64, qrow + t * kBM, bar);
      }
    };
    if (p.q_before_wait) load_queries();
    pdl_wait();
    if (!p.q_before_wait) load_queries();
    mbar_expect_tx(smem_u32(&bars->k_full[0]), TILE_BYTES);
    for (int c = 0; c < SUB; ++c) tma_load_2d(k_sm + c * SUB_BYTES, k_src(0), c * 64, tile_row(0), smem_u32(&bars->k_full[0]));
    mbar_expect_tx(smem_u32(&bars->v_full[0]), TILE_BYTES);
    for (int c = 0; c < SUB; ++c) tma_load_2d(v_sm + c * SUB_BYTES, v_src(0), c * 64, tile_row(0), smem_u32(&bars->v_full[0]));
  }
  if (warp == kMmaWarp) {
    tmem_alloc(smem_u32(&bars->tmem_base), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&bars->tmem_base);
  pdl_wait();     // everything above overlaps the tail of the previous kernel

  if (warp == kPvWarp) {
    // ------------------------------------------------------------------ issuer of the P V products
    // (a thread of its own: one thread issuing both products was the bottleneck of the CTA)
    reg_dec<kOtherRegs>();
    if (lane == 0) {
      constexpr uint32_t IDESC_PV = idesc_bf16_f32(kBM, D, 1);         // A = P (TMEM), B = V (MN-major)
      const uint64_t v_desc0 = smem_desc_sw128(v_sm, SUB_BYTES, 1024);
      bool ok = true;
      for (int j = 0; j < nblk && ok; ++j) {
        const int vs = j % kVStages;
        const uint64_t vd = v_desc0 + (uint64_t)((vs * TILE_BYTES) >> 4);
        for (int t = 0; t < ntile && ok; ++t) {
          ok = wait_bar(&bars->p_full[t], j & 1, bars, p.status, 5, wlim);
          if (ok && t == 0) ok = wait_bar(&bars->v_full[vs], (j / kVStages) & 1, bars, p.status, 6, wlim);
          if (!ok) break;
          tc_fence_after();
          mma_ts_chain4(tmem + O_COL + t * D, tmem + P_COL + t * 64, vd, IDESC_PV, j > 0);
          mma_ts_chain4(tmem + O_COL + t * D, tmem + P_COL + t * 64 + 32, vd + 4 * 128, IDESC_PV, 1);
          mma_commit(smem_u32(&bars->p_free[t]));             // P_t may be rewritten, O_t is up to date
          if (t == ntile - 1) mma_commit(smem_u32(&bars->v_empty[vs]));
          if (j + 1 == nblk) mma_commit(smem_u32(&bars->o_final[t]));
        }
      }
      if (!ok) {
        mma_commit(smem_u32(&bars->drain2));
        const uint32_t bar = smem_u32(&bars->drain2);
        for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(bar, 0); ++it) {}
      }
    }
  } else if (warp == kAppendWarp) {
    reg_dec<kOtherRegs>();
    if (p.append_new && len_b > 0 && dbg_ok(len_a >= 0 && len_a + len_b <= p.cap[type], p.status, 7)) {
      // Eq. 3 for this head: the new scale's rows go behind the len_a cache rows.  The rows are one
      // contiguous run in the caller's tensor and in the cache plane; the CTAs of the head share
      // them, and one thread moves this CTA's slice with bulk copies through two staging halves
      // (global -> shared -> global), so the append costs no registers and no issue slots.
      const int per_cta = (len_b + p.n_pairs - 1) / p.n_pairs;
      const int r0 = pair * per_cta, r1 = min(len_b, r0 + per_cta);
      for (int r = r0 + lane; r < r1; r += 32) p.pos_plane[krow + len_a + r] = p.pos_base + r;
      if (lane == 0 && r1 > r0) {
        const uint32_t row_bytes = (uint32_t)p.head_dim_pieces * 16;
        const size_t src_off = ((size_t)nrow + r0) * row_bytes, dst_off = ((size_t)krow + len_a + r0) * row_bytes;
        const uint32_t total = (uint32_t)(r1 - r0) * row_bytes;
        const uint32_t n_chunks = (total + kCopyChunk - 1) / kCopyChunk;
        bool ok = true;
        uint32_t n = 0;                              // chunk counter over both planes
        for (int plane = 0; plane < 2 && ok; ++plane) {
          const unsigned char* src = reinterpret_cast<const unsigned char*>(plane == 0 ? p.k_new : p.v_new) + src_off;
          unsigned char* dst = reinterpret_cast<unsigned char*>(plane == 0 ? p.k_plane : p.v_plane) + dst_off;
          for (uint32_t ch = 0; ch < n_chunks && ok; ++ch, ++n) {
            const uint32_t half = n & 1;
            const uint32_t bytes = min(kCopyChunk, total - ch * kCopyChunk);
            const uint32_t bar = smem_u32(&bars->copy_full[half]);
            bulk_wait_read<1>();                     // the store that last read this half (two chunks ago) is done with it
            mbar_expect_tx(bar, bytes);
            bulk_load(copy_sm + half * kCopyChunk, src + (size_t)ch * kCopyChunk, bytes, bar);
            ok = wait_bar(&bars->copy_full[half], (n >> 1) & 1, bars, p.status, 12, wlim);
            if (!ok) break;
            bulk_store(dst + (size_t)ch * kCopyChunk, copy_sm + half * kCopyChunk, bytes);
            bulk_commit();
          }
        }
        bulk_wait<0>();                              // every store has been performed before the CTA may leave
      }
    }
  } else if (warp == kProducerWarp) {
    // ------------------------------------------------------------------ TMA producer
    reg_dec<kOtherRegs>();
    if (lane == 0) {
      int k_issued = 1, v_issued = 1;               // Q and tile 0 of K and V are already on their way
      bool ok = true;
      for (int j = 1; j < nblk && ok; ++j) {
        {
          const int s = j % kKStages;
          ok = wait_bar(&bars->k_empty[s], ((j / kKStages) & 1) ^ 1, bars, p.status, 1, wlim);
          if (!ok) break;
          const uint32_t bar = smem_u32(&bars->k_full[s]);
          mbar_expect_tx(bar, TILE_BYTES);
          for (int c = 0; c < SUB; ++c)
            tma_load_2d(k_sm + s * TILE_BYTES + c * SUB_BYTES, k_src(j), c * 64, tile_row(j), bar);
          ++k_issued;
        }
        {
          const int s = j % kVStages;
          ok = wait_bar(&bars->v_empty[s], ((j / kVStages) & 1) ^ 1, bars, p.status, 2, wlim);
          if (!ok) break;
          const uint32_t bar = smem_u32(&bars->v_full[s]);
          mbar_expect_tx(bar, TILE_BYTES);
          for (int c = 0; c < SUB; ++c)
            tma_load_2d(v_sm + s * TILE_BYTES + c * SUB_BYTES, v_src(j), c * 64, tile_row(j), bar);
          ++v_issued;
        }
      }
      if (!ok) {
        // give the copies already in flight a bounded chance to land before the CTA leaves
        for (int t = 0; t < ntile; ++t) {
          const uint32_t bar = smem_u32(&bars->q_full[t]);
          for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(bar, 0); ++it) {}
        }
        for (int i = max(0, k_issued - kKStages); i < k_issued; ++i) {
          const uint32_t bar = smem_u32(&bars->k_full[i % kKStages]);
          for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(bar, (i / kKStages) & 1); ++it) {}
        }
        for (int i = max(0, v_issued - kVStages); i < v_issued; ++i) {
          const uint32_t bar = smem_u32(&bars->v_full[i % kVStages]);
          for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(bar, (i / kVStages) & 1); ++it) {}
        }
      }
    }
  } else if (warp == kMmaWarp) {
    // ------------------------------------------------------------------ issuer of the Q K^T products
    reg_dec<kOtherRegs>();
    if (lane == 0) {
      constexpr uint32_t IDESC_S = idesc_bf16_f32(kBM, kBN, 0);        // A = Q, B = K (both K-major)
      // descriptors of the tile bases; a k-step only adds a constant to the address field
      const uint64_t q_desc[2] = {smem_desc_sw128(q_sm, 16, 1024), smem_desc_sw128(q_sm + TILE_BYTES, 16, 1024)};
      const uint64_t k_desc0 = smem_desc_sw128(k_sm, 16, 1024);
      bool ok = true;
      // S = Q_t K_j^T into the one logit buffer; `use` counts the products issued so far, and product
      // number use needs the logits of product use - 1 to have left the buffer (s_free phase use - 1)
      int use = 0;
      auto issue_s = [&](int t, int j) -> bool {
        if (use > 0 && !wait_bar(&bars->s_free, (use - 1) & 1, bars, p.status, 10, wlim)) return false;
        tc_fence_after();
        const uint64_t kd = k_desc0 + (uint64_t)(((j % kKStages) * TILE_BYTES) >> 4);
        if constexpr (D == 128) mma_ss_chain8(tmem + S_COL, q_desc[t], kd, IDESC_S, 0);
        else mma_ss_chain4(tmem + S_COL, q_desc[t], kd, IDESC_S, 0);
        mma_commit(smem_u32(&bars->s_full[t]));
        ++use;
        return true;
      };
      for (int t = 0; t < ntile && ok; ++t) ok = wait_bar(&bars->q_full[t], 0, bars, p.status, 3, wlim);
      if (ok) ok = wait_bar(&bars->k_full[0], 0, bars, p.status, 4, wlim);
      for (int t = 0; t < ntile && ok; ++t) ok = issue_s(t, 0);
      if (ok) mma_commit(smem_u32(&bars->k_empty[0]));
      for (int j = 0; j < nblk && ok; ++j) {
        for (int t = 0; t < ntile && ok; ++t) {
          // the next logits of this tile: they only wait for the buffer, not for this tile's
          // softmax, and so run under it
          if (j + 1 < nblk) {
            if (t == 0) {
              ok = wait_bar(&bars->k_full[(j + 1) % kKStages], ((j + 1) / kKStages) & 1, bars, p.status, 7, wlim);
              if (!ok) break;
            }
            ok = issue_s(t, j + 1);
            if (!ok) break;
            if (t == ntile - 1) mma_commit(smem_u32(&bars->k_empty[(j + 1) % kKStages]));
          }
        }
      }
      if (!ok) {
        mma_commit(smem_u32(&bars->drain));
        const uint32_t bar = smem_u32(&bars->drain);
        for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(bar, 0); ++it) {}
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue
    reg_inc<kSoftmaxRegs>();
    const int t = (warp >> 2) - 1;                 // tile served by this warpgroup
    if (t < ntile) {
      const int r = tid & 127;                     // query row inside the tile == TMEM lane
      const uint32_t lane_addr = static_cast<uint32_t>((warp & 3) * 32) << 16;
      const uint32_t s_addr = tmem + lane_addr + S_COL;
      const uint32_t p_addr = tmem + lane_addr + P_COL + t * 64;
      const uint32_t o_addr = tmem + lane_addr + O_COL + t * D;
      const float c = p.scale_log2;
      float m_used = -INFINITY, l = 0.f;
      bool ok = true;
      for (int j = 0; j < nblk; ++j) {
        ok = __all_sync(0xffffffffu, wait_bar(&bars->s_full[t], j & 1, bars, p.status, 8, wlim));
        if (!ok) break;
        tc_fence_after();
        uint32_t sr[kBN];
#pragma unroll
        for (int ch = 0; ch < kBN / 32; ++ch) tmem_ld32(s_addr + ch * 32, sr + ch * 32);
        tmem_wait_ld();
        // the logits are in registers: the buffer goes back to the MMA warp at once
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars->s_free));
        // live keys of this tile: fewer than 128 only in the last tile of either segment
        const int valid = j < nblk_a ? len_a - j * kBN : len_b - (j - nblk_a) * kBN;
        if (valid < kBN) {
#pragma unroll
          for (int i = 0; i < kBN; ++i)
            if (i >= valid) sr[i] = 0xff800000u;   // -inf
        }
        // row maximum, kept apart for the pairs whose exponential runs on the FMA pipe (pair index
        // i with (i & 7) < kPolyOf8) and for the others: the row-sum correction below must form the
        // largest probability with the same instructions the loop uses for that element
        float mx_sfu[4], mx_fma[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          mx_sfu[u] = -INFINITY;
          mx_fma[u] = -INFINITY;
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float e0 = __uint_as_float(sr[u * 32 + 2 * i]), e1 = __uint_as_float(sr[u * 32 + 2 * i + 1]);
            if ((i & 7) < kPolyOf8) mx_fma[u] = max3(mx_fma[u], e0, e1);
            else mx_sfu[u] = max3(mx_sfu[u], e0, e1);
          }
        }
        const float mxs = fmaxf(fmaxf(mx_sfu[0], mx_sfu[1]), fmaxf(mx_sfu[2], mx_sfu[3]));
        const float mxf = fmaxf(fmaxf(mx_fma[0], mx_fma[1]), fmaxf(mx_fma[2], mx_fma[3]));
        const float mx = fmaxf(mxs, mxf);
        const bool grow = (mx - m_used) * c > kRescaleThreshold;     // always true in the first tile
        const bool any_grow = __any_sync(0xffffffffu, grow);
        float alpha = 1.f;
        if (any_grow) {
          const float m_new = grow ? mx : m_used;
          alpha = grow ? ex2((m_used - m_new) * c) : 1.f;
          l *= alpha;
          m_used = m_new;
        }
        const float2 c2 = make_float2(c, c);
        const float2 nmc2 = make_float2(-m_used * c, -m_used * c);
        float2 sum4[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
        uint32_t pk[kBN / 2];
#pragma unroll
        for (int i = 0; i < kBN / 2; ++i) {
          const float2 x = fma2(make_float2(__uint_as_float(sr[2 * i]), __uint_as_float(sr[2 * i + 1])), c2, nmc2);
          float2 pr;
          if ((i & 7) < kPolyOf8) {
            pr = ex2_poly2(x);
          } else {
            pr.x = ex2(x.x);
            pr.y = ex2(x.y);
          }
          sum4[i & 3] = add2(sum4[i & 3], pr);
          const __nv_bfloat162 hh = __floats2bfloat162_rn(pr.x, pr.y);
          pk[i] = *reinterpret_cast<const uint32_t*>(&hh);
        }
        const float2 sum2 = add2(add2(sum4[0], sum4[1]), add2(sum4[2], sum4[3]));
        l += sum2.x + sum2.y;
        {
          // The second MMA sees the probabilities rounded to bf16, the row sum does not.  With the
          // lazily raised reference maximum even a dominant key's probability is no power of two,
          // and its rounding error (up to 2^-9 of an output that can reach 4) would pass straight
          // into O.  The tile's largest probability is therefore entered into the sum as rounded,
          // which makes the weight of a dominant key exact; what is left is bounded by the weight
          // of the other keys.  Same instructions as the loop above uses for that element, hence the same bits.
          const float x_top = fmaf(mx, c, nmc2.x);
          float p_top = ex2(x_top);
          if (kPolyOf8 > 0 && mxf > mxs) p_top = ex2_poly2(make_float2(x_top, x_top)).x;
          l += __bfloat162float(__float2bfloat16_rn(p_top)) - p_top;
        }
        if (j > 0) {
          // P_t still feeds the product of the previous block, which also still adds to O_t
          ok = __all_sync(0xffffffffu, wait_bar(&bars->p_free[t], (j - 1) & 1, bars, p.status, 11, wlim));
          if (!ok) break;
          tc_fence_after();
          if (any_grow) {
#pragma unroll 1
            for (int ch = 0; ch < D / 8; ++ch) {             // rare path: kept light on registers
              uint32_t orr[8];
              tmem_ld8(o_addr + ch * 8, orr);
              tmem_wait_ld();
#pragma unroll
              for (int i = 0; i < 8; ++i) orr[i] = __float_as_uint(__uint_as_float(orr[i]) * alpha);
              tmem_st8(o_addr + ch * 8, orr);
            }
          }
        }
        tmem_st32(p_addr, pk);
        tmem_st32(p_addr + 32, pk + 32);
        tmem_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars->p_full[t]));
      }
      if (ok) ok = __all_sync(0xffffffffu, wait_bar(&bars->o_final[t], 0, bars, p.status, 9, wlim));
      // the four warps of the tile meet on a named barrier below, so they agree first on whether all of them got here
      uint32_t all_ok;
      asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.and.pred p, %2, 128, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                   : "=r"(all_ok) : "r"((uint32_t)ok), "r"(1 + t) : "memory");
      if (all_ok) {
        tc_fence_after();
        const int row = q0 + t * kBM + r;
        const float inv = 1.f / l;
        if (p.row_stats && row < p.n_new)
          *reinterpret_cast<float2*>(p.row_stats + (static_cast<size_t>(bh) * p.n_new + row) * 2) = make_float2(m_used, l);
        // The tile's output goes through its query tile's shared memory (the last Q K^T product has
        // read it), laid out as a tiled copy with the 128-byte swizzle expects it: thread r's 16-byte
        // pieces of a store instruction fall into different banks, and one tiled store per 64
        // columns writes whole rows (a thread storing its own row straight to memory wrote 32
        // half-used sectors per instruction: 3 us per CTA against 1).  Rows past the head's last
        // query lie outside the tensor and are not written.
        const uint32_t o_sm = q_sm + t * TILE_BYTES + r * 128;
#pragma unroll
        for (int ch = 0; ch < D / 32; ++ch) {
          uint32_t orr[32];
          tmem_ld32(o_addr + ch * 32, orr);
          tmem_wait_ld();
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(orr[v * 8 + 2 * e]) * inv,
                                                              __uint_as_float(orr[v * 8 + 2 * e + 1]) * inv);
              w[e] = *reinterpret_cast<const uint32_t*>(&hh);
            }
            const int piece = ch * 4 + v;                      // 16-byte piece of the row
            st_shared_v4(o_sm + (piece >> 3) * SUB_BYTES + (((piece & 7) ^ (r & 7)) << 4), w[0], w[1], w[2], w[3]);
          }
        }
        fence_proxy_async();                                   // the tiled store reads what these threads wrote
        asm volatile("bar.sync %0, 128;" ::"r"(1 + t) : "memory");
        if (r == 0) {
#pragma unroll
          for (int cc = 0; cc < SUB; ++cc) tma_store_3d(&tm_o, cc * 64, q0 + t * kBM, bh, q_sm + t * TILE_BYTES + cc * SUB_BYTES);
          bulk_commit();
          bulk_wait_read<0>();                                 // shared memory is read out before the CTA leaves
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  return fn;
}

template <int D>
size_t tc_smem_bytes() {
  return 1024 + (2 + kKStages + kVStages) * (size_t)(D / 64) * kBN * 128 + 2 * kCopyChunk + sizeof(Bars) + 64;
}

}  // namespace

// 2-D bf16 tensor map over `rows` x `head_dim`, box = 128 rows x 64 columns, 128-byte swizzle.
bool make_rows_map(void* out_map, const void* base, uint64_t rows, int head_dim) {
  EncodeTiledFn fn = encode_fn();
  if (!fn || rows == 0) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)head_dim, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)head_dim * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)kBN};
  const cuuint32_t estr[2] = {1, 1};
  return fn(static_cast<CUtensorMap*>(out_map), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims,
            strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

namespace {
// 3-D bf16 tensor map over the output [heads, n_new, head_dim] (boxes of 128 rows x 64 columns of one
// head, 128-byte swizzle): a tile that reaches past the head's last query row is clipped there.
bool make_out_map(CUtensorMap* out_map, const void* base, int heads, int n_new, int head_dim) {
  EncodeTiledFn fn = encode_fn();
  if (!fn || heads <= 0 || n_new <= 0) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)head_dim, (cuuint64_t)n_new, (cuuint64_t)heads};
  const cuuint64_t strides[2] = {(cuuint64_t)head_dim * 2, (cuuint64_t)n_new * head_dim * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)kBM, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(out_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
}  // namespace

int launch_attend_tc(const StepArgs& a, const void* k_map, const void* v_map, const int32_t* head_order,
                     const void* q, void* out, float* row_stats, const void* k_new, const void* v_new,
                     int n_heads_served, bool shares_gpu, cudaStream_t st, bool follows_compression) {
  CUtensorMap tm_q;
  if (!make_rows_map(&tm_q, q, (uint64_t)a.batch * a.n_heads * a.n_new, a.head_dim)) {
    set_error("attention: cuTensorMapEncodeTiled failed for the queries");
    return -1;
  }
  CUtensorMap tm_o;
  if (!make_out_map(&tm_o, out, a.batch * a.n_heads, a.n_new, a.head_dim)) {
    set_error("attention: cuTensorMapEncodeTiled failed for the output");
    return -1;
  }
  TcParams p;
  p.n_heads = a.n_heads;
  p.n_new = a.n_new;
  const int n_tiles = (a.n_new + kBM - 1) / kBM;
  // n_heads_served < all heads: only the first heads of head_order (those of one type) are served
  const int heads = n_heads_served > 0 ? n_heads_served : a.batch * a.n_heads;
  // one query tile per CTA while that still fits one wave: twice the CTAs, no idle SMs; a launch
  // that shares the GPU with the other head type's compression keeps two
  p.tiles_per_cta = (!shares_gpu && n_tiles * heads <= sm_count()) ? 1 : 2;
  p.n_pairs = (n_tiles + p.tiles_per_cta - 1) / p.tiles_per_cta;
  const CUtensorMap& tk = *static_cast<const CUtensorMap*>(k_map);
  const CUtensorMap& tv = *static_cast<const CUtensorMap*>(v_map);
  CUtensorMap tm_kn = tk, tm_vn = tv;       // placeholders unless a head type reads the caller's rows
  p.append_new = 0;
  for (int t = 0; t < 2; ++t) {
    const bool from_caller = k_new && v_new && a.seg_new[t];
    p.len_b[t] = from_caller ? a.n_new : 0;
    p.len_a[t] = a.kept[t] - p.len_b[t];
    if (from_caller) p.append_new = 1;
  }
  if (p.append_new) {
    const uint64_t rows = (uint64_t)a.batch * a.n_heads * a.n_new;
    if (!make_rows_map(&tm_kn, k_new, rows, a.head_dim) || !make_rows_map(&tm_vn, v_new, rows, a.head_dim)) {
      set_error("attention: cuTensorMapEncodeTiled failed for the new scale's keys or values");
      return -1;
    }
  }
  p.q_before_wait = follows_compression ? 1 : 0;
  p.pos_base = a.pos_base;
  p.head_dim_pieces = a.head_dim * 2 / 16;
  p.cap[0] = a.cap[0];
  p.cap[1] = a.cap[1];
  p.wait_cycles = a.wait_cycles;
  p.k_plane = static_cast<uint4*>(a.k_plane);
  p.v_plane = static_cast<uint4*>(a.v_plane);
  p.pos_plane = a.pos_plane;
  p.k_new = static_cast<const uint4*>(k_new);
  p.v_new = static_cast<const uint4*>(v_new);
  p.scale_log2 = a.sm_scale * 1.4426950408889634f;
  p.is_ctx = a.is_ctx;
  p.row_off = a.row_off;
  p.head_order = head_order;
  p.out = static_cast<__nv_bfloat16*>(out);
  p.row_stats = row_stats;
  p.status = a.status;
  const int grid = p.n_pairs * heads;
  if (a.head_dim == 128) {
    if (!allow_dynamic_smem(attend_tc_kernel<128>, tc_smem_bytes<128>())) return -1;
    launch_k(attend_tc_kernel<128>, grid, kThreadsTc, tc_smem_bytes<128>(), st, tm_q, tk, tv, tm_kn, tm_vn, tm_o, p);
  } else {
    if (!allow_dynamic_smem(attend_tc_kernel<64>, tc_smem_bytes<128>())) return -1;
    // the larger request keeps it at one CTA per SM (the kernel owns all 512 TMEM columns)
    launch_k(attend_tc_kernel<64>, grid, kThreadsTc, tc_smem_bytes<128>(), st, tm_q, tk, tv, tm_kn, tm_vn, tm_o, p);
  }
  return launched(1);
}

}  // namespace hack
