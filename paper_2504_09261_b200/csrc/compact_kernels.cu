// In-place compaction of the ragged per-head cache (the gathers of Eq. 10-11).
//
// Output row r of a head takes candidate idx[r]; the list is strictly ascending, so r <= idx[r]
// and the survivors that were already stored (idx[r] < L) form a prefix of the list, of length
// n_old.  Two launches:
//
//  * compact_move_kernel, rows [0, n_old): a stored row only ever moves towards the front.  One
//    CTA owns one (head, plane, column slice of 16-64 bytes) and walks the prefix front to back in
//    chunks; inside a chunk every thread first loads its 16-byte pieces into registers, the CTA
//    synchronises, then the pieces are stored.  A chunk's destinations lie at or before its own
//    sources, which lie before the next chunk's sources, so no row is overwritten before it has
//    been read and no second buffer is needed.  The kernel also publishes n_old per head.
//  * compact_copy_kernel, rows [n_old, kept): copies of the new scale's rows out of the caller's
//    K/V tensors, whole rows at a time, by as many CTAs as there are rows to fill.  It runs after
//    the moves (some of its destinations are sources of the moves), so it has no hazard at all.
//
// Steps that only append (no index list) have n_old = L: the copy kernel alone.
#include "hack_internal.h"

namespace hack {
namespace {

constexpr int kThreads = 256;
constexpr int kMoveUnroll = 16;       // rows in flight per thread while moving stored rows
constexpr int kCopyUnroll = 8;        // rows in flight per thread while copying new rows

// Number of list entries below `stored` (the list is ascending), found by the whole CTA: a round
// of probes finds the block of `step` entries that holds the boundary, then that block is counted
// (in slices of kThreads entries, so that any list length is served).
__device__ __forceinline__ int count_old(const int32_t* list, int n_keep, int stored) {
  const int tid = threadIdx.x;
  const int step = (n_keep + kThreads - 1) / kThreads;
  // probe the last entry of every block of `step` entries
  const int p = min((tid + 1) * step, n_keep) - 1;
  const bool below = tid * step < n_keep && list[p] < stored;
  const int full_blocks = __syncthreads_count(below);      // blocks that lie entirely below
  const int lo = full_blocks * step;
  int n = lo;
  for (int i0 = 0; i0 < step; i0 += kThreads) {
    const int i = i0 + tid;
    const bool below2 = i < step && lo + i < n_keep && list[lo + i] < stored;
    n += __syncthreads_count(below2);
  }
  return n;
}

// PIECES: 16-byte pieces per row handled by one CTA (64-byte slices measured best: narrower ones
// cover more rows per chunk but waste half of every 32-byte sector).
template <int PIECES>
__global__ void __launch_bounds__(kThreads)
compact_move_kernel(const StepArgs a, const int32_t* __restrict__ idx, int row_pieces) {
  pdl_wait();
  const int bh = blockIdx.z;
  const int ctx = a.is_ctx[bh % a.n_heads];
  const int stored = a.stored[ctx], n_keep = a.kept[ctx];
  const int32_t* list = idx + (size_t)bh * a.kept_stride;
  const int plane_id = blockIdx.y;                 // 0: K (slice 0 also moves the positions), 1: V
  const size_t off = a.row_off[bh];
  const int tid = threadIdx.x;
  const int n_old = count_old(list, n_keep, stored);
  if (blockIdx.x == 0 && plane_id == 0 && tid == 0) a.n_old[bh] = n_old;

  uint4* plane = reinterpret_cast<uint4*>(plane_id == 0 ? a.k_plane : a.v_plane) + off * row_pieces;
  constexpr int ROWS = kThreads / PIECES;          // rows per sub-step
  const int piece = blockIdx.x * PIECES + (tid % PIECES);
  const int rsub = tid / PIECES;
  for (int c0 = 0; c0 < n_old; c0 += ROWS * kMoveUnroll) {
    uint4 val[kMoveUnroll];
    bool mv[kMoveUnroll];
#pragma unroll
    for (int u = 0; u < kMoveUnroll; ++u) {
      const int r = c0 + u * ROWS + rsub;
      mv[u] = false;
      if (r < n_old) {
        const int src = list[r];
        if (src != r && dbg_ok(src > r && src < stored && r < a.cap[ctx], a.status, 1)) {
          val[u] = plane[(size_t)src * row_pieces + piece];
          mv[u] = true;
        }
      }
    }
    __syncthreads();
#pragma unroll
    for (int u = 0; u < kMoveUnroll; ++u)
      if (mv[u]) plane[(size_t)(c0 + u * ROWS + rsub) * row_pieces + piece] = val[u];
  }
  if (plane_id == 0 && blockIdx.x == 0) {
    // original positions of the same rows, same chunked load / synchronise / store scheme
    int32_t* pos = a.pos_plane + off;
    for (int c0 = 0; c0 < n_old; c0 += kThreads * kMoveUnroll) {
      int32_t val[kMoveUnroll];
      bool mv[kMoveUnroll];
#pragma unroll
      for (int u = 0; u < kMoveUnroll; ++u) {
        const int r = c0 + u * kThreads + tid;
        mv[u] = false;
        if (r < n_old) {
          const int src = list[r];
          if (src != r && dbg_ok(src > r && src < stored, a.status, 2)) { val[u] = pos[src]; mv[u] = true; }
        }
      }
      __syncthreads();
#pragma unroll
      for (int u = 0; u < kMoveUnroll; ++u)
        if (mv[u]) pos[c0 + u * kThreads + tid] = val[u];
    }
  }
}

__global__ void __launch_bounds__(kThreads)
compact_copy_kernel(const StepArgs a, const int32_t* __restrict__ idx, const uint4* __restrict__ k_new,
                    const uint4* __restrict__ v_new, int row_pieces) {
  pdl_wait();
  const int bh = blockIdx.z;
  const int ctx = a.is_ctx[bh % a.n_heads];
  if (a.seg_new[ctx]) return;                      // the attention launch appends this type's new rows
  const int stored = a.stored[ctx], n_keep = a.kept[ctx];
  const int32_t* list = idx ? idx + (size_t)bh * a.kept_stride : nullptr;
  const int n_old = list ? a.n_old[bh] : stored;
  const int plane_id = blockIdx.y;                 // 0: K (also writes the positions), 1: V
  const size_t off = a.row_off[bh];
  const int tid = threadIdx.x;
  int32_t* pos = a.pos_plane + off;
  uint4* plane = reinterpret_cast<uint4*>(plane_id == 0 ? a.k_plane : a.v_plane) + off * row_pieces;
  const uint4* fresh = (plane_id == 0 ? k_new : v_new) + (size_t)bh * a.n_new * row_pieces;
  const int rows_per_pass = kThreads / row_pieces;
  const int piece = tid % row_pieces;
  const int rsub = tid / row_pieces;
  for (int c0 = n_old + blockIdx.x * rows_per_pass * kCopyUnroll; c0 < n_keep;
       c0 += gridDim.x * rows_per_pass * kCopyUnroll) {
    uint4 val[kCopyUnroll];
    bool ok[kCopyUnroll];
#pragma unroll
    for (int u = 0; u < kCopyUnroll; ++u) {
      const int r = c0 + u * rows_per_pass + rsub;
      ok[u] = false;
      if (r < n_keep) {
        const int src = (list ? list[r] : r) - stored;
        ok[u] = dbg_ok(src >= 0 && src < a.n_new && r < a.cap[ctx], a.status, 3);
        if (!ok[u]) continue;
        val[u] = fresh[(size_t)src * row_pieces + piece];
        if (plane_id == 0 && piece == 0) pos[r] = a.pos_base + src;
      }
    }
#pragma unroll
    for (int u = 0; u < kCopyUnroll; ++u) {
      const int r = c0 + u * rows_per_pass + rsub;
      if (r < n_keep && ok[u]) plane[(size_t)r * row_pieces + piece] = val[u];
    }
  }
}

}  // namespace

int launch_compact(const StepArgs& a, int dtype, const int32_t* idx, int idx_all, const void* k_new,
                   const void* v_new, cudaStream_t st) {
  (void)idx_all;                                    // an index list, when given, covers every head
  const int elt = dtype == HACK_F32 ? 4 : 2;
  const int row_pieces = a.head_dim * elt / 16;    // 8, 16 or 32
  const int heads = a.batch * a.n_heads;
  int n = 0;
  if (idx) {
    launch_k(compact_move_kernel<4>, dim3(row_pieces / 4, 2, heads), dim3(kThreads), 0, st, a, idx, row_pieces);
    ++n;
  }
  // enough CTAs for the longest list in one pass (n_old is not known here), within a few waves
  const int rows_per_cta = (kThreads / row_pieces) * kCopyUnroll;
  if (a.seg_new[0] && a.seg_new[1]) return launched(n);       // no head has rows to copy here
  int most = a.n_new;
  if (idx) {
    most = 0;
    for (int t = 0; t < 2; ++t)
      if (!a.seg_new[t] && a.kept[t] > most) most = a.kept[t];
  }
  int n_copy = (most + rows_per_cta - 1) / rows_per_cta;
  const int cap = (16 * sm_count() + 2 * heads - 1) / (2 * heads);
  n_copy = n_copy < 1 ? 1 : (n_copy > cap ? cap : n_copy);
  launch_k(compact_copy_kernel, dim3(n_copy, 2, heads), dim3(kThreads), 0, st, a, idx,
           static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new), row_pieces);
  return launched(n + 1);
}

}  // namespace hack
