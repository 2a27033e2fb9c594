// In-place compaction of the ragged per-head cache (the gathers of Eq. 10-11).
//
// Output row r of a head takes candidate idx[r]; the list is strictly ascending, so r <= idx[r]
// and the survivors that were already stored (idx[r] < L) form a prefix of the list, of length
// n_old.  The two parts are served by different CTAs of the same launch:
//
//  * rows [0, n_old): a stored row only ever moves towards the front.  One CTA owns one
//    (head, plane, 64-byte column slice) and walks the prefix front to back in chunks; inside a
//    chunk every thread first loads its 16-byte pieces into registers, the CTA synchronises, then
//    the pieces are stored.  A chunk's destinations lie at or before its own sources, which lie
//    before the next chunk's sources, so no row is overwritten before it has been read and no
//    second buffer is needed.
//  * rows [n_old, min(L, kept)): new rows whose destination lies inside the old stored region.
//    Another slice's movers may still have to read those cache rows, so the CTA that owns the
//    slice writes them itself once its own moves are done.
//  * rows [L, kept): new rows landing beyond the old stored region, which no one reads in this
//    launch; any number of CTAs share them, whole rows at a time.
//
// New rows come from the caller's K/V tensors.  Heads that only append (no index list) have
// n_old = L and nothing to move.
#include "hack_internal.h"

namespace hack {
namespace {

constexpr int kThreads = 256;
constexpr int kPieces = 4;            // 16-byte pieces per thread group: one 64-byte column slice
constexpr int kMoveUnroll = 16;       // rows in flight per thread while moving stored rows
constexpr int kCopyUnroll = 8;        // rows in flight per thread while copying new rows

// Number of list entries below `stored` (the list is ascending), found by the whole CTA with two
// rounds of probes.  list == nullptr: the identity list.
__device__ __forceinline__ int count_old(const int32_t* list, int n_keep, int stored) {
  if (!list) return min(stored, n_keep);
  const int tid = threadIdx.x;
  const int step = (n_keep + kThreads - 1) / kThreads;
  // probe the last entry of every block of `step` entries
  const int p = min((tid + 1) * step, n_keep) - 1;
  const bool below = tid * step < n_keep && list[p] < stored;
  const int full_blocks = __syncthreads_count(below);      // blocks that lie entirely below
  const int lo = full_blocks * step;
  const bool below2 = tid < step && lo + tid < n_keep && list[lo + tid] < stored;
  return lo + __syncthreads_count(below2);
}

__global__ void __launch_bounds__(kThreads)
compact_kernel(const StepArgs a, const int32_t* __restrict__ idx, int idx_all,
               const uint4* __restrict__ k_new, const uint4* __restrict__ v_new, int row_pieces,
               int n_slices) {
  pdl_wait();
  const int bh = blockIdx.z;
  const int ctx = a.is_ctx[bh % a.n_heads];
  const int stored = a.stored[ctx], n_keep = a.kept[ctx];
  const bool use_idx = idx != nullptr && (a.trig[ctx] || idx_all);
  const int32_t* list = use_idx ? idx + (size_t)bh * a.kept_stride : nullptr;
  const int plane_id = blockIdx.y;                 // 0: K (its CTAs also keep the positions), 1: V
  const size_t off = a.row_off[bh];
  const int tid = threadIdx.x;
  const int n_old = count_old(list, n_keep, stored);

  int32_t* pos = a.pos_plane + off;
  uint4* plane = reinterpret_cast<uint4*>(plane_id == 0 ? a.k_plane : a.v_plane) + off * row_pieces;
  if ((int)blockIdx.x < n_slices) {
    // ---- stored rows moving towards the front, one 64-byte column slice per CTA
    if (!list) return;
    constexpr int ROWS = kThreads / kPieces;       // rows per sub-step
    const int piece = blockIdx.x * kPieces + (tid % kPieces);
    const int rsub = tid / kPieces;
    for (int c0 = 0; c0 < n_old; c0 += ROWS * kMoveUnroll) {
      uint4 val[kMoveUnroll];
      bool mv[kMoveUnroll];
#pragma unroll
      for (int u = 0; u < kMoveUnroll; ++u) {
        const int r = c0 + u * ROWS + rsub;
        mv[u] = false;
        if (r < n_old) {
          const int src = list[r];
          if (src != r) { val[u] = plane[(size_t)src * row_pieces + piece]; mv[u] = true; }
        }
      }
      __syncthreads();
#pragma unroll
      for (int u = 0; u < kMoveUnroll; ++u)
        if (mv[u]) plane[(size_t)(c0 + u * ROWS + rsub) * row_pieces + piece] = val[u];
    }
    // new rows that land inside the old stored region (this CTA has read all it needs from there)
    const uint4* fresh_s = (plane_id == 0 ? k_new : v_new) + (size_t)bh * a.n_new * row_pieces;
    const int in_end = min(stored, n_keep);
    for (int c0 = n_old; c0 < in_end; c0 += ROWS * kMoveUnroll) {
      uint4 val[kMoveUnroll];
#pragma unroll
      for (int u = 0; u < kMoveUnroll; ++u) {
        const int r = c0 + u * ROWS + rsub;
        if (r < in_end) val[u] = fresh_s[(size_t)(list[r] - stored) * row_pieces + piece];
      }
#pragma unroll
      for (int u = 0; u < kMoveUnroll; ++u) {
        const int r = c0 + u * ROWS + rsub;
        if (r < in_end) plane[(size_t)r * row_pieces + piece] = val[u];
      }
    }
    if (plane_id == 0 && blockIdx.x == 0) {
      // original positions of the same rows, same chunked load / synchronise / store scheme
      for (int c0 = 0; c0 < n_old; c0 += kThreads * kMoveUnroll) {
        int32_t val[kMoveUnroll];
        bool mv[kMoveUnroll];
#pragma unroll
        for (int u = 0; u < kMoveUnroll; ++u) {
          const int r = c0 + u * kThreads + tid;
          mv[u] = false;
          if (r < n_old) {
            const int src = list[r];
            if (src != r) { val[u] = pos[src]; mv[u] = true; }
          }
        }
        __syncthreads();
#pragma unroll
        for (int u = 0; u < kMoveUnroll; ++u)
          if (mv[u]) pos[c0 + u * kThreads + tid] = val[u];
      }
      for (int r = n_old + tid; r < in_end; r += kThreads) pos[r] = a.pos_base + (list[r] - stored);
    }
    return;
  }
  // ---- new rows beyond the old stored region: `rows_per_pass` whole rows at a time
  const uint4* fresh = (plane_id == 0 ? k_new : v_new) + (size_t)bh * a.n_new * row_pieces;
  const int n_copy_ctas = gridDim.x - n_slices;
  const int cta = blockIdx.x - n_slices;
  const int rows_per_pass = kThreads / row_pieces;
  const int piece = tid % row_pieces;
  const int rsub = tid / row_pieces;
  for (int c0 = stored + cta * rows_per_pass * kCopyUnroll; c0 < n_keep;
       c0 += n_copy_ctas * rows_per_pass * kCopyUnroll) {
    uint4 val[kCopyUnroll];
#pragma unroll
    for (int u = 0; u < kCopyUnroll; ++u) {
      const int r = c0 + u * rows_per_pass + rsub;
      if (r < n_keep) {
        const int src = (list ? list[r] : r) - stored;
        val[u] = fresh[(size_t)src * row_pieces + piece];
        if (plane_id == 0 && piece == 0) pos[r] = a.pos_base + src;
      }
    }
#pragma unroll
    for (int u = 0; u < kCopyUnroll; ++u) {
      const int r = c0 + u * rows_per_pass + rsub;
      if (r < n_keep) plane[(size_t)r * row_pieces + piece] = val[u];
    }
  }
}

}  // namespace

int launch_compact(const StepArgs& a, int dtype, const int32_t* idx, int idx_all, const void* k_new,
                   const void* v_new, cudaStream_t st) {
  const int elt = dtype == HACK_F32 ? 4 : 2;
  const int row_pieces = a.head_dim * elt / 16;    // 8, 16 or 32
  const int n_slices = row_pieces / kPieces;
  // copy CTAs per (head, plane): enough to cover the new rows of a head in about one pass, within
  // a grid of a few waves
  const int rows_per_cta = (kThreads / row_pieces) * kCopyUnroll;
  int beyond = 0;                                   // rows landing beyond the old stored region
  for (int t = 0; t < 2; ++t) beyond = a.kept[t] - a.stored[t] > beyond ? a.kept[t] - a.stored[t] : beyond;
  int n_copy = (beyond + rows_per_cta - 1) / rows_per_cta;
  const int heads = a.batch * a.n_heads;
  const int cap = (8 * 148 + 2 * heads - 1) / (2 * heads);
  n_copy = n_copy > cap ? cap : n_copy;
  dim3 grid(n_slices + n_copy, 2, heads);
  launch_k(compact_kernel, grid, kThreads, 0, st, a, idx, idx_all, static_cast<const uint4*>(k_new),
                                            static_cast<const uint4*>(v_new), row_pieces, n_slices);
  return launched(1);
}

}  // namespace hack
