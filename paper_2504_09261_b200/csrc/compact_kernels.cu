// In-place compaction of the ragged per-head cache (the gathers of Eq. 10-11).
//
// Output row r of a head takes candidate idx[r]; the list is strictly ascending, so r <= idx[r]:
// a surviving stored row only ever moves towards the front.  One CTA owns one (head, plane,
// 64-byte column slice) and walks the list front to back in chunks; inside a chunk every thread
// first loads its 16-byte pieces into registers, the CTA synchronises, then the pieces are
// stored.  A chunk's destinations lie at or before its own sources, which lie before the next
// chunk's sources, so no row is overwritten before it has been read and no second buffer is
// needed.  New-scale rows come from the caller's K/V tensors and have no hazard at all.
#include "hack_internal.h"

namespace hack {
namespace {

constexpr int kThreads = 256;
constexpr int kUnroll = 4;

// PIECES = 16-byte pieces of a row handled by this CTA (a 64-byte slice when PIECES = 4).
template <int PIECES>
__global__ void __launch_bounds__(kThreads)
compact_kernel(const StepArgs a, const int32_t* __restrict__ idx, int idx_all,
               const uint4* __restrict__ k_new, const uint4* __restrict__ v_new, int row_pieces) {
  const int bh = blockIdx.z;
  const int ctx = a.is_ctx[bh % a.n_heads];
  const int stored = a.stored[ctx], n_keep = a.kept[ctx];
  const bool use_idx = idx != nullptr && (a.trig[ctx] || idx_all);
  const int32_t* list = use_idx ? idx + (size_t)bh * a.kept_stride : nullptr;
  const int plane_id = blockIdx.y;                 // 0: K, 1: V, 2: positions
  const size_t off = a.row_off[bh];
  const int tid = threadIdx.x;
  // rows before `first` are already in place when the head only appends
  const int first = use_idx ? 0 : stored;

  if (plane_id == 2) {
    if (blockIdx.x != 0) return;
    int32_t* pos = a.pos_plane + off;
    for (int c0 = first; c0 < n_keep; c0 += kThreads * kUnroll) {
      int32_t val[kUnroll];
      bool mv[kUnroll];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int r = c0 + u * kThreads + tid;
        mv[u] = false;
        if (r < n_keep) {
          const int src = list ? list[r] : r;
          if (src >= stored) { val[u] = a.pos_base + (src - stored); mv[u] = true; }
          else if (src != r) { val[u] = pos[src]; mv[u] = true; }
        }
      }
      __syncthreads();
#pragma unroll
      for (int u = 0; u < kUnroll; ++u)
        if (mv[u]) pos[c0 + u * kThreads + tid] = val[u];
    }
    return;
  }

  constexpr int ROWS = kThreads / PIECES;          // rows per unrolled sub-step
  uint4* plane = reinterpret_cast<uint4*>(plane_id == 0 ? a.k_plane : a.v_plane) + off * row_pieces;
  const uint4* fresh = (plane_id == 0 ? k_new : v_new) + (size_t)bh * a.n_new * row_pieces;
  const int piece = blockIdx.x * PIECES + (tid % PIECES);
  const int rsub = tid / PIECES;
  for (int c0 = first; c0 < n_keep; c0 += ROWS * kUnroll) {
    uint4 val[kUnroll];
    bool mv[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int r = c0 + u * ROWS + rsub;
      mv[u] = false;
      if (r < n_keep) {
        const int src = list ? list[r] : r;
        if (src >= stored) { val[u] = fresh[(size_t)(src - stored) * row_pieces + piece]; mv[u] = true; }
        else if (src != r) { val[u] = plane[(size_t)src * row_pieces + piece]; mv[u] = true; }
      }
    }
    __syncthreads();
#pragma unroll
    for (int u = 0; u < kUnroll; ++u)
      if (mv[u]) plane[(size_t)(c0 + u * ROWS + rsub) * row_pieces + piece] = val[u];
  }
}

}  // namespace

int launch_compact(const StepArgs& a, int dtype, const int32_t* idx, int idx_all, const void* k_new,
                   const void* v_new, cudaStream_t st) {
  const int elt = dtype == HACK_F32 ? 4 : 2;
  const int row_pieces = a.head_dim * elt / 16;    // 8, 16 or 32
  constexpr int PIECES = 4;
  dim3 grid(row_pieces / PIECES, 3, a.batch * a.n_heads);
  compact_kernel<PIECES><<<grid, kThreads, 0, st>>>(a, idx, idx_all, static_cast<const uint4*>(k_new),
                                                     static_cast<const uint4*>(v_new), row_pieces);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace hack
