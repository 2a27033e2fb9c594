// Budgeted per-head selection (Eq. 10 for contextual heads, Eq. 11 for structural heads).
//
// One CTA per (batch, head).  The n largest keys are found exactly with an 8-bit-digit radix
// select over the fp32 bit patterns (4 histogram passes in shared memory), ties at the threshold
// going to the lower candidate index; protected candidates of structural heads carry the maximal
// key so that they are always inside the kept set.  A final ordered pass turns the keep flags
// into an ascending index list with a block-wide prefix sum.
#include "hack_internal.h"

namespace hack {
namespace {

constexpr int kSelThreads = 1024;

// Order-preserving map from fp32 bits to unsigned (larger float -> larger key).
__device__ __forceinline__ uint32_t orderable(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct HeadView {
  const float* s;
  int cand, stored, t_init, protect_new, structural;
  __device__ __forceinline__ uint32_t key(int j) const {
    if (structural && (j < t_init || (protect_new && j >= stored))) return 0xffffffffu;
    const uint32_t k = orderable(s[j]);
    return k == 0xffffffffu ? 0xfffffffeu : k;   // keep the top key for protected entries only
  }
};

// Exclusive prefix sum of one flag per thread over the CTA; also returns the CTA total.
__device__ __forceinline__ int block_exclusive_scan(int flag, int* warp_sums, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t ballot = __ballot_sync(0xffffffffu, flag);
  const int in_warp = __popc(ballot & ((1u << lane) - 1u));
  if (lane == 0) warp_sums[warp] = __popc(ballot);
  __syncthreads();
  if (warp == 0) {
    const int v = warp_sums[lane];
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += n;
    }
    warp_sums[lane] = incl - v;
    if (lane == 31) warp_sums[32] = incl;
  }
  __syncthreads();
  const int res = warp_sums[warp] + in_warp;
  total = warp_sums[32];
  __syncthreads();
  return res;
}

__global__ void __launch_bounds__(kSelThreads)
select_kernel(const StepArgs a, const float* __restrict__ scores, int32_t* __restrict__ idx,
              int32_t* __restrict__ kept_out) {
  const int bh = blockIdx.x;
  const int ctx = a.is_ctx[bh % a.n_heads];
  const int cand = a.cand[ctx], n_keep = a.kept[ctx];
  int32_t* out = idx + (size_t)bh * a.kept_stride;
  const int tid = threadIdx.x;
  if (tid == 0 && kept_out) kept_out[bh] = n_keep;
  if (!a.trig[ctx] || n_keep >= cand) {           // nothing to evict: identity list
    for (int j = tid; j < cand; j += kSelThreads) out[j] = j;
    return;
  }
  HeadView hv{scores + (size_t)bh * a.cand_stride, cand, a.stored[ctx], a.t_init, a.protect_new, ctx == 0};

  __shared__ int hist[256];
  __shared__ uint32_t sh_prefix;
  __shared__ int sh_need;
  __shared__ int warp_sums[33];

  uint32_t prefix = 0, mask = 0;
  int need = n_keep;                               // rank (from the top) still to be located
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    for (int j = tid; j < cand; j += kSelThreads) {
      const uint32_t k = hv.key(j);
      if ((k & mask) == prefix) atomicAdd(&hist[(k >> shift) & 255u], 1);
    }
    __syncthreads();
    if (tid == 0) {
      int cum = 0, digit = 0;
      for (int b = 255; b >= 0; --b) {
        if (cum + hist[b] >= need) { digit = b; break; }
        cum += hist[b];
      }
      sh_prefix = prefix | ((uint32_t)digit << shift);
      sh_need = need - cum;
    }
    __syncthreads();
    prefix = sh_prefix;
    need = sh_need;
    mask |= 255u << shift;
    __syncthreads();
  }
  // prefix = key of the n_keep-th largest element; `need` of the entries equal to it survive
  const uint32_t thr = prefix;
  int out_base = 0, eq_base = 0;
  for (int base = 0; base < cand; base += kSelThreads) {
    const int j = base + tid;
    uint32_t k = 0;
    const bool in = j < cand;
    if (in) k = hv.key(j);
    const int gt = in && k > thr;
    const int eq = in && k == thr;
    int eq_total, keep_total;
    const int eq_rank = block_exclusive_scan(eq, warp_sums, eq_total);
    const int keep = gt || (eq && (eq_base + eq_rank) < need);
    const int rank = block_exclusive_scan(keep, warp_sums, keep_total);
    if (keep) out[out_base + rank] = j;
    out_base += keep_total;
    eq_base += eq_total;
  }
}

}  // namespace

int launch_select(const StepArgs& a, const float* scores, int32_t* idx, int32_t* kept_out,
                  cudaStream_t st) {
  select_kernel<<<a.batch * a.n_heads, kSelThreads, 0, st>>>(a, scores, idx, kept_out);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace hack
