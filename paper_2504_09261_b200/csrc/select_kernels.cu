// Budgeted per-head selection (Eq. 10 for contextual heads, Eq. 11 for structural heads).
//
// One CTA per (batch, head).  The n largest keys are found exactly with an 8-bit-digit radix
// select over the fp32 bit patterns (4 histogram passes in shared memory), ties at the threshold
// going to the lower candidate index; protected candidates of structural heads carry the maximal
// key so that they are always inside the kept set.  A final ordered pass turns the keep flags
// into an ascending index list with a block-wide prefix sum.
//
// Fast path (up to kSelThreads * kMaxPerThread candidates): every thread keeps a contiguous run
// of keys in registers, histogram updates are aggregated per warp before they touch shared
// memory (scores of one head share their leading bits, so plain atomics would serialise), the
// digit holding the wanted rank is located by one warp, and the index list is produced with a
// single block scan.  Longer candidate lists take the general path that re-reads the scores.
#include "hack_internal.h"

namespace hack {
namespace {

constexpr int kSelThreads = 1024;
constexpr int kMaxPerThread = 16;

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

// Exclusive prefix sum of one value per thread over the CTA; also returns the CTA total.
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_sums, int& total) {
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
    const int w = warp_sums[lane];
    int wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += n;
    }
    warp_sums[lane] = wi - w;
    if (lane == 31) warp_sums[32] = wi;
  }
  __syncthreads();
  const int res = warp_sums[warp] + incl - v;
  total = warp_sums[32];
  __syncthreads();
  return res;
}

// Warp 0 finds the digit d (scanning from 255 down) at which the running count reaches `need`:
// sum_{b > d} hist[b] < need <= sum_{b >= d} hist[b].  Returns through shared memory.
__device__ __forceinline__ void locate_digit(const int* hist, int need, int* sh_digit, int* sh_need) {
  const int lane = threadIdx.x & 31;
  // lane l owns bins 255 - 8l ... 248 - 8l (descending), so lane order == descending bin order
  int c[8];
  int sum = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) { c[i] = hist[255 - 8 * lane - i]; sum += c[i]; }
  int incl = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += n;
  }
  const int before = incl - sum;               // keys in bins above this lane's bins
  if (before < need && need <= incl) {
    int cum = before;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (cum < need && need <= cum + c[i]) { *sh_digit = 255 - 8 * lane - i; *sh_need = need - cum; }
      cum += c[i];
    }
  }
}

template <int E>
__global__ void __launch_bounds__(kSelThreads)
select_reg_kernel(const StepArgs a, const float* __restrict__ scores, int32_t* __restrict__ idx,
                  int32_t* __restrict__ kept_out) {
  pdl_wait();
  const int bh = blockIdx.x;
  const int ctx = a.is_ctx[bh % a.n_heads];
  const int cand = a.cand[ctx], n_keep = a.kept[ctx];
  int32_t* out = idx + (size_t)bh * a.kept_stride;
  const int tid = threadIdx.x, lane = tid & 31;
  if (tid == 0 && kept_out) kept_out[bh] = n_keep;
  if (!a.trig[ctx] || n_keep >= cand) {           // nothing to evict: identity list
    for (int j = tid; j < cand; j += kSelThreads) out[j] = j;
    return;
  }
  HeadView hv{scores + (size_t)bh * a.cand_stride, cand, a.stored[ctx], a.t_init, a.protect_new, ctx == 0};

  __shared__ int hist[256];
  __shared__ int sh_digit, sh_need;
  __shared__ int warp_sums[33];

  // thread t owns candidates [t*E, t*E + E)
  const int j0 = tid * E;
  uint32_t key[E];
#pragma unroll
  for (int e = 0; e < E; ++e) key[e] = (j0 + e < cand) ? hv.key(j0 + e) : 0u;

  uint32_t prefix = 0, mask = 0;
  int need = n_keep;                               // rank (from the top) still to be located
#pragma unroll 1
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
#pragma unroll
    for (int e = 0; e < E; ++e) {
      const bool in = (j0 + e < cand) && ((key[e] & mask) == prefix);
      const uint32_t digit = in ? ((key[e] >> shift) & 255u) : 256u;
      const uint32_t peers = __match_any_sync(0xffffffffu, digit);
      if (in && lane == __ffs(peers) - 1) atomicAdd(&hist[digit], __popc(peers));
    }
    __syncthreads();
    if (tid < 32) locate_digit(hist, need, &sh_digit, &sh_need);
    __syncthreads();
    prefix |= (uint32_t)sh_digit << shift;
    need = sh_need;
    mask |= 255u << shift;
  }
  // prefix = key of the n_keep-th largest element; `need` of the entries equal to it survive
  const uint32_t thr = prefix;
  int gt = 0, eq = 0;
#pragma unroll
  for (int e = 0; e < E; ++e) {
    const bool in = j0 + e < cand;
    gt += in && key[e] > thr;
    eq += in && key[e] == thr;
  }
  int total;
  const int packed = block_exclusive_scan(gt | (eq << 16), warp_sums, total);
  int gt_before = packed & 0xffff, eq_before = packed >> 16;
#pragma unroll
  for (int e = 0; e < E; ++e) {
    const bool in = j0 + e < cand;
    if (in && key[e] > thr) {
      const int o = gt_before + min(eq_before, need);
      if (dbg_ok(o >= 0 && o < n_keep, a.status, 4)) out[o] = j0 + e;
      ++gt_before;
    } else if (in && key[e] == thr) {
      if (eq_before < need && dbg_ok(gt_before + eq_before < n_keep, a.status, 4)) out[gt_before + eq_before] = j0 + e;
      ++eq_before;
    }
  }
}

// General path: any candidate count; keys are recomputed from the scores in every pass.
__global__ void __launch_bounds__(kSelThreads)
select_kernel(const StepArgs a, const float* __restrict__ scores, int32_t* __restrict__ idx,
              int32_t* __restrict__ kept_out) {
  pdl_wait();
  const int bh = blockIdx.x;
  const int ctx = a.is_ctx[bh % a.n_heads];
  const int cand = a.cand[ctx], n_keep = a.kept[ctx];
  int32_t* out = idx + (size_t)bh * a.kept_stride;
  const int tid = threadIdx.x, lane = tid & 31;
  if (tid == 0 && kept_out) kept_out[bh] = n_keep;
  if (!a.trig[ctx] || n_keep >= cand) {
    for (int j = tid; j < cand; j += kSelThreads) out[j] = j;
    return;
  }
  HeadView hv{scores + (size_t)bh * a.cand_stride, cand, a.stored[ctx], a.t_init, a.protect_new, ctx == 0};

  __shared__ int hist[256];
  __shared__ int sh_digit, sh_need;
  __shared__ int warp_sums[33];

  uint32_t prefix = 0, mask = 0;
  int need = n_keep;
  const int rounds = (cand + kSelThreads - 1) / kSelThreads;
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    for (int r = 0; r < rounds; ++r) {
      const int j = r * kSelThreads + tid;
      uint32_t k = 0;
      const bool in = j < cand && (((k = hv.key(j)) & mask) == prefix);
      const uint32_t digit = in ? ((k >> shift) & 255u) : 256u;
      const uint32_t peers = __match_any_sync(0xffffffffu, digit);
      if (in && lane == __ffs(peers) - 1) atomicAdd(&hist[digit], __popc(peers));
    }
    __syncthreads();
    if (tid < 32) locate_digit(hist, need, &sh_digit, &sh_need);
    __syncthreads();
    prefix |= (uint32_t)sh_digit << shift;
    need = sh_need;
    mask |= 255u << shift;
  }
  const uint32_t thr = prefix;
  int out_base = 0, eq_base = 0;
  for (int base = 0; base < cand; base += kSelThreads) {
    const int j = base + tid;
    uint32_t k = 0;
    const bool in = j < cand;
    if (in) k = hv.key(j);
    const int gt = in && k > thr;
    const int eq = in && k == thr;
    int total;
    const int packed = block_exclusive_scan(gt | (eq << 16), warp_sums, total);
    const int gt_before = packed & 0xffff, eq_before = eq_base + (packed >> 16);
    // entries equal to the threshold are kept while their running rank is below `need`
    const int pos = out_base + gt_before + min(eq_before, need) - min(eq_base, need);
    if ((gt || (eq && eq_before < need)) && dbg_ok(pos >= 0 && pos < n_keep, a.status, 5)) out[pos] = j;
    out_base += (total & 0xffff) + min(eq_base + (total >> 16), need) - min(eq_base, need);
    eq_base += total >> 16;
  }
}

}  // namespace

int launch_select(const StepArgs& a, const float* scores, int32_t* idx, int32_t* kept_out,
                  cudaStream_t st) {
  const int grid = a.batch * a.n_heads;
  const int max_cand = a.cand[0] > a.cand[1] ? a.cand[0] : a.cand[1];
  const int per_thread = (max_cand + kSelThreads - 1) / kSelThreads;
  if (per_thread <= 4) launch_k(select_reg_kernel<4>, grid, kSelThreads, 0, st, a, scores, idx, kept_out);
  else if (per_thread <= 8) launch_k(select_reg_kernel<8>, grid, kSelThreads, 0, st, a, scores, idx, kept_out);
  else if (per_thread <= 12) launch_k(select_reg_kernel<12>, grid, kSelThreads, 0, st, a, scores, idx, kept_out);
  else if (per_thread <= kMaxPerThread) launch_k(select_reg_kernel<kMaxPerThread>, grid, kSelThreads, 0, st, a, scores, idx, kept_out);
  else launch_k(select_kernel, grid, kSelThreads, 0, st, a, scores, idx, kept_out);
  return launched(1);
}

}  // namespace hack
