// One-launch step for small scales: append the new scale's K/V rows to the per-head cache (Eq. 3)
// and attend over [stored rows ; new rows] (Eq. 4), for steps in which no head exceeds its budget
// and the scale has few queries.  Such steps are pure latency: two dependent launches and a
// tensor-core pipeline cost more than the arithmetic, so everything runs in one SIMT kernel.
//
// One warp serves one query row.  Scores: lane <-> key (a lane walks its key's row with 16-byte
// loads, the query row is broadcast from shared memory); softmax statistics with warp shuffles;
// output: lane <-> a run of head dimensions, the probabilities are broadcast lane by lane and the
// value rows are read coalesced.  Keys below the stored length come from the cache planes, the
// others straight from the caller's K/V tensors, so nothing depends on the append, which the
// same CTAs perform afterwards on cache rows no one reads in this launch.
#include "hack_internal.h"

namespace hack {
namespace {

constexpr int kWarps = 8;                       // query rows per CTA

template <typename T> struct Row;
template <> struct Row<float> {
  static constexpr int kPerVec = 4;
  __device__ static void unpack(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
    f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
  }
  __device__ static float load1(const float* p) { return *p; }
  __device__ static void store1(float* p, float v) { *p = v; }
};
template <> struct Row<__nv_bfloat16> {
  static constexpr int kPerVec = 8;
  __device__ static void unpack(const uint4& v, float* f) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  __device__ static float load1(const __nv_bfloat16* p) { return __bfloat162float(*p); }
  __device__ static void store1(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
};

// DL consecutive elements starting at p (DL * sizeof(T) bytes, naturally aligned) as floats.
template <typename T, int DL>
__device__ __forceinline__ void load_run(const T* p, float* f) {
  if constexpr (sizeof(T) == 4) {
    if constexpr (DL == 4) { const float4 v = *reinterpret_cast<const float4*>(p); f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w; }
    else { const float2 v = *reinterpret_cast<const float2*>(p); f[0] = v.x; f[1] = v.y; }
  } else {
    if constexpr (DL == 4) {
      const uint2 v = *reinterpret_cast<const uint2*>(p);
      f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
      f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
    } else {
      const uint32_t v = *reinterpret_cast<const uint32_t*>(p);
      f[0] = __uint_as_float(v << 16); f[1] = __uint_as_float(v & 0xffff0000u);
    }
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(kWarps * 32)
append_attend_small_kernel(const StepArgs a, const T* __restrict__ q, const T* __restrict__ k_new,
                           const T* __restrict__ v_new, T* __restrict__ out) {
  pdl_wait();
  constexpr int VEC = Row<T>::kPerVec;
  constexpr int DL = D / 32;                    // output dimensions per lane
  const int bh = blockIdx.y;
  const int ctx = a.is_ctx[bh % a.n_heads];
  const int stored = a.stored[ctx];
  const int total = stored + a.n_new;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qi = blockIdx.x * kWarps + warp;
  const size_t off = a.row_off[bh];
  const T* kc = static_cast<const T*>(a.k_plane) + off * D;
  const T* vc = static_cast<const T*>(a.v_plane) + off * D;
  const T* kn = k_new + (size_t)bh * a.n_new * D;
  const T* vn = v_new + (size_t)bh * a.n_new * D;

  __shared__ __align__(16) float qs[kWarps][D];
  if (qi < a.n_new) {
    const T* qp = q + ((size_t)bh * a.n_new + qi) * D;
    for (int d = lane; d < D; d += 32) qs[warp][d] = Row<T>::load1(qp + d);
  }
  __syncwarp();

  if (qi < a.n_new) {
    const float c = a.sm_scale * 1.4426950408889634f;          // work in log2 units
    float m = -INFINITY, l = 0.f;
    float o[DL];
#pragma unroll
    for (int i = 0; i < DL; ++i) o[i] = 0.f;
    for (int j0 = 0; j0 < total; j0 += 32) {
      const int j = j0 + lane;
      float z = -INFINITY;
      if (j < total) {
        const T* kr = j < stored ? kc + (size_t)j * D : kn + (size_t)(j - stored) * D;
        float acc = 0.f;
#pragma unroll
        for (int v = 0; v < D / VEC; ++v) {
          float kf[VEC];
          Row<T>::unpack(*reinterpret_cast<const uint4*>(kr + v * VEC), kf);
#pragma unroll
          for (int e = 0; e < VEC; e += 4) {
            const float4 qq = *reinterpret_cast<const float4*>(&qs[warp][v * VEC + e]);
            acc = fmaf(qq.x, kf[e], acc);
            acc = fmaf(qq.y, kf[e + 1], acc);
            acc = fmaf(qq.z, kf[e + 2], acc);
            acc = fmaf(qq.w, kf[e + 3], acc);
          }
        }
        z = acc * c;
      }
      float mt = z;
#pragma unroll
      for (int s = 16; s > 0; s >>= 1) mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, s));
      const float m_new = fmaxf(m, mt);
      const float corr = exp2f(m - m_new);                      // 0 in the first tile
      const float p = exp2f(z - m_new);                         // 0 for lanes past the end
      float ps = p;
#pragma unroll
      for (int s = 16; s > 0; s >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, s);
      l = l * corr + ps;
      m = m_new;
#pragma unroll
      for (int i = 0; i < DL; ++i) o[i] *= corr;
      // value rows in groups of eight, loads first: lanes past the end carry p = 0 and re-read the
      // last row, so no guard is needed
      const int n_in = min(32, total - j0);
      for (int u0 = 0; u0 < n_in; u0 += 8) {
        float vf[8][DL];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int ju = min(j0 + u0 + u, total - 1);
          const T* vr = (ju < stored ? vc + (size_t)ju * D : vn + (size_t)(ju - stored) * D) + lane * DL;
          load_run<T, DL>(vr, vf[u]);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const float pu = __shfl_sync(0xffffffffu, p, u0 + u);
#pragma unroll
          for (int i = 0; i < DL; ++i) o[i] = fmaf(pu, vf[u][i], o[i]);
        }
      }
    }
    const float inv = 1.f / l;
    T* op = out + ((size_t)bh * a.n_new + qi) * D + lane * DL;
#pragma unroll
    for (int i = 0; i < DL; ++i) Row<T>::store1(op + i, o[i] * inv);
  }

  // append: rows [stored, stored + n_new) of the cache take the new scale's rows; the CTAs of a
  // head share them, 16 bytes per thread
  constexpr int ROWV = D / VEC;                 // 16-byte pieces per row
  const int n_pieces = dbg_ok(stored + a.n_new <= a.cap[ctx], a.status, 6) ? a.n_new * ROWV : 0;
  const uint4* ksrc = reinterpret_cast<const uint4*>(kn);
  const uint4* vsrc = reinterpret_cast<const uint4*>(vn);
  uint4* kdst = reinterpret_cast<uint4*>(static_cast<T*>(a.k_plane) + (off + stored) * D);
  uint4* vdst = reinterpret_cast<uint4*>(static_cast<T*>(a.v_plane) + (off + stored) * D);
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n_pieces; i += gridDim.x * blockDim.x) {
    kdst[i] = ksrc[i];
    vdst[i] = vsrc[i];
  }
  if (blockIdx.x == 0 && n_pieces > 0)
    for (int r = threadIdx.x; r < a.n_new; r += blockDim.x) a.pos_plane[off + stored + r] = a.pos_base + r;
}

}  // namespace

int launch_append_attend_small(const StepArgs& a, int dtype, const void* q, const void* k_new,
                               const void* v_new, void* out, cudaStream_t st) {
  const dim3 grid((a.n_new + kWarps - 1) / kWarps, a.batch * a.n_heads);
  const dim3 block(kWarps * 32);
  if (dtype == HACK_F32) {
    const float* qp = static_cast<const float*>(q);
    const float* kp = static_cast<const float*>(k_new);
    const float* vp = static_cast<const float*>(v_new);
    float* op = static_cast<float*>(out);
    if (a.head_dim == 64) launch_k(append_attend_small_kernel<float, 64>, grid, block, 0, st, a, qp, kp, vp, op);
    else launch_k(append_attend_small_kernel<float, 128>, grid, block, 0, st, a, qp, kp, vp, op);
  } else {
    const __nv_bfloat16* qp = static_cast<const __nv_bfloat16*>(q);
    const __nv_bfloat16* kp = static_cast<const __nv_bfloat16*>(k_new);
    const __nv_bfloat16* vp = static_cast<const __nv_bfloat16*>(v_new);
    __nv_bfloat16* op = static_cast<__nv_bfloat16*>(out);
    if (a.head_dim == 64) launch_k(append_attend_small_kernel<__nv_bfloat16, 64>, grid, block, 0, st, a, qp, kp, vp, op);
    else launch_k(append_attend_small_kernel<__nv_bfloat16, 128>, grid, block, 0, st, a, qp, kp, vp, op);
  }
  return launched(1);
}

}  // namespace hack
