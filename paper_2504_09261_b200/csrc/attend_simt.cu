// Attention of the scale's queries over the compacted per-head cache (Eq. 4 on the compressed
// cache), plain fp32 arithmetic on the CUDA cores.  This is the exact-precision path (fp32
// workloads forbid TF32 at the required 1e-5) and the fallback for shapes the tensor-core kernel
// does not take.  Four threads share one query row (each owns a quarter of the head dimension);
// K/V tiles of 32 keys are staged in shared memory as fp32; softmax is the usual streaming
// (running max / running sum) form, rescaled once per group of 8 keys.
#include "hack_internal.h"

namespace hack {
namespace {

constexpr int kQPerCta = 32;
constexpr int kThreads = kQPerCta * 4;
constexpr int kTileK = 32;
constexpr int kGroup = 8;

template <typename T> struct Cvt;
template <> struct Cvt<float> {
  static constexpr int kPerVec = 4;
  __device__ static void unpack(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
    f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
  }
  __device__ static void store4(float* dst, const float* f) {
    *reinterpret_cast<float4*>(dst) = make_float4(f[0], f[1], f[2], f[3]);
  }
};
template <> struct Cvt<__nv_bfloat16> {
  static constexpr int kPerVec = 8;
  __device__ static void unpack(const uint4& v, float* f) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  __device__ static void store4(__nv_bfloat16* dst, const float* f) {
    __nv_bfloat162 a = __floats2bfloat162_rn(f[0], f[1]);
    __nv_bfloat162 b = __floats2bfloat162_rn(f[2], f[3]);
    uint2 p;
    p.x = *reinterpret_cast<uint32_t*>(&a);
    p.y = *reinterpret_cast<uint32_t*>(&b);
    *reinterpret_cast<uint2*>(dst) = p;
  }
};

template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
attend_simt_kernel(const StepArgs a, const T* __restrict__ q, T* __restrict__ out) {
  pdl_wait();
  constexpr int DQ = D / 4;                       // dims per thread
  constexpr int VEC = Cvt<T>::kPerVec;
  constexpr int ROWV = D / VEC;
  const int bh = blockIdx.y;
  const int ctx = a.is_ctx[bh % a.n_heads];
  const int len = a.kept[ctx];
  const int tid = threadIdx.x;
  const int qi = blockIdx.x * kQPerCta + tid / 4;
  const int part = tid % 4;
  const bool q_ok = qi < a.n_new;

  __shared__ __align__(16) float ks[kTileK][D];
  __shared__ __align__(16) float vs[kTileK][D];

  // this thread's slice of the query row: dims part*DQ .. part*DQ + DQ - 1
  float qr[DQ];
  if (q_ok) {
    const T* qp = q + ((size_t)bh * a.n_new + qi) * D + part * DQ;
#pragma unroll
    for (int c = 0; c < DQ / VEC; ++c) {
      Cvt<T>::unpack(*reinterpret_cast<const uint4*>(qp + c * VEC), qr + c * VEC);
    }
  } else {
#pragma unroll
    for (int d = 0; d < DQ; ++d) qr[d] = 0.f;
  }
  float o[DQ];
#pragma unroll
  for (int d = 0; d < DQ; ++d) o[d] = 0.f;
  float m = -INFINITY, l = 0.f;

  const T* kp = static_cast<const T*>(a.k_plane) + (size_t)a.row_off[bh] * D;
  const T* vp = static_cast<const T*>(a.v_plane) + (size_t)a.row_off[bh] * D;

  for (int t0 = 0; t0 < len; t0 += kTileK) {
    __syncthreads();
    for (int v = tid; v < kTileK * ROWV; v += kThreads) {
      const int r = v / ROWV, c = v % ROWV;
      float fk[VEC], fv[VEC];
      if (t0 + r < len) {
        Cvt<T>::unpack(*reinterpret_cast<const uint4*>(kp + (size_t)(t0 + r) * D + c * VEC), fk);
        Cvt<T>::unpack(*reinterpret_cast<const uint4*>(vp + (size_t)(t0 + r) * D + c * VEC), fv);
      } else {
#pragma unroll
        for (int e = 0; e < VEC; ++e) { fk[e] = 0.f; fv[e] = 0.f; }
      }
#pragma unroll
      for (int e = 0; e < VEC; ++e) { ks[r][c * VEC + e] = fk[e]; vs[r][c * VEC + e] = fv[e]; }
    }
    __syncthreads();
    const int n_in_tile = min(kTileK, len - t0);
    for (int g0 = 0; g0 < n_in_tile; g0 += kGroup) {
      float z[kGroup];
#pragma unroll
      for (int g = 0; g < kGroup; ++g) {
        float acc = 0.f;
        const float4* kr = reinterpret_cast<const float4*>(&ks[g0 + g][part * DQ]);
#pragma unroll
        for (int d4 = 0; d4 < DQ / 4; ++d4) {
          const float4 kk = kr[d4];
          acc = fmaf(qr[4 * d4 + 0], kk.x, acc);
          acc = fmaf(qr[4 * d4 + 1], kk.y, acc);
          acc = fmaf(qr[4 * d4 + 2], kk.z, acc);
          acc = fmaf(qr[4 * d4 + 3], kk.w, acc);
        }
        acc += __shfl_xor_sync(0xffffffffu, acc, 1);
        acc += __shfl_xor_sync(0xffffffffu, acc, 2);
        z[g] = (g0 + g < n_in_tile) ? acc * a.sm_scale : -INFINITY;
      }
      float m_new = m;
#pragma unroll
      for (int g = 0; g < kGroup; ++g) m_new = fmaxf(m_new, z[g]);
      const float corr = expf(m - m_new);           // exp(-inf) = 0 on the first group
      l *= corr;
#pragma unroll
      for (int d = 0; d < DQ; ++d) o[d] *= corr;
#pragma unroll
      for (int g = 0; g < kGroup; ++g) {
        const float p = expf(z[g] - m_new);
        l += p;
        const float4* vr = reinterpret_cast<const float4*>(&vs[g0 + g][part * DQ]);
#pragma unroll
        for (int d4 = 0; d4 < DQ / 4; ++d4) {
          const float4 vv = vr[d4];
          o[4 * d4 + 0] = fmaf(p, vv.x, o[4 * d4 + 0]);
          o[4 * d4 + 1] = fmaf(p, vv.y, o[4 * d4 + 1]);
          o[4 * d4 + 2] = fmaf(p, vv.z, o[4 * d4 + 2]);
          o[4 * d4 + 3] = fmaf(p, vv.w, o[4 * d4 + 3]);
        }
      }
      m = m_new;
    }
  }
  if (q_ok) {
    const float inv = 1.f / l;
    T* op = out + ((size_t)bh * a.n_new + qi) * D + part * DQ;
#pragma unroll
    for (int d4 = 0; d4 < DQ / 4; ++d4) {
      float f[4] = {o[4 * d4] * inv, o[4 * d4 + 1] * inv, o[4 * d4 + 2] * inv, o[4 * d4 + 3] * inv};
      Cvt<T>::store4(op + 4 * d4, f);
    }
  }
}

}  // namespace

int launch_attend_simt(const StepArgs& a, int dtype, const void* q, void* out, cudaStream_t st) {
  dim3 grid((a.n_new + kQPerCta - 1) / kQPerCta, a.batch * a.n_heads);
  if (dtype == HACK_F32) {
    if (a.head_dim == 64)
      launch_k(attend_simt_kernel<float, 64>, grid, kThreads, 0, st, a, static_cast<const float*>(q), static_cast<float*>(out));
    else
      launch_k(attend_simt_kernel<float, 128>, grid, kThreads, 0, st, a, static_cast<const float*>(q), static_cast<float*>(out));
  } else {
    if (a.head_dim == 64)
      launch_k(attend_simt_kernel<__nv_bfloat16, 64>, grid, kThreads, 0, st, 
          a, static_cast<const __nv_bfloat16*>(q), static_cast<__nv_bfloat16*>(out));
    else
      launch_k(attend_simt_kernel<__nv_bfloat16, 128>, grid, kThreads, 0, st, 
          a, static_cast<const __nv_bfloat16*>(q), static_cast<__nv_bfloat16*>(out));
  }
  return launched(1);
}

}  // namespace hack
