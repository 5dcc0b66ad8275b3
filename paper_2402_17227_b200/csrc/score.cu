// Row square-norms of dY and X (Sec. 4.1: ||G_n||_F is built from them; Sec. 4.2: the
// leverage scores ||G_hat_r|| ||X_r||).  HBM-bound: every input byte is read exactly once,
// with 128-bit loads, one warp per row, fp32 accumulation and a shuffle reduction.
#include "common.cuh"

namespace vcas {
namespace {

__device__ __forceinline__ float sq8(const uint4& v) {
  // eight bf16 values: widen by placing the 16 bits in the top half of a float
  float s = 0.f;
  const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float lo = __uint_as_float(u[i] << 16);
    const float hi = __uint_as_float(u[i] & 0xffff0000u);
    s = fmaf(lo, lo, s);
    s = fmaf(hi, hi, s);
  }
  return s;
}
__device__ __forceinline__ float sq4(const float4& v) {
  float s = v.x * v.x;
  s = fmaf(v.y, v.y, s);
  s = fmaf(v.z, v.z, s);
  s = fmaf(v.w, v.w, s);
  return s;
}

template <typename T> struct Vec;
template <> struct Vec<__nv_bfloat16> {
  using type = uint4;
  static constexpr int N = 8;
  static __device__ __forceinline__ float sq(const uint4& v) { return sq8(v); }
  static __device__ __forceinline__ float one(__nv_bfloat16 x) { const float f = __bfloat162float(x); return f * f; }
};
template <> struct Vec<float> {
  using type = float4;
  static constexpr int N = 4;
  static __device__ __forceinline__ float sq(const float4& v) { return sq4(v); }
  static __device__ __forceinline__ float one(float x) { return x * x; }
};

// Sum of squares of one row of d elements, accumulated by the 32 lanes of a warp (not yet reduced).
template <typename T>
__device__ __forceinline__ float row_partial(const T* __restrict__ src, int d, int lane) {
  using V = typename Vec<T>::type;
  constexpr int VN = Vec<T>::N;
  float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
  if ((d % VN) == 0) {
    const V* v = reinterpret_cast<const V*>(src);
    const int nv = d / VN;
    int i = lane;
    for (; i + 224 < nv; i += 256) {          // eight independent 16-byte loads in flight per lane
      const V x0 = __ldg(v + i), x1 = __ldg(v + i + 32), x2 = __ldg(v + i + 64), x3 = __ldg(v + i + 96);
      const V x4 = __ldg(v + i + 128), x5 = __ldg(v + i + 160), x6 = __ldg(v + i + 192), x7 = __ldg(v + i + 224);
      acc0 += Vec<T>::sq(x0); acc1 += Vec<T>::sq(x1); acc2 += Vec<T>::sq(x2); acc3 += Vec<T>::sq(x3);
      acc0 += Vec<T>::sq(x4); acc1 += Vec<T>::sq(x5); acc2 += Vec<T>::sq(x6); acc3 += Vec<T>::sq(x7);
    }
    for (; i + 96 < nv; i += 128) {
      const V x0 = __ldg(v + i), x1 = __ldg(v + i + 32), x2 = __ldg(v + i + 64), x3 = __ldg(v + i + 96);
      acc0 += Vec<T>::sq(x0); acc1 += Vec<T>::sq(x1); acc2 += Vec<T>::sq(x2); acc3 += Vec<T>::sq(x3);
    }
    for (; i < nv; i += 32) acc0 += Vec<T>::sq(__ldg(v + i));
  } else {
    for (int i = lane; i < d; i += 32) acc0 += Vec<T>::one(src[i]);
  }
  return (acc0 + acc1) + (acc2 + acc3);
}

// One warp per row r: a[r] = ||dY_r||^2, b[r] = ||X_r||^2, and two per-row values the sampling
// stage would otherwise compute on its single SM: lev[r] = ||dY_r|| ||X_r|| (the leverage score of
// Sec. 4.2 before the 1/p_n rescale) and u24[r], the 24-bit Philox uniform of SampleW for this row.
template <typename T>
__global__ void __launch_bounds__(256) rownorm_kernel(const T* __restrict__ dY, const T* __restrict__ X,
                                                      int R, int d_out, int d_in, uint64_t seed,
                                                      float* __restrict__ a, float* __restrict__ b,
                                                      float* __restrict__ lev, uint32_t* __restrict__ u24) {
  pdl_trigger();   // the next kernel may be scheduled now; it waits for this grid before reading
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= R) return;
  // the first four vectors per lane of the X row are requested before the dY row is touched
  using V = typename Vec<T>::type;
  constexpr int VN = Vec<T>::N;
  const T* xrow = X + (size_t)row * d_in;
  const bool xvec = (d_in % VN) == 0;
  const int nvx = xvec ? d_in / VN : 0;
  V xv[4];
#pragma unroll
  for (int k = 0; k < 4; ++k)
    if (lane + 32 * k < nvx) xv[k] = __ldg(reinterpret_cast<const V*>(xrow) + lane + 32 * k);
  const float pa = row_partial<T>(dY + (size_t)row * d_out, d_out, lane);
  float pb = 0.f;
  if (xvec) {
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (lane + 32 * k < nvx) pb += Vec<T>::sq(xv[k]);
    for (int i = lane + 128; i < nvx; i += 32) pb += Vec<T>::sq(__ldg(reinterpret_cast<const V*>(xrow) + i));
  } else {
    pb = row_partial<T>(xrow, d_in, lane);
  }
  const float sa = warp_sum(pa), sb = warp_sum(pb);
  if (lane == 0) {
    a[row] = sa;
    b[row] = sb;
    lev[row] = sqrtf(sa) * sqrtf(sb);
    u24[row] = philox_word0((uint32_t)row, 0u, 1u, 0u, (uint32_t)seed, (uint32_t)(seed >> 32)) >> 8;
  }
}

}  // namespace

cudaError_t launch_rownorms(Handle* h, const void* dY, const void* X, uint64_t seed, cudaStream_t st) {
  const vcas_layer_desc& d = h->desc;
  const int R = d.N * d.T;
  const int warps_per_block = 8;
  const int blocks = (R + warps_per_block - 1) / warps_per_block;
  if (d.dtype == VCAS_DTYPE_BF16) {
    rownorm_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>((const __nv_bfloat16*)dY, (const __nv_bfloat16*)X, R,
                                                          d.d_out, d.d_in, seed, h->ws.a, h->ws.b, h->ws.lev,
                                                          h->ws.u24);
  } else {
    rownorm_kernel<float><<<blocks, 256, 0, st>>>((const float*)dY, (const float*)X, R, d.d_out, d.d_in, seed,
                                                  h->ws.a, h->ws.b, h->ws.lev, h->ws.u24);
  }
  h->launches += 1;
  return cudaGetLastError();
}

}  // namespace vcas
