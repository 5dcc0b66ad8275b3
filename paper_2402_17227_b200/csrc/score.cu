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

// task t < R: row t of dY -> a[t];  task t >= R: row t-R of X -> b[t-R]
template <typename T>
__global__ void __launch_bounds__(256) rownorm_kernel(const T* __restrict__ dY, const T* __restrict__ X,
                                                      int R, int d_out, int d_in,
                                                      float* __restrict__ a, float* __restrict__ b) {
  using V = typename Vec<T>::type;
  constexpr int VN = Vec<T>::N;
  const int lane = threadIdx.x & 31;
  const int task = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (task >= 2 * R) return;
  const bool is_x = task >= R;
  const int row = is_x ? task - R : task;
  const int d = is_x ? d_in : d_out;
  const T* src = (is_x ? X : dY) + (size_t)row * d;
  float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
  if ((d % VN) == 0) {
    const V* v = reinterpret_cast<const V*>(src);
    const int nv = d / VN;
    int i = lane;
    for (; i + 96 < nv; i += 128) {
      const V x0 = __ldg(v + i), x1 = __ldg(v + i + 32), x2 = __ldg(v + i + 64), x3 = __ldg(v + i + 96);
      acc0 += Vec<T>::sq(x0); acc1 += Vec<T>::sq(x1); acc2 += Vec<T>::sq(x2); acc3 += Vec<T>::sq(x3);
    }
    for (; i < nv; i += 32) acc0 += Vec<T>::sq(__ldg(v + i));
  } else {
    for (int i = lane; i < d; i += 32) acc0 += Vec<T>::one(src[i]);
  }
  const float s = warp_sum((acc0 + acc1) + (acc2 + acc3));
  if (lane == 0) (is_x ? b : a)[row] = s;
}

}  // namespace

cudaError_t launch_rownorms(Handle* h, const void* dY, const void* X, cudaStream_t st) {
  const vcas_layer_desc& d = h->desc;
  const int R = d.N * d.T;
  const int warps_per_block = 8;
  const int blocks = (2 * R + warps_per_block - 1) / warps_per_block;
  if (d.dtype == VCAS_DTYPE_BF16) {
    rownorm_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>((const __nv_bfloat16*)dY, (const __nv_bfloat16*)X,
                                                          R, d.d_out, d.d_in, h->ws.a, h->ws.b);
  } else {
    rownorm_kernel<float><<<blocks, 256, 0, st>>>((const float*)dY, (const float*)X, R, d.d_out, d.d_in,
                                                  h->ws.a, h->ws.b);
  }
  h->launches += 1;
  return cudaGetLastError();
}

}  // namespace vcas
