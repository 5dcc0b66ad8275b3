// Row square-norms of dY and X (Sec. 4.1: ||G_n||_F is built from them; Sec. 4.2: the
// leverage scores ||G_hat_r|| ||X_r||).  HBM-bound: 128-bit loads, one warp per row, fp32
// accumulation and a shuffle reduction.  Two passes: every row of dY that can be non-zero is read
// once, before SampleA; of X only the rows of the data SampleA kept are read, after it.
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

// One warp per row: a[r] = ||dY_r||^2.  With a list of alive data only their rows are read (the rows of every
// other datum are known to be zero: they were dropped by a layer above).
// The result of row r goes to a[r * stride], followed by stride - 1 zeros (the layout of a producer's partial sums).
template <typename T>
__global__ void __launch_bounds__(256) rownorm_dy_kernel(const T* __restrict__ dY, int R, int Tn, int d_out,
                                                         const int32_t* __restrict__ alive,
                                                         const int32_t* __restrict__ alive_cnt, float* __restrict__ a,
                                                         int stride) {
  pdl_trigger();   // the next kernel may be scheduled now; it waits for this grid before reading
  const int lane = threadIdx.x & 31;
  const int wpb = blockDim.x >> 5;
  const int N = R / Tn;
  // a caller's list is not trusted: its length is clamped and entries outside [0, N) are skipped (SampleA
  // reports them in the status word)
  const int rows = alive != nullptr ? min(max(*alive_cnt, 0), N) * Tn : R;
  for (int c = blockIdx.x * wpb + (threadIdx.x >> 5); c < rows; c += gridDim.x * wpb) {
    int r = c;
    bool valid = true;
    if (alive != nullptr) {
      const int k = c / Tn;
      const int n = alive[k];
      valid = (unsigned)n < (unsigned)N;
      r = valid ? n * Tn + (c - k * Tn) : 0;
    }
    const float sa = warp_sum(row_partial<T>(dY + (size_t)r * d_out, d_out, lane));
    if (valid) {
      if (lane == 0) a[(size_t)r * stride] = sa;
      else if (lane < stride) a[(size_t)r * stride + lane] = 0.f;
    }
  }
}

// One warp per row of a kept datum, in compact order (entry c = k*T + t is token t of the k-th kept datum):
// ||X_r||^2, then the leverage score of the rescaled gradient, w = ||dY_r|| ||X_r|| / p_n (Sec. 4.2, Eq. 3),
// and the row's 24-bit Philox uniform of SampleW, so that the single-CTA stage that follows has no per-row
// transcendental or Philox work.  a_r is the sum of a_parts consecutive floats (partial sums of a producer).
template <typename T>
__global__ void __launch_bounds__(256) scores_x_kernel(const T* __restrict__ X, int Tn, int d_in,
                                                       const float* __restrict__ a, int a_parts,
                                                       const float* __restrict__ p, const int32_t* __restrict__ idxA,
                                                       const int32_t* __restrict__ counts, uint64_t seed, int sample_w,
                                                       float* __restrict__ wc, uint32_t* __restrict__ uc) {
  pdl_wait();      // the kept data come from the SampleA kernel
  pdl_trigger();
  const int lane = threadIdx.x & 31;
  const int wpb = blockDim.x >> 5;
  const int rows = counts[0] * Tn;
  for (int c = blockIdx.x * wpb + (threadIdx.x >> 5); c < rows; c += gridDim.x * wpb) {
    const int k = c / Tn;
    const int n = idxA[k];
    const int r = n * Tn + (c - k * Tn);
    const float sb = warp_sum(row_partial<T>(X + (size_t)r * d_in, d_in, lane));
    if (lane == 0) {
      float sa = 0.f;
      for (int j = 0; j < a_parts; ++j) sa += a[(size_t)r * a_parts + j];
      wc[c] = sqrtf(sa) * sqrtf(sb) / p[n];
      uc[c] = sample_w ? philox_word0((uint32_t)r, 0u, 1u, 0u, (uint32_t)seed, (uint32_t)(seed >> 32)) >> 8 : 0u;
    }
  }
}

// One warp per row, eight rows per CTA (the kernels stride over whatever the grid does not cover).  Not a
// persistent grid: the register count of these kernels leaves room for six or seven CTAs per SM, and a grid of
// whole waves at an assumed occupancy was measured slower than letting the hardware schedule one CTA per
// eight rows.
int row_grid(long rows) {
  long blocks = (rows + 7) / 8;
  if (blocks > (1l << 20)) blocks = 1l << 20;
  return (int)(blocks < 1 ? 1 : blocks);
}

}  // namespace

cudaError_t launch_rownorm_dy(Handle* h, const void* dY, const SamplerArgs& s, cudaStream_t st) {
  if (s.a_in != nullptr) return cudaSuccess;     // the producer of dY supplied its row norms
  const vcas_layer_desc& d = h->desc;
  const int R = d.N * d.T;
  const int blocks = row_grid(R);
  if (d.dtype == VCAS_DTYPE_BF16) {
    rownorm_dy_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>((const __nv_bfloat16*)dY, R, d.T, d.d_out, s.alive,
                                                             s.alive_cnt, h->ws.a, 1);
  } else {
    rownorm_dy_kernel<float><<<blocks, 256, 0, st>>>((const float*)dY, R, d.T, d.d_out, s.alive, s.alive_cnt, h->ws.a, 1);
  }
  h->launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_rownorm_out(Handle* h, const void* dX, float* a_out, cudaStream_t st) {
  const vcas_layer_desc& d = h->desc;
  const int R = d.N * d.T;
  const int blocks = row_grid(R);
  const int parts = a_out_parts(d.d_in);
  if (d.dtype == VCAS_DTYPE_BF16)
    rownorm_dy_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>((const __nv_bfloat16*)dX, R, d.T, d.d_in, nullptr, nullptr,
                                                             a_out, parts);
  else
    rownorm_dy_kernel<float><<<blocks, 256, 0, st>>>((const float*)dX, R, d.T, d.d_in, nullptr, nullptr, a_out, parts);
  h->launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_scores_x(Handle* h, const void* X, const SamplerArgs& s, bool programmatic, cudaStream_t st) {
  const vcas_layer_desc& d = h->desc;
  const Workspace& ws = h->ws;
  // the number of kept rows is only known on the device: the grid is sized for the expected share of rows
  // (at least a quarter) and strides over what there is
  double share = (double)s.rho * 1.5;
  if (share < 0.25) share = 0.25;
  if (share > 1.0) share = 1.0;
  const int blocks = row_grid((long)(share * (double)d.N * d.T) + 8);
  const float* a = s.a_in != nullptr ? s.a_in : ws.a;
  const int parts = s.a_in != nullptr ? s.a_parts : 1;
  cudaError_t e;
  if (d.dtype == VCAS_DTYPE_BF16)
    e = launch_maybe_after(programmatic, scores_x_kernel<__nv_bfloat16>, dim3(blocks), dim3(256), 0, st,
                           (const __nv_bfloat16*)X, d.T, d.d_in, a, parts, (const float*)ws.p, (const int32_t*)ws.idxA,
                           (const int32_t*)ws.counts, s.seed, s.sample_w, ws.wc, ws.uc);
  else
    e = launch_maybe_after(programmatic, scores_x_kernel<float>, dim3(blocks), dim3(256), 0, st, (const float*)X, d.T,
                           d.d_in, a, parts, (const float*)ws.p, (const int32_t*)ws.idxA, (const int32_t*)ws.counts,
                           s.seed, s.sample_w, ws.wc, ws.uc);
  h->launches += 1;
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace vcas
