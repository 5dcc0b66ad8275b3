// The two products of the sampled backward on plain fp32 FMA units (App. E: dX = G_hat W;
// Sec. 4.2: dW = G_tilde^T X).  Used for fp32 layers, where a tensor-core pass in tf32 could
// not meet a 1e-5 tolerance, and for bf16 layers whose sizes the tensor-core kernels do not
// take.  64x64 output tiles, 16-deep steps, 4x4 register tiles, fixed summation order.
#include "common.cuh"

namespace vcas {
namespace {

__device__ __forceinline__ float to_f(float x) { return x; }
__device__ __forceinline__ float to_f(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void from_f(float& d, float x) { d = x; }
__device__ __forceinline__ void from_f(__nv_bfloat16& d, float x) { d = __float2bfloat16_rn(x); }

// derivative of the erf-form GELU: Phi(x) + x phi(x)
__device__ __forceinline__ float gelu_prime(float x) {
  const float Phi = 0.5f * (1.0f + erff(x * 0.70710678118654752f));
  const float phi = 0.39894228040143268f * expf(-0.5f * x * x);
  return fmaf(x, phi, Phi);
}

constexpr int TM = 64, TN = 64, TK = 16;

// dX[rows of datum n] = scaleA[n] * dY[rows] W   (zero rows for dropped data)
template <typename T>
__global__ void __launch_bounds__(256) fma_dx_kernel(const T* __restrict__ dY, const T* __restrict__ W,
                                                     const float* __restrict__ scaleA,
                                                     const T* __restrict__ H, T* __restrict__ dX,
                                                     int N, int Tn, int d_in, int d_out) {
  __shared__ float As[TK][TM + 4];
  __shared__ float Bs[TK][TN + 4];
  const int chunks = (Tn + TM - 1) / TM;
  const int n = blockIdx.y / chunks, t0 = (blockIdx.y % chunks) * TM, i0 = blockIdx.x * TN;
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const float s = scaleA != nullptr ? scaleA[n] : 1.0f;
  const size_t row_base = (size_t)n * Tn + t0;
  float acc[4][4] = {};
  if (s != 0.f) {
    for (int k0 = 0; k0 < d_out; k0 += TK) {
      {
        const int row = tid >> 2, kk = (tid & 3) * 4;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          float v = 0.f;
          if (t0 + row < Tn && k0 + kk + j < d_out) v = to_f(dY[(row_base + row) * d_out + k0 + kk + j]);
          As[kk + j][row] = v;
        }
        const int kb = tid >> 4, col = (tid & 15) * 4;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          float v = 0.f;
          if (k0 + kb < d_out && i0 + col + j < d_in) v = to_f(W[(size_t)(k0 + kb) * d_in + i0 + col + j]);
          Bs[kb][col + j] = v;
        }
      }
      __syncthreads();
#pragma unroll
      for (int kk = 0; kk < TK; ++kk) {
        float av[4], bv[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) { av[j] = As[kk][ty * 4 + j]; bv[j] = Bs[kk][tx * 4 + j]; }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
      }
      __syncthreads();
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int t = t0 + ty * 4 + i;
    if (t >= Tn) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = i0 + tx * 4 + j;
      if (c >= d_in) continue;
      const size_t o = ((size_t)n * Tn + t) * d_in + c;
      float v = s * acc[i][j];
      if (H != nullptr && s != 0.f) v *= gelu_prime(to_f(H[o]));
      from_f(dX[o], v);
    }
  }
}

// dW[o, i] = sum_{k < cnt} scale[k] dY[idx[k], o] X[idx[k], i]   (idx == nullptr: identity, scale 1)
template <typename T>
__global__ void __launch_bounds__(256) fma_dw_kernel(const T* __restrict__ dY, const T* __restrict__ X,
                                                     const int32_t* __restrict__ idx,
                                                     const float* __restrict__ scale,
                                                     const int32_t* __restrict__ cnt_ptr,
                                                     float* __restrict__ dW, int d_in, int d_out) {
  __shared__ float As[TK][TM + 4];
  __shared__ float Bs[TK][TN + 4];
  const int cnt = *cnt_ptr;
  const int o0 = blockIdx.y * TM, i0 = blockIdx.x * TN;
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < cnt; k0 += TK) {
    {
      const int kk = tid >> 4, c4 = (tid & 15) * 4;
      const int k = k0 + kk;
      int row = 0;
      float sc = 0.f;
      if (k < cnt) { row = idx != nullptr ? idx[k] : k; sc = scale != nullptr ? scale[k] : 1.0f; }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float va = 0.f, vb = 0.f;
        if (k < cnt) {
          if (o0 + c4 + j < d_out) va = to_f(dY[(size_t)row * d_out + o0 + c4 + j]);
          if (i0 + c4 + j < d_in) vb = sc * to_f(X[(size_t)row * d_in + i0 + c4 + j]);
        }
        As[kk][c4 + j] = va;
        Bs[kk][c4 + j] = vb;
      }
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      float av[4], bv[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) { av[j] = As[kk][ty * 4 + j]; bv[j] = Bs[kk][tx * 4 + j]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int o = o0 + ty * 4 + i;
    if (o >= d_out) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = i0 + tx * 4 + j;
      if (c < d_in) dW[(size_t)o * d_in + c] = acc[i][j];
    }
  }
}

}  // namespace

cudaError_t launch_fma_dx(Handle* h, const void* dY, const void* W, const float* scaleA, const void* H,
                          void* dX, cudaStream_t st) {
  const vcas_layer_desc& d = h->desc;
  const dim3 grid((d.d_in + TN - 1) / TN, d.N * ((d.T + TM - 1) / TM));
  if (d.dtype == VCAS_DTYPE_BF16) {
    fma_dx_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)dY, (const __nv_bfloat16*)W, scaleA,
                                                       (const __nv_bfloat16*)H, (__nv_bfloat16*)dX, d.N, d.T,
                                                       d.d_in, d.d_out);
  } else {
    fma_dx_kernel<float><<<grid, 256, 0, st>>>((const float*)dY, (const float*)W, scaleA, (const float*)H,
                                               (float*)dX, d.N, d.T, d.d_in, d.d_out);
  }
  h->launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_fma_dw(Handle* h, const void* dY, const void* X, const int32_t* idx, const float* scale,
                          const int32_t* cnt, float* dW, cudaStream_t st) {
  const vcas_layer_desc& d = h->desc;
  const dim3 grid((d.d_in + TN - 1) / TN, (d.d_out + TM - 1) / TM);
  if (d.dtype == VCAS_DTYPE_BF16) {
    fma_dw_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)dY, (const __nv_bfloat16*)X, idx,
                                                       scale, cnt, dW, d.d_in, d.d_out);
  } else {
    fma_dw_kernel<float><<<grid, 256, 0, st>>>((const float*)dY, (const float*)X, idx, scale, cnt, dW, d.d_in,
                                               d.d_out);
  }
  h->launches += 1;
  return cudaGetLastError();
}

}  // namespace vcas
