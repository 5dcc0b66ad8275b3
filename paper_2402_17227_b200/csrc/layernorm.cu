// SampleA in front of a layer that is not a matrix product (Sec. 4: SampleA sits at every layer; App. E: the
// sampled, rescaled gradient is multiplied by the layer's exact Jacobian): the backward of
// Y = LayerNorm(X) * gamma + beta.  Only the rows of kept data are read and computed; rows of dropped data
// get dX = 0.  HBM-bound row-wise and column-wise passes, fixed summation orders.
#include "common.cuh"

namespace vcas {
namespace {

template <typename T> struct Ld;
template <> struct Ld<__nv_bfloat16> {
  static constexpr int N = 8;
  using V = uint4;
  static __device__ __forceinline__ void unpack(const uint4& v, float (&f)[8]) {
    const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) { f[2 * i] = __uint_as_float(u[i] << 16); f[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u); }
  }
  // rounds to bf16, returns the stored values' sum of squares
  static __device__ __forceinline__ float pack(const float (&f)[8], uint4& v) {
    uint32_t o[4];
    float sq = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 t = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
      o[i] = *reinterpret_cast<const uint32_t*>(&t);
      const float lo = __uint_as_float(o[i] << 16), hi = __uint_as_float(o[i] & 0xffff0000u);
      sq = fmaf(lo, lo, fmaf(hi, hi, sq));
    }
    v = make_uint4(o[0], o[1], o[2], o[3]);
    return sq;
  }
  static __device__ __forceinline__ float one(__nv_bfloat16 x) { return __bfloat162float(x); }
};
template <> struct Ld<float> {
  static constexpr int N = 4;
  using V = float4;
  static __device__ __forceinline__ void unpack(const float4& v, float (&f)[4]) { f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w; }
  static __device__ __forceinline__ float pack(const float (&f)[4], float4& v) {
    v = make_float4(f[0], f[1], f[2], f[3]);
    return fmaf(f[0], f[0], fmaf(f[1], f[1], fmaf(f[2], f[2], f[3] * f[3])));
  }
  static __device__ __forceinline__ float one(float x) { return x; }
};

struct LnParams {
  const void* X; const void* gamma; const void* dY; void* dX;
  const float* scaleA; const int32_t* idxA; const int32_t* dropA; const int32_t* counts;
  float* mu; float* rstd;          // [R] per-row statistics kept for the column pass
  float* a_out; int a_parts;       // optional row square-norms of the stored dX (first part; the others 0)
  float* partial;                  // [2][chunks][d] column partial sums
  float* dgamma; float* dbeta;
  int N, T, d, chunks, skip_dropped;
  float eps;
};

// One warp per row.  Work item c < cntA*T: token of a kept datum (compact order); the items after those are the
// rows of dropped data, which are zeroed (unless the caller's consumer never reads them).
template <typename T>
__global__ void __launch_bounds__(256) ln_row_kernel(LnParams P) {
  using L = Ld<T>;
  using V = typename L::V;
  constexpr int VN = L::N;
  pdl_wait();      // the kept data come from the SampleA kernel
  pdl_trigger();
  const int lane = threadIdx.x & 31, wpb = blockDim.x >> 5;
  const int cntA = P.counts[0], Tn = P.T, d = P.d;
  const int kept_rows = cntA * Tn;
  const int total = P.skip_dropped ? kept_rows : P.N * Tn;
  const int nv = d / VN;
  const float inv_d = 1.0f / (float)d;
  for (int c = blockIdx.x * wpb + (threadIdx.x >> 5); c < total; c += gridDim.x * wpb) {
    if (c >= kept_rows) {        // a row of a dropped datum
      const int i = c - kept_rows, k = i / Tn;
      const size_t r = (size_t)P.dropA[k] * Tn + (i - k * Tn);
      V z;
      float zero[VN];
#pragma unroll
      for (int e = 0; e < VN; ++e) zero[e] = 0.f;
      L::pack(zero, z);
      for (int j = lane; j < nv; j += 32) reinterpret_cast<V*>((T*)P.dX + r * d)[j] = z;
      if (P.a_out != nullptr && lane < P.a_parts) P.a_out[r * P.a_parts + lane] = 0.f;
      continue;
    }
    const int k = c / Tn;
    const int n = P.idxA[k];
    const size_t r = (size_t)n * Tn + (c - k * Tn);
    const float sc = P.scaleA[n];
    const V* xv = reinterpret_cast<const V*>((const T*)P.X + r * d);
    const V* gv = reinterpret_cast<const V*>((const T*)P.dY + r * d);
    const V* wv = reinterpret_cast<const V*>((const T*)P.gamma);
    // pass 1: the row's mean
    float s = 0.f;
    for (int j = lane; j < nv; j += 32) {
      float x[VN];
      L::unpack(__ldg(xv + j), x);
#pragma unroll
      for (int e = 0; e < VN; ++e) s += x[e];
    }
    const float mean = warp_sum(s) * inv_d;
    // pass 2: variance, and the two row sums of g_hat = G_hat * gamma that the Jacobian needs
    float v2 = 0.f, s1 = 0.f, s2 = 0.f;
    for (int j = lane; j < nv; j += 32) {
      float x[VN], g[VN], w[VN];
      L::unpack(__ldg(xv + j), x);
      L::unpack(__ldg(gv + j), g);
      L::unpack(__ldg(wv + j), w);
#pragma unroll
      for (int e = 0; e < VN; ++e) {
        const float xc = x[e] - mean, gh = sc * g[e] * w[e];
        v2 = fmaf(xc, xc, v2);
        s1 += gh;
        s2 = fmaf(gh, xc, s2);
      }
    }
    v2 = warp_sum(v2); s1 = warp_sum(s1); s2 = warp_sum(s2);
    const float rstd = rsqrtf(v2 * inv_d + P.eps);
    const float m1 = s1 * inv_d, m2 = s2 * rstd * inv_d;     // mean(g_hat), mean(g_hat * x_hat)
    // pass 3: dX
    float sq = 0.f;
    for (int j = lane; j < nv; j += 32) {
      float x[VN], g[VN], w[VN], o[VN];
      L::unpack(__ldg(xv + j), x);
      L::unpack(__ldg(gv + j), g);
      L::unpack(__ldg(wv + j), w);
#pragma unroll
      for (int e = 0; e < VN; ++e) {
        const float xh = (x[e] - mean) * rstd, gh = sc * g[e] * w[e];
        o[e] = (gh - m1 - xh * m2) * rstd;
      }
      V ov;
      sq += L::pack(o, ov);
      reinterpret_cast<V*>((T*)P.dX + r * d)[j] = ov;
    }
    sq = warp_sum(sq);
    if (lane == 0) {
      P.mu[r] = mean;
      P.rstd[r] = rstd;
      if (P.a_out != nullptr) P.a_out[r * P.a_parts] = sq;
    } else if (P.a_out != nullptr && lane < P.a_parts) {
      P.a_out[r * P.a_parts + lane] = 0.f;
    }
  }
}

// One thread per column, the kept rows cut into `chunks` contiguous ranges (blockIdx.y): partial sums of
// dgamma = sum_r G_hat_r * x_hat_r and dbeta = sum_r G_hat_r in row order.
template <typename T>
__global__ void __launch_bounds__(256) ln_col_kernel(LnParams P) {
  pdl_wait();
  pdl_trigger();
  const int col = blockIdx.x * blockDim.x + threadIdx.x;
  const int Tn = P.T, d = P.d;
  const int rows = P.counts[0] * Tn;
  const int per = (rows + P.chunks - 1) / P.chunks;
  const int c0 = blockIdx.y * per, c1 = min(rows, c0 + per);
  if (col >= d) return;
  float ag = 0.f, ab = 0.f;
  for (int c = c0; c < c1; ++c) {
    const int k = c / Tn;
    const int n = P.idxA[k];
    const size_t r = (size_t)n * Tn + (c - k * Tn);
    const float g = P.scaleA[n] * Ld<T>::one(((const T*)P.dY)[r * d + col]);
    const float xh = (Ld<T>::one(((const T*)P.X)[r * d + col]) - P.mu[r]) * P.rstd[r];
    ag = fmaf(g, xh, ag);
    ab += g;
  }
  P.partial[(size_t)blockIdx.y * d + col] = ag;
  P.partial[(size_t)(P.chunks + blockIdx.y) * d + col] = ab;
}

__global__ void __launch_bounds__(256) ln_col_reduce_kernel(LnParams P) {
  pdl_wait();
  const int col = blockIdx.x * blockDim.x + threadIdx.x;
  if (col >= P.d) return;
  float ag = 0.f, ab = 0.f;
  for (int ch = 0; ch < P.chunks; ++ch) {      // chunks in order
    ag += P.partial[(size_t)ch * P.d + col];
    ab += P.partial[(size_t)(P.chunks + ch) * P.d + col];
  }
  P.dgamma[col] = ag;
  P.dbeta[col] = ab;
}

}  // namespace

cudaError_t launch_layernorm_bwd(Handle* h, const void* X, const void* gamma, const void* dY, float eps, void* dX,
                                 float* a_out, bool skip_dropped, float* dgamma, float* dbeta, float rho_hint,
                                 cudaStream_t st) {
  const vcas_layer_desc& d = h->desc;
  const Workspace& ws = h->ws;
  LnParams P;
  P.X = X; P.gamma = gamma; P.dY = dY; P.dX = dX;
  P.scaleA = ws.scaleA; P.idxA = ws.idxA; P.dropA = ws.dropA; P.counts = ws.counts;
  P.mu = ws.w; P.rstd = ws.q;
  P.a_out = a_out; P.a_parts = a_out_parts(d.d_in);
  P.partial = ws.Gs;
  P.dgamma = dgamma; P.dbeta = dbeta;
  P.N = d.N; P.T = d.T; P.d = d.d_in; P.skip_dropped = skip_dropped ? 1 : 0;
  P.eps = eps;
  const int col_blocks = (d.d_in + 255) / 256;
  int chunks = (h->num_sms * 4) / col_blocks;
  if (chunks > d.d_in / 2) chunks = d.d_in / 2;       // the scratch holds d * d floats
  const long exp_rows = (long)((double)rho_hint * d.N * d.T) + 1;
  if (chunks > exp_rows / 16 + 1) chunks = (int)(exp_rows / 16 + 1);
  if (chunks < 1) chunks = 1;
  P.chunks = chunks;
  const long R = (long)d.N * d.T;
  long rb = (R + 7) / 8;
  if (rb > (1l << 20)) rb = 1l << 20;
  cudaError_t e;
  if (d.dtype == VCAS_DTYPE_BF16) {
    e = launch_after(ln_row_kernel<__nv_bfloat16>, dim3((unsigned)rb), dim3(256), 0, st, P);
    if (e == cudaSuccess) e = launch_after(ln_col_kernel<__nv_bfloat16>, dim3(col_blocks, chunks), dim3(256), 0, st, P);
  } else {
    e = launch_after(ln_row_kernel<float>, dim3((unsigned)rb), dim3(256), 0, st, P);
    if (e == cudaSuccess) e = launch_after(ln_col_kernel<float>, dim3(col_blocks, chunks), dim3(256), 0, st, P);
  }
  if (e == cudaSuccess) e = launch_after(ln_col_reduce_kernel, dim3(col_blocks), dim3(256), 0, st, P);
  h->launches += 3;
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace vcas
