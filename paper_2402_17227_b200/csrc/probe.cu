// Reductions of the variance probe (Alg. 1; App. D keeps only the exact gradient G_s,i, its
// running mean and a running second moment).  HBM-bound elementwise passes over
// [d_out, d_in] fp32 tensors, with block partials combined in a fixed order by the last block
// so that repeated runs give identical bits.
#include "common.cuh"

namespace vcas {
namespace {

// Running mean and running sum of squared deviations (Welford) of the exact gradients:
// after M updates, V_s = sum(m2) / (M - 1).
__global__ void welford_kernel(const float4* __restrict__ G, float4* __restrict__ mean, float4* __restrict__ m2,
                               size_t n4, float inv_count, int first) {
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < n4; e += (size_t)gridDim.x * blockDim.x) {
    const float4 x = G[e];
    if (first) {
      mean[e] = x;
      m2[e] = make_float4(0.f, 0.f, 0.f, 0.f);
    } else {
      float4 m = mean[e], s = m2[e];
      float d;
      d = x.x - m.x; m.x = fmaf(d, inv_count, m.x); s.x = fmaf(d, x.x - m.x, s.x);
      d = x.y - m.y; m.y = fmaf(d, inv_count, m.y); s.y = fmaf(d, x.y - m.y, s.y);
      d = x.z - m.z; m.z = fmaf(d, inv_count, m.z); s.z = fmaf(d, x.z - m.z, s.z);
      d = x.w - m.w; m.w = fmaf(d, inv_count, m.w); s.w = fmaf(d, x.w - m.w, s.w);
      mean[e] = m;
      m2[e] = s;
    }
  }
}

// mode 0: sum (A - B)^2 ; mode 1: sum A.  Adds the total to *acc.
__global__ void __launch_bounds__(256) reduce_kernel(const float4* __restrict__ A, const float4* __restrict__ B,
                                                     size_t n4, int mode, double* __restrict__ partial,
                                                     int32_t* __restrict__ ticket, double* __restrict__ acc) {
  __shared__ double sh[8];
  __shared__ int last;
  double s = 0.0;
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < n4; e += (size_t)gridDim.x * blockDim.x) {
    const float4 a = A[e];
    float t;
    if (mode == 0) {
      const float4 b = B[e];
      const float dx = a.x - b.x, dy = a.y - b.y, dz = a.z - b.z, dw = a.w - b.w;
      t = fmaf(dx, dx, fmaf(dy, dy, fmaf(dz, dz, dw * dw)));
    } else {
      t = (a.x + a.y) + (a.z + a.w);
    }
    s += (double)t;
  }
  s = warp_sum(s);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) sh[warp] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    double b = 0.0;
    for (int i = 0; i < 8; ++i) b += sh[i];
    partial[blockIdx.x] = b;
    __threadfence();
    last = (atomicAdd(ticket, 1) == (int)gridDim.x - 1);
  }
  __syncthreads();
  if (last) {
    // the last block adds the block partials: each thread a fixed strided subset, then a fixed tree
    __threadfence();
    double tot = 0.0;
    for (unsigned i = threadIdx.x; i < gridDim.x; i += blockDim.x) tot += __ldcg(partial + i);
    tot = warp_sum(tot);
    __syncthreads();
    if (lane == 0) sh[warp] = tot;
    __syncthreads();
    if (threadIdx.x == 0) {
      double b = 0.0;
      for (int i = 0; i < 8; ++i) b += sh[i];
      *acc += b;
      *ticket = 0;
    }
  }
}

// Eq. 4: p(s) = min{ n/N, n >= 1 : sum of the n largest norms >= s * sum of all norms }, for two values of s.
__global__ void __launch_bounds__(1024) sparsity_kernel(const float* __restrict__ g, float* __restrict__ sorted,
                                                        int N, double s_lo, double s_hi, double* __restrict__ acc) {
  // rank of g[i] in descending order (ties broken by index): a counting sort, N is a batch size
  for (int i = threadIdx.x; i < N; i += blockDim.x) {
    const float x = g[i];
    int rank = 0;
    for (int j = 0; j < N; ++j) {
      const float y = g[j];
      rank += (y > x) || (y == x && j < i);
    }
    sorted[rank] = x;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    double total = 0.0;
    for (int i = 0; i < N; ++i) total += (double)sorted[i];
    // n ranges over 1..N (the sum over i = 1..n of Eq. 4): at least one datum is always kept
    double res[2];
    const double ss[2] = {s_lo, s_hi};
    for (int k = 0; k < 2; ++k) {
      const double target = ss[k] * total;
      double cum = (double)sorted[0];
      int n = 1;
      while (cum < target && n < N) { cum += (double)sorted[n]; ++n; }
      res[k] = (double)n / (double)N;
    }
    acc[2] += res[0];
    acc[3] += res[1];
  }
}

// scale: d_out / (rows of the parameter gradient the sums were taken over) (App. D: a sample of the parameters)
__global__ void finalize_kernel(const double* __restrict__ acc, const double* __restrict__ acc2, int M, double scale,
                                float* V_s, float* V_act, float* V_w, float* p_lo, float* p_hi) {
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    const double mm = (double)M * (double)M;
    if (V_s) *V_s = (float)(scale * acc[4] / (double)(M - 1));
    if (V_act) *V_act = (float)(scale * (acc[0] + acc2[0]) / mm);     // even draws + odd draws
    if (V_w) *V_w = (float)((acc[1] + acc2[1]) / mm);
    if (p_lo) *p_lo = (float)(acc[2] / (double)M);
    if (p_hi) *p_hi = (float)(acc[3] / (double)M);
  }
}

// The columns `cols` of a row-major [R, d] matrix, compact: out[r, c] = in[r, cols[c]] (one warp per row).
template <typename T>
__global__ void __launch_bounds__(256) gather_cols_kernel(const T* __restrict__ in, int R, int d,
                                                          const int32_t* __restrict__ cols, int k, T* __restrict__ out) {
  const int lane = threadIdx.x & 31, wpb = blockDim.x >> 5;
  for (int r = blockIdx.x * wpb + (threadIdx.x >> 5); r < R; r += gridDim.x * wpb)
    for (int c = lane; c < k; c += 32) out[(size_t)r * k + c] = in[(size_t)r * d + cols[c]];
}

// A uniformly random subset of k of the d_out output features, ascending: feature i gets the Philox word of
// counter (i, 0, 2, 0) (sampler id 2) under the key (seed low, seed high); the k features with the smallest
// words are taken, ties by index.  One CTA; u is scratch of d_out words.
__global__ void __launch_bounds__(1024) subset_kernel(int d_out, int k, uint64_t seed, uint32_t* __restrict__ u,
                                                      int32_t* __restrict__ flag, int32_t* __restrict__ rows) {
  for (int i = threadIdx.x; i < d_out; i += blockDim.x)
    u[i] = philox_word0((uint32_t)i, 0u, 2u, 0u, (uint32_t)seed, (uint32_t)(seed >> 32));
  __syncthreads();
  for (int i = threadIdx.x; i < d_out; i += blockDim.x) {
    const uint32_t x = u[i];
    int rank = 0;
    for (int j = 0; j < d_out; ++j) {
      const uint32_t y = u[j];
      rank += (y < x) || (y == x && j < i);
    }
    flag[i] = rank < k ? 1 : 0;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int n = 0;
    for (int i = 0; i < d_out; ++i)
      if (flag[i]) rows[n++] = i;
  }
}

int reduce_blocks(size_t n4) {
  size_t b = (n4 + 256 * 4 - 1) / (256 * 4);
  if (b > 1024) b = 1024;
  if (b < 1) b = 1;
  return (int)b;
}

}  // namespace

cudaError_t launch_probe_reset(Handle* h, cudaStream_t st) {
  cudaError_t e = cudaMemsetAsync(h->ws.acc, 0, 16 * sizeof(double), st);
  if (e == cudaSuccess) e = cudaMemsetAsync(h->ws2.acc, 0, 16 * sizeof(double), st);
  if (e == cudaSuccess) e = cudaMemsetAsync(h->ws2.counts + 4, 0, sizeof(int32_t), st);
  if (e != cudaSuccess) return e;
  return cudaMemsetAsync(h->ws.counts + 4, 0, sizeof(int32_t), st);
}

cudaError_t launch_probe_welford(Handle* h, int i, cudaStream_t st) {
  const size_t n4 = (size_t)h->desc.d_out * h->desc.d_in / 4;
  welford_kernel<<<reduce_blocks(n4), 256, 0, st>>>((const float4*)h->ws.Gs, (float4*)h->ws.mean,
                                                    (float4*)h->ws.m2, n4, 1.0f / (float)(i + 1), i == 0);
  h->launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_probe_sqdiff(Handle* h, cudaStream_t st) {
  const size_t n4 = (size_t)h->desc.d_out * h->desc.d_in / 4;
  reduce_kernel<<<reduce_blocks(n4), 256, 0, st>>>((const float4*)h->ws.Gact, (const float4*)h->ws.Gs, n4, 0,
                                                   h->ws.partial, h->ws.counts + 4, h->ws.acc + 0);
  h->launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_probe_sparsity(Handle* h, double s_lo, double s_hi, cudaStream_t st) {
  sparsity_kernel<<<1, 1024, 0, st>>>(h->ws.g, h->ws.sorted, h->desc.N, s_lo, s_hi, h->ws.acc);
  h->launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_gather_cols(Handle* h, const void* in, int d, const int32_t* cols, int k, void* out, cudaStream_t st) {
  const int R = h->desc.N * h->desc.T;
  int blocks = (R + 7) / 8;
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (h->desc.dtype == VCAS_DTYPE_BF16)
    gather_cols_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>((const __nv_bfloat16*)in, R, d, cols, k, (__nv_bfloat16*)out);
  else
    gather_cols_kernel<float><<<blocks, 256, 0, st>>>((const float*)in, R, d, cols, k, (float*)out);
  h->launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_param_subset(Handle* h, int k, uint64_t seed, uint32_t* scratch_u, int32_t* scratch_flag,
                                int32_t* rows, cudaStream_t st) {
  subset_kernel<<<1, 1024, 0, st>>>(h->desc.d_out, k, seed, scratch_u, scratch_flag, rows);
  h->launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_probe_finalize(Handle* h, int M, double scale, float* V_s, float* V_act, float* V_w, float* p_lo,
                                  float* p_hi, cudaStream_t st) {
  const size_t n4 = (size_t)h->desc.d_out * h->desc.d_in / 4;
  reduce_kernel<<<reduce_blocks(n4), 256, 0, st>>>((const float4*)h->ws.m2, nullptr, n4, 1, h->ws.partial,
                                                   h->ws.counts + 4, h->ws.acc + 4);
  finalize_kernel<<<1, 32, 0, st>>>(h->ws.acc, h->ws2.acc, M, scale, V_s, V_act, V_w, p_lo, p_hi);
  h->launches += 2;
  return cudaGetLastError();
}

}  // namespace vcas
