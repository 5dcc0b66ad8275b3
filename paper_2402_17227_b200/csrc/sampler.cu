// Keep probabilities, Philox Bernoulli masks and compaction for SampleA and SampleW
// (Sec. 4.1, 4.2).  The arrays involved are tiny (N and R = N*T floats), so the whole stage is
// one CTA: latency-bound, not bandwidth-bound.  Everything stays on the device: the kept
// counts are written to the workspace and read by the product kernels.
#include "common.cuh"

namespace vcas {
namespace {

constexpr int SAMPLER_THREADS = 1024;

struct Scratch {
  double d[32];
  int i[32];
  int scan[33];
  double bd;
  int bi;
};

// Block-wide sum of one double and one int, result in every thread.
__device__ void block_sum(double& s, int& c, Scratch* sc) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  s = warp_sum(s);
  c = warp_sum(c);
  if (lane == 0) { sc->d[warp] = s; sc->i[warp] = c; }
  __syncthreads();
  if (warp == 0) {
    double x = lane < (int)(blockDim.x >> 5) ? sc->d[lane] : 0.0;
    int y = lane < (int)(blockDim.x >> 5) ? sc->i[lane] : 0;
    x = warp_sum(x);
    y = warp_sum(y);
    if (lane == 0) { sc->bd = x; sc->bi = y; }
  }
  __syncthreads();
  s = sc->bd;
  c = sc->bi;
  __syncthreads();
}

// Keep probabilities proportional to v, capped at 1, summing to `budget` (the minimiser of
// sum (1-p)/p v^2 under that budget): p = min(1, c v).  The saturated set is grown from
// empty; c only increases, so the iteration reaches the least fixed point, which is the
// unique solution.
__device__ void capped_prop_block(const float* v, int n, double budget, float* p, Scratch* sc) {
  const int tid = threadIdx.x, nt = blockDim.x;
  double S = 0.0;
  int nz = 0;
  for (int i = tid; i < n; i += nt) {
    const float x = v[i];
    if (x > 0.f) { S += (double)x; ++nz; }
  }
  block_sum(S, nz, sc);
  if (nz == 0 || budget <= 0.0) {
    for (int i = tid; i < n; i += nt) p[i] = 0.f;
    return;
  }
  if ((double)nz <= budget) {
    for (int i = tid; i < n; i += nt) p[i] = v[i] > 0.f ? 1.f : 0.f;
    return;
  }
  double c = budget / S;
  int k = 0;
  for (int iter = 0; iter < 128; ++iter) {
    double Su = 0.0;
    int ks = 0;
    for (int i = tid; i < n; i += nt) {
      const float x = v[i];
      if (x > 0.f) {
        if (c * (double)x >= 1.0) ++ks; else Su += (double)x;
      }
    }
    block_sum(Su, ks, sc);
    if (ks == k) break;
    k = ks;
    if (Su > 0.0) {
      const double cn = (budget - (double)k) / Su;
      c = cn > c ? cn : c;
    }
  }
  for (int i = tid; i < n; i += nt) {
    const float x = v[i];
    float r = 0.f;
    if (x > 0.f) {
      const double cx = c * (double)x;
      r = cx >= 1.0 ? 1.f : (float)cx;
    }
    p[i] = r;
  }
}

// Ordered compaction of the indices i < n with keep(i): emit(i, position).  Returns the count.
template <typename KeepFn, typename EmitFn>
__device__ int block_compact(int n, KeepFn keep, EmitFn emit, Scratch* sc) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nw = blockDim.x >> 5;
  int base = 0;
  for (int start = 0; start < n; start += blockDim.x) {
    const int i = start + tid;
    const bool k = (i < n) && keep(i);
    const unsigned ballot = __ballot_sync(0xffffffffu, k);
    const int wofs = __popc(ballot & ((1u << lane) - 1u));
    if (lane == 0) sc->scan[warp] = __popc(ballot);
    __syncthreads();
    if (warp == 0) {
      const int v = lane < nw ? sc->scan[lane] : 0;
      int incl = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
      }
      sc->scan[lane] = incl - v;
      if (lane == 31) sc->scan[32] = incl;
    }
    __syncthreads();
    if (k) emit(i, base + sc->scan[warp] + wofs);
    base += sc->scan[32];
    __syncthreads();
  }
  return base;
}

struct SamplerParams {
  const float* a; const float* b;
  float* g; float* p; float* w; float* q;
  float* scaleA; float* scaleW;
  int32_t* idxA; int32_t* dropA; int32_t* idxW; int32_t* counts;
  double* acc;
  const float* p_in; const float* q_in;
  int N, T;
  float rho, nu;
  uint64_t seed;
  int sample_w, accumulate_vw;
};

__global__ void __launch_bounds__(SAMPLER_THREADS) sampler_kernel(SamplerParams P) {
  __shared__ Scratch sc;
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
  const int N = P.N, T = P.T, R = N * T;

  // ---- SampleA: ||G_n||_F, p_n, mask, kept / dropped data lists (Sec. 4.1)
  for (int n = warp; n < N; n += nw) {
    double s = 0.0;
    for (int t = lane; t < T; t += 32) s += (double)P.a[(size_t)n * T + t];
    s = warp_sum(s);
    if (lane == 0) P.g[n] = (float)sqrt(s);
  }
  __syncthreads();
  if (P.p_in != nullptr) {
    for (int n = tid; n < N; n += nt) P.p[n] = P.p_in[n];
  } else {
    capped_prop_block(P.g, N, (double)N * (double)P.rho, P.p, &sc);
  }
  __syncthreads();
  for (int n = tid; n < N; n += nt) {
    const float pn = P.p[n];
    P.scaleA[n] = bernoulli_keep(pn, P.seed, 0u, (uint64_t)n) ? 1.0f / pn : 0.f;
  }
  __syncthreads();
  const int cntA = block_compact(N, [&](int n) { return P.scaleA[n] > 0.f; },
                                 [&](int n, int pos) { P.idxA[pos] = n; }, &sc);
  block_compact(N, [&](int n) { return !(P.scaleA[n] > 0.f); },
                [&](int n, int pos) { P.dropA[pos] = n; }, &sc);

  // ---- SampleW: leverage scores of G_hat, q_r, mask, kept rows (Sec. 4.2, Eq. 3)
  for (int r = tid; r < R; r += nt) {
    const int n = r / T;
    float wr = 0.f;
    if (P.scaleA[n] > 0.f) wr = (float)(sqrt((double)P.a[r] * (double)P.b[r]) / (double)P.p[n]);
    P.w[r] = wr;
  }
  __syncthreads();
  if (P.q_in != nullptr) {
    for (int r = tid; r < R; r += nt) P.q[r] = P.scaleA[r / T] > 0.f ? P.q_in[r] : 0.f;
  } else {
    capped_prop_block(P.w, R, (double)P.nu * (double)T * (double)cntA, P.q, &sc);
  }
  __syncthreads();
  if (P.accumulate_vw) {
    double vw = 0.0;
    int dummy = 0;
    for (int r = tid; r < R; r += nt) {
      const double qr = (double)P.q[r];
      if (qr > 0.0) {
        const double wr = (double)P.w[r];
        vw += (1.0 - qr) / qr * wr * wr;
      }
    }
    block_sum(vw, dummy, &sc);
    if (tid == 0) P.acc[1] += vw;
  }
  int cntW;
  if (P.sample_w) {
    cntW = block_compact(R,
        [&](int r) { const float qr = P.q[r]; return qr > 0.f && bernoulli_keep(qr, P.seed, 1u, (uint64_t)r); },
        [&](int r, int pos) { P.idxW[pos] = r; P.scaleW[pos] = P.scaleA[r / T] / P.q[r]; }, &sc);
  } else {
    cntW = block_compact(R, [&](int r) { return P.scaleA[r / T] > 0.f; },
        [&](int r, int pos) { P.idxW[pos] = r; P.scaleW[pos] = P.scaleA[r / T]; }, &sc);
  }
  if (tid == 0) { P.counts[0] = cntA; P.counts[1] = cntW; }
}

__global__ void __launch_bounds__(SAMPLER_THREADS)
mask_kernel(const float* __restrict__ p, int n, uint64_t seed, int sampler, uint8_t* keep, int32_t* idx,
            int32_t* cnt) {
  __shared__ Scratch sc;
  const int c = block_compact(n,
      [&](int i) {
        const bool k = bernoulli_keep(p[i], seed, (uint32_t)sampler, (uint64_t)i);
        if (keep != nullptr) keep[i] = k ? 1 : 0;
        return k;
      },
      [&](int i, int pos) { if (idx != nullptr) idx[pos] = i; }, &sc);
  if (threadIdx.x == 0 && cnt != nullptr) *cnt = c;
}

}  // namespace

cudaError_t launch_sampler(Handle* h, const SamplerArgs& a, cudaStream_t st) {
  const Workspace& ws = h->ws;
  SamplerParams P;
  P.a = ws.a; P.b = ws.b; P.g = ws.g; P.p = ws.p; P.w = ws.w; P.q = ws.q;
  P.scaleA = ws.scaleA; P.scaleW = ws.scaleW;
  P.idxA = ws.idxA; P.dropA = ws.dropA; P.idxW = ws.idxW; P.counts = ws.counts;
  P.acc = ws.acc;
  P.p_in = a.p_in; P.q_in = a.q_in;
  P.N = h->desc.N; P.T = h->desc.T;
  P.rho = a.rho; P.nu = a.nu; P.seed = a.seed;
  P.sample_w = a.sample_w; P.accumulate_vw = a.accumulate_vw;
  sampler_kernel<<<1, SAMPLER_THREADS, 0, st>>>(P);
  h->launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_mask_from_probs(Handle* h, const float* p, int n, uint64_t seed, int sampler,
                                   uint8_t* keep, int32_t* idx, int32_t* cnt, cudaStream_t st) {
  mask_kernel<<<1, SAMPLER_THREADS, 0, st>>>(p, n, seed, sampler, keep, idx, cnt);
  h->launches += 1;
  return cudaGetLastError();
}

}  // namespace vcas
