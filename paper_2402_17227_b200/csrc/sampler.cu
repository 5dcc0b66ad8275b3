// Keep probabilities, Philox Bernoulli masks and compaction for SampleA and SampleW
// (Sec. 4.1, 4.2).  The arrays involved are tiny (N and R = N*T floats), so the whole stage is
// one CTA: latency-bound, not bandwidth-bound.  Everything stays on the device: the kept
// counts are written to the workspace and read by the product kernels.
#include "common.cuh"

namespace vcas {
namespace {

constexpr int SAMPLER_THREADS = 1024;
static_assert(FAST_MAX_N <= SAMPLER_THREADS && FAST_MAX_R == 16 * SAMPLER_THREADS, "fast sampling limits");

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
  const float* lev; const uint32_t* u24;   // per-row leverage ||dY_r|| ||X_r|| and SampleW uniform (row-norm kernel)
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
  pdl_wait();      // the row norms come from the kernel before this one
  pdl_trigger();   // the product kernel may set itself up meanwhile
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

// ---------------------------------------------------------------------------------------
// Fast path for R <= 16 * 1024 rows and N <= 1024 data: every thread keeps its E consecutive
// rows in registers, SampleA runs inside warp 0 with shuffles only, and each water-filling
// iteration over the rows costs two block barriers.
// ---------------------------------------------------------------------------------------
struct FastShared {
  float part_f[2][32];
  int part_i[2][32];
  int warp_tot[32];
  float scaleA[1024];
  float pA[1024];
  int cntA;
};

// Block-wide sum of one float and one int in a fixed order (lanes by shuffle tree, then the 32
// warp totals by the same tree, which every warp runs for itself so that one barrier suffices; the
// buffers alternate with `parity`, and a buffer is rewritten only after a later barrier).  fp32 on
// purpose: this is a single-CTA kernel, and double-precision arithmetic concentrated on one SM was
// measured to dominate its run time; a tree sum of <= 16384 non-negative fp32 terms is accurate to
// about 1e-6, inside the 1e-5 the probabilities are specified to.
__device__ __forceinline__ void fast_sum(float& s, int& c, FastShared* sh, int parity) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  s = warp_sum(s);
  c = __reduce_add_sync(0xffffffffu, c);
  if (lane == 0) { sh->part_f[parity][warp] = s; sh->part_i[parity][warp] = c; }
  __syncthreads();
  s = warp_sum(sh->part_f[parity][lane]);
  c = __reduce_add_sync(0xffffffffu, sh->part_i[parity][lane]);
}

template <int E, int SLOTS>
__global__ void __launch_bounds__(SAMPLER_THREADS) sampler_fast_kernel(SamplerParams P) {
  __shared__ FastShared sh;
  pdl_wait();      // the row norms come from the kernel before this one
  pdl_trigger();   // the product kernel may set itself up meanwhile
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int N = P.N, T = P.T, R = N * T;
  // Element e of this thread is row (e / 4) * 4096 + tid * 4 + (e % 4): four consecutive rows per
  // thread and group, so that every 16-byte load or store of a warp covers 512 contiguous bytes.
  auto row_of = [&](int e) { return (e >> 2) * (4 * SAMPLER_THREADS) + tid * 4 + (e & 3); };

  // this thread's rows: the unscaled leverage score and the SampleW uniform, both made per row by
  // the row-norm kernel
  float ab[E];
#pragma unroll
  for (int e = 0; e < E; e += 4) {
    const int rb = row_of(e);
    if (rb + 3 < R) {
      const float4 v = *reinterpret_cast<const float4*>(P.lev + rb);
      ab[e] = v.x; ab[e + 1] = v.y; ab[e + 2] = v.z; ab[e + 3] = v.w;
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i) ab[e + i] = rb + i < R ? P.lev[rb + i] : 0.f;
    }
  }
  // The rows' SampleW uniforms: requested now, together with the scores, when the registers allow it
  // (E <= 8); with E = 16 they are loaded just before the masks are drawn.
  constexpr bool EARLY_U = E <= 8;
  uint32_t ue[EARLY_U ? E : 4];
  if (EARLY_U) {
#pragma unroll
    for (int e = 0; e < (EARLY_U ? E : 4); e += 4) {
      const int rb = row_of(e);
      ue[e] = ue[e + 1] = ue[e + 2] = ue[e + 3] = 0xffffffffu;
      if (P.sample_w) {
        if (rb + 3 < R) {
          const uint4 u = *reinterpret_cast<const uint4*>(P.u24 + rb);
          ue[e] = u.x; ue[e + 1] = u.y; ue[e + 2] = u.z; ue[e + 3] = u.w;
        } else {
#pragma unroll
          for (int i = 0; i < 4; ++i)
            if (rb + i < R) ue[e + i] = P.u24[rb + i];
        }
      }
    }
  }
  // Datum of each of this thread's rows, one division per group of four rows, kept as one word per
  // group (registers are scarce at 1024 threads): the first row's datum and three 2-bit increments.
  int ncode[E / 4];
#pragma unroll
  for (int e = 0; e < E; e += 4) {
    const int rb = row_of(e);
    const int n0 = rb / T;
    int n = n0, rem = rb - n0 * T, code = n0;
#pragma unroll
    for (int i = 1; i < 4; ++i) {
      if (++rem == T) { rem = 0; ++n; }
      code |= (n - n0) << (14 + 2 * i);
    }
    ncode[e >> 2] = code;
  }
  auto datum_of = [&](int e) {
    const int code = ncode[e >> 2];
    const int n = (code & 0xffff) + ((e & 3) ? ((code >> (14 + 2 * (e & 3))) & 3) : 0);
    return n < N ? n : N - 1;
  };

  // ---- ||G_n||_F: one warp per datum, fixed order
  for (int n = warp; n < N; n += 32) {
    const float s = datum_sqnorm_warp(P.a + (size_t)n * T, T, lane);
    if (lane == 0) { const float g = sqrtf(s); P.g[n] = g; sh.pA[n] = g; }
  }
  __syncthreads();
  // ---- SampleA inside warp 0 (Sec. 4.1): p_n, mask, kept / dropped lists
  if (warp == 0) {
    SampleAOut o;
    o.p = P.p; o.scaleA = P.scaleA; o.idxA = P.idxA; o.dropA = P.dropA;
    o.sh_p = sh.pA; o.sh_scaleA = sh.scaleA;
    const int kept = sample_a_warp<SLOTS>(sh.pA, N, P.rho, P.p_in, P.seed, o, lane);
    if (lane == 0) sh.cntA = kept;
  }
  __syncthreads();
  const int cntA = sh.cntA;

  // ---- SampleW (Sec. 4.2, Eq. 3): leverage scores of G_hat in registers
  float w[E];
#pragma unroll
  for (int e = 0; e < E; ++e) {
    const int n = datum_of(e);
    w[e] = (row_of(e) < R && sh.scaleA[n] > 0.f) ? ab[e] / sh.pA[n] : 0.f;
  }
#pragma unroll
  for (int e = 0; e < E; e += 4) {
    const int rb = row_of(e);
    if (rb + 3 < R) {
      *reinterpret_cast<float4*>(P.w + rb) = make_float4(w[e], w[e + 1], w[e + 2], w[e + 3]);
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (rb + i < R) P.w[rb + i] = w[e + i];
    }
  }
  float q[E];
  if (P.q_in != nullptr) {
#pragma unroll
    for (int e = 0; e < E; ++e) {
      const int r = row_of(e);
      q[e] = (r < R && sh.scaleA[datum_of(e)] > 0.f) ? P.q_in[r] : 0.f;
    }
  } else {
    const float budget = P.nu * (float)T * (float)cntA;
    float S = 0.f;
    int nz = 0;
#pragma unroll
    for (int e = 0; e < E; ++e)
      if (w[e] > 0.f) { S += w[e]; ++nz; }
    int parity = 0;
    fast_sum(S, nz, &sh, parity); parity ^= 1;
    if (nz == 0 || budget <= 0.f) {
#pragma unroll
      for (int e = 0; e < E; ++e) q[e] = 0.f;
    } else if ((float)nz <= budget) {
#pragma unroll
      for (int e = 0; e < E; ++e) q[e] = w[e] > 0.f ? 1.f : 0.f;
    } else {
      float c = budget / S;
      int k = 0;
      for (int iter = 0; iter < 128; ++iter) {
        float Su = 0.f;
        int ks = 0;
#pragma unroll
        for (int e = 0; e < E; ++e)
          if (w[e] > 0.f) {
            if (c * w[e] >= 1.0f) ++ks; else Su += w[e];
          }
        fast_sum(Su, ks, &sh, parity); parity ^= 1;
        if (ks == k) break;
        k = ks;
        if (Su > 0.f) {
          const float cn = (budget - (float)k) / Su;
          c = cn > c ? cn : c;
        }
      }
#pragma unroll
      for (int e = 0; e < E; ++e) {
        float r = 0.f;
        if (w[e] > 0.f) {
          const float cx = c * w[e];
          r = cx >= 1.0f ? 1.f : cx;
        }
        q[e] = r;
      }
    }
  }
#pragma unroll
  for (int e = 0; e < E; e += 4) {
    const int rb = row_of(e);
    if (rb + 3 < R) {
      *reinterpret_cast<float4*>(P.q + rb) = make_float4(q[e], q[e + 1], q[e + 2], q[e + 3]);
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (rb + i < R) P.q[rb + i] = q[e + i];
    }
  }

  if (P.accumulate_vw) {      // Eq. 3 at these probabilities (probe only)
    float vw = 0.f;
    int dummy = 0;
#pragma unroll
    for (int e = 0; e < E; ++e)
      if (q[e] > 0.f) vw += (1.0f - q[e]) / q[e] * w[e] * w[e];
    fast_sum(vw, dummy, &sh, 0);
    if (tid == 0) P.acc[1] += (double)vw;
  }

  // ---- mask and ordered compaction: rows ascend with (group, thread, k), so each group of 4096 rows
  // gets its own block-wide exclusive scan of the per-thread counts, on top of the groups before it
  unsigned keepbits = 0;
#pragma unroll
  for (int e = 0; e < E; e += 4) {
    const int rb = row_of(e);
    uint32_t ur[4] = {0xffffffffu, 0xffffffffu, 0xffffffffu, 0xffffffffu};   // the rows' SampleW uniforms
    if (EARLY_U) {
#pragma unroll
      for (int i = 0; i < 4; ++i) ur[i] = ue[(EARLY_U ? e : 0) + i];
    } else if (P.sample_w) {
      if (rb + 3 < R) {
        const uint4 u = *reinterpret_cast<const uint4*>(P.u24 + rb);
        ur[0] = u.x; ur[1] = u.y; ur[2] = u.z; ur[3] = u.w;
      } else {
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (rb + i < R) ur[i] = P.u24[rb + i];
      }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      bool k = false;
      if (rb + i < R) {
        if (P.sample_w) k = q[e + i] > 0.f && ur[i] < (uint32_t)floorf(q[e + i] * 16777216.0f);
        else k = sh.scaleA[datum_of(e + i)] > 0.f;
      }
      keepbits |= (k ? 1u : 0u) << (e + i);
    }
  }
  int total = 0;
#pragma unroll
  for (int g4 = 0; g4 < E / 4; ++g4) {
    const unsigned bits = (keepbits >> (g4 * 4)) & 0xfu;
    const int mine = __popc(bits);
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    __syncthreads();                       // warp_tot of the previous group has been read by everyone
    if (lane == 31) sh.warp_tot[warp] = incl;
    __syncthreads();
    const int wt = sh.warp_tot[lane];
    const int base0 = total + incl - mine + __reduce_add_sync(0xffffffffu, lane < warp ? wt : 0);
    total += __reduce_add_sync(0xffffffffu, wt);
    int base = base0;
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if (bits & (1u << i)) {
        const int e = g4 * 4 + i;
        P.idxW[base] = row_of(e);
        P.scaleW[base] = P.sample_w ? sh.scaleA[datum_of(e)] / q[e] : sh.scaleA[datum_of(e)];
        ++base;
      }
  }
  if (tid == 0) { P.counts[0] = cntA; P.counts[1] = total; }
}

// SampleA alone (Sec. 4.1), for the dX product: the same warp-level code as in the sampling kernels, so the
// masks are identical; results go to arrays of their own because the full sampling kernel runs at the
// same time on another stream.
constexpr int SAMPLE_A_THREADS = 512;
template <int SLOTS>
__global__ void __launch_bounds__(SAMPLE_A_THREADS)
sample_a_kernel(const float* __restrict__ a, int N, int T, float rho, const float* __restrict__ p_in, uint64_t seed,
                float* scaleA, int32_t* idxA, int32_t* dropA, int32_t* cnt) {
  __shared__ float s_g[32 * SLOTS];
  pdl_wait();      // the row norms come from the kernel before this one
  pdl_trigger();   // the dX product kernel may set itself up meanwhile
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int n = warp; n < N; n += SAMPLE_A_THREADS / 32) {
    const float s = datum_sqnorm_warp(a + (size_t)n * T, T, lane);
    if (lane == 0) s_g[n] = sqrtf(s);
  }
  __syncthreads();
  if (warp == 0) {
    SampleAOut o;
    o.p = nullptr; o.scaleA = scaleA; o.idxA = idxA; o.dropA = dropA;
    o.sh_p = nullptr; o.sh_scaleA = nullptr;
    const int kept = sample_a_warp<SLOTS>(s_g, N, rho, p_in, seed, o, lane);
    if (lane == 0) *cnt = kept;
  }
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

cudaError_t launch_sampler(Handle* h, const SamplerArgs& a, cudaStream_t st, bool after_event) {
  const Workspace& ws = h->ws;
  SamplerParams P;
  P.a = ws.a; P.b = ws.b; P.lev = ws.lev; P.u24 = ws.u24; P.g = ws.g; P.p = ws.p; P.w = ws.w; P.q = ws.q;
  P.scaleA = ws.scaleA; P.scaleW = ws.scaleW;
  P.idxA = ws.idxA; P.dropA = ws.dropA; P.idxW = ws.idxW; P.counts = ws.counts;
  P.acc = ws.acc;
  P.p_in = a.p_in; P.q_in = a.q_in;
  P.N = h->desc.N; P.T = h->desc.T;
  P.rho = a.rho; P.nu = a.nu; P.seed = a.seed;
  P.sample_w = a.sample_w; P.accumulate_vw = a.accumulate_vw;
  const int R = P.N * P.T;
  cudaError_t e = cudaSuccess;
  // after_event: the kernel before this one in the stream is not the producer of its inputs (those
  // arrive through an event from another stream), so it is launched without the programmatic attribute
  auto go = [&](void (*k)(SamplerParams)) {
    if (after_event) { k<<<1, SAMPLER_THREADS, 0, st>>>(P); return cudaSuccess; }
    return launch_after(k, dim3(1), dim3(SAMPLER_THREADS), 0, st, P);
  };
  if (fast_sampling(h->desc)) {
    const bool wide = P.N > 32;       // SampleA slots per lane of warp 0
    if (R <= 4 * SAMPLER_THREADS) e = go(wide ? sampler_fast_kernel<4, 32> : sampler_fast_kernel<4, 1>);
    else if (R <= 8 * SAMPLER_THREADS) e = go(wide ? sampler_fast_kernel<8, 32> : sampler_fast_kernel<8, 1>);
    else e = go(wide ? sampler_fast_kernel<16, 32> : sampler_fast_kernel<16, 1>);
  } else {
    e = go(sampler_kernel);
  }
  h->launches += 1;
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_sample_a(Handle* h, const SamplerArgs& a, cudaStream_t st) {
  const Workspace& ws = h->ws;
  const vcas_layer_desc& d = h->desc;
  if (!fast_sampling(d)) return cudaErrorInvalidValue;
  cudaError_t e;
  if (d.N <= 32)
    e = launch_after(sample_a_kernel<1>, dim3(1), dim3(SAMPLE_A_THREADS), 0, st, (const float*)ws.a, d.N, d.T, a.rho,
                     a.p_in, a.seed, ws.scaleA2, ws.idxA2, ws.dropA2, ws.counts + 6);
  else
    e = launch_after(sample_a_kernel<32>, dim3(1), dim3(SAMPLE_A_THREADS), 0, st, (const float*)ws.a, d.N, d.T, a.rho,
                     a.p_in, a.seed, ws.scaleA2, ws.idxA2, ws.dropA2, ws.counts + 6);
  h->launches += 1;
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_mask_from_probs(Handle* h, const float* p, int n, uint64_t seed, int sampler,
                                   uint8_t* keep, int32_t* idx, int32_t* cnt, cudaStream_t st) {
  mask_kernel<<<1, SAMPLER_THREADS, 0, st>>>(p, n, seed, sampler, keep, idx, cnt);
  h->launches += 1;
  return cudaGetLastError();
}

}  // namespace vcas
