// Keep probabilities, Philox Bernoulli masks and compaction for SampleA and SampleW
// (Sec. 4.1, 4.2).  Everything stays on the device: the kept counts are written to the workspace
// and read by the product kernels.  The stage is a chain of small kernels:
//   sample_a_kernel   one CTA: ||G_n||_F, p_n, mask, kept / dropped data (the dX product can start here);
//   scores_x_kernel   (score.cu) many CTAs: leverage scores and uniforms of the rows of kept data;
//   sample_w_kernel   one CTA, scores in shared memory: the water-filling for q = min(1, c w) - a handful
//                     of block-wide sums - then the masks' counts per chunk of 32 rows and their prefix sums;
//   emit_pack_kernel  many CTAs: kept-row list, 1/(p q), and the compact operands of the dW product.
// Only the scalar fixed point and a scan over R/32 counts run on a single SM.
#include <atomic>

#include "common.cuh"

namespace vcas {
namespace {

constexpr int SAMPLER_THREADS = 1024;
constexpr int WATER_ROUNDS = 128;     // rounds of the water-filling before it is reported as not converged

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
// unique solution.  Returns false if it has not converged after WATER_ROUNDS rounds.
__device__ bool capped_prop_block(const float* v, int n, double budget, float* p, Scratch* sc) {
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
    return true;
  }
  if ((double)nz <= budget) {
    for (int i = tid; i < n; i += nt) p[i] = v[i] > 0.f ? 1.f : 0.f;
    return true;
  }
  double c = budget / S;
  int k = 0;
  bool converged = false;
  for (int iter = 0; iter < WATER_ROUNDS; ++iter) {
    double Su = 0.0;
    int ks = 0;
    for (int i = tid; i < n; i += nt) {
      const float x = v[i];
      if (x > 0.f) {
        if (c * (double)x >= 1.0) ++ks; else Su += (double)x;
      }
    }
    block_sum(Su, ks, sc);
    if (ks == k) { converged = true; break; }
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
  return converged;
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

// ------------------------------------------------------------------------------ SampleA
struct SampleAParams {
  const float* a; int a_parts;
  const int32_t* alive; const int32_t* alive_cnt;
  int N, T;
  float rho;
  const float* p_in;
  uint64_t seed;
  float* g; float* p; float* scaleA;
  int32_t* idxA; int32_t* dropA; int32_t* counts;
  int32_t* kept_out; int32_t* kept_cnt_out;
  int32_t* status;
};

// SampleA (Sec. 4.1) for N <= 32 * SLOTS data: one warp per datum sums its T row square-norms (only the alive
// data are read; the others have norm 0), then warp 0 finds p, draws the masks and writes the lists.
constexpr int SAMPLE_A_THREADS = 512;
template <int SLOTS>
__global__ void __launch_bounds__(SAMPLE_A_THREADS) sample_a_kernel(SampleAParams P) {
  __shared__ float s_g[32 * SLOTS];
  pdl_wait();      // the row norms come from the kernel before this one
  pdl_trigger();   // the dX product kernel may set itself up meanwhile
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int n = threadIdx.x; n < 32 * SLOTS; n += SAMPLE_A_THREADS) s_g[n] = 0.f;
  __syncthreads();
  // a caller's list of alive data is not trusted: a length outside [0, N] or an entry outside [0, N) is reported
  // as VCAS_ERR_BAD_ARG in the status word and not followed
  int nd = P.N;
  if (P.alive != nullptr) {
    nd = *P.alive_cnt;
    if (nd < 0 || nd > P.N) {
      if (threadIdx.x == 0) atomicExch(P.status, (int32_t)VCAS_ERR_BAD_ARG);
      nd = min(max(nd, 0), P.N);
    }
  }
  const int len = P.T * P.a_parts;
  for (int k = warp; k < nd; k += SAMPLE_A_THREADS / 32) {
    const int n = P.alive != nullptr ? P.alive[k] : k;
    if ((unsigned)n >= (unsigned)P.N) {
      if (lane == 0) atomicExch(P.status, (int32_t)VCAS_ERR_BAD_ARG);
      continue;
    }
    const float s = datum_sqnorm_warp(P.a + (size_t)n * len, len, lane);
    if (lane == 0) s_g[n] = sqrtf(s);
  }
  __syncthreads();
  for (int n = threadIdx.x; n < P.N; n += SAMPLE_A_THREADS) P.g[n] = s_g[n];
  if (warp == 0) {
    SampleAOut o;
    o.p = P.p; o.scaleA = P.scaleA; o.idxA = P.idxA; o.dropA = P.dropA; o.idx_copy = P.kept_out;
    const int kept = sample_a_warp<SLOTS>(s_g, P.N, P.rho, P.p_in, P.seed, o, lane);
    if (lane == 0) {
      P.counts[0] = kept;
      if (P.kept_cnt_out != nullptr) *P.kept_cnt_out = kept;
    }
  }
}

// The same for batches of more than 1024 data: one CTA over global memory.
__global__ void __launch_bounds__(SAMPLER_THREADS) sample_a_big_kernel(SampleAParams P) {
  __shared__ Scratch sc;
  pdl_wait();
  pdl_trigger();
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
  const int N = P.N;
  for (int n = tid; n < N; n += nt) P.g[n] = 0.f;
  __syncthreads();
  int nd = N;
  if (P.alive != nullptr) {
    nd = *P.alive_cnt;
    if (nd < 0 || nd > N) {
      if (tid == 0) atomicExch(P.status, (int32_t)VCAS_ERR_BAD_ARG);
      nd = min(max(nd, 0), N);
    }
  }
  const int len = P.T * P.a_parts;
  for (int k = warp; k < nd; k += nw) {
    const int n = P.alive != nullptr ? P.alive[k] : k;
    if ((unsigned)n >= (unsigned)N) {
      if (lane == 0) atomicExch(P.status, (int32_t)VCAS_ERR_BAD_ARG);
      continue;
    }
    const float s = datum_sqnorm_warp(P.a + (size_t)n * len, len, lane);
    if (lane == 0) P.g[n] = sqrtf(s);
  }
  __syncthreads();
  if (P.p_in != nullptr) {
    for (int n = tid; n < N; n += nt) P.p[n] = P.p_in[n];
  } else if (!capped_prop_block(P.g, N, (double)N * (double)P.rho, P.p, &sc)) {
    if (tid == 0) atomicExch(P.status, (int32_t)VCAS_ERR_INTERNAL);
  }
  __syncthreads();
  for (int n = tid; n < N; n += nt) {
    const float pn = P.p[n];
    P.scaleA[n] = bernoulli_keep(pn, P.seed, 0u, (uint64_t)n) ? 1.0f / pn : 0.f;
  }
  __syncthreads();
  const int cntA = block_compact(N, [&](int n) { return P.scaleA[n] > 0.f; },
                                 [&](int n, int pos) { P.idxA[pos] = n; if (P.kept_out != nullptr) P.kept_out[pos] = n; },
                                 &sc);
  block_compact(N, [&](int n) { return !(P.scaleA[n] > 0.f); }, [&](int n, int pos) { P.dropA[pos] = n; }, &sc);
  if (tid == 0) {
    P.counts[0] = cntA;
    if (P.kept_cnt_out != nullptr) *P.kept_cnt_out = cntA;
  }
}

// ------------------------------------------------------------------------------ SampleW
// How q follows from a row's score once sample_w_kernel has run: fix[1] = mode, fix[0] = c.
constexpr int Q_ZERO = 0;     // nothing to keep (no score is positive, or the budget is 0)
constexpr int Q_ONES = 1;     // the budget covers every positive score: q = [w > 0]
constexpr int Q_CAPPED = 2;   // q = min(1, c w)
constexpr int Q_GIVEN = 3;    // q is read from the caller's q_in

__device__ __forceinline__ float q_of(int mode, float c, float w, const float* q_in, int r) {
  if (mode == Q_CAPPED) {
    if (!(w > 0.f)) return 0.f;
    const float cx = c * w;
    return cx >= 1.0f ? 1.f : cx;
  }
  if (mode == Q_ONES) return w > 0.f ? 1.f : 0.f;
  if (mode == Q_GIVEN) return q_in[r];
  return 0.f;
}
__device__ __forceinline__ bool row_kept(int sample_w, float q, uint32_t u) {
  return sample_w ? (q > 0.f && u < (uint32_t)floorf(q * 16777216.0f)) : true;
}

struct SampleWParams {
  const float* wc; const uint32_t* uc;     // compact scores and uniforms of the rows of kept data
  const float* q_in;
  const int32_t* idxA;
  int32_t* counts; int32_t* chunk_off; float* fix;
  double* acc; int32_t* status;
  int T;
  float nu;
  int sample_w, accumulate_vw;
  int smem_rows;                            // scores that fit the kernel's shared memory
};

struct WShared {
  float part_f[2][32];
  int part_i[2][32];
  int scan[33];
};

// Block-wide sum of one float and one int in a fixed order (lanes by shuffle tree, then the 32
// warp totals by the same tree, which every warp runs for itself so that one barrier suffices; the
// buffers alternate with `parity`, and a buffer is rewritten only after a later barrier).  fp32 on
// purpose: this is a single-CTA kernel, and double-precision arithmetic concentrated on one SM was
// measured to dominate its run time; a tree sum of non-negative fp32 terms is accurate to about
// 1e-6, inside the 2e-5 the probabilities are specified to.
__device__ __forceinline__ void fast_sum(float& s, int& c, WShared* sh, int parity) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  s = warp_sum(s);
  c = __reduce_add_sync(0xffffffffu, c);
  if (lane == 0) { sh->part_f[parity][warp] = s; sh->part_i[parity][warp] = c; }
  __syncthreads();
  s = warp_sum(sh->part_f[parity][lane]);
  c = __reduce_add_sync(0xffffffffu, sh->part_i[parity][lane]);
}

// SampleW's single-CTA part (Sec. 4.2, Eq. 3).  The n = T * (#kept data) scores sit in shared memory (in
// global memory beyond smem_rows: same code, slower loads).  1. c with sum_r min(1, c w_r) = nu * n by
// water-filling: every round is one pass over the scores and one block-wide sum.  2. Eq. 3 at these
// probabilities (probe only).  3. The number of kept rows in every chunk of 32 rows, and the exclusive
// prefix sums of these counts: emit_pack_kernel then places every chunk's rows without looking at others.
__global__ void __launch_bounds__(SAMPLER_THREADS) sample_w_kernel(SampleWParams P) {
  extern __shared__ __align__(16) float s_w[];
  __shared__ WShared sh;
  pdl_wait();      // the scores come from the kernel before this one
  pdl_trigger();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int cntA = P.counts[0];
  const int T = P.T;
  const int n = cntA * T;
  const bool in_smem = n <= P.smem_rows;
  if (in_smem) {
    const int n4 = n >> 2;
    for (int i = tid; i < n4; i += SAMPLER_THREADS)
      reinterpret_cast<float4*>(s_w)[i] = reinterpret_cast<const float4*>(P.wc)[i];
    for (int i = (n4 << 2) + tid; i < n; i += SAMPLER_THREADS) s_w[i] = P.wc[i];
    __syncthreads();
  }
  const float* w = in_smem ? s_w : P.wc;

  int mode = Q_GIVEN;
  float c = 0.f;
  if (P.q_in == nullptr) {
    const float budget = P.nu * (float)T * (float)cntA;
    float S = 0.f;
    int nz = 0;
    for (int i = tid; i < n; i += SAMPLER_THREADS) {
      const float x = w[i];
      if (x > 0.f) { S += x; ++nz; }
    }
    int parity = 0;
    fast_sum(S, nz, &sh, parity); parity ^= 1;
    if (nz == 0 || budget <= 0.f) {
      mode = Q_ZERO;
    } else if ((float)nz <= budget) {
      mode = Q_ONES;
    } else {
      mode = Q_CAPPED;
      c = budget / S;
      int k = 0;
      bool converged = false;
      for (int iter = 0; iter < WATER_ROUNDS; ++iter) {
        float Su = 0.f;
        int ks = 0;
        for (int i = tid; i < n; i += SAMPLER_THREADS) {
          const float x = w[i];
          if (x > 0.f) {
            if (c * x >= 1.0f) ++ks; else Su += x;
          }
        }
        fast_sum(Su, ks, &sh, parity); parity ^= 1;
        if (ks == k) { converged = true; break; }
        k = ks;
        if (Su > 0.f) {
          const float cn = (budget - (float)k) / Su;
          c = cn > c ? cn : c;
        }
      }
      if (!converged && tid == 0) atomicExch(P.status, (int32_t)VCAS_ERR_INTERNAL);
    }
  }
  __syncthreads();      // the reduction buffers are free again

  if (P.accumulate_vw) {      // Eq. 3 at these probabilities
    float vw = 0.f;
    int dummy = 0;
    for (int i = tid; i < n; i += SAMPLER_THREADS) {
      const int k = i / T;
      const float x = w[i];
      const float q = q_of(mode, c, x, P.q_in, P.q_in != nullptr ? P.idxA[k] * T + (i - k * T) : 0);
      if (q > 0.f) vw += (1.0f - q) / q * x * x;
    }
    fast_sum(vw, dummy, &sh, 0);
    if (tid == 0) P.acc[1] += (double)vw;
    __syncthreads();
  }

  // kept rows per chunk of 32 compact rows: chunk_off[ch] = count for now.  A warp takes four chunks at a time
  // and issues their loads together (one memory latency per four chunks instead of one per chunk).
  const int nchunks = (n + 31) >> 5;
  for (int ch0 = warp; ch0 < nchunks; ch0 += 4 * (SAMPLER_THREADS / 32)) {
    float wv[4];
    uint32_t uv[4];
#pragma unroll
    for (int k4 = 0; k4 < 4; ++k4) {
      const int i = ((ch0 + k4 * (SAMPLER_THREADS / 32)) << 5) + lane;
      wv[k4] = i < n ? w[i] : 0.f;
      uv[k4] = (i < n && P.sample_w) ? __ldg(P.uc + i) : 0u;
    }
#pragma unroll
    for (int k4 = 0; k4 < 4; ++k4) {
      const int ch = ch0 + k4 * (SAMPLER_THREADS / 32);
      if (ch >= nchunks) break;                    // warp-uniform
      const int i = (ch << 5) + lane;
      bool keep = false;
      if (i < n) {
        const int k = i / T;
        const float q = q_of(mode, c, wv[k4], P.q_in, P.q_in != nullptr ? P.idxA[k] * T + (i - k * T) : 0);
        keep = row_kept(P.sample_w, q, uv[k4]);
      }
      const unsigned b = __ballot_sync(0xffffffffu, keep);
      if (lane == 0) P.chunk_off[ch] = __popc(b);
    }
  }
  __syncthreads();
  // exclusive prefix sums over the chunk counts: every thread owns a contiguous segment
  const int seg = (nchunks + SAMPLER_THREADS - 1) / SAMPLER_THREADS;
  const int lo = tid * seg, hi = min(nchunks, lo + seg);
  int mine = 0;
  for (int ch = lo; ch < hi; ++ch) mine += P.chunk_off[ch];
  int incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) sh.scan[warp] = incl;
  __syncthreads();
  const int wt = sh.scan[lane];
  int base = incl - mine + __reduce_add_sync(0xffffffffu, lane < warp ? wt : 0);
  const int total = __reduce_add_sync(0xffffffffu, wt);
  for (int ch = lo; ch < hi; ++ch) {
    const int cnt = P.chunk_off[ch];
    P.chunk_off[ch] = base;
    base += cnt;
  }
  if (tid == 0) {
    P.counts[1] = total;
    P.fix[0] = c;
    P.fix[1] = (float)mode;
  }
}

struct EmitParams {
  const float* wc; const uint32_t* uc;
  const float* q_in;
  const float* scaleA;
  const int32_t* idxA; const int32_t* dropA;
  const int32_t* counts; const int32_t* chunk_off; const float* fix;
  float* w; float* q; float* scaleW; int32_t* idxW;
  const __nv_bfloat16* dY; const __nv_bfloat16* X;       // operands to pack
  __nv_bfloat16* packG; __nv_bfloat16* packX;            // compact operands (nullptr: no packing)
  int N, T, d_in, d_out;
  int sample_w;
  int parts;                                             // CTAs that share the packing of one chunk's rows
};

// Row k of packG = scaleW[k] * dY[idxW[k]] (G_tilde of Sec. 4.2, rounded to bf16), row k of packX = X[idxW[k]].
__device__ __forceinline__ uint4 scale8(const uint4& v, float sc) {
  const uint32_t u[4] = {v.x, v.y, v.z, v.w};
  uint32_t o[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const __nv_bfloat162 t = __floats2bfloat162_rn(sc * __uint_as_float(u[e] << 16), sc * __uint_as_float(u[e] & 0xffff0000u));
    o[e] = *reinterpret_cast<const uint32_t*>(&t);
  }
  return make_uint4(o[0], o[1], o[2], o[3]);
}
// One CTA per (chunk of 32 compact rows, part) (grid-strided): the chunk's kept rows go to positions
// chunk_off[ch]... of the ascending kept-row list with their rescale factors 1/(p_n q_r); q and w are written by
// global row (by part 0); the operands of the chunk's kept rows j with j % parts == part are packed for the dW
// product.  The rows of dropped data get w = q = 0, and the compact operands are padded with zero rows to a
// multiple of 64 (the product's last k-block then adds nothing).
constexpr int EMIT_THREADS = 256;
__global__ void __launch_bounds__(EMIT_THREADS) emit_pack_kernel(EmitParams P) {
  __shared__ int s_r[32], s_pos[32], s_cnt;
  __shared__ float s_sc[32];
  pdl_wait();      // c and the chunk offsets come from the kernel before this one
  pdl_trigger();   // the dW product kernel may set itself up; it waits for this grid before loading
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int cntA = P.counts[0], cntW = P.counts[1];
  const int T = P.T;
  const int n = cntA * T;
  const float c = P.fix[0];
  const int mode = (int)P.fix[1];
  const int nchunks = (n + 31) >> 5;
  const bool pack = P.packG != nullptr;
  const int parts = pack ? P.parts : 1;
  for (int u = blockIdx.x; u < nchunks * parts; u += gridDim.x) {
    const int ch = u / parts, part = u - ch * parts;
    if (warp == 0) {
      const int i = (ch << 5) + lane;
      bool keep = false;
      float q = 0.f, wv = 0.f, sa = 0.f;
      int r = 0;
      if (i < n) {
        const int k = i / T;
        const int nd = P.idxA[k];
        r = nd * T + (i - k * T);
        wv = P.wc[i];
        q = q_of(mode, c, wv, P.q_in, r);
        keep = row_kept(P.sample_w, q, P.sample_w ? P.uc[i] : 0u);
        sa = P.scaleA[nd];
        if (part == 0) { P.w[r] = wv; P.q[r] = q; }
      }
      const unsigned b = __ballot_sync(0xffffffffu, keep);
      if (keep) {
        const int j = __popc(b & ((1u << lane) - 1u));
        const int pos = P.chunk_off[ch] + j;
        const float sc = P.sample_w ? sa / q : sa;
        if (part == 0) { P.idxW[pos] = r; P.scaleW[pos] = sc; }
        s_r[j] = r; s_pos[j] = pos; s_sc[j] = sc;
      }
      if (lane == 0) s_cnt = __popc(b);
    }
    if (pack) {
      __syncthreads();
      // This part's rows j = part, part + parts, ...  A row's 16-byte pieces (first those of dY, then those of X)
      // are cut into segments of 128; a warp takes (row, segment) items in turn and moves a segment with four
      // independent loads per lane in flight.  One integer division per 2 KB moved, none per piece.
      const int m = s_cnt;
      const int mp = m > part ? (m - part + parts - 1) / parts : 0;
      const int vo = P.d_out / 8, vt = vo + P.d_in / 8;
      const int nseg = (vt + 127) >> 7;
      for (int item = warp; item < mp * nseg; item += EMIT_THREADS / 32) {
        const int jj = item / nseg, seg = item - jj * nseg;
        const int j = part + jj * parts;
        const size_t r = (size_t)s_r[j], pos = (size_t)s_pos[j];
        const float sc = s_sc[j];
        const uint4* srcG = reinterpret_cast<const uint4*>(P.dY + r * P.d_out);
        const uint4* srcX = reinterpret_cast<const uint4*>(P.X + r * P.d_in) - vo;
        uint4* dstG = reinterpret_cast<uint4*>(P.packG + pos * P.d_out);
        uint4* dstX = reinterpret_cast<uint4*>(P.packX + pos * P.d_in) - vo;
        const int p0 = (seg << 7) + lane;
        uint4 v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int piece = p0 + 32 * q;
          if (piece < vt) v[q] = __ldg(piece < vo ? srcG + piece : srcX + piece);
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int piece = p0 + 32 * q;
          if (piece < vt) {
            if (piece < vo) dstG[piece] = scale8(v[q], sc);
            else dstX[piece] = v[q];
          }
        }
      }
      __syncthreads();
    }
  }
  // rows of dropped data
  const int ndrop_rows = (P.N - cntA) * T;
  for (int i = blockIdx.x * EMIT_THREADS + tid; i < ndrop_rows; i += gridDim.x * EMIT_THREADS) {
    const int k = i / T;
    const int r = P.dropA[k] * T + (i - k * T);
    P.w[r] = 0.f;
    P.q[r] = 0.f;
  }
  // zero rows up to the next multiple of 64
  if (pack) {
    const int padded = (cntW + 63) / 64 * 64;
    for (int k = cntW + (int)blockIdx.x; k < padded; k += gridDim.x) {
      for (int i = tid; i < P.d_out / 8; i += EMIT_THREADS)
        reinterpret_cast<uint4*>(P.packG + (size_t)k * P.d_out)[i] = make_uint4(0u, 0u, 0u, 0u);
      for (int i = tid; i < P.d_in / 8; i += EMIT_THREADS)
        reinterpret_cast<uint4*>(P.packX + (size_t)k * P.d_in)[i] = make_uint4(0u, 0u, 0u, 0u);
    }
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

constexpr int SAMPLE_W_SMEM_ROWS = 56 * 1024;     // 224 KB of scores

}  // namespace

cudaError_t launch_sample_a(Handle* h, const SamplerArgs& a, bool programmatic, cudaStream_t st) {
  const Workspace& ws = h->ws;
  const vcas_layer_desc& d = h->desc;
  SampleAParams P;
  P.a = a.a_in != nullptr ? a.a_in : ws.a;
  P.a_parts = a.a_in != nullptr ? a.a_parts : 1;
  P.alive = a.alive; P.alive_cnt = a.alive_cnt;
  P.N = d.N; P.T = d.T; P.rho = a.rho; P.p_in = a.p_in; P.seed = a.seed;
  P.g = ws.g; P.p = ws.p; P.scaleA = ws.scaleA; P.idxA = ws.idxA; P.dropA = ws.dropA; P.counts = ws.counts;
  P.kept_out = a.kept_out; P.kept_cnt_out = a.kept_cnt_out;
  P.status = ws.status;
  cudaError_t e;
  if (d.N <= 32)
    e = launch_maybe_after(programmatic, sample_a_kernel<1>, dim3(1), dim3(SAMPLE_A_THREADS), 0, st, P);
  else if (d.N <= WARP_MAX_N)
    e = launch_maybe_after(programmatic, sample_a_kernel<32>, dim3(1), dim3(SAMPLE_A_THREADS), 0, st, P);
  else
    e = launch_maybe_after(programmatic, sample_a_big_kernel, dim3(1), dim3(SAMPLER_THREADS), 0, st, P);
  h->launches += 1;
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_sample_w(Handle* h, const SamplerArgs& a, cudaStream_t st) {
  static std::atomic<bool> attr_set[64];
  const Workspace& ws = h->ws;
  const vcas_layer_desc& d = h->desc;
  const long R = (long)d.N * d.T;
  // shared memory for the scores: enough for every row when that fits, else the kernel reads global memory
  // whenever the kept rows exceed it
  int rows = (int)(R < SAMPLE_W_SMEM_ROWS ? R : SAMPLE_W_SMEM_ROWS);
  rows = (rows + 3) & ~3;
  const size_t smem = (size_t)rows * sizeof(float);
  if (smem > 48 * 1024) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_set[dev].load(std::memory_order_acquire)) {
      e = cudaFuncSetAttribute(sample_w_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               SAMPLE_W_SMEM_ROWS * (int)sizeof(float));
      if (e != cudaSuccess) return e;
      attr_set[dev].store(true, std::memory_order_release);
    }
  }
  SampleWParams P;
  P.wc = ws.wc; P.uc = ws.uc; P.q_in = a.q_in; P.idxA = ws.idxA;
  P.counts = ws.counts; P.chunk_off = ws.chunk_off; P.fix = ws.fix; P.acc = ws.acc; P.status = ws.status;
  P.T = d.T; P.nu = a.nu; P.sample_w = a.sample_w; P.accumulate_vw = a.accumulate_vw;
  P.smem_rows = rows;
  const cudaError_t e = launch_after(sample_w_kernel, dim3(1), dim3(SAMPLER_THREADS), smem, st, P);
  h->launches += 1;
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_emit_pack(Handle* h, const void* dY, const void* X, const SamplerArgs& a, bool pack, cudaStream_t st) {
  const Workspace& ws = h->ws;
  const vcas_layer_desc& d = h->desc;
  EmitParams P;
  P.wc = ws.wc; P.uc = ws.uc; P.q_in = a.q_in; P.scaleA = ws.scaleA; P.idxA = ws.idxA; P.dropA = ws.dropA;
  P.counts = ws.counts; P.chunk_off = ws.chunk_off; P.fix = ws.fix;
  P.w = ws.w; P.q = ws.q; P.scaleW = ws.scaleW; P.idxW = ws.idxW;
  P.dY = (const __nv_bfloat16*)dY; P.X = (const __nv_bfloat16*)X;
  P.packG = pack ? ws.packG : nullptr;
  P.packX = pack ? ws.packX : nullptr;
  P.N = d.N; P.T = d.T; P.d_in = d.d_in; P.d_out = d.d_out;
  P.sample_w = a.sample_w;
  // The number of chunks with kept rows is only known on the device.  With packing, the grid has eight CTAs per
  // SM and the rows of a chunk are shared among as many CTAs as the expected number of chunks leaves room for.
  const long R = (long)d.N * d.T;
  const long cap = (long)(h->num_sms > 0 ? h->num_sms : 148) * 8;
  long expected = (long)((double)a.rho * (double)R / 32.0) + 1;
  long parts = pack ? cap / expected : 1;
  if (parts < 1) parts = 1;
  if (parts > 16) parts = 16;
  P.parts = (int)parts;
  long blocks = ((R + 31) / 32) * parts;
  if (blocks > cap) blocks = cap;
  const cudaError_t e = launch_after(emit_pack_kernel, dim3((unsigned)blocks), dim3(EMIT_THREADS), 0, st, P);
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
