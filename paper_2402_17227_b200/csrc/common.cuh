// Internal declarations shared by the kernels of libvcas (device helpers, workspace layout).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "vcas.h"

namespace vcas {

// ---------------------------------------------------------------------------------------
// Workspace: one allocation per handle, carved into these arrays at vcas_create.
// ---------------------------------------------------------------------------------------
struct Workspace {
  // scores (Sec. 4.1, 4.2)
  float* a;        // [R]  ||dY_r||^2 (rows of data that may be non-zero)
  float* wc;       // [R]  leverage scores ||G_hat_r|| ||X_r|| of the rows of kept data, compact: entry k*T + t is
                   //      token t of the k-th kept datum
  uint32_t* uc;    // [R]  SampleW's 24-bit uniform of those rows, same order
  float* g;        // [N]  ||G_n||_F
  float* p;        // [N]  SampleA keep probabilities
  float* w;        // [R]  leverage scores by global row (0 on rows of dropped data)
  float* q;        // [R]  SampleW keep probabilities by global row
  float* scaleA;   // [N]  1/p_n for kept data, 0 for dropped data
  float* scaleW;   // [R]  1/(p_n q_r) per compacted row
  float* sorted;   // [N]  data norms in descending order (Eq. 4)
  int32_t* idxA;   // [N]  kept data, ascending
  int32_t* dropA;  // [N]  dropped data, ascending
  int32_t* idxW;   // [R]  kept rows, ascending
  int32_t* chunk_off;  // [R/32 + 2] position in idxW of the first kept row of every chunk of 32 compact rows
  float* fix;      // [4]  0: the factor c of q = min(1, c w) found by the water-filling, 1: mode (see sample_w_kernel)
  int32_t* counts; // [8]  0: cntA, 1: cntW, 2: R (constant, for dense launches), 4: reduction ticket
  int32_t* status; // [1]  device status word
  double* acc;     // [16] probe accumulators (0: V_act, 1: V_w, 2: p_lo, 3: p_hi, 4: V_s)
  double* partial; // [PARTIAL_SLOTS] block partial sums of the probe reductions
  // compact operands of the weight-gradient product (tensor path)
  __nv_bfloat16* packG;  // [R_pad, d_out]
  __nv_bfloat16* packX;  // [R_pad, d_in]
  float* partial_tiles;  // [3][max_units][128 * 256] fp32 partial tiles of a split contraction: dX, dW, and the dW
                         // of the workspace's second set (see Handle::ws2)
  int32_t* tickets;      // [3][2 * max_units]: slices stored, slices finished, per tile
  int32_t* sched;        // [3][2]: next work item and finished CTAs of an unsliced product (dynamic tile order)
  // probe buffers (App. D: the exact gradient, its running mean and running squared deviation)
  float* Gs;       // [d_out, d_in]
  float* Gact;     // [d_out, d_in]
  float* mean;     // [d_out, d_in]
  float* m2;       // [d_out, d_in]
};

constexpr int PARTIAL_SLOTS = 4096;

// Tiling of one tensor-core product: tile width, slices of the contraction, and tile height
// (mh: 1 = 128-row tiles, 2 = 256-row tiles, 3 = 256-row tiles for whole waves + 128-row tiles for the rest).
struct Plan { int bn, split, mh; };
constexpr int PLAN_KEY_INTS = 9;
constexpr int PLAN_CACHE = 64;

struct Handle {
  vcas_layer_desc desc;
  vcas_config cfg;
  int device;
  int num_sms;
  bool tensor_path;
  int R_pad;
  int max_units;   // capacity of the split-contraction workspace, in (tile, slice) units
  void* base;
  size_t bytes;
  Workspace ws;
  // Second set of everything a sampled dW chain writes (sampler outputs, packed operands, G_act, counters,
  // accumulators, block partials, split-contraction slot); the row norms and G_s are shared.  The variance
  // probe runs its SampleA draws alternately on the two sets and two streams.
  Workspace ws2;
  uint64_t launches;
  // second stream and fork/join events: the dW branch (pack + product) runs beside the dX product
  cudaStream_t side_stream;
  cudaEvent_t ev_fork, ev_join;
  bool join_pending;   // the last call left its side-stream branch unjoined (vcas_chain_args::defer_join)
  // optional stage timing (vcas_set_profiling): rings of CUDA events around the stages
  bool prof_enabled;
  cudaEvent_t* ev;        // [PROF_RING][8]: stage boundaries of a sampled call (see vcas_stage_times)
  cudaEvent_t* ev_dense;  // [PROF_RING][4]: stage boundaries of a dense call
  int prof_calls, prof_dense_calls;
  // tuning overrides (vcas_set_tuning); 0 = choose automatically
  int tune_dx_tile_n, tune_dw_tile_n, tune_dx_split_k, tune_dw_split_k;
  // the last pair of plans made for the two products of a call, and what it was made for (plan_products)
  bool plan_valid;
  int plan_key[PLAN_KEY_INTS];
  Plan plan_dx, plan_dw;
  // ... and the pairs made before it (a handle shared by the layers of a stack sees a few dozen different
  // expected counts in turn): a small table replaced in round-robin order
  int plan_cache_key[PLAN_CACHE][PLAN_KEY_INTS];
  Plan plan_cache_dx[PLAN_CACHE], plan_cache_dw[PLAN_CACHE];
  int plan_cache_used, plan_cache_next;
  // the probe's sample of the parameters (App. D): sub_k rows of the parameter gradient (0: all of them)
  int sub_k;
  int32_t* sub_rows;   // [SUB_MAX] device, ascending
  void* sub_dY;        // [R, SUB_MAX] those columns of the current batch's dY, compact
  unsigned long long wait_limit_ns;   // bound of every device-side wait (default 2 s)
  int stall_once;    // test hook, see vcas_set_wait_limit
  int tune_dx_tile_m, tune_dw_tile_m;   // per product; 0 auto, 1: 128-row tiles only, 2: 256-row tiles whenever the width is 256, 3: 256-row tiles for
                     // whole waves of CTAs and 128-row tiles, their contraction sliced, for the rest
};
constexpr int PROF_RING = 2048;
constexpr int SUB_MAX = 256;     // most parameter rows the probe's subsample may hold

// ---------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplies.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t philox_word0(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                 uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  return c0;
}

// keep iff the 24-bit uniform of (seed, sampler, idx) is below floor(p * 2^24)
__device__ __forceinline__ bool bernoulli_keep(float p, uint64_t seed, uint32_t sampler, uint64_t idx) {
  const uint32_t u = philox_word0((uint32_t)idx, (uint32_t)(idx >> 32), sampler, 0u,
                                  (uint32_t)seed, (uint32_t)(seed >> 32)) >> 8;
  const uint32_t thr = (uint32_t)floorf(p * 16777216.0f);
  return u < thr;
}

// Programmatic dependent launch: a kernel launched with launch_after() may start while the kernel
// before it in the stream is still running; it must call pdl_wait() before it touches anything that
// kernel writes (the wait returns once that grid has completed and its writes are visible).
// pdl_trigger() in the earlier kernel lets the dependent grid be scheduled from that point on.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// programmatic = false: an ordinary launch (for a kernel whose inputs arrive through an event from
// another stream rather than from the kernel before it in its own stream).
template <typename... KArgs, typename... Args>
cudaError_t launch_maybe_after(bool programmatic, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                               cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = programmatic ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
template <typename... KArgs, typename... Args>
cudaError_t launch_after(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  return launch_maybe_after(true, kernel, grid, block, smem, st, args...);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ---------------------------------------------------------------------------------------
// SampleA inside one warp (Sec. 4.1), shared by the sampling kernel and the tail of the row-norm kernel.
// ---------------------------------------------------------------------------------------
// Sum of the T squared row norms of one datum by one warp, in a fixed order, result in every lane.  Up to
// sixteen independent loads per lane are in flight (a dependent chain of T/32 loads would cost a memory
// latency each).  The loads bypass L1: the values may have been written by other SMs of the same grid.
__device__ __forceinline__ float datum_sqnorm_warp(const float* an, int T, int lane) {
  float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
  int t = lane;
  for (; t + 480 < T; t += 512) {
    float v[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) v[k] = __ldcg(an + t + 32 * k);
#pragma unroll
    for (int k = 0; k < 16; k += 4) { s0 += v[k]; s1 += v[k + 1]; s2 += v[k + 2]; s3 += v[k + 3]; }
  }
  for (; t + 96 < T; t += 128) {
    s0 += __ldcg(an + t); s1 += __ldcg(an + t + 32); s2 += __ldcg(an + t + 64); s3 += __ldcg(an + t + 96);
  }
  for (; t < T; t += 32) s0 += __ldcg(an + t);
  return warp_sum((s0 + s1) + (s2 + s3));
}

// Keep probabilities proportional to v, capped at 1, summing to `budget` (the minimiser of
// sum (1-p)/p v^2 under that budget): p = min(1, c v).  The saturated set is grown from empty; c only
// increases, so the iteration reaches the least fixed point, which is the unique solution.  Value i of the
// array sits in lane i % 32, slot i / 32 of ONE warp; p is returned in place of v.
template <int SLOTS>
__device__ __forceinline__ void capped_prop_warp(float (&v)[SLOTS], float budget) {
  float S = 0.f;
  int nz = 0;
#pragma unroll
  for (int j = 0; j < SLOTS; ++j)
    if (v[j] > 0.f) { S += v[j]; ++nz; }
  S = warp_sum(S);
  nz = __reduce_add_sync(0xffffffffu, nz);
  if (nz == 0 || budget <= 0.f) {
#pragma unroll
    for (int j = 0; j < SLOTS; ++j) v[j] = 0.f;
    return;
  }
  if ((float)nz <= budget) {
#pragma unroll
    for (int j = 0; j < SLOTS; ++j) v[j] = v[j] > 0.f ? 1.f : 0.f;
    return;
  }
  float c = budget / S;
  int k = 0;
  for (int iter = 0; iter < 128; ++iter) {
    float Su = 0.f;
    int ks = 0;
#pragma unroll
    for (int j = 0; j < SLOTS; ++j)
      if (v[j] > 0.f) {
        if (c * v[j] >= 1.0f) ++ks; else Su += v[j];
      }
    Su = warp_sum(Su);
    ks = __reduce_add_sync(0xffffffffu, ks);
    if (ks == k) break;
    k = ks;
    if (Su > 0.f) {
      const float cn = (budget - (float)k) / Su;
      c = cn > c ? cn : c;
    }
  }
#pragma unroll
  for (int j = 0; j < SLOTS; ++j) {
    float r = 0.f;
    if (v[j] > 0.f) {
      const float cx = c * v[j];
      r = cx >= 1.0f ? 1.f : cx;
    }
    v[j] = r;
  }
}

// Where SampleA's results go: the workspace arrays, and optionally shared-memory copies of p and 1/p.
struct SampleAOut {
  float* p; float* scaleA; int32_t* idxA; int32_t* dropA;
  int32_t* idx_copy;   // optional second copy of the kept list (handed to the next layer of a chain)
};

// SampleA over N <= 32 * SLOTS data by one full warp: keep probabilities from the data norms g (or the
// given p_in), Philox masks (sampler 0), kept and dropped lists in ascending order.  Returns the number
// of kept data in every lane.
template <int SLOTS>
__device__ __forceinline__ int sample_a_warp(const float* g, int N, float rho, const float* p_in, uint64_t seed,
                                             const SampleAOut& o, int lane) {
  float v[SLOTS];
  if (p_in != nullptr) {
#pragma unroll
    for (int j = 0; j < SLOTS; ++j) { const int n = lane + 32 * j; v[j] = n < N ? p_in[n] : 0.f; }
  } else {
#pragma unroll
    for (int j = 0; j < SLOTS; ++j) { const int n = lane + 32 * j; v[j] = n < N ? g[n] : 0.f; }
    capped_prop_warp<SLOTS>(v, (float)N * rho);
  }
  int kept_before = 0, drop_before = 0;
#pragma unroll
  for (int j = 0; j < SLOTS; ++j) {
    const int n = lane + 32 * j;
    const bool in = n < N;
    const bool keep = in && bernoulli_keep(v[j], seed, 0u, (uint64_t)n);
    const unsigned bk = __ballot_sync(0xffffffffu, keep);
    const unsigned bd = __ballot_sync(0xffffffffu, in && !keep);
    const unsigned lower = (1u << lane) - 1u;
    if (in) {
      const float sc = keep ? 1.0f / v[j] : 0.f;
      o.p[n] = v[j];
      o.scaleA[n] = sc;
      if (keep) {
        const int pos = kept_before + __popc(bk & lower);
        o.idxA[pos] = n;
        if (o.idx_copy != nullptr) o.idx_copy[pos] = n;
      } else {
        o.dropA[drop_before + __popc(bd & lower)] = n;
      }
    }
    kept_before += __popc(bk);
    drop_before += __popc(bd);
  }
  return kept_before;
}

// SampleA runs inside one warp for up to this many data (32 lanes x 32 slots); larger batches take a
// block-wide kernel.
constexpr int WARP_MAX_N = 1024;

// ---------------------------------------------------------------------------------------
// Launchers (one per .cu file).  All enqueue on `st` and return a cudaError_t.
// ---------------------------------------------------------------------------------------
struct SamplerArgs {
  float rho, nu;
  uint64_t seed;
  const float* p_in;
  const float* q_in;
  int sample_w;      // 1: SampleW mask applied; 0: all rows of kept data survive (probe)
  int accumulate_vw; // 1: add Eq. 3 at ratio nu to acc[1]
  // Scoring handed down a stack of layers (the gradient gets sparser from layer to layer, Sec. 4):
  const float* a_in;        // row square-norms of dY made by its producer, a_r = sum of a_parts consecutive floats
  int a_parts;              // (nullptr: computed here from dY, one float per row)
  const int32_t* alive;     // data whose rows of dY may be non-zero (device list, ascending) and its length;
  const int32_t* alive_cnt; // every other datum is known to be zero and is never read (nullptr: all N data)
  int32_t* kept_out;        // optional copies of this call's kept-data list and count (device)
  int32_t* kept_cnt_out;
};
inline SamplerArgs sampler_args(float rho, float nu, uint64_t seed) {
  SamplerArgs a = {};
  a.rho = rho; a.nu = nu; a.seed = seed; a.sample_w = 1; a.a_parts = 1;
  return a;
}
// a_r = ||dY_r||^2 on the rows of alive data (nothing to do when the producer supplied them)
cudaError_t launch_rownorm_dy(Handle* h, const void* dY, const SamplerArgs& a, cudaStream_t st);
// row square-norms of a finished dX in the layout of the product kernels' partial sums (a_out_parts floats per
// row), for the products that do not emit them from their epilogue
cudaError_t launch_rownorm_out(Handle* h, const void* dX, float* a_out, cudaStream_t st);
// SampleA (Sec. 4.1): g, p, mask, kept / dropped lists, 1/p; programmatic: launched as a dependent of the
// kernel before it in the stream
cudaError_t launch_sample_a(Handle* h, const SamplerArgs& a, bool programmatic, cudaStream_t st);
// ||X_r|| on the rows of kept data, the leverage scores of G_hat and SampleW's uniforms, in compact order
cudaError_t launch_scores_x(Handle* h, const void* X, const SamplerArgs& a, bool programmatic, cudaStream_t st);
// SampleW (Sec. 4.2): the factor c of q = min(1, c w), the masks' counts per chunk of 32 compact rows
cudaError_t launch_sample_w(Handle* h, const SamplerArgs& a, cudaStream_t st);
// kept-row list, 1/(p q), q and w by global row and, with pack, the compact bf16 operands of the dW product
cudaError_t launch_emit_pack(Handle* h, const void* dY, const void* X, const SamplerArgs& a, bool pack, cudaStream_t st);
cudaError_t launch_mask_from_probs(Handle* h, const float* p, int n, uint64_t seed, int sampler,
                                   uint8_t* keep, int32_t* idx, int32_t* cnt, cudaStream_t st);

// fp32-FMA products
cudaError_t launch_fma_dx(Handle* h, const void* dY, const void* W, const float* scaleA,
                          const void* H, void* dX, cudaStream_t st);
cudaError_t launch_fma_dw(Handle* h, const void* dY, const void* X, const int32_t* idx,
                          const float* scale, const int32_t* cnt, float* dW, cudaStream_t st);

// tensor-core products
// spare_sms: SMs the persistent grid leaves free (for a kernel of another stream that must run beside it);
// pair_plan: the tiling chosen by plan_products for a call whose two products run at the same time
// (nullptr: chosen here, for this product alone)
// a_out: optional [R][a_out_parts(d_in)] partial row square-norms of the stored dX, written by the epilogue
// skip_dropped: the rows of dropped data are not written (a consumer with the kept-data list never reads them)
cudaError_t launch_umma_dx(Handle* h, const void* dY, const void* W, bool dense, float rho_hint,
                           const void* H, void* dX, float* a_out, bool skip_dropped, int spare_sms,
                           const Plan* pair_plan, cudaStream_t st);
inline int a_out_parts(int d_in) { return 2 * ((d_in + 255) / 256); }    // one per 256-column tile and epilogue group
// dW = A_rows^T B_rows over the first *cnt rows (A_rows [rows, d_out], B_rows [rows, d_in], bf16)
// cnt_hint: the expected *cnt, used on the host to pick the tiling
cudaError_t launch_umma_dw(Handle* h, const void* A_rows, const void* B_rows, int rows_capacity,
                           const int32_t* cnt, int cnt_hint, const Plan* pair_plan, float* dW, cudaStream_t st);
// Tilings of the dX and dW products of one call, chosen together because they share the SMs (cached in the
// handle until the expected kept counts or the tuning overrides change).
// row_norms_out: the dX product must emit row square-norms from its epilogue (unsliced 256-wide tiles only)
void plan_products(Handle* h, bool dense, float rho_hint, int cnt_hint, int spare_sms, bool row_norms_out, Plan* dx,
                   Plan* dw);

// LayerNorm backward over the rows of kept data (after SampleA): dX, optional row square-norms of dX, dgamma, dbeta
cudaError_t launch_layernorm_bwd(Handle* h, const void* X, const void* gamma, const void* dY, float eps, void* dX,
                                 float* a_out, bool skip_dropped, float* dgamma, float* dbeta, float rho_hint,
                                 cudaStream_t st);

// probe reductions
cudaError_t launch_probe_reset(Handle* h, cudaStream_t st);
cudaError_t launch_probe_welford(Handle* h, int i, cudaStream_t st);
cudaError_t launch_probe_sqdiff(Handle* h, cudaStream_t st);
cudaError_t launch_probe_sparsity(Handle* h, double s_lo, double s_hi, cudaStream_t st);
// adds the accumulators of the second set to the first (fixed order), then Alg. 1's averages
// scale: factor of V_s and V_act (d_out / sampled parameter rows)
cudaError_t launch_probe_finalize(Handle* h, int M, double scale, float* V_s, float* V_act, float* V_w,
                                  float* p_lo, float* p_hi, cudaStream_t st);
// out[r, c] = in[r, cols[c]] for the R rows of a [R, d] matrix of the layer dtype
cudaError_t launch_gather_cols(Handle* h, const void* in, int d, const int32_t* cols, int k, void* out, cudaStream_t st);
// k of the d_out output features chosen by Philox (ascending) into rows; scratch_u, scratch_flag: d_out words each
cudaError_t launch_param_subset(Handle* h, int k, uint64_t seed, uint32_t* scratch_u, int32_t* scratch_flag,
                                int32_t* rows, cudaStream_t st);

}  // namespace vcas
