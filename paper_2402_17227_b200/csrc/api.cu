// C ABI of libvcas (see vcas.h): argument checks, workspace, and the order in which the
// kernels of Eq. 2 and Alg. 1 are enqueued.  No arithmetic of the method happens on the host
// except vcas_update_ratios, which the paper defines on a handful of scalars.
#include <new>

#include "common.cuh"

using namespace vcas;

namespace {

inline Handle* H(vcas_handle h) { return reinterpret_cast<Handle*>(h); }
inline cudaStream_t S(vcas_stream s) { return reinterpret_cast<cudaStream_t>(s); }

size_t align_up(size_t x) { return (x + 255) & ~(size_t)255; }

template <typename T>
T* carve(uint8_t*& cur, size_t count) {
  T* p = reinterpret_cast<T*>(cur);
  cur += align_up(count * sizeof(T));
  return p;
}

bool ratio_ok(float r) { return r > 0.f && r <= 1.f; }

#define VCAS_CUDA(expr)                         \
  do {                                          \
    if ((expr) != cudaSuccess) return VCAS_ERR_CUDA; \
  } while (0)

// Lays the workspace out from `base` (base == nullptr: only measures).
size_t layout(Handle* h, uint8_t* base) {
  const vcas_layer_desc& d = h->desc;
  const size_t N = d.N, R = (size_t)d.N * d.T, DW = (size_t)d.d_out * d.d_in;
  uint8_t* cur = base;
  Workspace& w = h->ws;
  const size_t chunks = R / 32 + 2;
  w.a = carve<float>(cur, R);
  w.wc = carve<float>(cur, R);
  w.uc = carve<uint32_t>(cur, R);
  w.g = carve<float>(cur, N);
  w.p = carve<float>(cur, N);
  w.w = carve<float>(cur, R);
  w.q = carve<float>(cur, R);
  w.scaleA = carve<float>(cur, N);
  w.scaleW = carve<float>(cur, R);
  w.sorted = carve<float>(cur, N);
  w.idxA = carve<int32_t>(cur, N);
  w.dropA = carve<int32_t>(cur, N);
  w.idxW = carve<int32_t>(cur, R);
  w.chunk_off = carve<int32_t>(cur, chunks);
  w.fix = carve<float>(cur, 4);
  w.counts = carve<int32_t>(cur, 8);
  w.status = carve<int32_t>(cur, 1);
  w.acc = carve<double>(cur, 16);
  w.partial = carve<double>(cur, PARTIAL_SLOTS);
  if (h->tensor_path) {
    w.packG = carve<__nv_bfloat16>(cur, (size_t)h->R_pad * d.d_out);
    w.packX = carve<__nv_bfloat16>(cur, (size_t)h->R_pad * d.d_in);
    w.partial_tiles = carve<float>(cur, 3 * (size_t)h->max_units * 128 * 256);
    w.tickets = carve<int32_t>(cur, 6 * (size_t)h->max_units);
    w.sched = carve<int32_t>(cur, 8);
  } else {
    w.packG = nullptr;
    w.packX = nullptr;
    w.partial_tiles = nullptr;
    w.tickets = nullptr;
    w.sched = nullptr;
  }
  w.Gs = carve<float>(cur, DW);
  w.Gact = carve<float>(cur, DW);
  w.mean = carve<float>(cur, DW);
  w.m2 = carve<float>(cur, DW);
  // second set (variance probe): see Handle::ws2
  Workspace& v = h->ws2;
  v = w;
  v.wc = carve<float>(cur, R);
  v.uc = carve<uint32_t>(cur, R);
  v.g = carve<float>(cur, N);
  v.p = carve<float>(cur, N);
  v.w = carve<float>(cur, R);
  v.q = carve<float>(cur, R);
  v.scaleA = carve<float>(cur, N);
  v.scaleW = carve<float>(cur, R);
  v.idxA = carve<int32_t>(cur, N);
  v.dropA = carve<int32_t>(cur, N);
  v.idxW = carve<int32_t>(cur, R);
  v.chunk_off = carve<int32_t>(cur, chunks);
  v.fix = carve<float>(cur, 4);
  v.counts = carve<int32_t>(cur, 8);
  v.acc = carve<double>(cur, 16);
  v.partial = carve<double>(cur, PARTIAL_SLOTS);
  if (h->tensor_path) {
    v.packG = carve<__nv_bfloat16>(cur, (size_t)h->R_pad * d.d_out);
    v.packX = carve<__nv_bfloat16>(cur, (size_t)h->R_pad * d.d_in);
    v.partial_tiles = w.partial_tiles + (size_t)h->max_units * 128 * 256;   // dW slot of this set = third slot
    v.tickets = w.tickets + 2 * (size_t)h->max_units;
    v.sched = w.sched + 2;
  }
  v.Gact = carve<float>(cur, DW);
  h->sub_rows = carve<int32_t>(cur, SUB_MAX);
  h->sub_dY = carve<float>(cur, R * SUB_MAX * (d.dtype == VCAS_DTYPE_BF16 ? 2 : 4) / 4);
  return (size_t)(cur - base);
}

int copy_out(Handle* h, float* g, float* p, float* w, float* q, int32_t* idxA, int32_t* cntA, int32_t* idxW,
             int32_t* cntW, cudaStream_t st) {
  const size_t N = h->desc.N, R = (size_t)h->desc.N * h->desc.T;
  const Workspace& ws = h->ws;
  const cudaMemcpyKind k = cudaMemcpyDeviceToDevice;
  if (g) VCAS_CUDA(cudaMemcpyAsync(g, ws.g, N * sizeof(float), k, st));
  if (p) VCAS_CUDA(cudaMemcpyAsync(p, ws.p, N * sizeof(float), k, st));
  if (w) VCAS_CUDA(cudaMemcpyAsync(w, ws.w, R * sizeof(float), k, st));
  if (q) VCAS_CUDA(cudaMemcpyAsync(q, ws.q, R * sizeof(float), k, st));
  if (idxA) VCAS_CUDA(cudaMemcpyAsync(idxA, ws.idxA, N * sizeof(int32_t), k, st));
  if (cntA) VCAS_CUDA(cudaMemcpyAsync(cntA, ws.counts + 0, sizeof(int32_t), k, st));
  if (idxW) VCAS_CUDA(cudaMemcpyAsync(idxW, ws.idxW, R * sizeof(int32_t), k, st));
  if (cntW) VCAS_CUDA(cudaMemcpyAsync(cntW, ws.counts + 1, sizeof(int32_t), k, st));
  return VCAS_OK;
}

// SampleW, the kept-row list with its compact operands, and dW over those rows into `out`; follows SampleA
// on the workspace set that h->ws currently names.  first_programmatic: the first kernel is launched as a
// dependent of the kernel before it in `st` (false when its inputs arrive through an event).
int sample_w_and_dw(Handle* h, const void* X, const void* dY, const SamplerArgs& a, bool first_programmatic,
                    const Plan* plan, float* out, cudaStream_t st) {
  VCAS_CUDA(launch_scores_x(h, X, a, first_programmatic, st));
  VCAS_CUDA(launch_sample_w(h, a, st));
  VCAS_CUDA(launch_emit_pack(h, dY, X, a, h->tensor_path, st));
  if (h->tensor_path) {
    const float keep = a.sample_w ? a.rho * a.nu : a.rho;
    const int hint = (int)(keep * (float)(h->desc.N * h->desc.T)) + 1;
    VCAS_CUDA(launch_umma_dw(h, h->ws.packG, h->ws.packX, h->R_pad, h->ws.counts + 1, hint, plan, out, st));
  } else {
    VCAS_CUDA(launch_fma_dw(h, dY, X, h->ws.idxW, h->ws.scaleW, h->ws.counts + 1, out, st));
  }
  return VCAS_OK;
}

// A call that deferred its join left work on the side stream: everything that touches the handle's workspace
// or the outputs of that call waits for it first.
int join_pending(Handle* h, cudaStream_t st) {
  if (h->join_pending) {
    VCAS_CUDA(cudaStreamWaitEvent(st, h->ev_join, 0));
    h->join_pending = false;
  }
  return VCAS_OK;
}

// stage boundary k of the current sampled call (no-op unless profiling is on)
inline void mark(Handle* h, int k, cudaStream_t st) {
  if (h->prof_enabled && h->prof_calls < PROF_RING) cudaEventRecord(h->ev[h->prof_calls * 8 + k], st);
}
inline void mark_dense(Handle* h, int k, cudaStream_t st) {
  if (h->prof_enabled && h->prof_dense_calls < PROF_RING) cudaEventRecord(h->ev_dense[h->prof_dense_calls * 4 + k], st);
}

// plan: the tiling made for a call whose dX product runs beside it (nullptr: planned alone)
int dense_dw(Handle* h, const void* X, const void* dY, const Plan* plan, float* out, cudaStream_t st) {
  if (h->tensor_path) {
    VCAS_CUDA(launch_umma_dw(h, dY, X, h->desc.N * h->desc.T, h->ws.counts + 2, h->desc.N * h->desc.T, plan, out, st));
  } else {
    VCAS_CUDA(launch_fma_dw(h, dY, X, nullptr, nullptr, h->ws.counts + 2, out, st));
  }
  return VCAS_OK;
}

}  // namespace

extern "C" {

int vcas_version(void) { return 100; }

int vcas_default_config(vcas_config* cfg) {
  if (cfg == nullptr) return VCAS_ERR_BAD_ARG;
  cfg->F = 100;
  cfg->M = 2;
  cfg->tau_act = 0.025f;
  cfg->tau_w = 0.025f;
  cfg->alpha = 0.01f;
  cfg->beta = 0.95f;
  cfg->rho_min = 0.f;
  cfg->nu_min = 0.f;
  return VCAS_OK;
}

int vcas_create(vcas_handle* out, const vcas_layer_desc* desc, const vcas_config* cfg) {
  if (out == nullptr || desc == nullptr) return VCAS_ERR_BAD_ARG;
  *out = nullptr;
  if (desc->N <= 0 || desc->T <= 0 || desc->d_in <= 0 || desc->d_out <= 0) return VCAS_ERR_SHAPE;
  if ((desc->d_in % 8) != 0 || (desc->d_out % 8) != 0) return VCAS_ERR_SHAPE;
  if ((long long)desc->N * desc->T > (1ll << 30)) return VCAS_ERR_SHAPE;
  if (desc->dtype != VCAS_DTYPE_F32 && desc->dtype != VCAS_DTYPE_BF16) return VCAS_ERR_DTYPE;
  const bool tensor_ok = desc->dtype == VCAS_DTYPE_BF16 && (desc->d_in % 64) == 0 && (desc->d_out % 64) == 0;
  if (desc->gemm_path == VCAS_GEMM_TENSOR && !tensor_ok) return VCAS_ERR_SHAPE;
  if (desc->gemm_path < VCAS_GEMM_AUTO || desc->gemm_path > VCAS_GEMM_TENSOR) return VCAS_ERR_BAD_ARG;
  Handle* h = new (std::nothrow) Handle();
  if (h == nullptr) return VCAS_ERR_WORKSPACE;
  h->desc = *desc;
  if (cfg != nullptr) h->cfg = *cfg; else vcas_default_config(&h->cfg);
  h->tensor_path = tensor_ok && desc->gemm_path != VCAS_GEMM_FMA;
  h->R_pad = (desc->N * desc->T + 63) / 64 * 64;
  h->launches = 0;
  h->prof_enabled = false;
  h->ev = nullptr;
  h->ev_dense = nullptr;
  h->prof_calls = h->prof_dense_calls = 0;
  h->tune_dx_tile_n = h->tune_dw_tile_n = h->tune_dx_split_k = h->tune_dw_split_k = 0;
  h->tune_dx_tile_m = h->tune_dw_tile_m = 0;
  h->plan_valid = false;
  h->plan_cache_used = h->plan_cache_next = 0;
  h->wait_limit_ns = 2000000000ull;
  h->sub_k = 0;
  h->join_pending = false;
  h->stall_once = 0;
  cudaDeviceProp prop;
  if (cudaGetDevice(&h->device) != cudaSuccess || cudaGetDeviceProperties(&prop, h->device) != cudaSuccess) {
    delete h;
    return VCAS_ERR_CUDA;
  }
  h->num_sms = prop.multiProcessorCount;
  h->max_units = 2 * h->num_sms;
  if (h->tensor_path && prop.major != 10) { delete h; return VCAS_ERR_CUDA; }
  h->bytes = layout(h, nullptr);
  if (cudaMalloc(&h->base, h->bytes) != cudaSuccess) {
    cudaGetLastError();
    delete h;
    return VCAS_ERR_WORKSPACE;
  }
  layout(h, reinterpret_cast<uint8_t*>(h->base));
  const int32_t R = desc->N * desc->T;
  if (cudaMemset(h->base, 0, h->bytes) != cudaSuccess ||
      cudaMemcpy(h->ws.counts + 2, &R, sizeof(int32_t), cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(h->ws2.counts + 2, &R, sizeof(int32_t), cudaMemcpyHostToDevice) != cudaSuccess) {
    cudaFree(h->base);
    delete h;
    return VCAS_ERR_CUDA;
  }
  if (cudaStreamCreateWithFlags(&h->side_stream, cudaStreamNonBlocking) != cudaSuccess ||
      cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming) != cudaSuccess) {
    cudaFree(h->base);
    delete h;
    return VCAS_ERR_CUDA;
  }
  *out = reinterpret_cast<vcas_handle>(h);
  return VCAS_OK;
}

int vcas_destroy(vcas_handle hh) {
  if (hh == nullptr) return VCAS_ERR_BAD_ARG;
  Handle* h = H(hh);
  if (h->ev != nullptr) {
    for (int i = 0; i < PROF_RING * 8; ++i) cudaEventDestroy(h->ev[i]);
    for (int i = 0; i < PROF_RING * 4; ++i) cudaEventDestroy(h->ev_dense[i]);
    delete[] h->ev;
    delete[] h->ev_dense;
  }
  cudaStreamDestroy(h->side_stream);
  cudaEventDestroy(h->ev_fork);
  cudaEventDestroy(h->ev_join);
  const cudaError_t e = cudaFree(h->base);
  delete h;
  return e == cudaSuccess ? VCAS_OK : VCAS_ERR_CUDA;
}

int vcas_workspace_bytes(vcas_handle hh, size_t* bytes) {
  if (hh == nullptr || bytes == nullptr) return VCAS_ERR_BAD_ARG;
  *bytes = H(hh)->bytes;
  return VCAS_OK;
}

int vcas_launch_count(vcas_handle hh, uint64_t* launches) {
  if (hh == nullptr || launches == nullptr) return VCAS_ERR_BAD_ARG;
  *launches = H(hh)->launches;
  return VCAS_OK;
}

namespace {
// One sampled backward (Eq. 2).  `a` carries the ratios, the seed, the optional given probabilities and the
// optional scores handed down from the layer above; a_out: optional row square-norms of dX for the layer below.
int run_sampled(Handle* h, const void* X, const void* dY, const void* W, const SamplerArgs& a, const void* Hpre,
                void* dX, float* dW, float* a_out, bool skip_dropped, bool defer_join, cudaStream_t st) {
  if (join_pending(h, st) != VCAS_OK) return VCAS_ERR_CUDA;
  const int hint = (int)(a.rho * a.nu * (float)(h->desc.N * h->desc.T)) + 1;
  // The sampled dX grid leaves one SM free: SampleW's single-CTA kernel, which runs beside it on the side
  // stream, needs a whole SM's shared memory.
  const int spare = 1;
  Plan px = {256, 1, 1}, pw = {256, 1, 1};
  if (h->tensor_path) plan_products(h, false, a.rho, hint, spare, a_out != nullptr, &px, &pw);
  if (!h->tensor_path || h->prof_enabled) {
    // one stream, so that (with stage profiling) each pair of events brackets the kernels of one stage
    mark(h, 0, st);
    VCAS_CUDA(launch_rownorm_dy(h, dY, a, st));
    mark(h, 1, st);
    VCAS_CUDA(launch_sample_a(h, a, a.a_in == nullptr && !h->prof_enabled, st));
    VCAS_CUDA(launch_scores_x(h, X, a, !h->prof_enabled, st));
    VCAS_CUDA(launch_sample_w(h, a, st));
    mark(h, 2, st);
    if (h->tensor_path) {
      VCAS_CUDA(launch_umma_dx(h, dY, W, false, a.rho, Hpre, dX, a_out, skip_dropped, spare, &px, st));
    } else {
      VCAS_CUDA(launch_fma_dx(h, dY, W, h->ws.scaleA, Hpre, dX, st));     // always writes the zero rows
      if (a_out != nullptr) VCAS_CUDA(launch_rownorm_out(h, dX, a_out, st));
    }
    mark(h, 3, st);
    mark(h, 6, st);
    VCAS_CUDA(launch_emit_pack(h, dY, X, a, h->tensor_path, st));
    mark(h, 4, st);
    if (h->tensor_path) {
      VCAS_CUDA(launch_umma_dw(h, h->ws.packG, h->ws.packX, h->R_pad, h->ws.counts + 1, hint, &pw, dW, st));
    } else {
      VCAS_CUDA(launch_fma_dw(h, dY, X, h->ws.idxW, h->ws.scaleW, h->ws.counts + 1, dW, st));
    }
    mark(h, 5, st);
  } else {
    // The dX product needs SampleA only: on `st`, the row norms of dY, SampleA and the dX product follow one
    // another as programmatic dependent launches.  Everything SampleW needs (the norms of the kept rows of X,
    // the water-filling, the kept-row list and the compact operands) and the dW product run beside the dX
    // product on the handle's side stream and are joined back before the call's work ends on `st`.
    VCAS_CUDA(launch_rownorm_dy(h, dY, a, st));
    VCAS_CUDA(launch_sample_a(h, a, a.a_in == nullptr, st));
    VCAS_CUDA(cudaEventRecord(h->ev_fork, st));
    VCAS_CUDA(cudaStreamWaitEvent(h->side_stream, h->ev_fork, 0));
    VCAS_CUDA(launch_umma_dx(h, dY, W, false, a.rho, Hpre, dX, a_out, skip_dropped, spare, &px, st));
    const int rc = sample_w_and_dw(h, X, dY, a, false, &pw, dW, h->side_stream);
    if (rc != VCAS_OK) return rc;
    VCAS_CUDA(cudaEventRecord(h->ev_join, h->side_stream));
    if (defer_join) h->join_pending = true;       // dW and the sampling record are complete only after vcas_join
    else VCAS_CUDA(cudaStreamWaitEvent(st, h->ev_join, 0));
  }
  if (h->prof_enabled && h->prof_calls < PROF_RING) h->prof_calls += 1;
  return VCAS_OK;
}
}  // namespace

int vcas_linear_bwd_ex(vcas_handle hh, const void* X, const void* dY, const void* W, float rho, float nu,
                       uint64_t seed, const float* p_in, const float* q_in, const void* Hpre, void* dX, float* dW,
                       vcas_stream stream) {
  if (hh == nullptr || X == nullptr || dY == nullptr || W == nullptr || dX == nullptr || dW == nullptr)
    return VCAS_ERR_BAD_ARG;
  if (!ratio_ok(rho) || !ratio_ok(nu)) return VCAS_ERR_BAD_ARG;
  SamplerArgs a = sampler_args(rho, nu, seed);
  a.p_in = p_in; a.q_in = q_in;
  return run_sampled(H(hh), X, dY, W, a, Hpre, dX, dW, nullptr, false, false, S(stream));
}

int vcas_linear_bwd_chain(vcas_handle hh, const void* X, const void* dY, const void* W, float rho, float nu,
                          uint64_t seed, const vcas_chain_args* c, void* dX, float* dW, vcas_stream stream) {
  if (hh == nullptr || X == nullptr || dY == nullptr || W == nullptr || dX == nullptr || dW == nullptr || c == nullptr)
    return VCAS_ERR_BAD_ARG;
  if (!ratio_ok(rho) || !ratio_ok(nu)) return VCAS_ERR_BAD_ARG;
  if ((c->alive_in == nullptr) != (c->alive_cnt_in == nullptr)) return VCAS_ERR_BAD_ARG;
  if ((c->kept_out == nullptr) != (c->kept_cnt_out == nullptr)) return VCAS_ERR_BAD_ARG;
  if (c->a_in != nullptr && c->a_in_parts < 1) return VCAS_ERR_BAD_ARG;
  SamplerArgs a = sampler_args(rho, nu, seed);
  a.a_in = c->a_in; a.a_parts = c->a_in != nullptr ? c->a_in_parts : 1;
  a.alive = c->alive_in; a.alive_cnt = c->alive_cnt_in;
  a.kept_out = c->kept_out; a.kept_cnt_out = c->kept_cnt_out;
  return run_sampled(H(hh), X, dY, W, a, c->H, dX, dW, c->a_out, c->skip_dropped_rows != 0, c->defer_join != 0,
                     S(stream));
}

int vcas_layernorm_bwd(vcas_handle hh, const void* X, const void* gamma, const void* dY, float eps, float rho,
                       uint64_t seed, const vcas_chain_args* c, void* dX, float* dgamma, float* dbeta,
                       vcas_stream stream) {
  if (hh == nullptr || X == nullptr || gamma == nullptr || dY == nullptr || dX == nullptr || dgamma == nullptr ||
      dbeta == nullptr)
    return VCAS_ERR_BAD_ARG;
  if (!ratio_ok(rho) || !(eps >= 0.f)) return VCAS_ERR_BAD_ARG;
  Handle* h = H(hh);
  if (h->desc.d_in != h->desc.d_out) return VCAS_ERR_SHAPE;      // a handle made with d_in = d_out = the normalised width
  if (h->desc.d_in < 2 * a_out_parts(h->desc.d_in)) return VCAS_ERR_SHAPE;
  SamplerArgs a = sampler_args(rho, 1.0f, seed);
  float* a_out = nullptr;
  bool skip = false;
  if (c != nullptr) {
    if ((c->alive_in == nullptr) != (c->alive_cnt_in == nullptr)) return VCAS_ERR_BAD_ARG;
    if ((c->kept_out == nullptr) != (c->kept_cnt_out == nullptr)) return VCAS_ERR_BAD_ARG;
    if (c->a_in != nullptr && c->a_in_parts < 1) return VCAS_ERR_BAD_ARG;
    a.a_in = c->a_in; a.a_parts = c->a_in != nullptr ? c->a_in_parts : 1;
    a.alive = c->alive_in; a.alive_cnt = c->alive_cnt_in;
    a.kept_out = c->kept_out; a.kept_cnt_out = c->kept_cnt_out;
    a_out = c->a_out;
    skip = c->skip_dropped_rows != 0;
  }
  cudaStream_t st = S(stream);
  if (join_pending(h, st) != VCAS_OK) return VCAS_ERR_CUDA;
  VCAS_CUDA(launch_rownorm_dy(h, dY, a, st));
  VCAS_CUDA(launch_sample_a(h, a, a.a_in == nullptr, st));
  VCAS_CUDA(launch_layernorm_bwd(h, X, gamma, dY, eps, dX, a_out, skip, dgamma, dbeta, rho, st));
  return VCAS_OK;
}

int vcas_join(vcas_handle hh, vcas_stream stream) {
  if (hh == nullptr) return VCAS_ERR_BAD_ARG;
  return join_pending(H(hh), S(stream));
}

int vcas_chain_parts(vcas_handle hh, int32_t* parts) {
  if (hh == nullptr || parts == nullptr) return VCAS_ERR_BAD_ARG;
  *parts = a_out_parts(H(hh)->desc.d_in);
  return VCAS_OK;
}

int vcas_linear_bwd(vcas_handle hh, const void* X, const void* dY, const void* W, float rho, float nu,
                    uint64_t seed, void* dX, float* dW, vcas_stream stream) {
  return vcas_linear_bwd_ex(hh, X, dY, W, rho, nu, seed, nullptr, nullptr, nullptr, dX, dW, stream);
}

int vcas_dense_bwd(vcas_handle hh, const void* X, const void* dY, const void* W, void* dX, float* dW,
                   vcas_stream stream) {
  return vcas_dense_bwd_ex(hh, X, dY, W, nullptr, dX, dW, stream);
}

int vcas_dense_bwd_ex(vcas_handle hh, const void* X, const void* dY, const void* W, const void* Hpre, void* dX,
                      float* dW, vcas_stream stream) {
  if (hh == nullptr || X == nullptr || dY == nullptr || W == nullptr || dX == nullptr || dW == nullptr)
    return VCAS_ERR_BAD_ARG;
  Handle* h = H(hh);
  cudaStream_t st = S(stream);
  if (join_pending(h, st) != VCAS_OK) return VCAS_ERR_CUDA;
  cudaStream_t sw = st;
  const bool fork = h->tensor_path && !h->prof_enabled;
  if (fork) {
    VCAS_CUDA(cudaEventRecord(h->ev_fork, st));
    VCAS_CUDA(cudaStreamWaitEvent(h->side_stream, h->ev_fork, 0));
    sw = h->side_stream;
  }
  Plan px = {256, 1, 1}, pw = {256, 1, 1};
  if (h->tensor_path) plan_products(h, true, 1.0f, h->desc.N * h->desc.T, 0, false, &px, &pw);
  mark_dense(h, 0, st);
  if (h->tensor_path) {
    VCAS_CUDA(launch_umma_dx(h, dY, W, true, 1.0f, Hpre, dX, nullptr, false, 0, &px, st));
  } else {
    VCAS_CUDA(launch_fma_dx(h, dY, W, nullptr, Hpre, dX, st));
  }
  mark_dense(h, 1, st);
  mark_dense(h, 3, sw);
  const int rc = dense_dw(h, X, dY, h->tensor_path ? &pw : nullptr, dW, sw);
  mark_dense(h, 2, sw);
  if (fork) {
    VCAS_CUDA(cudaEventRecord(h->ev_join, sw));
    VCAS_CUDA(cudaStreamWaitEvent(st, h->ev_join, 0));
  }
  if (h->prof_enabled && h->prof_dense_calls < PROF_RING) h->prof_dense_calls += 1;
  return rc;
}

int vcas_score(vcas_handle hh, const void* X, const void* dY, float rho, float nu, uint64_t seed, float* g,
               float* p, float* w, float* q, int32_t* idxA, int32_t* cntA, int32_t* idxW, int32_t* cntW,
               vcas_stream stream) {
  if (hh == nullptr || X == nullptr || dY == nullptr) return VCAS_ERR_BAD_ARG;
  if (!ratio_ok(rho) || !ratio_ok(nu)) return VCAS_ERR_BAD_ARG;
  Handle* h = H(hh);
  cudaStream_t st = S(stream);
  if (join_pending(h, st) != VCAS_OK) return VCAS_ERR_CUDA;
  const SamplerArgs a = sampler_args(rho, nu, seed);
  VCAS_CUDA(launch_rownorm_dy(h, dY, a, st));
  VCAS_CUDA(launch_sample_a(h, a, true, st));
  VCAS_CUDA(launch_scores_x(h, X, a, true, st));
  VCAS_CUDA(launch_sample_w(h, a, st));
  VCAS_CUDA(launch_emit_pack(h, dY, X, a, false, st));
  return copy_out(h, g, p, w, q, idxA, cntA, idxW, cntW, st);
}

int vcas_last_sampling(vcas_handle hh, float* g, float* p, float* w, float* q, int32_t* idxA, int32_t* cntA,
                       int32_t* idxW, int32_t* cntW, vcas_stream stream) {
  if (hh == nullptr) return VCAS_ERR_BAD_ARG;
  if (join_pending(H(hh), S(stream)) != VCAS_OK) return VCAS_ERR_CUDA;
  return copy_out(H(hh), g, p, w, q, idxA, cntA, idxW, cntW, S(stream));
}

int vcas_mask_from_probs(vcas_handle hh, const float* p, int32_t n, uint64_t seed, int32_t sampler_id,
                         uint8_t* keep, int32_t* idx, int32_t* cnt, vcas_stream stream) {
  if (hh == nullptr || p == nullptr || n < 0) return VCAS_ERR_BAD_ARG;
  if (sampler_id < 0) return VCAS_ERR_BAD_ARG;
  VCAS_CUDA(launch_mask_from_probs(H(hh), p, n, seed, sampler_id, keep, idx, cnt, S(stream)));
  return VCAS_OK;
}

int vcas_variance_probe(vcas_handle hh, int32_t M, const void* const* X_i, const void* const* dY_i, const void* W,
                        float rho, float nu, float s, uint64_t seed, float* V_s, float* V_act, float* V_w,
                        float* p_lo, float* p_hi, vcas_stream stream) {
  if (hh == nullptr || X_i == nullptr || dY_i == nullptr || W == nullptr) return VCAS_ERR_BAD_ARG;
  if (M < 2 || !ratio_ok(rho) || !ratio_ok(nu) || !(s >= 0.f && s <= 1.f)) return VCAS_ERR_BAD_ARG;
  for (int i = 0; i < M; ++i)
    if (X_i[i] == nullptr || dY_i[i] == nullptr) return VCAS_ERR_BAD_ARG;
  Handle* h = H(hh);
  cudaStream_t st = S(stream);
  if (join_pending(h, st) != VCAS_OK) return VCAS_ERR_CUDA;
  const double alpha = (double)h->cfg.alpha;
  double s_lo = (double)s - alpha, s_hi = (double)s + alpha;
  if (s_lo < 0.0) s_lo = 0.0;
  if (s_hi > 1.0) s_hi = 1.0;
  // App. D: with a subsample set (vcas_set_probe_subsample) the exact and the SampleA-only gradients are formed
  // on sub_k rows of the parameter gradient only: the products run through a copy of the handle whose d_out is
  // sub_k, on those columns of dY; scoring and sampling still see the whole of dY.
  const bool sub = h->sub_k > 0;
  Handle hs = *h;
  if (sub) hs.desc.d_out = h->sub_k;
  hs.plan_valid = false;
  Handle* hp = sub ? &hs : h;
  const uint64_t launches0 = hs.launches;
  VCAS_CUDA(launch_probe_reset(h, st));
  for (int i = 0; i < M; ++i) {
    const void* dYp = dY_i[i];
    if (sub) {
      VCAS_CUDA(launch_gather_cols(h, dY_i[i], h->desc.d_out, h->sub_rows, h->sub_k, h->sub_dY, st));
      dYp = h->sub_dY;
    }
    int rc = dense_dw(hp, X_i[i], dYp, nullptr, h->ws.Gs, st);   // G_s,i
    if (rc != VCAS_OK) return rc;
    VCAS_CUDA(launch_probe_welford(hp, i, st));
    SamplerArgs a = sampler_args(rho, nu, 0);
    a.sample_w = 0;          // the probe draws no SampleW mask: G_act keeps every row of the kept data,
    a.accumulate_vw = 1;     // and Eq. 3 is accumulated analytically at ratio nu
    VCAS_CUDA(launch_rownorm_dy(h, dY_i[i], a, st));
    // The M draws of SampleA for this batch are independent chains (SampleA, scores, SampleW's probabilities,
    // kept rows, product, squared difference): even draws run on `st` with the first workspace set, odd draws
    // on the side stream with the second, so that the latency-bound kernels of one chain overlap the product
    // of the other.
    VCAS_CUDA(cudaEventRecord(h->ev_fork, st));
    VCAS_CUDA(cudaStreamWaitEvent(h->side_stream, h->ev_fork, 0));
    const Workspace first = h->ws;
    for (int j = 0; j < M; ++j) {
      const bool second = (j & 1) != 0;
      cudaStream_t sj = second ? h->side_stream : st;
      h->ws = second ? h->ws2 : first;
      h->ws.a = first.a;
      hs.ws = h->ws;
      a.seed = seed + (uint64_t)(i * M + j + 1) * 0x9E3779B97F4A7C15ull;
      cudaError_t e = launch_sample_a(h, a, !second, sj);
      if (e == cudaSuccess && j == 0) e = launch_probe_sparsity(h, s_lo, s_hi, sj);
      if (e == cudaSuccess) rc = sample_w_and_dw(hp, X_i[i], dYp, a, true, nullptr, h->ws.Gact, sj);   // G_act,ij
      if (e == cudaSuccess && rc == VCAS_OK) e = launch_probe_sqdiff(hp, sj);
      h->ws = first;
      hs.ws = first;
      if (e != cudaSuccess) return VCAS_ERR_CUDA;
      if (rc != VCAS_OK) return rc;
    }
    VCAS_CUDA(cudaEventRecord(h->ev_join, h->side_stream));
    VCAS_CUDA(cudaStreamWaitEvent(st, h->ev_join, 0));
  }
  const double scale = sub ? (double)h->desc.d_out / (double)h->sub_k : 1.0;
  VCAS_CUDA(launch_probe_finalize(hp, M, scale, V_s, V_act, V_w, p_lo, p_hi, st));
  if (sub) h->launches += hs.launches - launches0;
  return VCAS_OK;
}

int vcas_update_ratios(vcas_state* state, int32_t L, const float* V_s, const float* V_act, const float* V_w,
                       const float* p_lo, const float* p_hi, const vcas_config* cfg) {
  if (state == nullptr || cfg == nullptr || V_s == nullptr || V_act == nullptr || V_w == nullptr ||
      p_lo == nullptr || p_hi == nullptr || state->rho == nullptr || state->nu == nullptr)
    return VCAS_ERR_BAD_ARG;
  if (L <= 0 || L != state->L) return VCAS_ERR_BAD_ARG;
  if (!(cfg->beta > 0.f && cfg->beta < 1.f) || !(cfg->alpha > 0.f)) return VCAS_ERR_BAD_ARG;
  double sum_act = 0.0, sum_s = 0.0;
  for (int l = 0; l < L; ++l) { sum_act += (double)V_act[l]; sum_s += (double)V_s[l]; }
  const bool up = sum_act - (double)cfg->tau_act * sum_s >= 0.0;   // Eq. 5, sign(0) = +1
  double s = (double)state->s + (up ? (double)cfg->alpha : -(double)cfg->alpha);
  s = s < 0.0 ? 0.0 : (s > 1.0 ? 1.0 : s);
  state->s = (float)s;
  double run = 0.0;                                                  // Eq. 4: running maximum from layer 1 up
  for (int l = 0; l < L; ++l) {
    const double cand = (double)(up ? p_hi[l] : p_lo[l]);
    run = cand > run ? cand : run;
    const double r = run > (double)cfg->rho_min ? run : (double)cfg->rho_min;
    state->rho[l] = (float)r;
  }
  for (int l = 0; l < L; ++l) {                                      // Eq. 7
    double nu = (double)state->nu[l];
    if ((double)V_w[l] - (double)cfg->tau_w * (double)V_s[l] >= 0.0) {
      nu = nu / (double)cfg->beta;
      if (nu > 1.0) nu = 1.0;
    } else {
      nu = nu * (double)cfg->beta;
    }
    if (nu < (double)cfg->nu_min) nu = (double)cfg->nu_min;
    state->nu[l] = (float)nu;
  }
  return VCAS_OK;
}

int vcas_set_tuning(vcas_handle hh, int32_t dx_tile_n, int32_t dw_tile_n, int32_t dx_split_k, int32_t dw_split_k,
                    int32_t dx_tile_m, int32_t dw_tile_m) {
  if (hh == nullptr) return VCAS_ERR_BAD_ARG;
  auto tile_ok = [](int32_t t) { return t == 0 || t == 64 || t == 128 || t == 256; };
  if (!tile_ok(dx_tile_n) || !tile_ok(dw_tile_n) || dx_split_k < 0 || dx_split_k > 16 ||
      dw_split_k < 0 || dw_split_k > 16 || dx_tile_m < 0 || dx_tile_m > 3 || dw_tile_m < 0 || dw_tile_m > 3)
    return VCAS_ERR_BAD_ARG;
  Handle* h = H(hh);
  h->tune_dx_tile_n = dx_tile_n;
  h->tune_dw_tile_n = dw_tile_n;
  h->tune_dx_split_k = dx_split_k;
  h->tune_dw_split_k = dw_split_k;
  h->tune_dx_tile_m = dx_tile_m;
  h->tune_dw_tile_m = dw_tile_m;
  return VCAS_OK;
}

int vcas_last_plan(vcas_handle hh, int32_t* plan) {
  if (hh == nullptr || plan == nullptr) return VCAS_ERR_BAD_ARG;
  Handle* h = H(hh);
  if (!h->tensor_path || !h->plan_valid) return VCAS_ERR_BAD_ARG;
  plan[0] = h->plan_dx.bn; plan[1] = h->plan_dx.split; plan[2] = h->plan_dx.mh;
  plan[3] = h->plan_dw.bn; plan[4] = h->plan_dw.split; plan[5] = h->plan_dw.mh;
  return VCAS_OK;
}

int vcas_set_probe_subsample(vcas_handle hh, int32_t rows, uint64_t seed) {
  if (hh == nullptr || rows < 0) return VCAS_ERR_BAD_ARG;
  Handle* h = H(hh);
  if (rows == 0) { h->sub_k = 0; return VCAS_OK; }
  const int unit = h->tensor_path ? 64 : 8;
  if (rows > SUB_MAX || (rows % unit) != 0 || rows >= h->desc.d_out) return VCAS_ERR_BAD_ARG;
  // scratch: the probe's gradient buffers are free between probes
  VCAS_CUDA(launch_param_subset(h, rows, seed, reinterpret_cast<uint32_t*>(h->ws.Gs),
                                reinterpret_cast<int32_t*>(h->ws.Gact), h->sub_rows, nullptr));
  VCAS_CUDA(cudaDeviceSynchronize());
  h->sub_k = rows;
  return VCAS_OK;
}

int vcas_get_probe_subsample(vcas_handle hh, int32_t* rows_host, int32_t* count) {
  if (hh == nullptr || count == nullptr) return VCAS_ERR_BAD_ARG;
  Handle* h = H(hh);
  *count = h->sub_k;
  if (rows_host != nullptr && h->sub_k > 0)
    VCAS_CUDA(cudaMemcpy(rows_host, h->sub_rows, (size_t)h->sub_k * sizeof(int32_t), cudaMemcpyDeviceToHost));
  return VCAS_OK;
}

int vcas_set_wait_limit(vcas_handle hh, uint64_t limit_ns, int32_t stall_once) {
  if (hh == nullptr || limit_ns == 0) return VCAS_ERR_BAD_ARG;
  H(hh)->wait_limit_ns = limit_ns;
  H(hh)->stall_once = stall_once != 0 ? 1 : 0;
  return VCAS_OK;
}

int vcas_set_profiling(vcas_handle hh, int32_t enable) {
  if (hh == nullptr) return VCAS_ERR_BAD_ARG;
  Handle* h = H(hh);
  if (enable && h->ev == nullptr) {
    h->ev = new (std::nothrow) cudaEvent_t[PROF_RING * 8];
    h->ev_dense = new (std::nothrow) cudaEvent_t[PROF_RING * 4];
    if (h->ev == nullptr || h->ev_dense == nullptr) return VCAS_ERR_WORKSPACE;
    for (int i = 0; i < PROF_RING * 8; ++i) VCAS_CUDA(cudaEventCreate(&h->ev[i]));
    for (int i = 0; i < PROF_RING * 4; ++i) VCAS_CUDA(cudaEventCreate(&h->ev_dense[i]));
  }
  h->prof_enabled = enable != 0;
  h->prof_calls = h->prof_dense_calls = 0;
  return VCAS_OK;
}

int vcas_stage_times(vcas_handle hh, float* ms, int32_t* calls) {
  if (hh == nullptr || ms == nullptr || calls == nullptr) return VCAS_ERR_BAD_ARG;
  Handle* h = H(hh);
  for (int k = 0; k < 8; ++k) ms[k] = 0.f;
  calls[0] = h->prof_calls;
  calls[1] = h->prof_dense_calls;
  if (h->ev == nullptr) return VCAS_OK;
  VCAS_CUDA(cudaDeviceSynchronize());
  // stage k lies between events (from, to): row norms 0-1, sampler 1-2, dX 2-3, pack 6-4, dW 4-5
  const int from[5] = {0, 1, 2, 6, 4}, to[5] = {1, 2, 3, 4, 5};
  for (int c = 0; c < h->prof_calls; ++c)
    for (int k = 0; k < 5; ++k) {
      float t = 0.f;
      VCAS_CUDA(cudaEventElapsedTime(&t, h->ev[c * 8 + from[k]], h->ev[c * 8 + to[k]]));
      ms[k] += t;
    }
  for (int c = 0; c < h->prof_dense_calls; ++c) {      // dense dX between events 0-1, dense dW between 3-2
    float t = 0.f;
    VCAS_CUDA(cudaEventElapsedTime(&t, h->ev_dense[c * 4 + 0], h->ev_dense[c * 4 + 1]));
    ms[5] += t;
    VCAS_CUDA(cudaEventElapsedTime(&t, h->ev_dense[c * 4 + 3], h->ev_dense[c * 4 + 2]));
    ms[6] += t;
  }
  h->prof_calls = h->prof_dense_calls = 0;
  return VCAS_OK;
}

int vcas_last_device_status(vcas_handle hh, int32_t* status) {
  if (hh == nullptr || status == nullptr) return VCAS_ERR_BAD_ARG;
  Handle* h = H(hh);
  VCAS_CUDA(cudaDeviceSynchronize());
  h->join_pending = false;
  VCAS_CUDA(cudaMemcpy(status, h->ws.status, sizeof(int32_t), cudaMemcpyDeviceToHost));
  VCAS_CUDA(cudaMemset(h->ws.status, 0, sizeof(int32_t)));
  if (*status != VCAS_OK && h->tensor_path) {
    // a product kernel that gave up may have left its slice tickets and work counters non-zero
    VCAS_CUDA(cudaMemset(h->ws.tickets, 0, 6 * (size_t)h->max_units * sizeof(int32_t)));
    VCAS_CUDA(cudaMemset(h->ws.sched, 0, 8 * sizeof(int32_t)));
  }
  return VCAS_OK;
}

}  // extern "C"
