// vcas_score_static: the scoring / sampling stage for callers that cannot allocate device
// memory.  Same kernels as vcas_score; the intermediate arrays live in a fixed device array
// that is part of the library image instead of a handle's workspace.
#include <mutex>

#include "common.cuh"

using namespace vcas;

namespace {

constexpr int STATIC_MAX_R = 16384;   // rows (N*T) the fixed scratch can serve
constexpr int STATIC_MAX_N = 4096;    // data
constexpr size_t kRowArrays = 8;      // a, wc, w, q, scaleW (float), idxW, chunk_off (int32), uc (uint32), each [STATIC_MAX_R]
constexpr size_t kDatumArrays = 6;    // g, p, scaleA, sorted (float) and idxA, dropA (int32), each [STATIC_MAX_N]
constexpr size_t kTailBytes = 768;    // counts [8] int32, acc [16] double, fix [4] float + status word, 256-byte slots
constexpr size_t kScratchBytes = kRowArrays * STATIC_MAX_R * 4 + kDatumArrays * STATIC_MAX_N * 4 + kTailBytes;

// Lives in every GPU that loads the library until the process exits (about 0.6 MB).  In host
// code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_score_scratch[kScratchBytes];

std::mutex g_mu;
unsigned char* g_scratch_addr[64] = {};   // device address of g_score_scratch, per device ordinal

// Resolves the device address of the scratch array on the current device (once per device).
cudaError_t scratch_for_current_device(unsigned char** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mu);
  if (g_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_score_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_addr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" int vcas_score_static(int32_t N, int32_t T, int32_t d_in, int32_t d_out, int32_t dtype, const void* X,
                                 const void* dY, float rho, float nu, uint64_t seed, float* g, float* p, float* w,
                                 float* q, int32_t* idxA, int32_t* cntA, int32_t* idxW, int32_t* cntW,
                                 vcas_stream stream) {
  if (X == nullptr || dY == nullptr) return VCAS_ERR_BAD_ARG;
  if (!(rho > 0.f && rho <= 1.f) || !(nu > 0.f && nu <= 1.f)) return VCAS_ERR_BAD_ARG;
  if (dtype != VCAS_DTYPE_F32 && dtype != VCAS_DTYPE_BF16) return VCAS_ERR_DTYPE;
  if (N <= 0 || T <= 0 || d_in <= 0 || d_out <= 0 || (d_in % 8) != 0 || (d_out % 8) != 0) return VCAS_ERR_SHAPE;
  if (N > STATIC_MAX_N || (long long)N * T > STATIC_MAX_R) return VCAS_ERR_SHAPE;   // beyond the fixed scratch

  unsigned char* base = nullptr;
  if (scratch_for_current_device(&base) != cudaSuccess) return VCAS_ERR_CUDA;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);

  // A stack-only handle whose "workspace" points into the fixed array; nothing is allocated.
  Handle h = {};
  h.desc.N = N; h.desc.T = T; h.desc.d_in = d_in; h.desc.d_out = d_out; h.desc.dtype = dtype;
  h.desc.gemm_path = VCAS_GEMM_FMA;
  float* fr = reinterpret_cast<float*>(base);
  Workspace& ws = h.ws;
  ws.a = fr + 0 * STATIC_MAX_R;
  ws.wc = fr + 1 * STATIC_MAX_R;
  ws.w = fr + 2 * STATIC_MAX_R;
  ws.q = fr + 3 * STATIC_MAX_R;
  ws.scaleW = fr + 4 * STATIC_MAX_R;
  ws.idxW = reinterpret_cast<int32_t*>(fr + 5 * STATIC_MAX_R);
  ws.chunk_off = reinterpret_cast<int32_t*>(fr + 6 * STATIC_MAX_R);
  ws.uc = reinterpret_cast<uint32_t*>(fr + 7 * STATIC_MAX_R);
  float* fn = fr + kRowArrays * STATIC_MAX_R;
  ws.g = fn + 0 * STATIC_MAX_N;
  ws.p = fn + 1 * STATIC_MAX_N;
  ws.scaleA = fn + 2 * STATIC_MAX_N;
  ws.sorted = fn + 3 * STATIC_MAX_N;
  ws.idxA = reinterpret_cast<int32_t*>(fn + 4 * STATIC_MAX_N);
  ws.dropA = reinterpret_cast<int32_t*>(fn + 5 * STATIC_MAX_N);
  unsigned char* tail = reinterpret_cast<unsigned char*>(fn + kDatumArrays * STATIC_MAX_N);
  ws.counts = reinterpret_cast<int32_t*>(tail);
  ws.acc = reinterpret_cast<double*>(tail + 256);
  ws.fix = reinterpret_cast<float*>(tail + 512);
  ws.status = reinterpret_cast<int32_t*>(tail + 512 + 64);

  // The array keeps the previous call's contents: the counters and accumulators start at zero.
  if (cudaMemsetAsync(tail, 0, kTailBytes, st) != cudaSuccess) return VCAS_ERR_CUDA;
  const SamplerArgs a = sampler_args(rho, nu, seed);
  if (launch_rownorm_dy(&h, dY, a, st) != cudaSuccess) return VCAS_ERR_CUDA;
  if (launch_sample_a(&h, a, true, st) != cudaSuccess) return VCAS_ERR_CUDA;
  if (launch_scores_x(&h, X, a, true, st) != cudaSuccess) return VCAS_ERR_CUDA;
  if (launch_sample_w(&h, a, st) != cudaSuccess) return VCAS_ERR_CUDA;
  if (launch_emit_pack(&h, dY, X, a, false, st) != cudaSuccess) return VCAS_ERR_CUDA;

  const size_t R = (size_t)N * T;
  const cudaMemcpyKind k = cudaMemcpyDeviceToDevice;
#define COPY_OUT(dst, src, bytes) \
  if ((dst) != nullptr && cudaMemcpyAsync((dst), (src), (bytes), k, st) != cudaSuccess) return VCAS_ERR_CUDA
  COPY_OUT(g, ws.g, N * sizeof(float));
  COPY_OUT(p, ws.p, N * sizeof(float));
  COPY_OUT(w, ws.w, R * sizeof(float));
  COPY_OUT(q, ws.q, R * sizeof(float));
  COPY_OUT(idxA, ws.idxA, N * sizeof(int32_t));
  COPY_OUT(cntA, ws.counts + 0, sizeof(int32_t));
  COPY_OUT(idxW, ws.idxW, R * sizeof(int32_t));
  COPY_OUT(cntW, ws.counts + 1, sizeof(int32_t));
#undef COPY_OUT
  return VCAS_OK;
}
