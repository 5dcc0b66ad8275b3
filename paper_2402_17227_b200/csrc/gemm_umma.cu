// The two products of the sampled backward on the 5th-generation tensor cores (tcgen05):
//   dX[rows of kept data] = (1/p_n) dY[rows] W          (App. E; rows of dropped data are zero-filled)
//   dW = A_rows^T B_rows over the compacted kept rows    (Sec. 4.2: G_tilde^T X)
// One persistent CTA per SM works through tiles whose number depends on the kept counts, which
// are read from device memory.  Per CTA: warps 0-3 and 6-9 are the epilogue (TMEM -> registers ->
// shared memory -> global; the two warps that reach the same TMEM lanes split a tile's columns), warp 4
// issues TMA loads into a ring of shared-memory stages, warp 5
// issues tcgen05.mma into TMEM accumulators (two of 128 rows, so that the epilogue of a tile overlaps
// the main loop of the next one, or one of 256 rows).  bf16 operands, fp32 accumulation.  Outputs leave
// through 128-byte-swizzled shared-memory staging and TMA / bulk stores.  Three instances per tile
// shape: two unsliced ones (tiles in CTA order, or drawn from a device-wide counter); the sliced one cuts
// each contraction into slices, stores every slice's fp32 partial tile, and a reduction launch that follows
// it adds the slices in a fixed order on all SMs.  No CTA waits for another CTA.  Every wait on an mbarrier
// is bounded: when it runs out the CTA records VCAS_ERR_TIMEOUT in the status word and leaves.
#include <cuda.h>

#include <atomic>

#include "common.cuh"

namespace vcas {
namespace {

constexpr int BM = 128;          // tile rows (UMMA M)
constexpr int BK = 64;           // k-block: 64 bf16 = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int A_BYTES = BM * BK * 2;
constexpr int CHUNK_BYTES = 64 * BK * 2;   // one 64-wide MN chunk of an MN-major operand
constexpr int NUM_THREADS = 320;          // 8 epilogue warps, 1 TMA producer warp, 1 MMA warp
constexpr int EPI_THREADS = 256;          // two groups of four epilogue warps
// Register cap of the product kernels: a CTA of 320 threads must leave room on its SM for the CTAs of the
// scoring and packing kernels of the call's other branch, which run beside it.
constexpr int MAX_REGS = 128;
constexpr int TMEM_COLS = 512;
constexpr int EPI_WARP_BYTES = 32 * 128;                // one staging buffer: 32 rows of 128 bytes, 128B-swizzled
constexpr int EPI_BYTES = 8 * EPI_WARP_BYTES;           // one buffer for each of the eight epilogue warps

// MH = number of 128-row halves of a tile (1 or 2).  A 256-row tile reuses each B stage for two
// accumulators, which cuts the shared-memory fill per FLOP by a third (the fill rate of one SM is
// what bounds a 128 x 256 tile); it uses all 512 TMEM columns, so its epilogue does not overlap the
// next main loop.  It is used for large problems only and never with a sliced contraction.
template <int BN, int MH> struct TileCfg {
  static constexpr int B_BYTES = BN * BK * 2;
  static constexpr int AT_BYTES = MH * A_BYTES;                       // the A part of a stage
  static constexpr int STAGE_BYTES = AT_BYTES + B_BYTES;
  static constexpr int STAGES = MH == 2 ? 3 : (BN == 256 ? 4 : (BN == 128 ? 6 : 8));
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + EPI_BYTES + 256 /*barriers*/;
};

// --------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Waits for the phase with the given parity; gives up after the wait limit (the 64-bit word 20 bytes after abort_flag, nanoseconds,
// put there at set-up) or when another role of this CTA has given up.  Returns false in that case.
__device__ __noinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int32_t* status) {
  const unsigned long long limit = *reinterpret_cast<volatile unsigned long long*>(abort_flag + 5);
  unsigned long long t0 = 0;
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 0xfffu) == 0) {
      if (*abort_flag) return false;
      const unsigned long long now = global_ns();
      if (t0 == 0) {
        t0 = now;
      } else if (now - t0 > limit) {
        *abort_flag = 1;
        atomicExch(status, (int32_t)VCAS_ERR_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int c0, int c1, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(c0), "r"(c1), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, int c0, int c1, int c2, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(smem_u32(bar)) : "memory");
}

// ---- asynchronous bulk stores (shared -> global), tracked in per-thread bulk groups
__device__ __forceinline__ void bulk_store(void* gdst, const void* ssrc, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_u32(ssrc)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, const void* ssrc, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(map), "r"(smem_u32(ssrc)), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, const void* ssrc, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(map), "r"(smem_u32(ssrc)), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// all groups of this thread are complete (their global writes are performed)
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t* holder, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(holder)), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
// D[tmem] (+)= A[smem] B[smem], bf16 x bf16 -> fp32
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate) : "memory");
}
// the mbarrier gets one arrival when all tcgen05.mma issued so far by this thread have finished
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// 32 lanes x 32 consecutive fp32 columns: thread i of the warp gets lane (base + i)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// ---------------------------------------------------------------------- UMMA descriptors
// Shared-memory matrix descriptor, 128-byte swizzle: bits [0,14) start address >> 4,
// [16,30) leading byte offset >> 4, [32,46) stride byte offset >> 4, [46,48) version = 1,
// [61,64) layout type (2 = SWIZZLE_128B).
//  K-major operand (rows of 64 bf16 = 128 B, 8-row groups 1024 B apart): SBO = 1024, LBO unused.
//  MN-major operand (each k-row holds 64 MN elements = 128 B; 8-k groups 1024 B apart;
//  64-wide MN chunks CHUNK_BYTES apart): SBO = 1024, LBO = CHUNK_BYTES.
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3ffffu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3ffffu) >> 4) | ((uint64_t)(CHUNK_BYTES >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
// Instruction descriptor (kind::f16): [4,6) D format (1 = f32), [7,10) A format (1 = bf16),
// [10,13) B format, bit 15 A major (1 = MN), bit 16 B major, [17,23) N >> 3, [24,29) M >> 4.
__host__ __device__ constexpr uint32_t make_idesc(int n, bool a_mn, bool b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

constexpr int QD = 2;   // depth of the work queue: the producer may be this many items ahead of the other roles
struct SmemLayout {
  uint8_t* stages;
  uint64_t* full;
  uint64_t* empty;
  uint64_t* tmem_full;
  uint64_t* tmem_empty;
  uint64_t* q_full;   // work queue (unsliced instance): slot holds a work item
  uint64_t* q_empty;  // ... slot has been read by the MMA thread and the 128 epilogue threads
  uint32_t* tmem_holder;
  int* abort_flag;
  int* flag;          // epilogue broadcast slot
  int* tile_q;        // [QD] work items handed from the producer thread to the other roles
  uint8_t* epi;       // [4 warps][2][32 rows][128 B] staging for bulk / TMA stores
};

template <int BN, int MH>
__device__ __forceinline__ SmemLayout carve(uint8_t* raw) {
  using C = TileCfg<BN, MH>;
  SmemLayout s;
  uint8_t* base = (uint8_t*)(((uintptr_t)raw + 1023) & ~(uintptr_t)1023);
  s.stages = base;
  s.epi = base + C::STAGES * C::STAGE_BYTES;                       // 1024-byte aligned (swizzle atom)
  uint64_t* bars = (uint64_t*)(s.epi + EPI_BYTES);
  s.full = bars;
  s.empty = bars + C::STAGES;
  s.tmem_full = bars + 2 * C::STAGES;
  s.tmem_empty = bars + 2 * C::STAGES + 2;
  s.q_full = bars + 2 * C::STAGES + 4;
  s.q_empty = bars + 2 * C::STAGES + 4 + QD;
  s.tmem_holder = (uint32_t*)(bars + 2 * C::STAGES + 4 + 2 * QD);
  s.abort_flag = (int*)(s.tmem_holder + 1);
  s.flag = s.abort_flag + 1;
  s.tile_q = s.flag + 1;
  return s;
}

template <int BN, int MH>
__device__ __forceinline__ uint32_t setup(const SmemLayout& s, int warp, int tid, bool with_queue,
                                          unsigned long long wait_limit_ns) {
  using C = TileCfg<BN, MH>;
  if (tid == 0) {
    for (int i = 0; i < C::STAGES; ++i) { mbar_init(&s.full[i], 1); mbar_init(&s.empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&s.tmem_full[i], 1); mbar_init(&s.tmem_empty[i], EPI_THREADS); }
    if (with_queue)
      for (int i = 0; i < QD; ++i) { mbar_init(&s.q_full[i], 1); mbar_init(&s.q_empty[i], EPI_THREADS + 1); }
    *s.abort_flag = 0;
    *reinterpret_cast<unsigned long long*>(s.abort_flag + 5) = wait_limit_ns;   // read by mbar_wait
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 5) tmem_alloc(s.tmem_holder, TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  return *(volatile uint32_t*)s.tmem_holder;
}

// GELU'(x) = Phi(x) + x phi(x) (erf form) as a polynomial: GELU'(x) - 1/2 is odd, so GELU'(x) = 1/2 + x Q(x^2);
// Q is a degree-11 polynomial in t = 2 x^2 / 25 - 1 (a Chebyshev least-squares fit on |x| <= 5, converted to
// powers of t, whose coefficients stay below 0.15), and |x| is clamped to 5, beyond which GELU' is 0 or 1 to
// within 1e-5.  Maximum absolute error 3e-5 in fp32 Horner form against the erf form in double precision, far
// inside the bf16 rounding of the product it scales.  No special-function unit: with an exponential and a
// reciprocal per element the epilogue of a wide dX tile took longer than its products (the exponential alone
// cost as much as all other arithmetic); thirteen fused multiply-adds, issued for two elements at a time
// (fma.rn.f32x2), cost less.
#define VCAS_GELU_PRIME_COEFFS                                                                   \
  {1.421275400e-01f, -7.508027066e-02f, 6.700628620e-02f, -7.250861119e-02f, 7.542644430e-02f,  \
   -7.929997715e-02f, 1.003925139e-01f, -8.373814972e-02f, 1.450312277e-02f, -1.099747622e-02f, \
   4.948262191e-02f, -2.731859035e-02f}
__device__ __forceinline__ float gelu_prime(float x) {
  constexpr float GP_C[12] = VCAS_GELU_PRIME_COEFFS;
  const float ax = fminf(fabsf(x), 5.0f);
  const float t = fmaf(ax * ax, 0.08f, -1.0f);
  float p = GP_C[11];
#pragma unroll
  for (int k = 10; k >= 0; --k) p = fmaf(p, t, GP_C[k]);
  return fmaf(copysignf(ax, x), p, 0.5f);
}
__device__ __forceinline__ uint64_t pack2(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// r[e] *= GELU'(h_e) for the eight bf16 pre-activations in hv: the same polynomial as gelu_prime, the four pairs
// side by side and every step of Horner's rule issued for all of them before the next (independent chains).
__device__ __forceinline__ void gelu_prime8(const uint4& hv, float (&r)[8]) {
  constexpr float GP_C[12] = VCAS_GELU_PRIME_COEFFS;
  const uint32_t hu[4] = {hv.x, hv.y, hv.z, hv.w};
  float x[8], ax[8];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    x[2 * e] = __uint_as_float(hu[e] << 16);
    x[2 * e + 1] = __uint_as_float(hu[e] & 0xffff0000u);
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) ax[e] = fminf(fabsf(x[e]), 5.0f);
  uint64_t t[4], p[4];
  const uint64_t c08 = pack2(0.08f, 0.08f), cm1 = pack2(-1.0f, -1.0f);
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const uint64_t a2 = pack2(ax[2 * e], ax[2 * e + 1]);
    t[e] = fma2(mul2(a2, a2), c08, cm1);
    p[e] = pack2(GP_C[11], GP_C[11]);
  }
#pragma unroll
  for (int k = 10; k >= 0; --k) {
    const uint64_t ck = pack2(GP_C[k], GP_C[k]);
#pragma unroll
    for (int e = 0; e < 4; ++e) p[e] = fma2(p[e], t[e], ck);
  }
  const uint64_t half2 = pack2(0.5f, 0.5f);
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const uint64_t xc = pack2(copysignf(ax[2 * e], x[2 * e]), copysignf(ax[2 * e + 1], x[2 * e + 1]));
    const uint64_t g = fma2(xc, p[e], half2);
    const uint64_t o = mul2(pack2(r[2 * e], r[2 * e + 1]), g);
    unpack2(o, r[2 * e], r[2 * e + 1]);
  }
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// ----------------------------------------------------------------------- the two products
// One kernel template serves both products; MODE selects operand staging and the epilogue.
//
// Work decomposition (all derived on the device from the kept counts): `gemm_tiles` output
// tiles, each cut along the contraction into S slices of kb_per k-blocks -> units; a unit is
// (tile, slice).  In the sliced instance every unit stores its fp32 partial tile to the workspace;
// slice_reduce_kernel, launched behind the product, adds the S partials of every tile in slice order
// (a fixed order: results do not depend on timing) and writes the output.
constexpr int MODE_DX = 0, MODE_DW = 1;
constexpr int KIND_SLICED = 0, KIND_STATIC = 1, KIND_DYNAMIC = 2;

struct GemmParams {
  int32_t* status;
  float* partial;          // [max_units][128 * BN] fp32 partial tiles (split contraction)
  int32_t* sched;          // [2]: next work item, CTAs that have finished (unsliced instance); zero between launches
  int split_k;             // slices requested by the host
  int grid_ctas;           // CTAs of the product launch (the slicing is derived from it, also by the reduction launch)
  int max_units;
  unsigned long long wait_limit_ns;   // every mbarrier wait gives up after this long
  int stall_once;          // test hook: CTA 0 leaves out the loads of its first k-block, so that a wait runs out
  // Whole waves and remainder (256-wide tiles): part 1 is the launch with 256-row tiles, which takes only as
  // many tiles as fill its head_ctas CTAs a whole number of times (when the rest is at most half a wave);
  // part 2 is a second launch with 128-row tiles that covers the remaining 256-row tiles, two tiles each,
  // the contraction cut into as many slices as fill its grid once.  0: one launch does everything.
  int part, head_ctas;
  int d_in, d_out;
  // dX: A = dY viewed [N][T][d_out] (K-major, one TMA box = 128 tokens x 64 k of one datum),
  //     B = W [d_out][d_in] (MN-major: n contiguous)
  const int32_t* idxA;     // kept data
  const int32_t* dropA;    // dropped data
  const int32_t* counts;   // counts[0] = number of kept data
  const float* scaleA;     // 1/p_n per datum
  const __nv_bfloat16* H;  // optional GELU pre-activation [R, d_in]
  __nv_bfloat16* dX;       // [R, d_in]
  float* a_out;            // optional [R][a_parts]: square-norm of the stored row of dX, one partial sum per 256-column
  int a_parts;             // tile (unsliced 256-wide tiles only); the layer below adds the partials in order
  int N, T;
  int dense;               // 1: every datum kept with scale 1
  int skip_dropped;        // 1: the rows of dropped data are left unwritten (the consumer knows they are zero)
  int a_tx_bytes;          // bytes one A box delivers (min(T, 128) token rows of 128 B)
  // dW: A = rows x d_out, B = rows x d_in (both MN-major, gathered along k by the pack step)
  const int32_t* cnt;      // number of valid rows (the contraction length)
  float* dW;               // [d_out, d_in]
};

struct Decomp {
  int gemm_tiles, zero_tiles, kblocks, S, kb_per, units;
  int upi;                 // units taken per pass of the grid: a multiple of S, so that the S slices of a tile
                           // are always worked on at the same time by S neighbouring CTAs
  int per_datum, ntiles;   // dX: tiles per datum; both: column tiles
  int head256, per_datum256;   // parts 1 and 2: 256-row tiles left to part 1; dX: 256-row tiles per datum
};

template <int MODE, int BN, int MH, bool LEAN>
__device__ __forceinline__ Decomp decompose(const GemmParams& P) {
  constexpr int BMT = BM * MH;
  Decomp d;
  d.ntiles = (P.d_in + BN - 1) / BN;
  if (MODE == MODE_DX) {
    const int cntA = P.dense ? P.N : P.counts[0];
    d.per_datum = ((P.T + BMT - 1) / BMT) * d.ntiles;
    d.gemm_tiles = cntA * d.per_datum;
    d.zero_tiles = P.skip_dropped ? 0 : (P.N - cntA) * d.per_datum;
    d.kblocks = (P.d_out + BK - 1) / BK;
  } else {
    d.per_datum = 0;
    const int tiles = ((P.d_out + BMT - 1) / BMT) * d.ntiles;
    d.kblocks = (*P.cnt + BK - 1) / BK;
    d.gemm_tiles = d.kblocks > 0 ? tiles : 0;   // nothing kept: every tile is a zero tile
    d.zero_tiles = d.kblocks > 0 ? 0 : tiles;
  }
  int split_req = P.split_k;
  d.head256 = 0;
  d.per_datum256 = 0;
  if (P.part != 0) {
    int total256;
    if (MODE == MODE_DX) {
      d.per_datum256 = ((P.T + 2 * BM - 1) / (2 * BM)) * d.ntiles;
      total256 = (P.dense ? P.N : P.counts[0]) * d.per_datum256;
    } else {
      total256 = d.kblocks > 0 ? ((P.d_out + 2 * BM - 1) / (2 * BM)) * d.ntiles : 0;
    }
    const int frac = total256 % P.head_ctas;
    const int tail256 = 2 * frac <= P.head_ctas ? frac : 0;
    d.head256 = total256 - tail256;
    if (P.part == 1) {
      d.gemm_tiles = d.head256;
    } else {
      d.gemm_tiles = 2 * tail256;
      d.zero_tiles = 0;                      // part 1 writes them
      split_req = d.gemm_tiles > 0 ? P.grid_ctas / d.gemm_tiles : 1;
      if (split_req > 8) split_req = 8;
      if (split_req > d.kblocks / 4) split_req = d.kblocks / 4;      // slices of at least four k-blocks
    }
  }
  int S = (split_req < 1 || MH == 2 || LEAN) ? 1 : split_req;
  if (S > d.kblocks) S = d.kblocks > 0 ? d.kblocks : 1;
  if (d.gemm_tiles > 0 && (long)d.gemm_tiles * S > P.max_units) S = P.max_units / d.gemm_tiles;
  if (S > P.grid_ctas) S = P.grid_ctas;
  if (S < 1) S = 1;
  d.kb_per = d.kblocks > 0 ? (d.kblocks + S - 1) / S : 0;
  d.S = d.kb_per > 0 ? (d.kblocks + d.kb_per - 1) / d.kb_per : 1;   // every slice non-empty
  d.units = d.gemm_tiles * d.S;
  d.upi = (P.grid_ctas / d.S) * d.S;
  return d;
}

// Product tile -> (kept datum k [dX], row chunk c0 in units of this kernel's tile height, column tile c1).
// In part 2 tile j is half (j & 1) of the 256-row tile head256 + j / 2.
template <int MODE>
__device__ __forceinline__ void tile_coords(const GemmParams& P, const Decomp& D, int tile, int& k, int& c0, int& c1) {
  k = 0;
  if (P.part == 2) {
    const int t = D.head256 + (tile >> 1), half = tile & 1;
    if (MODE == MODE_DX) {
      k = t / D.per_datum256;
      const int rem = t % D.per_datum256;
      c0 = 2 * (rem / D.ntiles) + half; c1 = rem % D.ntiles;
    } else {
      c0 = 2 * (t / D.ntiles) + half; c1 = t % D.ntiles;
    }
  } else if (MODE == MODE_DX) {
    k = tile / D.per_datum;
    const int rem = tile % D.per_datum;
    c0 = rem / D.ntiles; c1 = rem % D.ntiles;
  } else {
    c0 = tile / D.ntiles; c1 = tile % D.ntiles;
  }
}


// KIND: three instances per tile shape.  KIND_STATIC and KIND_DYNAMIC are for unsliced contractions (S = 1)
// and carry no code of the slice exchange; the static one takes work items blockIdx.x, + gridDim.x, ...,
// the dynamic one draws them from a device-wide counter (chosen when there are more items than CTAs) and
// hands them to the MMA and epilogue roles through a small queue in shared memory, so that CTAs which start
// late - the SMs are shared with the call's other product - or get cheap items simply take fewer.
// KIND_SLICED has only the slice exchange (a contraction that ends up in one slice still goes through it).
// Separate instances because the product kernels are short: code that a launch never runs still costs it
// time.
template <int MODE, int BN, int MH, int KIND>
__global__ void __maxnreg__(MAX_REGS)
umma_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
            const __grid_constant__ CUtensorMap tmC, GemmParams P) {
  using C = TileCfg<BN, MH>;
  constexpr int BMT = BM * MH;          // rows of a tile
  constexpr int NACC = MH == 2 ? 1 : 2;  // accumulator sets in TMEM
  extern __shared__ uint8_t smem_raw[];
  const SmemLayout s = carve<BN, MH>(smem_raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t tmem_base = setup<BN, MH>(s, warp, tid, KIND == KIND_DYNAMIC, P.wait_limit_ns);
  volatile int* abort_flag = s.abort_flag;
  pdl_wait();      // barriers and TMEM are set up; the counts and operands come from earlier kernels
  constexpr bool LEAN = KIND != KIND_SLICED;
  constexpr bool DYN = KIND == KIND_DYNAMIC;
  const Decomp D = decompose<MODE, BN, MH, LEAN>(P);
  const int total_items = D.units + D.zero_tiles;     // unsliced instances: product tiles, then zero tiles

  if (warp == 4) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      bool ok = true, stalled = false;
      int qi = 0; uint32_t qph = 0;
      // next unit of this CTA, or -1 (see KIND above)
      auto next_unit = [&](int prev) -> int {
        if constexpr (DYN) {
          if (!mbar_wait(&s.q_empty[qi], qph ^ 1u, abort_flag, P.status)) { ok = false; return -1; }
          int t = atomicAdd(P.sched, 1);
          if (t >= D.units + D.zero_tiles) t = -1;
          *(volatile int*)&s.tile_q[qi] = t;
          mbar_arrive(&s.q_full[qi]);
          if (++qi == QD) { qi = 0; qph ^= 1u; }
          return t;
        } else if constexpr (LEAN) {
          const int u = prev < 0 ? (int)blockIdx.x : prev + (int)gridDim.x;
          return u < total_items ? u : -1;
        } else {
          const int u = prev < 0 ? (int)blockIdx.x : prev + D.upi;
          return ((int)blockIdx.x < D.upi && u < D.units) ? u : -1;
        }
      };
      for (int u = next_unit(-1); u >= 0 && ok; u = next_unit(u)) {
        if (LEAN && u >= D.units) continue;    // a zero tile: nothing to load
        const int tile = u / D.S, slice = u % D.S;
        const int kb0 = slice * D.kb_per;
        const int kb1 = min(D.kblocks, kb0 + D.kb_per);
        int c0 = 0, c1 = 0, n = 0;   // dX: token chunk, column tile, datum; dW: row tile, column tile
        {
          int k;
          tile_coords<MODE>(P, D, tile, k, c0, c1);
          if (MODE == MODE_DX) n = P.dense ? k : P.idxA[k];
        }
        for (int kb = kb0; kb < kb1; ++kb) {
          ok = mbar_wait(&s.empty[stage], phase ^ 1u, abort_flag, P.status);
          if (!ok) break;
          uint8_t* sa = s.stages + stage * C::STAGE_BYTES;
          if (P.stall_once != 0 && blockIdx.x == 0 && !stalled) {
            stalled = true;                    // nothing will ever arrive for this stage: the MMA role's wait runs out
            if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
            continue;
          }
          if (MODE == MODE_DX) {
            mbar_expect_tx(&s.full[stage], (uint32_t)(MH * P.a_tx_bytes + C::B_BYTES));
#pragma unroll
            for (int hh = 0; hh < MH; ++hh)
              tma_load_3d(sa + hh * A_BYTES, &tmA, kb * BK, c0 * BMT + hh * BM, n, &s.full[stage]);
          } else {
            mbar_expect_tx(&s.full[stage], C::STAGE_BYTES);
#pragma unroll
            for (int j = 0; j < BMT / 64; ++j)
              tma_load_2d(sa + j * CHUNK_BYTES, &tmA, c0 * BMT + j * 64, kb * BK, &s.full[stage]);
          }
#pragma unroll
          for (int j = 0; j < BN / 64; ++j)
            tma_load_2d(sa + C::AT_BYTES + j * CHUNK_BYTES, &tmB, c1 * BN + j * 64, kb * BK, &s.full[stage]);
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if constexpr (DYN) {
        if (ok) {        // the last CTA to run out of work re-arms the counters for the next launch
          __threadfence();
          if (atomicAdd(P.sched + 1, 1) == (int)gridDim.x - 1) { P.sched[0] = 0; P.sched[1] = 0; }
        }
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc(BN, MODE == MODE_DW, true);
      constexpr uint32_t a_step = MODE == MODE_DW ? (UMMA_K * 128 >> 4) : (UMMA_K * 2 >> 4);
      int stage = 0; uint32_t phase = 0; int lt = 0;
      bool ok = true;
      int qi = 0; uint32_t qph = 0;
      auto next_unit = [&](int prev) -> int {
        if constexpr (DYN) {
          if (!mbar_wait(&s.q_full[qi], qph, abort_flag, P.status)) { ok = false; return -1; }
          const int t = *(volatile int*)&s.tile_q[qi];
          mbar_arrive(&s.q_empty[qi]);
          if (++qi == QD) { qi = 0; qph ^= 1u; }
          return t;
        } else if constexpr (LEAN) {
          const int u = prev < 0 ? (int)blockIdx.x : prev + (int)gridDim.x;
          return u < total_items ? u : -1;
        } else {
          const int u = prev < 0 ? (int)blockIdx.x : prev + D.upi;
          return ((int)blockIdx.x < D.upi && u < D.units) ? u : -1;
        }
      };
      for (int u = next_unit(-1); u >= 0 && ok; u = next_unit(u)) {
        if (LEAN && u >= D.units) continue;    // a zero tile: the epilogue warps write it
        const int lt_now = lt++;
        const int slice = u % D.S;
        const int nkb = min(D.kblocks, (slice + 1) * D.kb_per) - slice * D.kb_per;
        const int buf = lt_now % NACC; const uint32_t use = (uint32_t)(lt_now / NACC) & 1u;
        ok = mbar_wait(&s.tmem_empty[buf], use ^ 1u, abort_flag, P.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);   // half hh of a 256-row tile: + hh * BN
        for (int kb = 0; kb < nkb; ++kb) {
          ok = mbar_wait(&s.full[stage], phase, abort_flag, P.status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sa = smem_u32(s.stages + stage * C::STAGE_BYTES);
          const uint64_t db = desc_mnmajor(sa + C::AT_BYTES);
#pragma unroll
          for (int hh = 0; hh < MH; ++hh) {
            const uint64_t da = MODE == MODE_DW ? desc_mnmajor(sa + hh * A_BYTES) : desc_kmajor(sa + hh * A_BYTES);
#pragma unroll
            for (int k4 = 0; k4 < BK / UMMA_K; ++k4)
              umma_bf16(d_tmem + (uint32_t)(hh * BN), da + (uint64_t)(k4 * a_step),
                        db + (uint64_t)(k4 * (UMMA_K * 128 >> 4)), idesc, (kb | k4) != 0 ? 1u : 0u);
          }
          umma_commit(&s.empty[stage]);
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit(&s.tmem_full[buf]);
      }
    }
  } else {
    // -------------------------------------------------------------------- epilogue
    // Two groups of four epilogue warps (warps 0-3 and 6-9).  A warp reaches the 32 TMEM lanes of quarter
    // (warp % 4), so the two warps of a quarter share its rows and split the tile's column chunks between
    // them (even chunks / odd chunks): two warps per scheduler hide each other's TMEM, arithmetic and store
    // latencies, which a single warp per scheduler cannot.
    const int eq = warp & 3;                  // TMEM lane quarter
    const int eg = warp < 4 ? 0 : 1;          // epilogue group: which column chunks
    const int row = eq * 32 + lane;           // this thread's row of a 128-row half
    const size_t ld = (size_t)P.d_in;
    // output rows [row0, row0 + rows_valid) x columns [col0, col0 + BN) of the tile; sc = 1/p_n
    auto geometry = [&](int tile, bool is_gemm, size_t& row0, int& rows_valid, int& col0, float& sc, int& n_out,
                        int& t_out) {
      sc = 1.0f; n_out = 0; t_out = 0;
      if (MODE == MODE_DX) {
        int k, c, nt;
        if (is_gemm) {
          tile_coords<MODE>(P, D, tile, k, c, nt);
        } else {
          k = tile / D.per_datum;
          const int rem = tile % D.per_datum;
          c = rem / D.ntiles; nt = rem % D.ntiles;
        }
        const int n = is_gemm ? (P.dense ? k : P.idxA[k]) : P.dropA[k];
        row0 = (size_t)n * P.T + (size_t)c * BMT;
        rows_valid = min(BMT, P.T - c * BMT);
        col0 = nt * BN;
        n_out = n; t_out = c * BMT;
        if (is_gemm && !P.dense) sc = P.scaleA[n];
      } else {
        int k, mt, nt;
        if (is_gemm) { tile_coords<MODE>(P, D, tile, k, mt, nt); } else { mt = tile / D.ntiles; nt = tile % D.ntiles; }
        row0 = (size_t)mt * BMT;
        rows_valid = min(BMT, P.d_out - mt * BMT);
        col0 = nt * BN;
      }
    };
    const uint32_t swz = (uint32_t)(lane & 7);                   // 128-byte swizzle: 16-byte slot ^= row & 7
    int lt = 0;
    bool ok = true;
    int qi = 0; uint32_t qph = 0;
    auto next_unit = [&](int prev) -> int {
      if constexpr (DYN) {
        if (!mbar_wait(&s.q_full[qi], qph, abort_flag, P.status)) { ok = false; return -1; }
        const int t = *(volatile int*)&s.tile_q[qi];
        mbar_arrive(&s.q_empty[qi]);
        if (++qi == QD) { qi = 0; qph ^= 1u; }
        return t;
      } else if constexpr (LEAN) {
        const int u = prev < 0 ? (int)blockIdx.x : prev + (int)gridDim.x;
        return u < total_items ? u : -1;
      } else {
        const int u = prev < 0 ? (int)blockIdx.x : prev + D.upi;
        return ((int)blockIdx.x < D.upi && u < D.units) ? u : -1;
      }
    };
    // Writes the zero tile z (rows of dropped data; nothing kept at all): every warp clears one of its staging
    // buffers and stores it, by TMA, to each 32-row x 128-byte piece of its slab of the tile.  The tensor map
    // clips rows beyond T and columns beyond d_in.  No per-element work: the epilogue warps are free again at once.
    uint8_t* stage0 = s.epi + (eg * 4 + eq) * EPI_WARP_BYTES;    // this warp's staging buffer
    auto zero_tile = [&](int z) {
      size_t row0; int rows_valid, col0, n_out, t_out; float sc;
      geometry(z, false, row0, rows_valid, col0, sc, n_out, t_out);
      reinterpret_cast<uint4*>(stage0)[lane] = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
      for (int k8 = 1; k8 < EPI_WARP_BYTES / 512; ++k8)
        reinterpret_cast<uint4*>(stage0)[k8 * 32 + lane] = make_uint4(0u, 0u, 0u, 0u);
      fence_async_smem();
      __syncwarp();
      constexpr int COLS = MODE == MODE_DX ? 64 : 32;             // columns per 128-byte staged row
      if (lane == 0) {
#pragma unroll 1
        for (int hh = 0; hh < MH; ++hh) {
          if (hh * BM + eq * 32 >= rows_valid) break;
          for (int j = eg; j < BN / COLS; j += 2) {
            if (col0 + j * COLS >= P.d_in) break;
            if (MODE == MODE_DX) tma_store_3d(&tmC, stage0, col0 + j * COLS, t_out + hh * BM + eq * 32, n_out);
            else tma_store_2d(&tmC, stage0, col0 + j * COLS, (int)row0 + hh * BM + eq * 32);
          }
        }
        bulk_commit();
        bulk_wait_read_0();                  // the buffer may be rewritten; the global writes finish on their own
      }
      __syncwarp();
      if (MODE == MODE_DX && P.a_out != nullptr) {
#pragma unroll 1
        for (int hh = 0; hh < MH; ++hh)
          if (hh * BM + row < rows_valid) P.a_out[(row0 + hh * BM + row) * P.a_parts + (col0 / 256) * 2 + eg] = 0.f;
      }
    };
    for (int u = next_unit(-1); u >= 0 && ok; u = next_unit(u)) {
      if (LEAN && u >= D.units) { zero_tile(u - D.units); continue; }
      const int lt_now = lt++;
      const int tile = u / D.S;
      size_t row0; int rows_valid, col0, n_out, t_out; float sc;
      geometry(tile, true, row0, rows_valid, col0, sc, n_out, t_out);
      const int buf = lt_now % NACC; const uint32_t use = (uint32_t)(lt_now / NACC) & 1u;
      if constexpr (LEAN && MODE == MODE_DX) {
        // GELU' epilogue: while the tile's products are still running, ask L2 for the pre-activations of this
        // thread's rows
        if (P.H != nullptr) {
#pragma unroll
          for (int hh = 0; hh < MH; ++hh) {
            const int hrow = hh * BM + row;
            if (hrow < rows_valid) {
              const __nv_bfloat16* hp = P.H + (row0 + hrow) * ld + col0;
#pragma unroll
              for (int j = eg; j < BN / 64; j += 2)
                if (col0 + j * 64 < P.d_in) asm volatile("prefetch.global.L2 [%0];" ::"l"(hp + j * 64));
            }
          }
        }
      }
      bool got = mbar_wait(&s.tmem_full[buf], use, abort_flag, P.status);
      if constexpr (!LEAN) {
        // the epilogue threads give up together or not at all
        uint32_t all;
        asm volatile(
            "{\n\t.reg .pred p, q;\n\t"
            "setp.ne.u32 p, %1, 0;\n\t"
            "bar.red.and.pred q, 1, 256, p;\n\t"
            "selp.u32 %0, 1, 0, q;\n\t}"
            : "=r"(all) : "r"(got ? 1u : 0u) : "memory");
        got = all != 0;
      }
      if (!got) { ok = false; break; }
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(eq * 32) << 16) + (uint32_t)(buf * BN);
      if constexpr (LEAN) {
        // ---- whole contraction in this unit: accumulator -> (rescale, GELU', convert) -> swizzled
        // shared memory -> TMA store of 32 rows x 128 bytes per warp (rows / columns outside the
        // tensor are clipped by the tensor map, so rows of the next datum are never touched)
        constexpr int COLS = MODE == MODE_DX ? 64 : 32;             // columns per 128-byte staged row
        int nbuf = 0;
        float rowsq[MH];                                            // square-norm of this thread's row(s), as stored
#pragma unroll
        for (int hh = 0; hh < MH; ++hh) rowsq[hh] = 0.f;
        // GELU' epilogue: this thread's 64 pre-activations of a chunk (eight 16-byte loads, its own row) are
        // requested at the top of the chunk, in front of the TMEM load; they were prefetched to L2 before the
        // wait for the accumulator, and the other warp of this quarter covers what latency is left.  (Staging
        // them through shared memory with coalesced copies was measured slower.)
        uint4 hq[8];
#pragma unroll 1
        for (int hj = eg; hj < MH * (BN / COLS); hj += 2, ++nbuf) {      // this group's chunks
          const int hh = hj / (BN / COLS), j = hj % (BN / COLS);    // 128-row half of the tile, column chunk
          const uint32_t taddr_h = taddr + (uint32_t)(hh * BN);
          if (col0 + j * COLS >= P.d_in) { --nbuf; continue; }      // warp-uniform
          uint8_t* buf8 = stage0;
          uint4* myrow = reinterpret_cast<uint4*>(buf8 + lane * 128);
          // the store of this warp's chunk before must have read the buffer before it is refilled (the wait sits
          // behind the TMEM load, where it costs little; the other warp of this quarter works meanwhile)
          auto buffer_free = [&]() { if (nbuf >= 1) { if (lane == 0) bulk_wait_read_0(); __syncwarp(); } };
          const bool with_h = MODE == MODE_DX && P.H != nullptr;
          if (with_h) {
            // rows beyond the tile's valid rows read a valid row instead: their outputs are clipped by the store
            const int hrow = min(hh * BM + row, rows_valid - 1);
            const uint4* src = reinterpret_cast<const uint4*>(P.H + (row0 + hrow) * ld + col0 + j * 64);
#pragma unroll
            for (int k8 = 0; k8 < 8; ++k8) hq[k8] = __ldg(src + k8);
          }
          if (MODE == MODE_DX) {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              uint32_t v[32];
              tmem_ld32(taddr_h + (uint32_t)(j * 64 + half * 32), v);
              if (half == 0) buffer_free();
#pragma unroll
              for (int g8 = 0; g8 < 4; ++g8) {
                float r[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) r[e] = sc * __uint_as_float(v[g8 * 8 + e]);
                if (with_h) gelu_prime8(hq[half * 4 + g8], r);
                uint4 o;
                o.x = pack_bf16(r[0], r[1]); o.y = pack_bf16(r[2], r[3]);
                o.z = pack_bf16(r[4], r[5]); o.w = pack_bf16(r[6], r[7]);
                myrow[(uint32_t)(half * 4 + g8) ^ swz] = o;
                if (P.a_out != nullptr) {
                  const uint32_t ou[4] = {o.x, o.y, o.z, o.w};
                  float sq = 0.f;
#pragma unroll
                  for (int e = 0; e < 4; ++e) {
                    const float lo = __uint_as_float(ou[e] << 16), hi = __uint_as_float(ou[e] & 0xffff0000u);
                    sq = fmaf(lo, lo, sq);
                    sq = fmaf(hi, hi, sq);
                  }
#pragma unroll
                  for (int h2 = 0; h2 < MH; ++h2)
                    if (h2 == hh) rowsq[h2] += sq;
                }
              }
            }
          } else {
            uint32_t v[32];
            tmem_ld32(taddr_h + (uint32_t)(j * 32), v);
            buffer_free();
#pragma unroll
            for (int g4 = 0; g4 < 8; ++g4)
              myrow[(uint32_t)g4 ^ swz] = make_uint4(v[g4 * 4], v[g4 * 4 + 1], v[g4 * 4 + 2], v[g4 * 4 + 3]);
          }
          fence_async_smem();
          __syncwarp();
          if (lane == 0) {
            if (MODE == MODE_DX) tma_store_3d(&tmC, buf8, col0 + j * 64, t_out + hh * BM + eq * 32, n_out);
            else tma_store_2d(&tmC, buf8, col0 + j * 32, (int)row0 + hh * BM + eq * 32);
            bulk_commit();
          }
        }
        tc_fence_before();
        mbar_arrive(&s.tmem_empty[buf]);
        if (MODE == MODE_DX && P.a_out != nullptr) {
#pragma unroll
          for (int hh = 0; hh < MH; ++hh)
            if (hh * BM + row < rows_valid)
              P.a_out[(row0 + hh * BM + row) * P.a_parts + (col0 / 256) * 2 + eg] = rowsq[hh];
        }
        if (lane == 0) bulk_wait_all();        // staging buffers are reused by the next unit
        __syncwarp();
        continue;
      }
      if constexpr (!LEAN) {
      // ---- one slice of the contraction: store the fp32 partial tile.  Layout in the workspace:
      // [32-column chunk][row][32 floats], the eight 16-byte slots of a row swizzled by (row & 7) as
      // staged in shared memory, so each warp moves its 32 rows of a chunk with one 4 KB bulk copy.
      float* part = P.partial + (size_t)u * (BM * BN);
#pragma unroll 1
      for (int j = eg; j < BN / 32; j += 2) {                       // this group's chunks
        if (col0 + j * 32 >= P.d_in) break;                         // warp-uniform
        uint8_t* buf8 = stage0;
        uint32_t v[32];
        tmem_ld32(taddr + (uint32_t)(j * 32), v);
        if (j >= 2) { if (lane == 0) bulk_wait_read_0(); __syncwarp(); }
        uint4* myrow = reinterpret_cast<uint4*>(buf8 + lane * 128);
#pragma unroll
        for (int g4 = 0; g4 < 8; ++g4)
          myrow[(uint32_t)g4 ^ swz] = make_uint4(v[g4 * 4], v[g4 * 4 + 1], v[g4 * 4 + 2], v[g4 * 4 + 3]);
        fence_async_smem();
        __syncwarp();
        if (lane == 0) {
          bulk_store(part + (size_t)j * (BM * 32) + (size_t)(eq * 32) * 32, buf8, EPI_WARP_BYTES);
          bulk_commit();
        }
      }
      tc_fence_before();
      mbar_arrive(&s.tmem_empty[buf]);          // the accumulator is free again
      if (lane == 0) bulk_wait_all();           // this warp's part of the partial tile is in global memory;
      __syncwarp();                             // the launch that follows adds the slices (slice_reduce_kernel)
      }  // !LEAN
    }
    // sliced instance: zero tiles are taken from the far end of the grid first, where CTAs have no product units
    if constexpr (!LEAN) {
      for (int z = (int)gridDim.x - 1 - (int)blockIdx.x; z < D.zero_tiles && ok; z += gridDim.x) zero_tile(z);
    }
  }
  if (warp != 4 && warp != 5 && lane == 0) bulk_wait_all();     // the bulk stores of zero tiles are only waited for here
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (warp == 5) { tc_fence_after(); tmem_dealloc(tmem_base, TMEM_COLS); }
}

// Adds the S partial tiles of every product tile of a sliced launch in slice order and writes the output
// (dX: rescaled by 1/p_n, optional GELU', rounded to bf16; dW: fp32).  Launched behind the product kernel as a
// programmatic dependent; it derives the same tiles and slices from the device-resident counts.  One thread per
// 8 consecutive columns of one output row: it reads two 16-byte slots of every slice (through L2, where the
// product has just put them) and stores 16 or 32 bytes, so consecutive threads write consecutive bytes.  A partial
// tile is laid out [32-column chunk][row][32 floats] with the eight 16-byte slots of a row swizzled by (row & 7),
// as the product's epilogue staged it.
constexpr int REDUCE_THREADS = 256;
template <int MODE, int BN>
__global__ void __launch_bounds__(REDUCE_THREADS) slice_reduce_kernel(GemmParams P) {
  pdl_wait();      // the partial tiles come from the product kernel before this one
  pdl_trigger();
  const Decomp D = decompose<MODE, BN, 1, false>(P);
  if (D.gemm_tiles <= 0) return;
  constexpr int C8 = BN / 8;                       // 8-column groups per tile row
  constexpr int PER_TILE = BM * C8;
  const long total = (long)D.gemm_tiles * PER_TILE;
  const size_t ld = (size_t)P.d_in;
  for (long it = (long)blockIdx.x * REDUCE_THREADS + threadIdx.x; it < total; it += (long)gridDim.x * REDUCE_THREADS) {
    const int tile = (int)(it / PER_TILE);
    const int rem = (int)(it - (long)tile * PER_TILE);
    const int r = rem / C8, c8 = rem - r * C8;
    int k, c0, c1;
    tile_coords<MODE>(P, D, tile, k, c0, c1);
    size_t row0;
    int rows_valid;
    float sc = 1.0f;
    if (MODE == MODE_DX) {
      const int n = P.dense ? k : P.idxA[k];
      row0 = (size_t)n * P.T + (size_t)c0 * BM;
      rows_valid = min(BM, P.T - c0 * BM);
      if (!P.dense) sc = P.scaleA[n];
    } else {
      row0 = (size_t)c0 * BM;
      rows_valid = min(BM, P.d_out - c0 * BM);
    }
    const int col = c1 * BN + c8 * 8;
    if (r >= rows_valid || col >= P.d_in) continue;
    const float* tile_part = P.partial + (size_t)tile * D.S * (BM * BN);
    const size_t chunk = (size_t)(c8 >> 2) * (BM * 32) + (size_t)r * 32;
    const size_t o0 = chunk + (size_t)((((c8 & 3) * 2 + 0) ^ (r & 7)) * 4);
    const size_t o1 = chunk + (size_t)((((c8 & 3) * 2 + 1) ^ (r & 7)) * 4);
    float f[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int sl0 = 0; sl0 < D.S; sl0 += 4) {         // slices in order, four at a time in flight
      float4 x[4][2];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float* src = tile_part + (size_t)min(sl0 + q, D.S - 1) * (BM * BN);
        x[q][0] = __ldcg(reinterpret_cast<const float4*>(src + o0));
        x[q][1] = __ldcg(reinterpret_cast<const float4*>(src + o1));
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        if (sl0 + q < D.S) {
          f[0] += x[q][0].x; f[1] += x[q][0].y; f[2] += x[q][0].z; f[3] += x[q][0].w;
          f[4] += x[q][1].x; f[5] += x[q][1].y; f[6] += x[q][1].z; f[7] += x[q][1].w;
        }
      }
    }
    const size_t off = (row0 + r) * ld + col;
    if (MODE == MODE_DX) {
      float v[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) v[e] = sc * f[e];
      if (P.H != nullptr) {
        const uint4 hv = __ldg(reinterpret_cast<const uint4*>(P.H + off));
        const uint32_t hu[4] = {hv.x, hv.y, hv.z, hv.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          v[2 * e] *= gelu_prime(__uint_as_float(hu[e] << 16));
          v[2 * e + 1] *= gelu_prime(__uint_as_float(hu[e] & 0xffff0000u));
        }
      }
      uint4 o;
      o.x = pack_bf16(v[0], v[1]); o.y = pack_bf16(v[2], v[3]);
      o.z = pack_bf16(v[4], v[5]); o.w = pack_bf16(v[6], v[7]);
      *reinterpret_cast<uint4*>(P.dX + off) = o;
    } else {
      *reinterpret_cast<float4*>(P.dW + off) = make_float4(f[0], f[1], f[2], f[3]);
      *reinterpret_cast<float4*>(P.dW + off + 4) = make_float4(f[4], f[5], f[6], f[7]);
    }
  }
}

// ------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static const EncodeTiledFn fn = []() -> EncodeTiledFn {     // initialised once, thread-safe
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      return (EncodeTiledFn)p;
    return nullptr;
  }();
  return fn;
}

// tensor of `rank` dims (innermost first), 128-byte swizzle; out-of-bounds reads give 0, out-of-bounds
// parts of a store are dropped
bool make_map(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
              const uint32_t* box, CUtensorMapDataType dtype = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t gd[3]; cuuint64_t gs[2]; cuuint32_t bx[3]; cuuint32_t es[3] = {1, 1, 1};
  for (int i = 0; i < rank; ++i) { gd[i] = dims[i]; bx[i] = box[i]; }
  for (int i = 0; i + 1 < rank; ++i) gs[i] = strides_bytes[i];
  return fn(m, dtype, (cuuint32_t)rank, const_cast<void*>(base), gd, gs, bx, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tile shape and number of contraction slices from a small cost model of the kernel instances (per
// unit of work, so independent of the layer's shape), fitted to serialised stage times of every tiling
// on five layer shapes on B200: a k-block costs about 0.50 / 0.45 / 0.43 us for 256 / 128 / 64 wide
// 128-row tiles (the shared-memory fill rate of one SM bounds it, so narrow tiles only pay off when
// they fill more SMs); a unit costs about 4 us of set-up, pipeline fill and output store; a sliced unit
// stores its partial tile instead, and the reduction launch that follows adds the slices on all SMs:
// together about 11 us + 1 us per slice; a 256 x 256 tile (mh = 2) costs about 0.66 us per k-block for
// twice the work, and 7 us per tile.
constexpr double SLICED_US = 11.0, SLICED_PER_SLICE_US = 1.0;
struct Cand {
  Plan plan;
  long units;      // (tile, slice) units
  double unit;     // time of one unit, us
  double alone;    // time of the product when it has the GPU to itself, us
};
constexpr int MAX_CANDS = 64;
constexpr int MAX_DEVICES = 64;

// row_tiles128: number of 128-row tile rows (for dX: kept data x 128-token chunks); a 256-row tile covers two.
// remainder_ok: 256-row tiles may leave a last partial wave to a second launch with 128-row tiles (mh = 3).
int enumerate_plans(long row_tiles128, long row_tiles256, int n_extent, int kblocks, int num_sms, int max_units,
                    int force_bn, int force_split, bool remainder_ok, Cand* out) {
  const int widths[3] = {256, 128, 64};
  const double c_kb[3] = {0.50, 0.45, 0.43};
  int n = 0;
  if (kblocks < 1) kblocks = 1;
  for (int i = 0; i < 3; ++i) {
    if (force_bn != 0 && widths[i] != force_bn) continue;
    if (force_bn == 0 && widths[i] > 64 && n_extent <= widths[i] / 2) continue;   // mostly padding
    const long ntiles = (n_extent + widths[i] - 1) / widths[i];
    const long tiles = row_tiles128 * ntiles;
    for (int sp = 1; sp <= 16; ++sp) {
      if (force_split != 0 && sp != force_split) continue;
      if (force_split == 0 && sp > 4 && (sp & 1) != 0) continue;       // 1, 2, 3, 4, 6, 8, ... 16
      if (sp > 1 && tiles * sp > max_units) continue;
      if (sp > 1 && force_split == 0 && kblocks / sp < 4) continue;   // slices too short to pay off
      const long units = tiles * sp;
      const double waves = (double)((units + num_sms - 1) / num_sms);
      const double unit = (double)((kblocks + sp - 1) / sp) * c_kb[i] + (sp > 1 ? SLICED_US + SLICED_PER_SLICE_US * sp : 4.0);
      if (n < MAX_CANDS) out[n++] = {{widths[i], sp, 1}, units, unit, waves * unit};
    }
    if (widths[i] == 256 && force_split <= 1) {                        // 256 x 256 tiles, never sliced
      const long units = row_tiles256 * ntiles;
      const double wave = (double)kblocks * 0.66 + 7.0;
      if (n < MAX_CANDS) out[n++] = {{256, 1, 2}, units, wave, (double)((units + num_sms - 1) / num_sms) * wave};
      const long frac = units % num_sms;
      if (remainder_ok && frac > 0 && 2 * frac <= num_sms) {            // whole waves, then the rest as sliced 128-row tiles
        long sp = num_sms / (2 * frac);
        if (sp > 8) sp = 8;
        if (sp > kblocks / 4) sp = kblocks / 4;
        if (sp < 1) sp = 1;
        // the second launch always runs the sliced instance (its tiles go through the slice exchange even when
        // a contraction ends up in one slice), and costs a launch of its own
        const double tail = (double)((kblocks + sp - 1) / sp) * 0.50 + SLICED_US + SLICED_PER_SLICE_US * (double)sp + 4.0;
        if (n < MAX_CANDS) out[n++] = {{256, 1, 3}, units, wave, (double)(units / num_sms) * wave + tail};
      }
    }
  }
  if (n == 0) out[n++] = {{256, 1, 1}, 1, 1.0, 1.0};
  return n;
}

// the tile-height override of vcas_set_tuning, applied to a chosen plan
Plan apply_tile_m(int tile_m, Plan plan, bool remainder_ok) {
  if (tile_m == 1) plan.mh = 1;
  if (tile_m == 2 && plan.bn == 256) { plan.mh = 2; plan.split = 1; }
  if (tile_m == 3 && plan.bn == 256 && remainder_ok) { plan.mh = 3; plan.split = 1; }
  return plan;
}

Plan best_alone(const Cand* c, int n) {
  int b = 0;
  for (int i = 1; i < n; ++i)
    if (c[i].alone < c[b].alone - 1e-9) b = i;
  return c[b].plan;
}

// The two products of one call run at the same time on two streams.  Model: the first product's CTAs are
// resident from time 0 and leave after their last unit (a grid whose last wave is partial frees the CTAs without
// a unit in it one unit time earlier); the second product becomes ready `offset` us later and works its units
// off on the SMs that are free at the time - a persistent CTA of the second grid simply starts when an SM frees
// up and draws units until none are left.  (Measured on the BERT-base layer: a dense call takes 63 us when the
// two grids together exceed the SMs and every unit of the second waits for the first, 52 us when the dW product
// runs as 36 tiles of 256 x 256 beside the 96 CTAs of the dX product.)
constexpr double KERNEL_US = 3.0;   // launch ramp and exit of a product kernel, on top of its units (timeline measurements)

// Finish time of the second product: `units` units of `unit` us each, ready at `ready`, on the SMs the first
// product (g1 CTAs, `units1` units of `unit1` us) leaves free.
// slices > 1: the sliced instance assigns its units to CTAs in advance (CTA i takes units i, i + upi, ...), so the
// CTAs that start first are also the ones with the most units.
double second_end(long units, double unit, long g2, int slices, double ready, long g1, long units1, double unit1,
                  int num_sms) {
  const long full = units1 / g1, rest = units1 % g1;
  // phases of the first product: [0, full * unit1) all g1 CTAs busy; [full * unit1, (full + 1) * unit1) only
  // `rest` of them (if any); afterwards none
  const double t_a = (double)full * unit1 + KERNEL_US;
  const double t_b = rest > 0 ? t_a + unit1 : t_a;
  const long busy[3] = {g1, rest, 0};
  const double from[3] = {0.0, t_a, t_b};
  const double to[3] = {t_a, t_b, 1e30};
  long left = units;
  double end = ready;
  bool started = false;
  for (int ph = 0; ph < 3 && left > 0; ++ph) {
    long sms = num_sms - busy[ph];
    if (sms > g2) sms = g2;
    const double t0 = ready > from[ph] ? ready : from[ph];
    if (sms <= 0 || t0 >= to[ph]) continue;
    if (!started && slices > 1) {
      const long upi = (g2 / slices) * slices;
      const long most = upi > 0 ? (units + upi - 1) / upi : units;
      end = t0 + (double)most * unit;
    }
    started = true;
    // units that start in this phase (a unit started before the phase ends is finished by its CTA)
    const double span = to[ph] - t0;
    long rounds = ph == 2 ? (left + sms - 1) / sms : (long)(span / unit) + 1;
    long can = rounds * sms;
    if (can > left) { can = left; rounds = (left + sms - 1) / sms; }
    left -= can;
    const double e = t0 + (double)rounds * unit;
    if (e > end) end = e;
  }
  return end + KERNEL_US;
}

void best_pair(const Cand* c1, int n1, int ctas1, const Cand* c2, int n2, int ctas2, int num_sms, double offset,
               Plan* p1, Plan* p2) {
  double best = 1e30;
  *p1 = c1[0].plan; *p2 = c2[0].plan;
  for (int i = 0; i < n1; ++i) {
    const bool split1 = c1[i].plan.mh == 3;
    const long g1 = split1 || c1[i].units > ctas1 ? ctas1 : c1[i].units;
    const double d1 = (split1 ? c1[i].alone : (double)((c1[i].units + g1 - 1) / g1) * c1[i].unit) + KERNEL_US;
    for (int j = 0; j < n2; ++j) {
      const bool split2 = c2[j].plan.mh == 3;
      const long g2 = split2 || c2[j].units > ctas2 ? ctas2 : c2[j].units;
      double end2;
      if (split1 || split2) {
        // a product in two launches: its time alone, after the first product unless both grids fit side by side
        const double d2 = (split2 ? c2[j].alone : (double)((c2[j].units + g2 - 1) / g2) * c2[j].unit) + KERNEL_US;
        const double start2 = g2 <= num_sms - g1 ? offset : (offset > d1 ? offset : d1);
        end2 = start2 + d2;
      } else {
        end2 = second_end(c2[j].units, c2[j].unit, g2, c2[j].plan.split, offset, g1, c1[i].units, c1[i].unit, num_sms);
      }
      const double end = d1 > end2 ? d1 : end2;
      // ties: the pair whose products finish earlier, then the one with less SM time
      const double sm_time = (double)c1[i].units * c1[i].unit + (double)c2[j].units * c2[j].unit;
      const double t = end + 0.02 * (d1 + end2) + 1e-3 * sm_time / num_sms;
      if (t < best - 1e-9) { best = t; *p1 = c1[i].plan; *p2 = c2[j].plan; }
    }
  }
}

template <int MODE, int BN, int MH, int KIND>
cudaError_t run_gemm_k(Handle* h, const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& c, const GemmParams& P0,
                     long max_items, int ctas, bool pdl, cudaStream_t st) {
  // the opt-in to large dynamic shared memory is a per-device attribute of the kernel
  static std::atomic<bool> attr_set[MAX_DEVICES];
  if (h->device < 0 || h->device >= MAX_DEVICES) return cudaErrorInvalidDevice;
  if (!attr_set[h->device].load(std::memory_order_acquire)) {
    cudaError_t e = cudaFuncSetAttribute(umma_kernel<MODE, BN, MH, KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         TileCfg<BN, MH>::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attr_set[h->device].store(true, std::memory_order_release);
  }
  GemmParams P = P0;
  P.grid_ctas = (int)(max_items < ctas ? max_items : ctas);
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  cfg.blockDim = dim3(NUM_THREADS);
  cfg.dynamicSmemBytes = (size_t)TileCfg<BN, MH>::SMEM_BYTES;
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = 0;
  int grid = (int)(max_items < ctas ? max_items : ctas);
  if (pdl) {
    attr[cfg.numAttrs].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[cfg.numAttrs].val.programmaticStreamSerializationAllowed = 1;
    cfg.numAttrs += 1;
  }
  cfg.gridDim = dim3((unsigned)grid);
  cudaError_t e = cudaLaunchKernelEx(&cfg, umma_kernel<MODE, BN, MH, KIND>, a, b, c, P);
  h->launches += 1;
  if (e != cudaSuccess) return e;
  if constexpr (KIND == KIND_SLICED) {
    // the slices are added by a launch of their own on all SMs: one thread per 8 columns of an output row of the
    // most tiles the product can have (the kernel strides over what the device-resident counts leave)
    const long max_tiles = P.split_k > 0 ? max_items / P.split_k : max_items;
    long blocks = (max_tiles * BM * (BN / 8) + REDUCE_THREADS - 1) / REDUCE_THREADS;
    const long cap = (long)h->num_sms * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    e = launch_after(slice_reduce_kernel<MODE, BN>, dim3((unsigned)blocks), dim3(REDUCE_THREADS), 0, st, P);
    h->launches += 1;
    if (e != cudaSuccess) return e;
  }
  return cudaGetLastError();
}

template <int MODE, int BN, int MH>
cudaError_t run_gemm(Handle* h, const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& c, const GemmParams& P,
                     long max_items, int ctas, bool pdl, cudaStream_t st) {
  const bool many = max_items > ctas;      // more work items than CTAs: dynamic order
  if constexpr (MH == 2) {
    if (many) return run_gemm_k<MODE, BN, MH, KIND_DYNAMIC>(h, a, b, c, P, max_items, ctas, pdl, st);
    return run_gemm_k<MODE, BN, MH, KIND_STATIC>(h, a, b, c, P, max_items, ctas, pdl, st);
  } else {
    if (P.split_k != 1) return run_gemm_k<MODE, BN, MH, KIND_SLICED>(h, a, b, c, P, max_items, ctas, pdl, st);
    if (many) return run_gemm_k<MODE, BN, MH, KIND_DYNAMIC>(h, a, b, c, P, max_items, ctas, pdl, st);
    return run_gemm_k<MODE, BN, MH, KIND_STATIC>(h, a, b, c, P, max_items, ctas, pdl, st);
  }
}

template <int MODE>
cudaError_t run_gemm_bn(Handle* h, const Plan& plan, const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& c,
                        const GemmParams& P, long max_items, int ctas, bool pdl, cudaStream_t st) {
  if (plan.mh == 3) {
    // whole waves of 256-row tiles, then the remaining tiles as 128-row tiles with a sliced contraction
    // (both launches derive the same division from the device-resident counts)
    GemmParams Q = P;
    Q.split_k = 1;
    Q.part = 1;
    Q.head_ctas = (int)(max_items < ctas ? max_items : ctas);
    const cudaError_t e = run_gemm<MODE, 256, 2>(h, a, b, c, Q, max_items, ctas, pdl, st);
    if (e != cudaSuccess) return e;
    Q.part = 2;
    Q.split_k = 0;
    return run_gemm<MODE, 256, 1>(h, a, b, c, Q, (long)ctas, ctas, true, st);
  }
  if (plan.mh == 2) return run_gemm<MODE, 256, 2>(h, a, b, c, P, max_items, ctas, pdl, st);
  switch (plan.bn) {
    case 256: return run_gemm<MODE, 256, 1>(h, a, b, c, P, max_items, ctas, pdl, st);
    case 128: return run_gemm<MODE, 128, 1>(h, a, b, c, P, max_items, ctas, pdl, st);
    default: return run_gemm<MODE, 64, 1>(h, a, b, c, P, max_items, ctas, pdl, st);
  }
}

void common_params(Handle* h, GemmParams& P, int which) {
  P = GemmParams();
  P.status = h->ws.status;
  P.partial = h->ws.partial_tiles + (size_t)which * h->max_units * (BM * 256);
  P.sched = h->ws.sched + which * 2;
  P.max_units = h->max_units;
  P.wait_limit_ns = h->wait_limit_ns;
  P.stall_once = h->stall_once;
  P.d_in = h->desc.d_in;
  P.d_out = h->desc.d_out;
}

}  // namespace

namespace {
struct DxShape { long row_tiles128, row_tiles256; int kblocks; bool rem_ok; };
DxShape dx_shape(const Handle* h, bool dense, float rho_hint) {
  const vcas_layer_desc& d = h->desc;
  double kept = dense ? (double)d.N : (double)rho_hint * d.N;
  if (kept < 1.0) kept = 1.0;
  const long nk = (long)(kept + 0.5);
  DxShape g;
  g.row_tiles128 = nk * ((d.T + BM - 1) / BM);
  g.row_tiles256 = nk * ((d.T + 2 * BM - 1) / (2 * BM));
  g.kblocks = (d.d_out + BK - 1) / BK;
  // the halves of a 256-row tile must both hold rows for the remainder launch to take them over
  g.rem_ok = h->tune_dx_tile_m != 2 && ((d.T % (2 * BM)) == 0 || (d.T % (2 * BM)) > BM);
  return g;
}
bool dw_remainder_ok(const Handle* h) {
  const int d_out = h->desc.d_out;
  return h->tune_dw_tile_m != 2 && ((d_out % (2 * BM)) == 0 || (d_out % (2 * BM)) > BM);
}
}  // namespace

void plan_products(Handle* h, bool dense, float rho_hint, int cnt_hint, int spare_sms, bool row_norms_out, Plan* dx,
                   Plan* dw) {
  const vcas_layer_desc& d = h->desc;
  const DxShape g = dx_shape(h, dense, rho_hint);
  const int kb_w = (cnt_hint + BK - 1) / BK;
  const int key[PLAN_KEY_INTS] = {(dense ? 1 : 0) | (row_norms_out ? 2 : 0), (int)g.row_tiles128, kb_w, spare_sms,
                                  h->tune_dx_tile_n, h->tune_dw_tile_n, h->tune_dx_split_k, h->tune_dw_split_k,
                                  h->tune_dx_tile_m + 4 * h->tune_dw_tile_m};
  bool hit = h->plan_valid;
  for (int i = 0; i < PLAN_KEY_INTS && hit; ++i) hit = h->plan_key[i] == key[i];
  if (!hit) {
    for (int e = 0; e < h->plan_cache_used && !hit; ++e) {
      bool same = true;
      for (int i = 0; i < PLAN_KEY_INTS && same; ++i) same = h->plan_cache_key[e][i] == key[i];
      if (same) {
        h->plan_dx = h->plan_cache_dx[e];
        h->plan_dw = h->plan_cache_dw[e];
        for (int i = 0; i < PLAN_KEY_INTS; ++i) h->plan_key[i] = key[i];
        h->plan_valid = true;
        hit = true;
      }
    }
  }
  if (!hit) {
    const int ctas = h->num_sms - spare_sms > 1 ? h->num_sms - spare_sms : 1;
    Cand cx[MAX_CANDS], cw[MAX_CANDS];
    // the epilogue emits row square-norms of dX only from unsliced 256-wide tiles (one partial sum per tile)
    const int nx = enumerate_plans(g.row_tiles128, g.row_tiles256, d.d_in, g.kblocks, ctas, h->max_units,
                                   row_norms_out ? 256 : h->tune_dx_tile_n, row_norms_out ? 1 : h->tune_dx_split_k,
                                   g.rem_ok && !row_norms_out, cx);
    const bool rem_w = dw_remainder_ok(h);
    const int nw = enumerate_plans((d.d_out + BM - 1) / BM, (d.d_out + 2 * BM - 1) / (2 * BM), d.d_in, kb_w, h->num_sms,
                                   h->max_units, h->tune_dw_tile_n, h->tune_dw_split_k, rem_w, cw);
    // A sampled dW product becomes ready later than the dX product by the time of the kernels in front of it
    // on the side stream (fitted to their ncu durations on three layer shapes): the norms of the kept rows of X
    // (HBM-bound), SampleW's single-CTA fixed point over the rows of kept data, and the emit + pack pass, which
    // moves the kept rows of both operands twice.  The dense products start together.
    double offset = 0.0;
    if (!dense) {
      const double rows_a = (double)rho_hint * d.N * d.T;
      const double scores_us = 4.0 + rows_a * d.d_in * 2.0 / 3.5e6;
      const double sample_w_us = 6.0 + rows_a * 0.0013;
      const double pack_us = 6.0 + 2.0 * (double)cnt_hint * (d.d_in + d.d_out) * 2.0 / 3.0e6;
      offset = scores_us + sample_w_us + pack_us;
    }
    Plan px, pw;
    best_pair(cx, nx, ctas, cw, nw, h->num_sms, h->num_sms, offset, &px, &pw);
    h->plan_dx = apply_tile_m(h->tune_dx_tile_m, px, g.rem_ok && !row_norms_out);
    h->plan_dw = apply_tile_m(h->tune_dw_tile_m, pw, rem_w);
    for (int i = 0; i < PLAN_KEY_INTS; ++i) h->plan_key[i] = key[i];
    h->plan_valid = true;
    const int e = h->plan_cache_next;
    for (int i = 0; i < PLAN_KEY_INTS; ++i) h->plan_cache_key[e][i] = key[i];
    h->plan_cache_dx[e] = h->plan_dx;
    h->plan_cache_dw[e] = h->plan_dw;
    h->plan_cache_next = (e + 1) % PLAN_CACHE;
    if (h->plan_cache_used < PLAN_CACHE) h->plan_cache_used += 1;
  }
  *dx = h->plan_dx;
  *dw = h->plan_dw;
}

cudaError_t launch_umma_dx(Handle* h, const void* dY, const void* W, bool dense, float rho_hint, const void* H,
                           void* dX, float* a_out, bool skip_dropped, int spare_sms, const Plan* pair_plan,
                           cudaStream_t st) {
  const vcas_layer_desc& d = h->desc;
  CUtensorMap tmA, tmB, tmC;
  {
    const uint64_t dims[3] = {(uint64_t)d.d_out, (uint64_t)d.T, (uint64_t)d.N};
    const uint64_t strides[2] = {(uint64_t)d.d_out * 2, (uint64_t)d.T * d.d_out * 2};
    const uint32_t box[3] = {BK, (uint32_t)(d.T < BM ? d.T : BM), 1};
    if (!make_map(&tmA, dY, 3, dims, strides, box)) return cudaErrorInvalidValue;
  }
  {
    const uint64_t dims[2] = {(uint64_t)d.d_in, (uint64_t)d.d_out};
    const uint64_t strides[1] = {(uint64_t)d.d_in * 2};
    const uint32_t box[2] = {64, BK};
    if (!make_map(&tmB, W, 2, dims, strides, box)) return cudaErrorInvalidValue;
  }
  {
    const uint64_t dims[3] = {(uint64_t)d.d_in, (uint64_t)d.T, (uint64_t)d.N};
    const uint64_t strides[2] = {(uint64_t)d.d_in * 2, (uint64_t)d.T * d.d_in * 2};
    const uint32_t box[3] = {64, (uint32_t)(d.T < 32 ? d.T : 32), 1};
    if (!make_map(&tmC, dX, 3, dims, strides, box)) return cudaErrorInvalidValue;
  }
  GemmParams P;
  common_params(h, P, 0);
  P.idxA = h->ws.idxA; P.dropA = h->ws.dropA; P.counts = h->ws.counts; P.scaleA = h->ws.scaleA;
  P.a_out = a_out; P.a_parts = a_out_parts(d.d_in);
  P.H = (const __nv_bfloat16*)H; P.dX = (__nv_bfloat16*)dX;
  P.N = d.N; P.T = d.T; P.dense = dense ? 1 : 0;
  P.skip_dropped = skip_dropped ? 1 : 0;
  P.a_tx_bytes = (d.T < BM ? d.T : BM) * BK * 2;
  const int chunks = (d.T + BM - 1) / BM, chunks2 = (d.T + 2 * BM - 1) / (2 * BM);
  const int ctas = h->num_sms - spare_sms > 1 ? h->num_sms - spare_sms : 1;
  Plan plan;
  if (pair_plan != nullptr) {
    plan = *pair_plan;
  } else {
    DxShape g = dx_shape(h, dense, rho_hint);
    Cand cands[MAX_CANDS];
    const bool rn = a_out != nullptr;
    const int n = enumerate_plans(g.row_tiles128, g.row_tiles256, d.d_in, g.kblocks, ctas, h->max_units,
                                  rn ? 256 : h->tune_dx_tile_n, rn ? 1 : h->tune_dx_split_k, g.rem_ok && !rn, cands);
    plan = apply_tile_m(h->tune_dx_tile_m, best_alone(cands, n), g.rem_ok && !rn);
  }
  P.split_k = plan.split;
  // upper bound of work items: every datum kept and split, or every datum a zero tile
  const long max_items = (long)d.N * (plan.mh >= 2 ? chunks2 : chunks) * ((d.d_in + plan.bn - 1) / plan.bn) * plan.split;
  return run_gemm_bn<MODE_DX>(h, plan, tmA, tmB, tmC, P, max_items, ctas, true, st);
}

cudaError_t launch_umma_dw(Handle* h, const void* A_rows, const void* B_rows, int rows_capacity, const int32_t* cnt,
                           int cnt_hint, const Plan* pair_plan, float* dW, cudaStream_t st) {
  const vcas_layer_desc& d = h->desc;
  CUtensorMap tmA, tmB, tmC;
  {
    const uint64_t dims[2] = {(uint64_t)d.d_out, (uint64_t)rows_capacity};
    const uint64_t strides[1] = {(uint64_t)d.d_out * 2};
    const uint32_t box[2] = {64, BK};
    if (!make_map(&tmA, A_rows, 2, dims, strides, box)) return cudaErrorInvalidValue;
  }
  {
    const uint64_t dims[2] = {(uint64_t)d.d_in, (uint64_t)rows_capacity};
    const uint64_t strides[1] = {(uint64_t)d.d_in * 2};
    const uint32_t box[2] = {64, BK};
    if (!make_map(&tmB, B_rows, 2, dims, strides, box)) return cudaErrorInvalidValue;
  }
  {
    const uint64_t dims[2] = {(uint64_t)d.d_in, (uint64_t)d.d_out};
    const uint64_t strides[1] = {(uint64_t)d.d_in * 4};
    const uint32_t box[2] = {32, 32};
    if (!make_map(&tmC, dW, 2, dims, strides, box, CU_TENSOR_MAP_DATA_TYPE_FLOAT32)) return cudaErrorInvalidValue;
  }
  GemmParams P;
  common_params(h, P, 1);
  P.cnt = cnt; P.dW = dW;
  const long mtiles = (d.d_out + BM - 1) / BM, mtiles2 = (d.d_out + 2 * BM - 1) / (2 * BM);
  Plan plan;
  if (pair_plan != nullptr) {
    plan = *pair_plan;
  } else {
    const bool rem_ok = dw_remainder_ok(h);
    Cand cands[MAX_CANDS];
    const int n = enumerate_plans(mtiles, mtiles2, d.d_in, (cnt_hint + BK - 1) / BK, h->num_sms, h->max_units,
                                  h->tune_dw_tile_n, h->tune_dw_split_k, rem_ok, cands);
    plan = apply_tile_m(h->tune_dw_tile_m, best_alone(cands, n), rem_ok);
  }
  P.split_k = plan.split;
  const long max_items = (plan.mh >= 2 ? mtiles2 : mtiles) * ((d.d_in + plan.bn - 1) / plan.bn) * plan.split;
  return run_gemm_bn<MODE_DW>(h, plan, tmA, tmB, tmC, P, max_items, h->num_sms, true, st);
}

}  // namespace vcas
