// The two products of the sampled backward on the 5th-generation tensor cores (tcgen05):
//   dX[rows of kept data] = (1/p_n) dY[rows] W          (App. E; rows of dropped data are zero-filled)
//   dW = A_rows^T B_rows over the compacted kept rows    (Sec. 4.2: G_tilde^T X)
// One persistent CTA per SM walks a tile list whose length depends on the kept counts, which
// are read from device memory.  Per CTA: warps 0-3 are the epilogue (TMEM -> registers ->
// global), warp 4 issues TMA loads into a ring of shared-memory stages, warp 5 issues
// tcgen05.mma into one of two TMEM accumulators, so the epilogue of a tile overlaps the main
// loop of the next one.  bf16 operands, fp32 accumulation.  Every mbarrier wait is bounded:
// when it runs out the CTA records VCAS_ERR_TIMEOUT in the status word and leaves.
#include <cuda.h>

#include "common.cuh"

namespace vcas {
namespace {

constexpr int BM = 128;          // tile rows (UMMA M)
constexpr int BK = 64;           // k-block: 64 bf16 = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int A_BYTES = BM * BK * 2;
constexpr int CHUNK_BYTES = 64 * BK * 2;   // one 64-wide MN chunk of an MN-major operand
constexpr int NUM_THREADS = 192;
constexpr int TMEM_COLS = 512;
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;

template <int BN> struct TileCfg {
  static constexpr int B_BYTES = BN * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = BN == 256 ? 4 : (BN == 128 ? 6 : 8);
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
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
// Waits for the phase with the given parity; gives up after WAIT_LIMIT_NS or when another
// role of this CTA has given up.  Returns false in that case.
__device__ __noinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int32_t* status) {
  unsigned long long t0 = 0;
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 0xfffu) == 0) {
      if (*abort_flag) return false;
      const unsigned long long now = global_ns();
      if (t0 == 0) {
        t0 = now;
      } else if (now - t0 > WAIT_LIMIT_NS) {
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

struct SmemLayout {
  uint8_t* stages;
  uint64_t* full;
  uint64_t* empty;
  uint64_t* tmem_full;
  uint64_t* tmem_empty;
  uint32_t* tmem_holder;
  int* abort_flag;
};

template <int BN>
__device__ __forceinline__ SmemLayout carve(uint8_t* raw) {
  using C = TileCfg<BN>;
  SmemLayout s;
  uint8_t* base = (uint8_t*)(((uintptr_t)raw + 1023) & ~(uintptr_t)1023);
  s.stages = base;
  uint64_t* bars = (uint64_t*)(base + C::STAGES * C::STAGE_BYTES);
  s.full = bars;
  s.empty = bars + C::STAGES;
  s.tmem_full = bars + 2 * C::STAGES;
  s.tmem_empty = bars + 2 * C::STAGES + 2;
  s.tmem_holder = (uint32_t*)(bars + 2 * C::STAGES + 4);
  s.abort_flag = (int*)(s.tmem_holder + 1);
  return s;
}

template <int BN>
__device__ __forceinline__ uint32_t setup(const SmemLayout& s, int warp, int tid) {
  using C = TileCfg<BN>;
  if (tid == 0) {
    for (int i = 0; i < C::STAGES; ++i) { mbar_init(&s.full[i], 1); mbar_init(&s.empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&s.tmem_full[i], 1); mbar_init(&s.tmem_empty[i], 128); }
    *s.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 5) tmem_alloc(s.tmem_holder, TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  return *(volatile uint32_t*)s.tmem_holder;
}

__device__ __forceinline__ float gelu_prime(float x) {
  const float Phi = 0.5f * (1.0f + erff(x * 0.70710678118654752f));
  const float phi = 0.39894228040143268f * expf(-0.5f * x * x);
  return fmaf(x, phi, Phi);
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// ------------------------------------------------------------------------------ dX kernel
struct DxParams {
  const int32_t* idxA;     // kept data
  const int32_t* dropA;    // dropped data
  const int32_t* counts;   // counts[0] = number of kept data
  const float* scaleA;     // 1/p_n per datum
  const __nv_bfloat16* H;  // optional GELU pre-activation [R, d_in]
  __nv_bfloat16* dX;       // [R, d_in]
  int32_t* status;
  int N, T, d_in, d_out;
  int dense;               // 1: every datum kept with scale 1
  int a_tx_bytes;          // bytes one A box delivers (min(T, 128) token rows of 128 B)
};

// A = dY viewed [N][T][d_out] (K-major, one TMA box = 128 tokens x 64 k of one datum),
// B = W [d_out][d_in] (MN-major: n contiguous), D = 128 x BN fp32 in TMEM.
template <int BN>
__global__ void __launch_bounds__(NUM_THREADS, 1)
umma_dx_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, DxParams P) {
  using C = TileCfg<BN>;
  extern __shared__ uint8_t smem_raw[];
  const SmemLayout s = carve<BN>(smem_raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t tmem_base = setup<BN>(s, warp, tid);
  volatile int* abort_flag = s.abort_flag;

  const int cntA = P.dense ? P.N : P.counts[0];
  const int chunks = (P.T + BM - 1) / BM;
  const int ntiles = (P.d_in + BN - 1) / BN;
  const int per_datum = chunks * ntiles;
  const int gemm_tiles = cntA * per_datum;
  const int total_tiles = P.N * per_datum;
  const int kblocks = (P.d_out + BK - 1) / BK;

  if (warp == 4) {
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      for (int tile = blockIdx.x; tile < gemm_tiles; tile += gridDim.x) {
        const int k = tile / per_datum, rem = tile % per_datum;
        const int c = rem / ntiles, nt = rem % ntiles;
        const int n = P.dense ? k : P.idxA[k];
        bool ok = true;
        for (int kb = 0; kb < kblocks && ok; ++kb) {
          ok = mbar_wait(&s.empty[stage], phase ^ 1u, abort_flag, P.status);
          if (!ok) break;
          uint8_t* sa = s.stages + stage * C::STAGE_BYTES;
          mbar_expect_tx(&s.full[stage], (uint32_t)(P.a_tx_bytes + C::B_BYTES));
          tma_load_3d(sa, &tmA, kb * BK, c * BM, n, &s.full[stage]);
#pragma unroll
          for (int j = 0; j < BN / 64; ++j)
            tma_load_2d(sa + A_BYTES + j * CHUNK_BYTES, &tmB, nt * BN + j * 64, kb * BK, &s.full[stage]);
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
      }
    }
  } else if (warp == 5) {
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc(BN, false, true);
      int stage = 0; uint32_t phase = 0; int lt = 0;
      for (int tile = blockIdx.x; tile < gemm_tiles; tile += gridDim.x, ++lt) {
        const int buf = lt & 1; const uint32_t use = (uint32_t)(lt >> 1) & 1u;
        bool ok = mbar_wait(&s.tmem_empty[buf], use ^ 1u, abort_flag, P.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
        for (int kb = 0; kb < kblocks; ++kb) {
          ok = mbar_wait(&s.full[stage], phase, abort_flag, P.status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sa = smem_u32(s.stages + stage * C::STAGE_BYTES);
          const uint64_t da = desc_kmajor(sa), db = desc_mnmajor(sa + A_BYTES);
#pragma unroll
          for (int k4 = 0; k4 < BK / UMMA_K; ++k4)
            umma_bf16(d_tmem, da + (uint64_t)(k4 * (UMMA_K * 2 >> 4)), db + (uint64_t)(k4 * (UMMA_K * 128 >> 4)), idesc,
                      (kb | k4) != 0 ? 1u : 0u);
          umma_commit(&s.empty[stage]);
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit(&s.tmem_full[buf]);
      }
    }
  } else {
    // epilogue: thread (warp, lane) owns accumulator lane warp*32 + lane = tile row
    int lt = 0;
    const int row = warp * 32 + lane;
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
      const bool is_gemm = tile < gemm_tiles;
      const int t2 = is_gemm ? tile : tile - gemm_tiles;
      const int k = t2 / per_datum, rem = t2 % per_datum;
      const int c = rem / ntiles, nt = rem % ntiles;
      const int n = is_gemm ? (P.dense ? k : P.idxA[k]) : P.dropA[k];
      const int t = c * BM + row;
      const bool valid = t < P.T;
      const size_t off = ((size_t)n * P.T + (valid ? t : 0)) * P.d_in + (size_t)nt * BN;
      __nv_bfloat16* out = P.dX + off;
      if (!is_gemm) {
        if (valid) {
#pragma unroll
          for (int j = 0; j < BN / 8; ++j)
            if (nt * BN + j * 8 < P.d_in) *reinterpret_cast<uint4*>(out + j * 8) = make_uint4(0u, 0u, 0u, 0u);
        }
        continue;
      }
      const int buf = lt & 1; const uint32_t use = (uint32_t)(lt >> 1) & 1u;
      ++lt;
      if (!mbar_wait(&s.tmem_full[buf], use, abort_flag, P.status)) break;
      tc_fence_after();
      const float sc = P.dense ? 1.0f : P.scaleA[n];
      const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(buf * BN);
#pragma unroll 1
      for (int j = 0; j < BN / 32; ++j) {
        uint32_t v[32];
        tmem_ld32(taddr + (uint32_t)(j * 32), v);
        if (valid) {
#pragma unroll
          for (int g8 = 0; g8 < 4; ++g8) {
            const int col = nt * BN + j * 32 + g8 * 8;
            if (col < P.d_in) {
              float f[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) f[e] = sc * __uint_as_float(v[g8 * 8 + e]);
              if (P.H != nullptr) {
                const uint4 hv = *reinterpret_cast<const uint4*>(P.H + off + j * 32 + g8 * 8);
                const uint32_t hu[4] = {hv.x, hv.y, hv.z, hv.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  f[2 * e] *= gelu_prime(__uint_as_float(hu[e] << 16));
                  f[2 * e + 1] *= gelu_prime(__uint_as_float(hu[e] & 0xffff0000u));
                }
              }
              uint4 o;
              o.x = pack_bf16(f[0], f[1]); o.y = pack_bf16(f[2], f[3]);
              o.z = pack_bf16(f[4], f[5]); o.w = pack_bf16(f[6], f[7]);
              *reinterpret_cast<uint4*>(out + j * 32 + g8 * 8) = o;
            }
          }
        }
      }
      tc_fence_before();
      mbar_arrive(&s.tmem_empty[buf]);
    }
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (warp == 5) { tc_fence_after(); tmem_dealloc(tmem_base, TMEM_COLS); }
}

// ------------------------------------------------------------------------------ dW kernel
struct DwParams {
  const int32_t* cnt;   // number of valid rows (the contraction length)
  float* dW;            // [d_out, d_in]
  int32_t* status;
  int d_in, d_out;
};

// A = rows x d_out (MN-major: m contiguous), B = rows x d_in (MN-major), both gathered along k
// by the pack step (or the original tensors for the dense product).
template <int BN>
__global__ void __launch_bounds__(NUM_THREADS, 1)
umma_dw_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, DwParams P) {
  using C = TileCfg<BN>;
  extern __shared__ uint8_t smem_raw[];
  const SmemLayout s = carve<BN>(smem_raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t tmem_base = setup<BN>(s, warp, tid);
  volatile int* abort_flag = s.abort_flag;

  const int cnt = *P.cnt;
  const int kblocks = (cnt + BK - 1) / BK;
  const int mtiles = (P.d_out + BM - 1) / BM;
  const int ntiles = (P.d_in + BN - 1) / BN;
  const int total_tiles = mtiles * ntiles;

  if (warp == 4) {
    if (lane == 0 && kblocks > 0) {
      int stage = 0; uint32_t phase = 0;
      for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
        const int mt = tile / ntiles, nt = tile % ntiles;
        bool ok = true;
        for (int kb = 0; kb < kblocks; ++kb) {
          ok = mbar_wait(&s.empty[stage], phase ^ 1u, abort_flag, P.status);
          if (!ok) break;
          uint8_t* sa = s.stages + stage * C::STAGE_BYTES;
          mbar_expect_tx(&s.full[stage], C::STAGE_BYTES);
#pragma unroll
          for (int j = 0; j < BM / 64; ++j)
            tma_load_2d(sa + j * CHUNK_BYTES, &tmA, mt * BM + j * 64, kb * BK, &s.full[stage]);
#pragma unroll
          for (int j = 0; j < BN / 64; ++j)
            tma_load_2d(sa + A_BYTES + j * CHUNK_BYTES, &tmB, nt * BN + j * 64, kb * BK, &s.full[stage]);
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
      }
    }
  } else if (warp == 5) {
    if (lane == 0 && kblocks > 0) {
      constexpr uint32_t idesc = make_idesc(BN, true, true);
      int stage = 0; uint32_t phase = 0; int lt = 0;
      for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++lt) {
        const int buf = lt & 1; const uint32_t use = (uint32_t)(lt >> 1) & 1u;
        bool ok = mbar_wait(&s.tmem_empty[buf], use ^ 1u, abort_flag, P.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
        for (int kb = 0; kb < kblocks; ++kb) {
          ok = mbar_wait(&s.full[stage], phase, abort_flag, P.status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sa = smem_u32(s.stages + stage * C::STAGE_BYTES);
          const uint64_t da = desc_mnmajor(sa), db = desc_mnmajor(sa + A_BYTES);
#pragma unroll
          for (int k4 = 0; k4 < BK / UMMA_K; ++k4)
            umma_bf16(d_tmem, da + (uint64_t)(k4 * (UMMA_K * 128 >> 4)), db + (uint64_t)(k4 * (UMMA_K * 128 >> 4)), idesc,
                      (kb | k4) != 0 ? 1u : 0u);
          umma_commit(&s.empty[stage]);
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit(&s.tmem_full[buf]);
      }
    }
  } else {
    int lt = 0;
    const int row = warp * 32 + lane;
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++lt) {
      const int mt = tile / ntiles, nt = tile % ntiles;
      const int o = mt * BM + row;
      const bool valid = o < P.d_out;
      float* out = P.dW + (size_t)(valid ? o : 0) * P.d_in + (size_t)nt * BN;
      if (kblocks == 0) {
        if (valid) {
#pragma unroll
          for (int j = 0; j < BN / 4; ++j)
            if (nt * BN + j * 4 < P.d_in) *reinterpret_cast<float4*>(out + j * 4) = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        continue;
      }
      const int buf = lt & 1; const uint32_t use = (uint32_t)(lt >> 1) & 1u;
      if (!mbar_wait(&s.tmem_full[buf], use, abort_flag, P.status)) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(buf * BN);
#pragma unroll 1
      for (int j = 0; j < BN / 32; ++j) {
        uint32_t v[32];
        tmem_ld32(taddr + (uint32_t)(j * 32), v);
        if (valid) {
#pragma unroll
          for (int g4 = 0; g4 < 8; ++g4) {
            const int col = nt * BN + j * 32 + g4 * 4;
            if (col < P.d_in)
              *reinterpret_cast<uint4*>(out + j * 32 + g4 * 4) = make_uint4(v[g4 * 4], v[g4 * 4 + 1], v[g4 * 4 + 2], v[g4 * 4 + 3]);
          }
        }
      }
      tc_fence_before();
      mbar_arrive(&s.tmem_empty[buf]);
    }
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (warp == 5) { tc_fence_after(); tmem_dealloc(tmem_base, TMEM_COLS); }
}

// ---------------------------------------------------------------------------- pack kernel
// Compact operands of the weight-gradient product: row k of packG = scaleW[k] * dY[idxW[k]]
// (G_tilde of Sec. 4.2, rounded to bf16), row k of packX = X[idxW[k]]; rows up to the next
// multiple of 64 are zero so that the last k-block of the product contributes nothing.
__global__ void __launch_bounds__(256) pack_kernel(const __nv_bfloat16* __restrict__ dY, const __nv_bfloat16* __restrict__ X,
                                                   const int32_t* __restrict__ idxW, const float* __restrict__ scaleW,
                                                   const int32_t* __restrict__ counts, __nv_bfloat16* __restrict__ packG,
                                                   __nv_bfloat16* __restrict__ packX, int d_out, int d_in) {
  const int cnt = counts[1];
  const int padded = (cnt + BK - 1) / BK * BK;
  const int vo = d_out / 8, vi = d_in / 8;
  for (int k = blockIdx.x; k < padded; k += gridDim.x) {
    uint4* og = reinterpret_cast<uint4*>(packG + (size_t)k * d_out);
    uint4* ox = reinterpret_cast<uint4*>(packX + (size_t)k * d_in);
    if (k < cnt) {
      const int r = idxW[k];
      const float sc = scaleW[k];
      const uint4* ig = reinterpret_cast<const uint4*>(dY + (size_t)r * d_out);
      const uint4* ix = reinterpret_cast<const uint4*>(X + (size_t)r * d_in);
      for (int i = threadIdx.x; i < vo; i += blockDim.x) {
        const uint4 v = __ldg(ig + i);
        const uint32_t u[4] = {v.x, v.y, v.z, v.w};
        uint32_t o[4];
#pragma unroll
        for (int e = 0; e < 4; ++e)
          o[e] = pack_bf16(sc * __uint_as_float(u[e] << 16), sc * __uint_as_float(u[e] & 0xffff0000u));
        og[i] = make_uint4(o[0], o[1], o[2], o[3]);
      }
      for (int i = threadIdx.x; i < vi; i += blockDim.x) ox[i] = __ldg(ix + i);
    } else {
      for (int i = threadIdx.x; i < vo; i += blockDim.x) og[i] = make_uint4(0u, 0u, 0u, 0u);
      for (int i = threadIdx.x; i < vi; i += blockDim.x) ox[i] = make_uint4(0u, 0u, 0u, 0u);
    }
  }
}

// ------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

// bf16 tensor of `rank` dims (innermost first), 128-byte swizzle, out-of-bounds reads give 0
bool make_map(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
              const uint32_t* box) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t gd[3]; cuuint64_t gs[2]; cuuint32_t bx[3]; cuuint32_t es[3] = {1, 1, 1};
  for (int i = 0; i < rank; ++i) { gd[i] = dims[i]; bx[i] = box[i]; }
  for (int i = 0; i + 1 < rank; ++i) gs[i] = strides_bytes[i];
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gd, gs, bx, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tile width: fewest waves of the persistent grid, weighted by the per-tile cost of each width
// (narrow tiles reuse the A stage less and run the tensor pipe below its peak rate).
int pick_bn(long row_tiles, int n_extent, int num_sms) {
  const int widths[3] = {256, 128, 64};
  const double cost[3] = {1.0, 0.56, 0.36};
  int best = 256; double best_t = 1e30;
  for (int i = 0; i < 3; ++i) {
    const long tiles = row_tiles * ((n_extent + widths[i] - 1) / widths[i]);
    const double t = (double)((tiles + num_sms - 1) / num_sms) * cost[i];
    if (t < best_t - 1e-9) { best_t = t; best = widths[i]; }
  }
  return best;
}

template <int BN>
cudaError_t run_dx(Handle* h, const CUtensorMap& a, const CUtensorMap& b, const DxParams& P, cudaStream_t st) {
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(umma_dx_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, TileCfg<BN>::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  const long total = (long)P.N * ((P.T + BM - 1) / BM) * ((P.d_in + BN - 1) / BN);
  const int grid = (int)(total < h->num_sms ? total : h->num_sms);
  umma_dx_kernel<BN><<<grid, NUM_THREADS, TileCfg<BN>::SMEM_BYTES, st>>>(a, b, P);
  h->launches += 1;
  return cudaGetLastError();
}

template <int BN>
cudaError_t run_dw(Handle* h, const CUtensorMap& a, const CUtensorMap& b, const DwParams& P, cudaStream_t st) {
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(umma_dw_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, TileCfg<BN>::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  const long total = (long)((P.d_out + BM - 1) / BM) * ((P.d_in + BN - 1) / BN);
  const int grid = (int)(total < h->num_sms ? total : h->num_sms);
  umma_dw_kernel<BN><<<grid, NUM_THREADS, TileCfg<BN>::SMEM_BYTES, st>>>(a, b, P);
  h->launches += 1;
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_umma_dx(Handle* h, const void* dY, const void* W, bool dense, float rho_hint, const void* H,
                           void* dX, cudaStream_t st) {
  const vcas_layer_desc& d = h->desc;
  CUtensorMap tmA, tmB;
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
  DxParams P;
  P.idxA = h->ws.idxA; P.dropA = h->ws.dropA; P.counts = h->ws.counts; P.scaleA = h->ws.scaleA;
  P.H = (const __nv_bfloat16*)H; P.dX = (__nv_bfloat16*)dX; P.status = h->ws.status;
  P.N = d.N; P.T = d.T; P.d_in = d.d_in; P.d_out = d.d_out; P.dense = dense ? 1 : 0;
  P.a_tx_bytes = (d.T < BM ? d.T : BM) * BK * 2;
  double kept = dense ? (double)d.N : (double)rho_hint * d.N;
  if (kept < 1.0) kept = 1.0;
  const long row_tiles = (long)(kept + 0.5) * ((d.T + BM - 1) / BM);
  switch (h->tune_dx_tile_n != 0 ? h->tune_dx_tile_n : pick_bn(row_tiles, d.d_in, h->num_sms)) {
    case 256: return run_dx<256>(h, tmA, tmB, P, st);
    case 128: return run_dx<128>(h, tmA, tmB, P, st);
    default: return run_dx<64>(h, tmA, tmB, P, st);
  }
}

cudaError_t launch_pack(Handle* h, const void* dY, const void* X, cudaStream_t st) {
  const vcas_layer_desc& d = h->desc;
  int blocks = h->num_sms * 8;
  if (blocks > h->R_pad) blocks = h->R_pad;
  pack_kernel<<<blocks, 256, 0, st>>>((const __nv_bfloat16*)dY, (const __nv_bfloat16*)X, h->ws.idxW, h->ws.scaleW,
                                      h->ws.counts, h->ws.packG, h->ws.packX, d.d_out, d.d_in);
  h->launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_umma_dw(Handle* h, const void* A_rows, const void* B_rows, int rows_capacity, const int32_t* cnt,
                           float* dW, cudaStream_t st) {
  const vcas_layer_desc& d = h->desc;
  CUtensorMap tmA, tmB;
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
  DwParams P;
  P.cnt = cnt; P.dW = dW; P.status = h->ws.status; P.d_in = d.d_in; P.d_out = d.d_out;
  switch (h->tune_dw_tile_n != 0 ? h->tune_dw_tile_n : pick_bn((d.d_out + BM - 1) / BM, d.d_in, h->num_sms)) {
    case 256: return run_dw<256>(h, tmA, tmB, P, st);
    case 128: return run_dw<128>(h, tmA, tmB, P, st);
    default: return run_dw<64>(h, tmA, tmB, P, st);
  }
}

}  // namespace vcas
