// Varlen GEMM with fused epilogue on tcgen05 / TMEM, fed by TMA.
//   out[M,N] = act(A[M,K] * Wt[N,K]^T + bias[N]) (+ residual[M,N]),  bf16 in, fp32 accumulate, bf16 out.
// M is the run-time row count (sum of the requests' rows); the A tensor map is encoded for
// exactly M rows, so rows past M read as zeros and are never stored.
// One 128 x BN output tile per CTA, BK = 64 (one 128-byte swizzle atom of bf16 per row).
// Warp 0 lane 0 streams tiles with TMA through a STAGES-deep mbarrier ring, warp 1 lane 0 issues
// tcgen05.mma into a TMEM accumulator, then all four warps drain TMEM (warp w owns lanes
// 32w..32w+31 = tile rows) through the epilogue. Two CTAs fit per SM, so one CTA's epilogue
// overlaps the other's main loop.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include "ptx.cuh"

namespace sod2 {
namespace k {

enum Act : int { ACT_NONE = 0, ACT_GELU = 1, ACT_RELU = 2 };

struct GemmEpilogue {
  const __nv_bfloat16* bias;      // [N] or nullptr
  const __nv_bfloat16* residual;  // [M, ldr] or nullptr (added after the activation)
  long long ldr;
  __nv_bfloat16* out;             // [M, ldo]
  long long ldo;
  int act;
  int* status;                    // device word; set non-zero if a bounded wait ran out
};

constexpr int GEMM_BM = 128;
constexpr int GEMM_BK = 64;

template <int BN, int STAGES>
struct GemmSmem {
  static constexpr int A_BYTES = GEMM_BM * GEMM_BK * 2;
  static constexpr int B_BYTES = BN * GEMM_BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int TOTAL = STAGES * STAGE_BYTES + 1024 /*align slack*/ + 256 /*barriers*/;
};

__device__ __forceinline__ float gelu_erf(float x) { return 0.5f * x * (1.0f + erff(x * 0.70710678118654752f)); }

template <int BN, int STAGES>
__global__ void __launch_bounds__(128)
gemm_bf16_tcgen05(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                  int M, int N, int K, GemmEpilogue ep) {
  using S = GemmSmem<BN, STAGES>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full = reinterpret_cast<uint64_t*>(tiles + STAGES * S::STAGE_BYTES);
  uint64_t* empty = full + STAGES;
  uint64_t* accum = empty + STAGES;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(accum + 1);
  volatile int* dead = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tiles_m = (M + GEMM_BM - 1) / GEMM_BM;
  const int tm = blockIdx.x % tiles_m, tn = blockIdx.x / tiles_m;
  const int m0 = tm * GEMM_BM, n0 = tn * BN;
  const int kblocks = (K + GEMM_BK - 1) / GEMM_BK;
  constexpr uint32_t TMEM_COLS = BN < 32 ? 32 : BN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { ptx::mbar_init(&full[s], 1); ptx::mbar_init(&empty[s], 1); }
    ptx::mbar_init(accum, 1);
    *dead = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
    ptx::prefetch_tmap(&tmA);
    ptx::prefetch_tmap(&tmB);
  }
  if (warp == 0) { ptx::tmem_alloc(tmem_slot, TMEM_COLS); ptx::tmem_relinquish(); }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0 && lane == 0) {
    // ---- TMA producer
    for (int kb = 0; kb < kblocks; ++kb) {
      const int s = kb % STAGES;
      if (kb >= STAGES) ptx::mbar_wait(&empty[s], ((kb / STAGES) - 1) & 1, dead);
      uint8_t* a = tiles + s * S::STAGE_BYTES;
      ptx::mbar_expect_tx(&full[s], S::STAGE_BYTES);
      ptx::tma_load_2d(a, &tmA, kb * GEMM_BK, m0, &full[s]);
      ptx::tma_load_2d(a + S::A_BYTES, &tmB, kb * GEMM_BK, n0, &full[s]);
    }
  } else if (warp == 1 && lane == 0) {
    // ---- MMA issuer
    constexpr uint32_t idesc = ptx::idesc_bf16(GEMM_BM, BN);
    for (int kb = 0; kb < kblocks; ++kb) {
      const int s = kb % STAGES;
      ptx::mbar_wait(&full[s], (kb / STAGES) & 1, dead);
      ptx::tc_fence_after();
      const uint32_t a = ptx::smem_u32(tiles + s * S::STAGE_BYTES);
      const uint64_t ad = ptx::smem_desc_sw128(a), bd = ptx::smem_desc_sw128(a + S::A_BYTES);
#pragma unroll
      for (int kk = 0; kk < GEMM_BK / 16; ++kk)
        ptx::mma_bf16(tmem, ad + 2 * kk, bd + 2 * kk, idesc, (kb | kk) != 0);
      ptx::mma_commit(&empty[s]);  // frees the stage once these MMAs have read it
    }
    ptx::mma_commit(accum);
  }
  __syncwarp();

  // ---- epilogue: all four warps
  ptx::mbar_wait(accum, 0, dead);
  __syncwarp();
  ptx::tc_fence_after();
  const int row = m0 + warp * 32 + lane;
  const bool row_ok = row < M;
#pragma unroll 1
  for (int c = 0; c < BN; c += 32) {
    uint32_t r[32];
    ptx::tmem_ld32(tmem + (static_cast<uint32_t>(warp * 32) << 16) + c, r);
    ptx::tmem_ld_wait();
    const int col0 = n0 + c;
    if (row_ok && col0 < N) {
      float v[32];
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
      const bool fullc = (col0 + 32 <= N);
      if (ep.bias) {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (fullc || col0 + j < N) v[j] += __bfloat162float(ep.bias[col0 + j]);
      }
      if (ep.act == ACT_GELU) {
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = gelu_erf(v[j]);
      } else if (ep.act == ACT_RELU) {
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = fmaxf(v[j], 0.0f);
      }
      __nv_bfloat16* o = ep.out + static_cast<long long>(row) * ep.ldo + col0;
      if (fullc && ((reinterpret_cast<uintptr_t>(o) & 15) == 0) &&
          (!ep.residual || ((reinterpret_cast<uintptr_t>(ep.residual + static_cast<long long>(row) * ep.ldr + col0) & 15) == 0))) {
        if (ep.residual) {
          const uint4* rp = reinterpret_cast<const uint4*>(ep.residual + static_cast<long long>(row) * ep.ldr + col0);
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            uint4 rv = rp[q];
            const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&rv);
#pragma unroll
            for (int t = 0; t < 4; ++t) {
              float2 f = __bfloat1622float2(h[t]);
              v[q * 8 + 2 * t] += f.x;
              v[q * 8 + 2 * t + 1] += f.y;
            }
          }
        }
        uint4* op = reinterpret_cast<uint4*>(o);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint4 ov;
          __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&ov);
#pragma unroll
          for (int t = 0; t < 4; ++t) h[t] = __floats2bfloat162_rn(v[q * 8 + 2 * t], v[q * 8 + 2 * t + 1]);
          op[q] = ov;
        }
      } else {
        for (int j = 0; j < 32; ++j) {
          if (col0 + j < N) {
            float x = v[j];
            if (ep.residual) x += __bfloat162float(ep.residual[static_cast<long long>(row) * ep.ldr + col0 + j]);
            o[j] = __float2bfloat16_rn(x);
          }
        }
      }
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 0) ptx::tmem_dealloc(tmem, TMEM_COLS);
  if (threadIdx.x == 0 && *dead && ep.status) atomicExch(ep.status, 1);
}

}  // namespace k
}  // namespace sod2
