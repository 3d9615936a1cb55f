// Varlen GEMM with fused epilogue on tcgen05 / TMEM, fed by TMA.
//   out[M,N] = act2( act(A[M,K] * Wt[N,K]^T + bias[N]) + residual[M,N] ),  bf16 in, fp32 accumulate, bf16 out.
// M is the run-time row count (sum of the requests' rows); the tensor maps are encoded for exactly
// M rows, so rows past M read as zeros and the TMA store clips them.
//
// Persistent, warp-specialised, one CTA per SM.  Tile 128 x BN; one pipeline stage holds KCH
// k-chunks of 64 (each chunk = one 128-byte swizzle atom per row).  Measured on B200: one thread
// can issue a tcgen05.mma about every 65-80 cycles and a barrier wait in the issue loop costs about
// 170 cycles, so a stage must carry >= 512 cycles of MMA work to hide them: (BN=256, KCH=1) or
// (BN=128, KCH=2).
//   warp 0      TMA producer for A (STAGES-deep mbarrier ring; one 3-D box per stage)
//   warp 1      TMA producer for B (a thread sustains about one TMA instruction per 170 ns, so A
//               and B get a thread each)
//   warp 2      MMA issuer: tcgen05.mma into one of two TMEM accumulators (double buffered)
//   warps 3..10 epilogue, in passes of 128 columns: drain TMEM (warp w owns lanes 32*(w%4)..), add
//               bias from shared memory, activation, residual (TMA-loaded into the staging tile and
//               updated in place), pack to bf16 into the swizzled staging tile, TMA store
// so the epilogue of tile i overlaps the main loop of tile i+1.  Every wait is bounded (ptx.cuh).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include "ptx.cuh"

namespace sod2 {
namespace k {

enum Act : int { ACT_NONE = 0, ACT_GELU = 1, ACT_RELU = 2 };

struct GemmEpilogue {
  const __nv_bfloat16* bias;  // [N] or nullptr
  int has_residual;           // residual arrives through its own tensor map
  int act2;                   // applied after the residual add (ACT_NONE or ACT_RELU); the pre-residual one is a template parameter
  int* status;                // device word; set non-zero if a bounded wait ran out
};

constexpr int GEMM_BM = 128;
constexpr int GEMM_THREADS = 352;
constexpr int GEMM_PASS_COLS = 128;                       // epilogue pass width
constexpr int GEMM_STAGE_OUT = GEMM_BM * GEMM_PASS_COLS * 2;  // 32 KB staging tile: 2 boxes of [128 rows x 128 B]

template <int BN, int KCH, int STAGES>
struct GemmSmem {
  static constexpr int A_BYTES = KCH * GEMM_BM * 128;
  static constexpr int B_BYTES = KCH * BN * 128;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int TOTAL = STAGES * STAGE_BYTES + GEMM_STAGE_OUT + 896 /*align slack: the window is at least 128-B aligned*/ + 2048 /*bias*/ + 128 /*barriers*/;
};

// erf by the rational approximation 7.1.26 of Abramowitz & Stegun (|error| <= 1.5e-7), far inside
// the bf16 output rounding; cheaper than erff on the epilogue warps.
__device__ __forceinline__ float gelu_erf(float x) {
  const float z = fabsf(x) * 0.70710678118654752f;
  float t;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t) : "f"(fmaf(0.3275911f, z, 1.0f)));
  float p = fmaf(1.061405429f, t, -1.453152027f);
  p = fmaf(p, t, 1.421413741f);
  p = fmaf(p, t, -0.284496736f);
  p = fmaf(p, t, 0.254829592f);
  const float e = 1.0f - p * t * __expf(-z * z);   // erf(|x|/sqrt2)
  return 0.5f * x * (1.0f + copysignf(e, x));
}
// The activation is a template parameter: a run-time switch inside the unrolled element loops
// turns every element into its own basic block and serialises the dependent FMA / MUFU chains.
template <int ACT>
__device__ __forceinline__ float apply_act(float v) {
  if constexpr (ACT == ACT_GELU) return gelu_erf(v);
  else if constexpr (ACT == ACT_RELU) return fmaxf(v, 0.0f);
  else return v;
}

__device__ __forceinline__ void tma_store_2d(const void* tmap, const void* src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(tmap), "r"(ptx::smem_u32(src)), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// tmA / tmB are 3-D views {64, rows, K/64} of the row-major operands (K % 64 == 0), box
// {64, 128 or BN, KCH}: one instruction fills KCH consecutive swizzled [rows x 64] chunks.
template <int BN, int KCH, int STAGES, int ACT>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_bf16_tcgen05(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                  const __grid_constant__ CUtensorMap tmOut, const __grid_constant__ CUtensorMap tmRes,
                  int M, int N, int K, GemmEpilogue ep) {
  using S = GemmSmem<BN, KCH, STAGES>;
  constexpr int PASSES = BN / GEMM_PASS_COLS;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* out_stage = tiles + STAGES * S::STAGE_BYTES;
  float* bias_s = reinterpret_cast<float*>(out_stage + GEMM_STAGE_OUT);  // [2][256]
  uint64_t* full = reinterpret_cast<uint64_t*>(bias_s + 512);
  uint64_t* empty = full + STAGES;
  uint64_t* tmem_full = empty + STAGES;   // [2]
  uint64_t* tmem_empty = tmem_full + 2;   // [2]
  uint64_t* res_full = tmem_empty + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(res_full + 1);
  volatile int* dead = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tiles_m = (M + GEMM_BM - 1) / GEMM_BM, tiles_n = (N + BN - 1) / BN;
  const int num_tiles = tiles_m * tiles_n;
  const int kchunks = K / 64;
  const int kstages = (kchunks + KCH - 1) / KCH;
  constexpr uint32_t TMEM_COLS = 2 * BN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { ptx::mbar_init(&full[s], 2); ptx::mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { ptx::mbar_init(&tmem_full[b], 1); ptx::mbar_init(&tmem_empty[b], 8); }
    ptx::mbar_init(res_full, 1);
    *dead = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
    ptx::prefetch_tmap(&tmA);
    ptx::prefetch_tmap(&tmB);
    ptx::prefetch_tmap(&tmOut);
    if (ep.has_residual) ptx::prefetch_tmap(&tmRes);
  }
  if (warp == 2) { ptx::tmem_alloc(tmem_slot, TMEM_COLS); ptx::tmem_relinquish(); }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // everything above touched only this CTA's own state; the operands may still be in flight
  ptx::pdl_wait();
  ptx::pdl_launch();

  if (warp == 0) {
    if (lane == 0) {
      // ---- TMA producer: A stages
      int n = 0;
      for (int t = blockIdx.x; t < num_tiles; t += gridDim.x) {
        const int m0 = (t % tiles_m) * GEMM_BM;
        for (int ks = 0; ks < kstages; ++ks, ++n) {
          const int s = n % STAGES;
          if (n >= STAGES) ptx::mbar_wait(&empty[s], ((n / STAGES) - 1) & 1, dead);
          ptx::mbar_expect_tx(&full[s], S::A_BYTES);
          ptx::tma_load_3d(tiles + s * S::STAGE_BYTES, &tmA, 0, m0, ks * KCH, &full[s]);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---- TMA producer: B stages
      int n = 0;
      for (int t = blockIdx.x; t < num_tiles; t += gridDim.x) {
        const int n0 = (t / tiles_m) * BN;
        for (int ks = 0; ks < kstages; ++ks, ++n) {
          const int s = n % STAGES;
          if (n >= STAGES) ptx::mbar_wait(&empty[s], ((n / STAGES) - 1) & 1, dead);
          ptx::mbar_expect_tx(&full[s], S::B_BYTES);
          ptx::tma_load_3d(tiles + s * S::STAGE_BYTES + S::A_BYTES, &tmB, 0, n0, ks * KCH, &full[s]);
        }
      }
    }
  } else if (warp == 2) {
    if (lane == 0) {
      // ---- MMA issuer
      constexpr uint32_t idesc = ptx::idesc_bf16(GEMM_BM, BN);
      int n = 0, j = 0;
      for (int t = blockIdx.x; t < num_tiles; t += gridDim.x, ++j) {
        const int acc = j & 1;
        if (j >= 2) ptx::mbar_wait(&tmem_empty[acc], ((j >> 1) - 1) & 1, dead);
        ptx::tc_fence_after();
        const uint32_t d = tmem + acc * BN;
        for (int ks = 0; ks < kstages; ++ks, ++n) {
          const int s = n % STAGES;
          ptx::mbar_wait(&full[s], (n / STAGES) & 1, dead);
          ptx::tc_fence_after();
          const uint32_t a = ptx::smem_u32(tiles + s * S::STAGE_BYTES);
#pragma unroll
          for (int c = 0; c < KCH; ++c) {
            if (ks * KCH + c < kchunks) {
              const uint64_t ad = ptx::smem_desc_sw128(a + c * (GEMM_BM * 128));
              const uint64_t bd = ptx::smem_desc_sw128(a + S::A_BYTES + c * (BN * 128));
#pragma unroll
              for (int kk = 0; kk < 4; ++kk) ptx::mma_bf16(d, ad + 2 * kk, bd + 2 * kk, idesc, (ks | c | kk) != 0);
            }
          }
          ptx::mma_commit(&empty[s]);  // frees the stage once these MMAs have read it
        }
        ptx::mma_commit(&tmem_full[acc]);
      }
    }
  } else {
    // ---- epilogue warps 3..10
    const int e = warp - 3;
    const int q = warp & 3;          // TMEM lane quarter this warp may access
    const int half = e >> 2;         // which 64-column half of the pass
    const int et = threadIdx.x - 96; // 0..255
    const int row = q * 32 + lane;   // row inside the tile
    int j = 0, rp = 0;               // rp counts residual loads (phase of res_full)
    auto load_bias = [&](int t) -> float {
      const int idx = (t / tiles_m) * BN + et;
      return (ep.bias && et < BN && t < num_tiles && idx < N) ? __bfloat162float(ep.bias[idx]) : 0.0f;
    };
    float bias_next = load_bias(blockIdx.x);
    const float relu2_floor = ep.act2 == ACT_RELU ? 0.0f : -INFINITY;  // post-residual activation, branch-free
    for (int t = blockIdx.x; t < num_tiles; t += gridDim.x, ++j) {
      const int acc = j & 1;
      const int m0 = (t % tiles_m) * GEMM_BM, n0 = (t / tiles_m) * BN;
      float* bias_t = bias_s + (j & 1) * 256;      // this tile's bias, prefetched during the last tile
      bias_t[et] = bias_next;
      bias_next = load_bias(t + gridDim.x);
      epi_bar_sync();
      ptx::mbar_wait(&tmem_full[acc], (j >> 1) & 1, dead);
      __syncwarp();
      ptx::tc_fence_after();
#pragma unroll 1
      for (int ps = 0; ps < PASSES; ++ps) {
        const int np = n0 + ps * GEMM_PASS_COLS;   // first global column of this pass
        const bool live = np < N;
        const bool res = ep.has_residual && live;
        if (res) {
          // the residual tile is TMA-loaded into the staging tile (once the previous store has
          // finished reading it) and updated in place
          if (et == 0) {
            bulk_wait_read0();
            ptx::mbar_expect_tx(res_full, GEMM_STAGE_OUT);
            ptx::tma_load_2d(out_stage, &tmRes, np, m0, res_full);
            ptx::tma_load_2d(out_stage + 16384, &tmRes, np + 64, m0, res_full);
          }
          ptx::mbar_wait(res_full, rp & 1, dead);
          __syncwarp();
          ++rp;
        }
        uint8_t* obase = out_stage + half * 16384 + row * 128;
        uint4 pk[8];
        if (live) {
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            const int col = half * 64 + c * 32;  // column inside the pass
            uint32_t r[32];
            ptx::tmem_ld32(tmem + (static_cast<uint32_t>(q * 32) << 16) + acc * BN + ps * GEMM_PASS_COLS + col, r);
            ptx::tmem_ld_wait();
            const float* bp = bias_t + ps * GEMM_PASS_COLS + col;
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              float v[8];
#pragma unroll
              for (int i = 0; i < 8; ++i) v[i] = apply_act<ACT>(__uint_as_float(r[g * 8 + i]) + bp[g * 8 + i]);
              if (res) {
                const uint4 rv = *reinterpret_cast<const uint4*>(obase + (((c * 4 + g) ^ (row & 7)) << 4));
                const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&rv);
#pragma unroll
                for (int i = 0; i < 4; ++i) { const float2 f = __bfloat1622float2(h[i]); v[2 * i] += f.x; v[2 * i + 1] += f.y; }
#pragma unroll
                for (int i = 0; i < 8; ++i) v[i] = fmaxf(v[i], relu2_floor);
              }
              __nv_bfloat162* oh = reinterpret_cast<__nv_bfloat162*>(&pk[c * 4 + g]);
#pragma unroll
              for (int i = 0; i < 4; ++i) oh[i] = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
            }
          }
        }
        // the math above overlapped the previous pass's TMA store; now the staging tile must be free
        if (!res) {
          if (et == 0) bulk_wait_read0();
          epi_bar_sync();
        }
        if (live) {
#pragma unroll
          for (int g = 0; g < 8; ++g) *reinterpret_cast<uint4*>(obase + ((g ^ (row & 7)) << 4)) = pk[g];
        }
        // publish the staging tile to the async proxy; after the last pass the accumulator is free
        ptx::tc_fence_before();
        ptx::fence_proxy_async();
        __syncwarp();
        if (ps == PASSES - 1 && lane == 0) ptx::mbar_arrive(&tmem_empty[acc]);
        epi_bar_sync();
        if (et == 0 && live) {
          tma_store_2d(&tmOut, out_stage, np, m0);
          if (np + 64 < N) tma_store_2d(&tmOut, out_stage + 16384, np + 64, m0);
          bulk_commit();
        }
      }
    }
    if (et == 0) bulk_wait0();
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 2) ptx::tmem_dealloc(tmem, TMEM_COLS);
  if (threadIdx.x == 0 && *dead && ep.status) atomicExch(ep.status, 1);
}

}  // namespace k
}  // namespace sod2
