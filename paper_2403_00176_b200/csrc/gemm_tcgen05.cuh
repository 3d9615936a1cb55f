// Varlen GEMM with fused epilogue on tcgen05 / TMEM, fed by TMA.
//   out[M,N] = act2( act(A[M,K] * Wt[N,K]^T + bias[N]) + residual[M,N] ),  bf16 in, fp32 accumulate, bf16 out.
// M is the run-time row count (sum of the requests' rows); the tensor maps are encoded for exactly
// M rows, so rows past M read as zeros and the TMA store clips them.
//
// Persistent, warp-specialised, one CTA per SM.  Tile 128 x BN; one pipeline stage holds KCH
// k-chunks of 64 (each chunk = one 128-byte swizzle atom per row).  Measured on B200: a
// tcgen05.mma occupies the tensor pipe for max(~48, BN/2) cycles, and a barrier wait between MMAs
// leaves the pipe idle for about 320 cycles unless the MMAs queued before it are long enough to
// cover it, so a stage must carry >= 512 cycles of MMA work: (BN=256, KCH=1) or (BN=128, KCH=2).
// An SM takes in about 70 bytes per clock from L2, which bounds the main loop of a 128 x 256 tile
// at about 75 % of the tensor peak.
//   warp 0      TMA producer for A (STAGES-deep mbarrier ring; one 3-D box per stage)
//   warp 1      TMA producer for B (a thread sustains about one TMA instruction per 170 ns, so A
//               and B get a thread each); B is constant, so it does not wait for the previous kernel
//   warp 2      MMA issuer: tcgen05.mma into one of two TMEM accumulators (double buffered)
//   warps 3..10 epilogue, in passes of 64 columns: drain TMEM (warp w owns lanes 32*(w%4)..), add
//               bias from shared memory, activation, residual (already in the staging buffer,
//               updated in place), pack to bf16 into the swizzled staging buffer
//   warp 11     staging agent: residual TMA loads ahead of the epilogue, TMA stores behind it
// so the epilogue of tile i overlaps the main loop of tile i+1 and no epilogue thread waits on a
// TMA round trip.  Every wait is bounded (ptx.cuh).
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
  int splits;                 // split-K kernels: number of K ranges per tile (work item = tile x range), else unused
  int stages_per_split;       // split-K kernels: pipeline stages per K range
  // ---- LayerNorm folded into the GEMM (template parameters LN / EMIT).  Row statistics are (mean, M2) pairs,
  // M2 = sum of squared deviations from that mean, one pair per row and slot of `ln_cols` consecutive columns;
  // slot s of row i is at [s * pitch + i], i counted from this launch's first row.
  const float2* ln_stats;     // LN != 0: statistics of the rows being normalised (A rows for LN = 1, residual rows for LN = 2)
  long long ln_pitch;
  int ln_slots, ln_cols;      // slots per row and columns per slot (slots * cols = normalised width)
  float ln_eps;
  const float* ln_c1;         // LN = 1: [N] column sums of the gamma-scaled weights
  const float* ln_c2;         // LN = 1: [N] beta . W + bias (replaces `bias`)
  const __nv_bfloat16* ln_gamma;  // LN = 2: [N]
  const __nv_bfloat16* ln_beta;   // LN = 2: [N]
  float2* emit_stats;         // EMIT: receives the statistics of the stored output rows: slot = 2 * n-tile + column half
  long long emit_pitch;
};

// One row's LayerNorm statistics from its partial (mean, M2) pairs, merged in slot order (pairwise update of
// mean and sum of squared deviations): the same result whichever kernel reads them.
__device__ __forceinline__ void ln_merge_stats(const float2* st, long long pitch, int slots, int cols, float eps, float* mean_out, float* rstd_out) {
  float n = 0.f, mean = 0.f, m2 = 0.f;
  const float c = static_cast<float>(cols);
  for (int s = 0; s < slots; ++s) {
    const float2 q = st[s * pitch];
    const float nn = n + c;
    const float d = q.x - mean;
    mean = fmaf(d, c / nn, mean);
    m2 += q.y + d * d * (n * c / nn);
    n = nn;
  }
  *mean_out = mean;
  *rstd_out = 1.0f / sqrtf(m2 / n + eps);
}

constexpr int GEMM_BM = 128;
constexpr int GEMM_THREADS = 384;
constexpr int GEMM_PASS_COLS = 64;                            // epilogue pass width: one 128-byte swizzled row
constexpr int GEMM_STAGE_OUT = GEMM_BM * GEMM_PASS_COLS * 2;  // 16 KB staging buffer: [128 rows x 128 B]
constexpr int GEMM_NSB = 2;                                   // staging buffers

template <int BN, int KCH, int STAGES>
struct GemmSmem {
  static constexpr int A_BYTES = KCH * GEMM_BM * 128;
  static constexpr int B_BYTES = KCH * BN * 128;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int USED = STAGES * STAGE_BYTES + GEMM_NSB * GEMM_STAGE_OUT + 2048 /*bias*/ + 136 /*barriers, TMEM slot, dead flag*/;
  // plus the pad that brings the tiles to a 1024-byte boundary; the kernel checks the pad it really
  // needs against the launch's dynamic size and reports an error instead of running past the end
  static constexpr int TOTAL = USED + 888;
};

// GELU(x) = x * Phi(x) with Phi written as 0.5 * (1 + tanh(u(x))), u(x) = atanh(erf(x / sqrt 2)).
// u is odd; x * (c0 + c1 x^2 + c2 x^4) fitted by least squares on [-8, 8] reproduces the erf form of
// GELU to 3e-5 absolute, and the hardware tanh adds a relative 2^-11: both far inside the bf16 output
// rounding.  x^2 is clamped where the quintic would turn over (|x| > 7; tanh is saturated there).
// Eight instructions per element instead of seventeen for a polynomial erf: the epilogue of a
// GELU GEMM is bound by instruction issue.
__device__ __forceinline__ float gelu_erf(float x) {
  const float x2 = fminf(x * x, 50.0f);
  const float u = x * fmaf(x2, fmaf(x2, -0.00035873236f, 0.037050345f), 0.79745847f);
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(u));
  const float hx = 0.5f * x;
  return fmaf(hx, t, hx);
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
__device__ __forceinline__ void tma_store_3d(const void* tmap, const void* src, int x, int y, int z) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(tmap), "r"(ptx::smem_u32(src)), "r"(x), "r"(y), "r"(z) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// tmA / tmB are 3-D views {64, rows, K/64} of the row-major operands (K % 64 == 0), box
// {64, 128 or BN, KCH}: one instruction fills KCH consecutive swizzled [rows x 64] chunks.
// B must be a constant of the graph (prepacked weights): its producer does not wait for the
// previous kernel in the stream.
// RES: the group adds a residual tile (a compile-time switch: a run-time branch inside the unrolled
// element loops splits them into basic blocks and exposes every shared-memory latency).
// SPLITK: a work item is (tile, K range); the epilogue stores the raw fp32 partial tile into slab
// `range` of an fp32 [ranges, M, N] workspace (tmOut is then a 3-D fp32 map with boxes of 32 columns)
// and a finishing kernel adds the slabs in a fixed order and applies bias, residual and LayerNorm.
// This spreads a GEMM with few output tiles and a long K over all SMs, deterministically.
// LN = 1: A is the raw input of a folded LayerNorm and the weights carry its gamma: the epilogue computes
//   rstd_i * (acc - mean_i * c1[n]) + c2[n]   (= LayerNorm(A) * W + bias) before the activation.
// LN = 2 (with RES): the staged residual tile holds raw rows; the epilogue adds (r - mean_i) * rstd_i * gamma[n] + beta[n].
// EMIT: the epilogue also writes the statistics of the rows it stores (of the bf16 values as stored), one
// (mean, M2) pair per row, n-tile and 32-column-per-pass half; needs N % BN == 0.
// With LN != 0 the per-column vectors (bias / c2, c1 / gamma, beta) live single-buffered in the 2 KB vector area,
// guarded by a second barrier of the epilogue warps per tile; LN = 2 needs BN <= 128 to fit three of them.
template <int BN, int KCH, int STAGES, int ACT, bool SPLITK = false, bool RES = false, int LN = 0, bool EMIT = false>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_bf16_tcgen05(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                  const __grid_constant__ CUtensorMap tmOut, const __grid_constant__ CUtensorMap tmRes,
                  int M, int N, int K, GemmEpilogue ep) {
  using S = GemmSmem<BN, KCH, STAGES>;
  constexpr int PASSES = SPLITK ? BN / 32 : BN / GEMM_PASS_COLS;   // split-K passes are 32 fp32 columns (128-byte rows)
  constexpr int NSB = GEMM_NSB;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* out_stage = tiles + STAGES * S::STAGE_BYTES;
  float* bias_s = reinterpret_cast<float*>(out_stage + NSB * GEMM_STAGE_OUT);  // [2][256]
  uint64_t* full = reinterpret_cast<uint64_t*>(bias_s + 512);
  uint64_t* empty = full + STAGES;
  uint64_t* tmem_full = empty + STAGES;   // [2]
  uint64_t* tmem_empty = tmem_full + 2;   // [2]
  uint64_t* buf_ready = tmem_empty + 2;   // [NSB] staging buffer handed to the epilogue warps (residual loaded, or just free)
  uint64_t* buf_filled = buf_ready + NSB; // [NSB] epilogue warps have written the buffer
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(buf_filled + NSB);
  volatile int* dead = reinterpret_cast<volatile int*>(tmem_slot + 1);

  {
    uint32_t dyn;
    asm("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn));
    if (static_cast<uint32_t>(tiles - smem_raw) + S::USED > dyn) {   // uniform over the CTA
      if (threadIdx.x == 0 && ep.status) atomicExch(ep.status, 2);
      return;
    }
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tiles_m = (M + GEMM_BM - 1) / GEMM_BM, tiles_n = (N + BN - 1) / BN;
  const int kchunks = K / 64;
  const int kstages = (kchunks + KCH - 1) / KCH;
  const int out_tiles = tiles_m * tiles_n;
  const int num_tiles = SPLITK ? out_tiles * ep.splits : out_tiles;   // work items; item w = (tile w % out_tiles, K range w / out_tiles)
  auto k_range = [&](int w, int* ks0, int* ks1) {
    if (SPLITK) { *ks0 = (w / out_tiles) * ep.stages_per_split; *ks1 = min(kstages, *ks0 + ep.stages_per_split); }
    else { *ks0 = 0; *ks1 = kstages; }
  };
  constexpr uint32_t TMEM_COLS = 2 * BN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { ptx::mbar_init(&full[s], 2); ptx::mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { ptx::mbar_init(&tmem_full[b], 1); ptx::mbar_init(&tmem_empty[b], 8); }
    for (int b = 0; b < NSB; ++b) { ptx::mbar_init(&buf_ready[b], 1); ptx::mbar_init(&buf_filled[b], SPLITK ? 4 : 8); }
    *dead = 0;
    ptx::fence_barrier_init();
    // without a residual the staging buffers start out free: their first phase is completed here, before the
    // block-wide barrier below, so the epilogue need not wait for its first NSB units at all
    if (!SPLITK && !RES) { for (int b = 0; b < NSB; ++b) ptx::mbar_arrive(&buf_ready[b]); }
    ptx::fence_proxy_async();
    ptx::prefetch_tmap(&tmA);
    ptx::prefetch_tmap(&tmB);
    ptx::prefetch_tmap(&tmOut);
    if (RES) ptx::prefetch_tmap(&tmRes);
  }
  if (warp == 2) { ptx::tmem_alloc(tmem_slot, TMEM_COLS); ptx::tmem_relinquish(); }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  if (threadIdx.x == 0) { SOD2_TRACE(0, 1) }
  // Everything above touched only this CTA's own state.  Each role waits for the previous kernel
  // only where it touches that kernel's data: the A producer and the epilogue warps do, the B
  // producer (constant weights) and the MMA issuer (shared memory and TMEM only) do not, so the
  // weight stages stream in while the previous kernel drains.
  ptx::pdl_launch();

  if (warp == 0) {
    if (lane == 0) {
      // ---- TMA producer: A stages
      ptx::pdl_wait();
      SOD2_TRACE(0, 2)
      int n = 0;
      for (int w = blockIdx.x; w < num_tiles; w += gridDim.x) {
        const int t = SPLITK ? w % out_tiles : w;
        const int m0 = (t % tiles_m) * GEMM_BM;
        int ks0, ks1;
        k_range(w, &ks0, &ks1);
        for (int ks = ks0; ks < ks1; ++ks, ++n) {
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
      for (int w = blockIdx.x; w < num_tiles; w += gridDim.x) {
        const int t = SPLITK ? w % out_tiles : w;
        const int n0 = (t / tiles_m) * BN;
        int ks0, ks1;
        k_range(w, &ks0, &ks1);
        for (int ks = ks0; ks < ks1; ++ks, ++n) {
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
      for (int w = blockIdx.x; w < num_tiles; w += gridDim.x, ++j) {
        const int acc = j & 1;
        if (j >= 2) ptx::mbar_wait(&tmem_empty[acc], ((j >> 1) - 1) & 1, dead);
        ptx::tc_fence_after();
        const uint32_t d = tmem + acc * BN;
        int ks0, ks1;
        k_range(w, &ks0, &ks1);
        for (int ks = ks0; ks < ks1; ++ks, ++n) {
          const int s = n % STAGES;
          ptx::mbar_wait(&full[s], (n / STAGES) & 1, dead);
          ptx::tc_fence_after();
          if (ks == 0) { SOD2_TRACE(1, 10 + j) }
          const uint32_t a = ptx::smem_u32(tiles + s * S::STAGE_BYTES);
#pragma unroll
          for (int c = 0; c < KCH; ++c) {
            if (ks * KCH + c < kchunks) {
              const uint64_t ad = ptx::smem_desc_sw128(a + c * (GEMM_BM * 128));
              const uint64_t bd = ptx::smem_desc_sw128(a + S::A_BYTES + c * (BN * 128));
#pragma unroll
              for (int kk = 0; kk < 4; ++kk) ptx::mma_bf16(d, ad + 2 * kk, bd + 2 * kk, idesc, (ks > ks0) || c != 0 || kk != 0);
            }
          }
          ptx::mma_commit(&empty[s]);  // frees the stage once these MMAs have read it
        }
        ptx::mma_commit(&tmem_full[acc]);
        SOD2_TRACE(1, 20 + j)
      }
    }
  } else if (warp == 11) {
    if (lane == 0) {
      // ---- staging agent: owns the staging buffers' TMA traffic so that no epilogue thread waits on a
      // TMA round trip.  A unit is one 64-column pass of one tile; unit u uses buffer u % NSB.
      // prepare(u) hands the buffer to the epilogue warps: with a residual it is TMA-loaded into the
      // buffer (the epilogue updates it in place), otherwise a plain arrive.  Once the epilogue warps
      // have filled the buffer the agent stores it and, after the store has read the buffer, prepares
      // unit u + NSB.  The kernel may end once the last store has read shared memory.
      ptx::pdl_wait();
      int my_tiles = 0;
      for (int t = blockIdx.x; t < num_tiles; t += gridDim.x) ++my_tiles;
      const int U = my_tiles * PASSES;
      constexpr int PASS_COLS = SPLITK ? 32 : GEMM_PASS_COLS;
      auto prepare = [&](int u) {
        const int w = blockIdx.x + (u / PASSES) * gridDim.x;
        const int t = SPLITK ? w % out_tiles : w;
        const int m0 = (t % tiles_m) * GEMM_BM, np = (t / tiles_m) * BN + (u % PASSES) * PASS_COLS;
        const int bsel = u % NSB;
        if (!SPLITK && RES && np < N) {
          ptx::mbar_expect_tx(&buf_ready[bsel], GEMM_STAGE_OUT);
          ptx::tma_load_2d(out_stage + bsel * GEMM_STAGE_OUT, &tmRes, np, m0, &buf_ready[bsel]);
        } else {
          ptx::mbar_arrive(&buf_ready[bsel]);
        }
      };
      if (SPLITK || RES) { for (int u = 0; u < NSB && u < U; ++u) prepare(u); }   // else: done at barrier initialisation
      for (int u = 0; u < U; ++u) {
        const int bsel = u % NSB;
        ptx::mbar_wait(&buf_filled[bsel], (u / NSB) & 1, dead);
        const int w = blockIdx.x + (u / PASSES) * gridDim.x;
        const int t = SPLITK ? w % out_tiles : w;
        const int m0 = (t % tiles_m) * GEMM_BM, np = (t / tiles_m) * BN + (u % PASSES) * PASS_COLS;
        if (np < N) {
          if (SPLITK) tma_store_3d(&tmOut, out_stage + bsel * GEMM_STAGE_OUT, np, m0, w / out_tiles);
          else tma_store_2d(&tmOut, out_stage + bsel * GEMM_STAGE_OUT, np, m0);
          bulk_commit();
        }
        if (u + NSB < U) {
          bulk_wait_read0();
          prepare(u + NSB);
        }
      }
      SOD2_TRACE(2, 40)
      bulk_wait_read0();
      SOD2_TRACE(2, 41)
    }
  } else {
    // ---- epilogue warps 3..10: TMEM -> +bias -> act -> (+residual, act2) -> bf16 -> swizzled staging.
    // Warp (q, half) owns TMEM lanes 32q..32q+31 (a warp may only read its own lane quarter) and the
    // 32-column half of every 64-column pass; a thread holds one output row.
    const int e = warp - 3;
    const int q = warp & 3;
    const int half = e >> 2;
    const int et = threadIdx.x - 96; // 0..255
    const int row = q * 32 + lane;   // row inside the tile
    ptx::pdl_wait();
    if constexpr (SPLITK) {
      // raw fp32 partial sums, 32 columns per pass; the warps of column half h take the passes of
      // parity h, which are exactly the units of staging buffer h
      int j = 0;
      for (int w = blockIdx.x; w < num_tiles; w += gridDim.x, ++j) {
        const int acc = j & 1;
        const int n0 = ((w % out_tiles) / tiles_m) * BN;
        ptx::mbar_wait_warp(&tmem_full[acc], (j >> 1) & 1, dead);
        ptx::tc_fence_after();
        const uint32_t taddr = tmem + (static_cast<uint32_t>(q * 32) << 16) + acc * BN;
        uint32_t r[2][32];
        ptx::tmem_ld32(taddr + half * 32, r[0]);
#pragma unroll
        for (int i = 0; i < PASSES / 2; ++i) {
          const int ps = 2 * i + half;
          const int u = j * PASSES + ps;
          ptx::tmem_ld_wait();
          if (i + 1 < PASSES / 2) {
            ptx::tmem_ld32(taddr + (ps + 2) * 32, r[(i + 1) & 1]);
          } else {
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&tmem_empty[acc]);
          }
          ptx::mbar_wait_warp(&buf_ready[half], (u / NSB) & 1, dead);
          if (n0 + ps * 32 < N) {
            uint8_t* obase = out_stage + half * GEMM_STAGE_OUT + row * 128;
#pragma unroll
            for (int g = 0; g < 8; ++g)
              *reinterpret_cast<uint4*>(obase + ((g ^ (row & 7)) << 4)) =
                  make_uint4(r[i & 1][4 * g], r[i & 1][4 * g + 1], r[i & 1][4 * g + 2], r[i & 1][4 * g + 3]);
          }
          ptx::fence_proxy_async();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&buf_filled[half]);
        }
      }
    } else {
    static_assert(LN == 0 || !SPLITK, "folded LayerNorm and split-K do not combine");
    static_assert(LN != 2 || (RES && BN <= 128), "a normalised residual needs the residual path and three vectors of BN floats");
    static_assert(LN != 1 || !RES, "a normalised A operand is not combined with a residual");
    constexpr int NVEC = LN == 1 ? 2 : LN == 2 ? 3 : 1;
    int j = 0, u = 0;
    // column vectors of tile t: v0 = bias (LN = 1: c2), v1 = c1 (LN = 1) or gamma (LN = 2), v2 = beta (LN = 2)
    auto load_vec = [&](int t, int which) -> float {
      const int idx = (t / tiles_m) * BN + et;
      if (!(et < BN && t < num_tiles && idx < N)) return 0.0f;
      if (which == 0) {
        if constexpr (LN == 1) return ep.ln_c2[idx];
        else return ep.bias ? __bfloat162float(ep.bias[idx]) : 0.0f;
      }
      if (which == 1) {
        if constexpr (LN == 1) return ep.ln_c1[idx];
        else return __bfloat162float(ep.ln_gamma[idx]);
      }
      return __bfloat162float(ep.ln_beta[idx]);
    };
    float vec_next[NVEC];
#pragma unroll
    for (int w = 0; w < NVEC; ++w) vec_next[w] = load_vec(blockIdx.x, w);
    const float relu2_floor = ep.act2 == ACT_RELU ? 0.0f : -INFINITY;  // post-residual activation, branch-free
    for (int t = blockIdx.x; t < num_tiles; t += gridDim.x, ++j) {
      const int acc = j & 1;
      float* bias_t;
      if constexpr (LN == 0) {
        bias_t = bias_s + (j & 1) * 256;           // this tile's bias, prefetched during the last tile
        bias_t[et] = vec_next[0];
      } else {
        bias_t = bias_s;                           // single-buffered vectors: every warp has left the previous tile
        epi_bar_sync();
        if (et < BN) {
#pragma unroll
          for (int w = 0; w < NVEC; ++w) bias_t[w * BN + et] = vec_next[w];
        }
      }
#pragma unroll
      for (int w = 0; w < NVEC; ++w) vec_next[w] = load_vec(t + gridDim.x, w);
      // statistics of this thread's row (hidden behind the main loop of the tile)
      const int grow = (t % tiles_m) * GEMM_BM + row;
      float ln_mean = 0.f, ln_rstd = 0.f;
      if constexpr (LN != 0) {
        if (grow < M) ln_merge_stats(ep.ln_stats + grow, ep.ln_pitch, ep.ln_slots, ep.ln_cols, ep.ln_eps, &ln_mean, &ln_rstd);
      }
      float em_n = 0.f, em_mean = 0.f, em_m2 = 0.f;    // EMIT: running statistics of this thread's columns of the row
      // one warp polls for the accumulator, the others park at the hardware barrier: seven more polling
      // lanes cost the main loop 3-4 % of its issue slots
      if (warp == 3) ptx::mbar_wait_warp(&tmem_full[acc], (j >> 1) & 1, dead);
      epi_bar_sync();
      ptx::tc_fence_after();
      if (et == 0) { SOD2_TRACE(2, 30 + j) }
      const uint32_t taddr = tmem + (static_cast<uint32_t>(q * 32) << 16) + acc * BN + half * 32;
      uint32_t r[2][32];
      ptx::tmem_ld32(taddr, r[0]);
#pragma unroll
      for (int ps = 0; ps < PASSES; ++ps, ++u) {
        const int bsel = u % NSB;
        uint8_t* obase = out_stage + bsel * GEMM_STAGE_OUT + row * 128;
        ptx::tmem_ld_wait();
        if (ps + 1 < PASSES) {
          ptx::tmem_ld32(taddr + (ps + 1) * GEMM_PASS_COLS, r[(ps + 1) & 1]);
        } else {
          // every column of this warp's share has left TMEM: the accumulator may be overwritten
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&tmem_empty[acc]);
        }
        // everything that does not need the staging buffer happens before the wait for it: bias and
        // activation (and, without a residual, the bf16 packing); columns past N compute harmless
        // values that the agent never stores
        const float* bp = bias_t + ps * GEMM_PASS_COLS + half * 32;
        float v[32];
        if constexpr (LN == 1) {
          const float nmr = -ln_mean * ln_rstd;    // rstd * (acc - mean * c1) + c2
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = apply_act<ACT>(fmaf(ln_rstd, __uint_as_float(r[ps & 1][i]), fmaf(nmr, bp[BN + i], bp[i])));
        } else {
          // the 32 bias values as eight 16-byte broadcast loads (the offset is a multiple of 128 bytes)
          const float4* bp4 = reinterpret_cast<const float4*>(bp);
#pragma unroll
          for (int i4 = 0; i4 < 8; ++i4) {
            const float4 b4 = bp4[i4];
            v[4 * i4] = apply_act<ACT>(__uint_as_float(r[ps & 1][4 * i4]) + b4.x);
            v[4 * i4 + 1] = apply_act<ACT>(__uint_as_float(r[ps & 1][4 * i4 + 1]) + b4.y);
            v[4 * i4 + 2] = apply_act<ACT>(__uint_as_float(r[ps & 1][4 * i4 + 2]) + b4.z);
            v[4 * i4 + 3] = apply_act<ACT>(__uint_as_float(r[ps & 1][4 * i4 + 3]) + b4.w);
          }
        }
        uint4 pk[4];
        if constexpr (!RES) {
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            __nv_bfloat162* oh = reinterpret_cast<__nv_bfloat162*>(&pk[g]);
#pragma unroll
            for (int i = 0; i < 4; ++i) oh[i] = __floats2bfloat162_rn(v[g * 8 + 2 * i], v[g * 8 + 2 * i + 1]);
          }
        }
        // without a residual the first NSB units find their buffers free (first phase completed at barrier
        // initialisation): even a satisfied wait costs a barrier round trip on the epilogue's critical path
        if (RES || u >= NSB) ptx::mbar_wait_warp(&buf_ready[bsel], (u / NSB) & 1, dead);
        if constexpr (RES) {
          // the four residual loads first, then the arithmetic, then the four stores: loads and stores go
          // to the same buffer, so interleaved the compiler keeps each load behind the previous store
          uint4 rv[4];
#pragma unroll
          for (int g = 0; g < 4; ++g) rv[g] = *reinterpret_cast<const uint4*>(obase + (((half * 4 + g) ^ (row & 7)) << 4));
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&rv[g]);
            __nv_bfloat162* oh = reinterpret_cast<__nv_bfloat162*>(&pk[g]);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              float2 f = __bfloat1622float2(h[i]);
              if constexpr (LN == 2) {
                const int cidx = g * 8 + 2 * i;
                f.x = fmaf(f.x - ln_mean, ln_rstd * bp[BN + cidx], bp[2 * BN + cidx]);
                f.y = fmaf(f.y - ln_mean, ln_rstd * bp[BN + cidx + 1], bp[2 * BN + cidx + 1]);
              }
              oh[i] = __floats2bfloat162_rn(fmaxf(v[g * 8 + 2 * i] + f.x, relu2_floor), fmaxf(v[g * 8 + 2 * i + 1] + f.y, relu2_floor));
            }
          }
        }
#pragma unroll
        for (int g = 0; g < 4; ++g) *reinterpret_cast<uint4*>(obase + (((half * 4 + g) ^ (row & 7)) << 4)) = pk[g];
        ptx::fence_proxy_async();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&buf_filled[bsel]);
        if constexpr (EMIT) {
          // statistics of the 32 values just stored (as rounded to bf16), merged into the row's running pair
          float xs[32];
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            const __nv_bfloat162* oh = reinterpret_cast<const __nv_bfloat162*>(&pk[g]);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float2 f = __bfloat1622float2(oh[i]);
              xs[g * 8 + 2 * i] = f.x;
              xs[g * 8 + 2 * i + 1] = f.y;
            }
          }
          float sum = 0.f;
#pragma unroll
          for (int i = 0; i < 32; ++i) sum += xs[i];
          const float mb = sum * (1.0f / 32.0f);
          float qb = 0.f;
#pragma unroll
          for (int i = 0; i < 32; ++i) { const float d = xs[i] - mb; qb = fmaf(d, d, qb); }
          const float nn = em_n + 32.0f;
          const float d = mb - em_mean;
          em_mean = fmaf(d, 32.0f / nn, em_mean);
          em_m2 += qb + d * d * (em_n * 32.0f / nn);
          em_n = nn;
        }
      }
      if constexpr (EMIT) {
        if (grow < M) ep.emit_stats[(static_cast<long long>(t / tiles_m) * 2 + half) * ep.emit_pitch + grow] = make_float2(em_mean, em_m2);
      }
    }
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 2) ptx::tmem_dealloc(tmem, TMEM_COLS);
  if (threadIdx.x == 0 && *dead && ep.status) atomicExch(ep.status, 1);
  SOD2_TRACE_DUMP()
}

}  // namespace k
}  // namespace sod2
