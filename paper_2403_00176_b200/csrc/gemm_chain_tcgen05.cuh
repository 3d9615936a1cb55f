// A chain of dependent GEMMs as ONE persistent kernel.
//
// With a few thousand rows every GEMM of a transformer layer is one or two waves of tiles, so as a kernel of
// its own it pays its pipeline fill and the epilogue of its last tile in full, and SMs idle wherever the tile
// count does not divide by the SM count.  Here consecutive GEMM groups of the plan whose operands depend on
// each other row block by row block (the A operand or the residual of one is the output of an earlier one,
// LayerNorm between them folded into the epilogues) run as one launch:
//   - the tiles of all problems form one list, problem after problem, row block after row block inside a
//     problem; CTA b owns tiles b, b + grid, b + 2 grid, ... and its warps keep their roles, barriers, TMEM
//     and pipeline across problem boundaries, so the weights of the next problem stream in while the last
//     tiles of the previous one are multiplied and stored;
//   - a tile that reads rows written by an earlier problem of the chain waits until every tile of that row
//     block of the producer is stored: one counter per (problem, row block) in the arena header, bumped with
//     release semantics by the staging agent once its TMA stores have completed, polled with acquire
//     semantics (bounded) by the thread that issues the dependent TMA loads;
//   - no wait can be circular: a tile only waits for tiles that come earlier in the list, every CTA works
//     through its tiles in list order, and all CTAs of the grid are resident (grid <= SM count, one CTA per SM).
// All problems share the row count M and the tile version 128 x 128, two k-chunks per stage, three stages
// (the version whose epilogue vectors fit every epilogue form); epilogue forms are chosen per problem from
// the versions instantiated below.
#pragma once
#include "gemm_tcgen05.cuh"

// Timeline hook for probes: expands to nothing in the library build.
#ifndef SOD2_CHAIN_TRACE
#define SOD2_CHAIN_TRACE(who, tag)
#endif

namespace sod2 {
namespace k {

constexpr int CHAIN_MAX = 4;          // problems per chain
constexpr int CHAIN_BN = 128, CHAIN_KCH = 2, CHAIN_STAGES = 3;

struct GemmChainProblem {
  int N, K;
  int tiles_n;
  int tile0;        // index of the problem's first tile in the chain's tile list
  int epi;          // epilogue version (ChainEpi)
  int dep_a;        // problem that writes this problem's A rows (and their row statistics); -1: written before the launch
  int dep_r;        // problem that writes this problem's residual rows (and their row statistics); -1: before the launch
  GemmEpilogue ep;
};
struct GemmChainParams {
  int n;            // problems
  int M, tiles_m, total_tiles;
  unsigned* done;   // [n][tiles_m] stored tiles per (problem, row block); zero when the kernel starts
  GemmChainProblem p[CHAIN_MAX];
};
struct GemmChainMaps { CUtensorMap a[CHAIN_MAX], b[CHAIN_MAX], o[CHAIN_MAX], r[CHAIN_MAX]; };

// epilogue versions: activation, residual, folded LayerNorm (1 = on A, 2 = on the residual), row statistics out
enum ChainEpi : int {
  CE_PLAIN = 0,        // (none, -, -, -)
  CE_RES,              // (none, residual, -, -)
  CE_GELU,             // (gelu, -, -, -)
  CE_RES_EMIT,         // (none, residual, -, stats)
  CE_RES_LN2,          // (none, residual, normalised residual, -)
  CE_RES_LN2_EMIT,     // (none, residual, normalised residual, stats)
  CE_LN1,              // (none, -, normalised A, -)
  CE_LN1_GELU,         // (gelu, -, normalised A, -)
  CE_COUNT
};
__host__ __device__ constexpr bool chain_epi_has_res(int e) { return e == CE_RES || e == CE_RES_EMIT || e == CE_RES_LN2 || e == CE_RES_LN2_EMIT; }

// Bounded acquire-poll of a dependency counter.
__device__ __forceinline__ bool chain_wait(const unsigned* ctr, unsigned target, volatile int* dead) {
  for (uint32_t i = 0; i < (1u << 22); ++i) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ctr) : "memory");
    if (v >= target) return true;
    if ((i & 15u) == 15u) {
      if (*dead) return false;
      __nanosleep(100);
    }
  }
  *dead = 1;
  return false;
}
__device__ __forceinline__ void chain_signal(unsigned* ctr) {
  asm volatile("fence.proxy.async;" ::: "memory");   // the tile was written through the async proxy (TMA stores, completed)
  asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(ctr) : "memory");
}

// The epilogue of one 128 x 128 tile (two passes of 64 columns) for the eight epilogue warps.  Same arithmetic
// as the epilogue of gemm_bf16_tcgen05; the per-column vectors are single-buffered in `vec` (3 x 128 floats).
template <int ACT, bool RES, int LN, bool EMIT>
__device__ __forceinline__ void chain_epilogue_tile(const GemmChainProblem& P, const GemmChainParams& cp, int m_blk, int n_blk, uint32_t tmem_acc, float* vec,
                                                    uint8_t* out_stage, uint64_t* tmem_full_b, uint32_t tmem_full_parity, uint64_t* tmem_empty_b,
                                                    uint64_t* buf_ready, uint64_t* buf_filled, int& u, volatile int* dead) {
  constexpr int BN = CHAIN_BN, PASSES = BN / GEMM_PASS_COLS, NSB = GEMM_NSB;
  constexpr int NVEC = LN == 1 ? 2 : LN == 2 ? 3 : 1;
  const GemmEpilogue& ep = P.ep;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q = warp & 3, half = (warp - 3) >> 2, et = threadIdx.x - 96, row = q * 32 + lane;
  const int n0 = n_blk * BN;
  // column vectors: v0 = bias (LN = 1: c2), v1 = c1 (LN = 1) or gamma (LN = 2), v2 = beta (LN = 2)
  float vv[NVEC];
  {
    const int idx = n0 + et;
    const bool in = et < BN && idx < P.N;
#pragma unroll
    for (int w = 0; w < NVEC; ++w) {
      float x = 0.f;
      if (in) {
        if (w == 0) x = LN == 1 ? ep.ln_c2[idx] : (ep.bias ? __bfloat162float(ep.bias[idx]) : 0.0f);
        else if (w == 1) x = LN == 1 ? ep.ln_c1[idx] : __bfloat162float(ep.ln_gamma[idx]);
        else x = __bfloat162float(ep.ln_beta[idx]);
      }
      vv[w] = x;
    }
  }
  epi_bar_sync();                 // every warp has left the previous tile's vectors
  if (et < BN) {
#pragma unroll
    for (int w = 0; w < NVEC; ++w) vec[w * BN + et] = vv[w];
  }
  const int grow = m_blk * GEMM_BM + row;
  float ln_mean = 0.f, ln_rstd = 0.f;
  if constexpr (LN != 0) {
    // the statistics were written by the problem that wrote the normalised rows
    const int dep = LN == 1 ? P.dep_a : P.dep_r;
    if (dep >= 0) {
      if (lane == 0) chain_wait(cp.done + dep * cp.tiles_m + m_blk, static_cast<unsigned>(cp.p[dep].tiles_n), dead);
      __syncwarp();
    }
    if (grow < cp.M) ln_merge_stats(ep.ln_stats + grow, ep.ln_pitch, ep.ln_slots, ep.ln_cols, ep.ln_eps, &ln_mean, &ln_rstd);
  }
  float em_n = 0.f, em_mean = 0.f, em_m2 = 0.f;
  if (warp == 3) ptx::mbar_wait_warp(tmem_full_b, tmem_full_parity, dead);
  epi_bar_sync();
  ptx::tc_fence_after();
  const uint32_t taddr = tmem_acc + (static_cast<uint32_t>(q * 32) << 16) + half * 32;
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
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(tmem_empty_b);
    }
    const float* bp = vec + ps * GEMM_PASS_COLS + half * 32;
    float v[32];
    if constexpr (LN == 1) {
      const float nmr = -ln_mean * ln_rstd;
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] = apply_act<ACT>(fmaf(ln_rstd, __uint_as_float(r[ps & 1][i]), fmaf(nmr, bp[BN + i], bp[i])));
    } else {
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] = apply_act<ACT>(__uint_as_float(r[ps & 1][i]) + bp[i]);
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
    ptx::mbar_wait_warp(&buf_ready[bsel], (u / NSB) & 1, dead);
    if constexpr (RES) {
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
          oh[i] = __floats2bfloat162_rn(v[g * 8 + 2 * i] + f.x, v[g * 8 + 2 * i + 1] + f.y);
        }
      }
    }
#pragma unroll
    for (int g = 0; g < 4; ++g) *reinterpret_cast<uint4*>(obase + (((half * 4 + g) ^ (row & 7)) << 4)) = pk[g];
    if constexpr (EMIT) {
      // statistics of the 32 values just stored (as rounded to bf16), merged into the row's running pair; the
      // pair is written before the last pass is handed to the agent, whose release publishes it with the tile
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
      if (ps + 1 == PASSES && grow < cp.M)
        ep.emit_stats[(static_cast<long long>(n_blk) * 2 + half) * ep.emit_pitch + grow] = make_float2(em_mean, em_m2);
    }
    ptx::fence_proxy_async();
    __syncwarp();
    if (lane == 0) ptx::mbar_arrive(&buf_filled[bsel]);
  }
}

__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_chain_bf16_tcgen05(const __grid_constant__ GemmChainMaps maps, const __grid_constant__ GemmChainParams cp, int* status) {
  constexpr int BN = CHAIN_BN, KCH = CHAIN_KCH, STAGES = CHAIN_STAGES;
  using S = GemmSmem<BN, KCH, STAGES>;
  constexpr int PASSES = BN / GEMM_PASS_COLS;
  constexpr int NSB = GEMM_NSB;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* out_stage = tiles + STAGES * S::STAGE_BYTES;
  float* vec = reinterpret_cast<float*>(out_stage + NSB * GEMM_STAGE_OUT);  // [3][128]
  uint64_t* full = reinterpret_cast<uint64_t*>(vec + 512);
  uint64_t* empty = full + STAGES;
  uint64_t* tmem_full = empty + STAGES;   // [2]
  uint64_t* tmem_empty = tmem_full + 2;   // [2]
  uint64_t* buf_ready = tmem_empty + 2;   // [NSB]
  uint64_t* buf_filled = buf_ready + NSB; // [NSB]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(buf_filled + NSB);
  volatile int* dead = reinterpret_cast<volatile int*>(tmem_slot + 1);
  {
    uint32_t dyn;
    asm("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn));
    if (static_cast<uint32_t>(tiles - smem_raw) + S::USED > dyn) {
      if (threadIdx.x == 0 && status) atomicExch(status, 2);
      return;
    }
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr uint32_t TMEM_COLS = 2 * BN;
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { ptx::mbar_init(&full[s], 2); ptx::mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { ptx::mbar_init(&tmem_full[b], 1); ptx::mbar_init(&tmem_empty[b], 8); }
    for (int b = 0; b < NSB; ++b) { ptx::mbar_init(&buf_ready[b], 1); ptx::mbar_init(&buf_filled[b], 8); }
    *dead = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
    for (int i = 0; i < cp.n; ++i) {
      ptx::prefetch_tmap(&maps.a[i]);
      ptx::prefetch_tmap(&maps.b[i]);
      ptx::prefetch_tmap(&maps.o[i]);
      if (chain_epi_has_res(cp.p[i].epi)) ptx::prefetch_tmap(&maps.r[i]);
    }
  }
  if (warp == 2) { ptx::tmem_alloc(tmem_slot, TMEM_COLS); ptx::tmem_relinquish(); }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  ptx::pdl_launch();

  // tile s of the list -> (problem, row block, column block)
  auto locate = [&](int s, int* m_blk, int* n_blk) -> int {
    int pi = 0;
    while (pi + 1 < cp.n && s >= cp.p[pi + 1].tile0) ++pi;
    const int lt = s - cp.p[pi].tile0;
    *m_blk = lt / cp.p[pi].tiles_n;
    *n_blk = lt - *m_blk * cp.p[pi].tiles_n;
    return pi;
  };

  if (warp == 0) {
    if (lane == 0) {
      // ---- TMA producer: A stages (rows written by the previous kernel, or by an earlier problem of the chain)
      ptx::pdl_wait();
      int n = 0;
      for (int s = blockIdx.x; s < cp.total_tiles; s += gridDim.x) {
        int m_blk, n_blk;
        const int pi = locate(s, &m_blk, &n_blk);
        const GemmChainProblem& P = cp.p[pi];
        SOD2_CHAIN_TRACE(0, s * 4 + 0)
        if (P.dep_a >= 0) {
          chain_wait(cp.done + P.dep_a * cp.tiles_m + m_blk, static_cast<unsigned>(cp.p[P.dep_a].tiles_n), dead);
          asm volatile("fence.proxy.async;" ::: "memory");
        }
        SOD2_CHAIN_TRACE(0, s * 4 + 1)
        const int kstages = (P.K / 64 + KCH - 1) / KCH;
        for (int ks = 0; ks < kstages; ++ks, ++n) {
          const int st = n % STAGES;
          if (n >= STAGES) ptx::mbar_wait(&empty[st], ((n / STAGES) - 1) & 1, dead);
          ptx::mbar_expect_tx(&full[st], S::A_BYTES);
          ptx::tma_load_3d(tiles + st * S::STAGE_BYTES, &maps.a[pi], 0, m_blk * GEMM_BM, ks * KCH, &full[st]);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---- TMA producer: B stages (constant weights: never waits for another kernel or problem)
      int n = 0;
      for (int s = blockIdx.x; s < cp.total_tiles; s += gridDim.x) {
        int m_blk, n_blk;
        const int pi = locate(s, &m_blk, &n_blk);
        const int kstages = (cp.p[pi].K / 64 + KCH - 1) / KCH;
        for (int ks = 0; ks < kstages; ++ks, ++n) {
          const int st = n % STAGES;
          if (n >= STAGES) ptx::mbar_wait(&empty[st], ((n / STAGES) - 1) & 1, dead);
          ptx::mbar_expect_tx(&full[st], S::B_BYTES);
          ptx::tma_load_3d(tiles + st * S::STAGE_BYTES + S::A_BYTES, &maps.b[pi], 0, n_blk * BN, ks * KCH, &full[st]);
        }
      }
    }
  } else if (warp == 2) {
    if (lane == 0) {
      // ---- MMA issuer
      constexpr uint32_t idesc = ptx::idesc_bf16(GEMM_BM, BN);
      int n = 0, j = 0;
      for (int s = blockIdx.x; s < cp.total_tiles; s += gridDim.x, ++j) {
        int m_blk, n_blk;
        const int pi = locate(s, &m_blk, &n_blk);
        const int kchunks = cp.p[pi].K / 64;
        const int kstages = (kchunks + KCH - 1) / KCH;
        const int acc = j & 1;
        if (j >= 2) ptx::mbar_wait(&tmem_empty[acc], ((j >> 1) - 1) & 1, dead);
        ptx::tc_fence_after();
        const uint32_t d = tmem + acc * BN;
        for (int ks = 0; ks < kstages; ++ks, ++n) {
          const int st = n % STAGES;
          ptx::mbar_wait(&full[st], (n / STAGES) & 1, dead);
          ptx::tc_fence_after();
          if (ks == 0) { SOD2_CHAIN_TRACE(1, s * 4 + 0) }
          const uint32_t a = ptx::smem_u32(tiles + st * S::STAGE_BYTES);
#pragma unroll
          for (int c = 0; c < KCH; ++c) {
            if (ks * KCH + c < kchunks) {
              const uint64_t ad = ptx::smem_desc_sw128(a + c * (GEMM_BM * 128));
              const uint64_t bd = ptx::smem_desc_sw128(a + S::A_BYTES + c * (BN * 128));
#pragma unroll
              for (int kk = 0; kk < 4; ++kk) ptx::mma_bf16(d, ad + 2 * kk, bd + 2 * kk, idesc, (ks > 0) || c != 0 || kk != 0);
            }
          }
          ptx::mma_commit(&empty[st]);
        }
        ptx::mma_commit(&tmem_full[acc]);
        SOD2_CHAIN_TRACE(1, s * 4 + 1)
      }
    }
  } else if (warp == 11) {
    if (lane == 0) {
      // ---- staging agent: residual loads ahead of the epilogue, stores behind it, and the row-block counters
      ptx::pdl_wait();
      int my_tiles = 0;
      for (int s = blockIdx.x; s < cp.total_tiles; s += gridDim.x) ++my_tiles;
      const int U = my_tiles * PASSES;
      auto prepare = [&](int u) {
        int m_blk, n_blk;
        const int pi = locate(blockIdx.x + (u / PASSES) * gridDim.x, &m_blk, &n_blk);
        const GemmChainProblem& P = cp.p[pi];
        const int np = n_blk * BN + (u % PASSES) * GEMM_PASS_COLS;
        const int bsel = u % NSB;
        if (chain_epi_has_res(P.epi) && np < P.N) {
          if (P.dep_r >= 0 && (u % PASSES) == 0) {
            chain_wait(cp.done + P.dep_r * cp.tiles_m + m_blk, static_cast<unsigned>(cp.p[P.dep_r].tiles_n), dead);
            asm volatile("fence.proxy.async;" ::: "memory");
          }
          ptx::mbar_expect_tx(&buf_ready[bsel], GEMM_STAGE_OUT);
          ptx::tma_load_2d(out_stage + bsel * GEMM_STAGE_OUT, &maps.r[pi], np, m_blk * GEMM_BM, &buf_ready[bsel]);
        } else {
          ptx::mbar_arrive(&buf_ready[bsel]);
        }
      };
      // A unit whose residual comes from an earlier problem of the chain is prepared only once every earlier tile
      // of this CTA has been published: the tile it waits for may be one of them, and this thread is the one that
      // publishes.  Units are prepared in order, each as soon as its buffer is free (the store of unit u - NSB has
      // read it) and that condition holds.
      int prepared = 0, published = 0;
      auto eligible = [&](int u) {
        int m_blk, n_blk;
        const int pi = locate(blockIdx.x + (u / PASSES) * gridDim.x, &m_blk, &n_blk);
        return !(chain_epi_has_res(cp.p[pi].epi) && cp.p[pi].dep_r >= 0) || published >= u / PASSES;
      };
      while (prepared < NSB && prepared < U && eligible(prepared)) prepare(prepared++);
      for (int u = 0; u < U; ++u) {
        const int bsel = u % NSB;
        ptx::mbar_wait(&buf_filled[bsel], (u / NSB) & 1, dead);
        int m_blk, n_blk;
        const int pi = locate(blockIdx.x + (u / PASSES) * gridDim.x, &m_blk, &n_blk);
        const int np = n_blk * BN + (u % PASSES) * GEMM_PASS_COLS;
        if (np < cp.p[pi].N) {
          tma_store_2d(&maps.o[pi], out_stage + bsel * GEMM_STAGE_OUT, np, m_blk * GEMM_BM);
          bulk_commit();
        }
        if ((u % PASSES) == PASSES - 1) {
          // the tile is complete once its stores have been performed; then it is published
          bulk_wait0();
          chain_signal(cp.done + pi * cp.tiles_m + m_blk);
          ++published;
          SOD2_CHAIN_TRACE(3, (blockIdx.x + (u / PASSES) * gridDim.x) * 4 + 0)
        }
        bool drained = false;
        while (prepared < U && prepared <= u + NSB && eligible(prepared)) {
          if (!drained) { bulk_wait_read0(); drained = true; }
          prepare(prepared++);
        }
      }
      bulk_wait0();
    }
  } else {
    // ---- epilogue warps 3..10
    ptx::pdl_wait();
    int j = 0, u = 0;
    for (int s = blockIdx.x; s < cp.total_tiles; s += gridDim.x, ++j) {
      int m_blk, n_blk;
      const int pi = locate(s, &m_blk, &n_blk);
      const GemmChainProblem& P = cp.p[pi];
      const int acc = j & 1;
      const uint32_t tacc = tmem + acc * BN;
      const uint32_t par = (j >> 1) & 1;
#define SOD2_CE(ACT_, RES_, LN_, EMIT_) \
      chain_epilogue_tile<ACT_, RES_, LN_, EMIT_>(P, cp, m_blk, n_blk, tacc, vec, out_stage, &tmem_full[acc], par, &tmem_empty[acc], buf_ready, buf_filled, u, dead)
      if (threadIdx.x == 96) { SOD2_CHAIN_TRACE(2, s * 4 + 0) }
      switch (P.epi) {
        case CE_PLAIN: SOD2_CE(ACT_NONE, false, 0, false); break;
        case CE_RES: SOD2_CE(ACT_NONE, true, 0, false); break;
        case CE_GELU: SOD2_CE(ACT_GELU, false, 0, false); break;
        case CE_RES_EMIT: SOD2_CE(ACT_NONE, true, 0, true); break;
        case CE_RES_LN2: SOD2_CE(ACT_NONE, true, 2, false); break;
        case CE_RES_LN2_EMIT: SOD2_CE(ACT_NONE, true, 2, true); break;
        case CE_LN1: SOD2_CE(ACT_NONE, false, 1, false); break;
        default: SOD2_CE(ACT_GELU, false, 1, false); break;
      }
      if (threadIdx.x == 96) { SOD2_CHAIN_TRACE(2, s * 4 + 1) }
#undef SOD2_CE
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 2) ptx::tmem_dealloc(tmem, TMEM_COLS);
  if (threadIdx.x == 0 && *dead && status) atomicExch(status, 1);
}

}  // namespace k
}  // namespace sod2
