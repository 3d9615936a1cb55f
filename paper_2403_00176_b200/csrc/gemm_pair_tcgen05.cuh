// The varlen GEMM on CTA PAIRS: tcgen05.mma.cta_group::2.
//   out[M,N] = act(A[M,K] * Wt[N,K]^T + bias[N]) (+ residual[M,N]),  bf16 in, fp32 accumulate, bf16 out.
// A 128 x 256 tile needs 48 KB of operands per 64-wide k-chunk and 512 cycles of MMA.  Here two CTAs of a thread-block
// cluster share a 256 x BN tile: each loads its own 128 rows of A and only HALF of the weight tile (BN / 2 rows), and one
// tcgen05.mma.cta_group::2 issued by the even CTA of the pair multiplies the pair's operands out of both CTAs'
// shared memory into both CTAs' tensor memory (each CTA's TMEM holds its 128 rows x BN columns).  Operand bytes per
// flop drop by a third (BN = 256: 32 KB per CTA and k-chunk) to a half (BN = 128 against single-CTA 128 x 128).
// Protocol (one pipeline, driven by the even CTA, "leader"):
//   - both CTAs' TMA producers load their own operand slices into their own shared memory with the cta_group::2 form
//     of the load, whose completion bytes go to the LEADER's `full` barrier (no multicast anywhere: every CTA fetches
//     its own slice); the leader's producers post the expected bytes of both CTAs;
//   - the leader's MMA thread waits on `full`, issues the MMAs, and commits to `empty` of BOTH CTAs (tcgen05.commit with
//     a two-CTA multicast mask), which frees the stage for both CTAs' producers; the accumulator-full barrier is
//     committed to both CTAs the same way;
//   - each CTA's epilogue warps drain their own TMEM through the same staging / TMA-store path as the single-CTA
//     kernel and arrive on the LEADER's accumulator-empty barrier (a remote mbarrier arrive for the odd CTA);
//   - tensor memory is allocated and freed by one warp of EACH CTA with the cta_group::2 forms; a cluster barrier after
//     the barrier initialisation and one before the release keep both CTAs alive while the other can still reach them.
// Every wait is bounded (ptx.cuh).  Launch: cluster dimension 2, grid = 2 x min(pairs of tiles, SM count / 2).
// Measured: the pair's MMA instructions run at the single-CTA rate (128 cycles per 256 x 256 x 16, 74 per 256 x 128 x 16,
// issue-rate probe), and kernel time against K has the same slope as the single-CTA kernel's (0.30 us per 64-wide k-stage
// at N = 2304): the single-CTA main loop does not wait for operands at a few thousand rows, so loading fewer of them
// gains nothing, and the cluster launch, the two cluster barriers and the paired tensor-memory allocation add 0.5 - 1.5 us
// per kernel.  The planner uses this kernel only on request.
#pragma once
#include "gemm_tcgen05.cuh"

// Timeline hook for probes: expands to nothing in the library build.
#ifndef SOD2_PAIR_TRACE
#define SOD2_PAIR_TRACE(who, tag)
#endif

namespace sod2 {
namespace k {

__device__ __forceinline__ uint32_t cluster_ctarank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ uint32_t cluster_id_x() { uint32_t r; asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r)); return r; }
__device__ __forceinline__ uint32_t cluster_count_x() { uint32_t r; asm volatile("mov.u32 %0, %%nclusterid.x;" : "=r"(r)); return r; }
// shared::cluster address of the same shared-memory location in CTA `rank` of this cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// 3-D tiled TMA load into this CTA's shared memory whose completion is signalled on a barrier given by its
// shared::cluster address (the leader's): the cta_group::2 form, no multicast
__device__ __forceinline__ void tma_load_3d_pair(void* dst, const void* tmap, int x, int y, int z, uint32_t bar_cluster_addr) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(ptx::smem_u32(dst)), "l"(tmap), "r"(x), "r"(y), "r"(z), "r"(bar_cluster_addr)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(ptx::smem_u32(dst_smem)), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() { asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// D[tmem of both CTAs] (+)= A[smem of both CTAs] * B[smem of both CTAs]; issued by one thread of the leader
__device__ __forceinline__ void mma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrive on the barrier at this shared-memory offset in BOTH CTAs of the pair once the MMAs issued so far are done
__device__ __forceinline__ void mma_commit_pair(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(ptx::smem_u32(bar)), "h"(static_cast<uint16_t>(3)) : "memory");
}

template <int BN, int KCH, int STAGES>
struct GemmPairSmem {
  static constexpr int A_BYTES = KCH * GEMM_BM * 128;          // this CTA's 128 rows
  static constexpr int B_BYTES = KCH * (BN / 2) * 128;         // this CTA's half of the weight tile
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int USED = STAGES * STAGE_BYTES + GEMM_NSB * GEMM_STAGE_OUT + 2048 /*bias*/ + 8 * (2 * STAGES + 4 + 2 * GEMM_NSB) + 16;
  // plus the pad that brings the tiles to a 1024-byte boundary (the kernel checks what it really needs)
  static constexpr int TOTAL = USED + 848;
};

// tmA: {64, rows, K/64} box {64, 128, KCH}; tmB: the same view of the K-major weights, box {64, BN/2, KCH}.
template <int BN, int KCH, int STAGES, int ACT, bool RES>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_pair_bf16_tcgen05(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                       const __grid_constant__ CUtensorMap tmOut, const __grid_constant__ CUtensorMap tmRes,
                       int M, int N, int K, GemmEpilogue ep) {
  using S = GemmPairSmem<BN, KCH, STAGES>;
  constexpr int PASSES = BN / GEMM_PASS_COLS;
  constexpr int NSB = GEMM_NSB;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* out_stage = tiles + STAGES * S::STAGE_BYTES;
  float* bias_s = reinterpret_cast<float*>(out_stage + NSB * GEMM_STAGE_OUT);  // [2][256]
  uint64_t* full = reinterpret_cast<uint64_t*>(bias_s + 512);
  uint64_t* empty = full + STAGES;
  uint64_t* tmem_full = empty + STAGES;   // [2]
  uint64_t* tmem_empty = tmem_full + 2;   // [2]
  uint64_t* buf_ready = tmem_empty + 2;   // [NSB]
  uint64_t* buf_filled = buf_ready + NSB; // [NSB]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(buf_filled + NSB);
  volatile int* dead = reinterpret_cast<volatile int*>(tmem_slot + 1);
  {
    // the shared-memory layout must be the same in both CTAs of a pair (the MMA addresses both by one descriptor):
    // the dynamic window starts at the same offset in every CTA of a kernel, so the aligned base is the same too
    uint32_t dyn;
    asm("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn));
    if (static_cast<uint32_t>(tiles - smem_raw) + S::USED > dyn) {   // uniform over the grid
      if (threadIdx.x == 0 && ep.status) atomicExch(ep.status, 2);
      return;
    }
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();          // 0 = leader
  const bool leader = rank == 0;
  const int tiles_m2 = (M + 2 * GEMM_BM - 1) / (2 * GEMM_BM), tiles_n = (N + BN - 1) / BN;
  const int kchunks = K / 64;
  const int kstages = (kchunks + KCH - 1) / KCH;
  const int num_tiles = tiles_m2 * tiles_n;          // pair tiles of 256 x BN
  const int first = static_cast<int>(cluster_id_x()), step = static_cast<int>(cluster_count_x());
  constexpr uint32_t TMEM_COLS = 2 * BN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { ptx::mbar_init(&full[s], 2); ptx::mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { ptx::mbar_init(&tmem_full[b], 1); ptx::mbar_init(&tmem_empty[b], 16); }   // 8 epilogue warps of each CTA
    for (int b = 0; b < NSB; ++b) { ptx::mbar_init(&buf_ready[b], 1); ptx::mbar_init(&buf_filled[b], 8); }
    *dead = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
    ptx::prefetch_tmap(&tmA);
    ptx::prefetch_tmap(&tmB);
    ptx::prefetch_tmap(&tmOut);
    if (RES) ptx::prefetch_tmap(&tmRes);
  }
  if (warp == 2) { tmem_alloc_pair(tmem_slot, TMEM_COLS); tmem_relinquish_pair(); }
  ptx::tc_fence_before();
  __syncthreads();
  cluster_sync_all();               // both CTAs' barriers exist before anything of the other CTA can reach them
  ptx::tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  ptx::pdl_launch();
  if (threadIdx.x == 96) { SOD2_PAIR_TRACE(2, 1) }

  if (warp == 0) {
    if (lane == 0) {
      // ---- TMA producer: this CTA's A rows; completion on the leader's barrier
      ptx::pdl_wait();
      int n = 0;
      for (int w = first; w < num_tiles; w += step) {
        const int m0 = ((w % tiles_m2) * 2 + static_cast<int>(rank)) * GEMM_BM;
        for (int ks = 0; ks < kstages; ++ks, ++n) {
          const int s = n % STAGES;
          if (n >= STAGES) ptx::mbar_wait(&empty[s], ((n / STAGES) - 1) & 1, dead);
          SOD2_PAIR_TRACE(0, n)
          if (leader) ptx::mbar_expect_tx(&full[s], 2 * S::A_BYTES);
          tma_load_3d_pair(tiles + s * S::STAGE_BYTES, &tmA, 0, m0, ks * KCH, map_to_cta(ptx::smem_u32(&full[s]), 0));
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---- TMA producer: this CTA's half of the weight tile (constants: no wait for the previous kernel)
      int n = 0;
      for (int w = first; w < num_tiles; w += step) {
        const int n0 = (w / tiles_m2) * BN + static_cast<int>(rank) * (BN / 2);
        for (int ks = 0; ks < kstages; ++ks, ++n) {
          const int s = n % STAGES;
          if (n >= STAGES) ptx::mbar_wait(&empty[s], ((n / STAGES) - 1) & 1, dead);
          if (leader) ptx::mbar_expect_tx(&full[s], 2 * S::B_BYTES);
          tma_load_3d_pair(tiles + s * S::STAGE_BYTES + S::A_BYTES, &tmB, 0, n0, ks * KCH, map_to_cta(ptx::smem_u32(&full[s]), 0));
        }
      }
    }
  } else if (warp == 2) {
    if (lane == 0 && leader) {
      // ---- MMA issuer (leader only): 256 x BN x 16 per instruction over both CTAs
      constexpr uint32_t idesc = ptx::idesc_bf16(2 * GEMM_BM, BN);
      int n = 0, j = 0;
      for (int w = first; w < num_tiles; w += step, ++j) {
        const int acc = j & 1;
        if (j >= 2) ptx::mbar_wait(&tmem_empty[acc], ((j >> 1) - 1) & 1, dead);
        ptx::tc_fence_after();
        const uint32_t d = tmem + acc * BN;
        for (int ks = 0; ks < kstages; ++ks, ++n) {
          const int s = n % STAGES;
          ptx::mbar_wait(&full[s], (n / STAGES) & 1, dead);
          ptx::tc_fence_after();
          SOD2_PAIR_TRACE(1, n)
          const uint32_t a = ptx::smem_u32(tiles + s * S::STAGE_BYTES);
#pragma unroll
          for (int c = 0; c < KCH; ++c) {
            if (ks * KCH + c < kchunks) {
              const uint64_t ad = ptx::smem_desc_sw128(a + c * (GEMM_BM * 128));
              const uint64_t bd = ptx::smem_desc_sw128(a + S::A_BYTES + c * ((BN / 2) * 128));
#pragma unroll
              for (int kk = 0; kk < 4; ++kk) mma_bf16_pair(d, ad + 2 * kk, bd + 2 * kk, idesc, (ks > 0) || c != 0 || kk != 0);
            }
          }
          mma_commit_pair(&empty[s]);     // frees the stage in both CTAs
        }
        mma_commit_pair(&tmem_full[acc]);
      }
    }
  } else if (warp == 11) {
    if (lane == 0) {
      // ---- staging agent (as in the single-CTA kernel): this CTA's 128 rows
      ptx::pdl_wait();
      int my_tiles = 0;
      for (int t = first; t < num_tiles; t += step) ++my_tiles;
      const int U = my_tiles * PASSES;
      auto coords = [&](int u, int* m0, int* np) {
        const int w = first + (u / PASSES) * step;
        *m0 = ((w % tiles_m2) * 2 + static_cast<int>(rank)) * GEMM_BM;
        *np = (w / tiles_m2) * BN + (u % PASSES) * GEMM_PASS_COLS;
      };
      auto prepare = [&](int u) {
        int m0, np;
        coords(u, &m0, &np);
        const int bsel = u % NSB;
        if (RES && np < N && m0 < M) {
          ptx::mbar_expect_tx(&buf_ready[bsel], GEMM_STAGE_OUT);
          ptx::tma_load_2d(out_stage + bsel * GEMM_STAGE_OUT, &tmRes, np, m0, &buf_ready[bsel]);
        } else {
          ptx::mbar_arrive(&buf_ready[bsel]);
        }
      };
      for (int u = 0; u < NSB && u < U; ++u) prepare(u);
      for (int u = 0; u < U; ++u) {
        const int bsel = u % NSB;
        ptx::mbar_wait(&buf_filled[bsel], (u / NSB) & 1, dead);
        int m0, np;
        coords(u, &m0, &np);
        if (np < N && m0 < M) {
          tma_store_2d(&tmOut, out_stage + bsel * GEMM_STAGE_OUT, np, m0);
          bulk_commit();
        }
        if (u + NSB < U) {
          bulk_wait_read0();
          prepare(u + NSB);
        }
      }
      bulk_wait_read0();
    }
  } else {
    // ---- epilogue warps 3..10 of each CTA: its own TMEM lanes (its 128 rows)
    const int e = warp - 3;
    const int q = warp & 3;
    const int half = e >> 2;
    const int et = threadIdx.x - 96;
    const int row = q * 32 + lane;
    ptx::pdl_wait();
    const uint32_t empty_leader[2] = {map_to_cta(ptx::smem_u32(&tmem_empty[0]), 0), map_to_cta(ptx::smem_u32(&tmem_empty[1]), 0)};
    int j = 0, u = 0;
    auto load_bias = [&](int w) -> float {
      const int idx = (w / tiles_m2) * BN + et;
      return (ep.bias && et < BN && w < num_tiles && idx < N) ? __bfloat162float(ep.bias[idx]) : 0.0f;
    };
    float bias_next = load_bias(first);
    for (int w = first; w < num_tiles; w += step, ++j) {
      const int acc = j & 1;
      float* bias_t = bias_s + (j & 1) * 256;
      bias_t[et] = bias_next;
      bias_next = load_bias(w + step);
      if (warp == 3) ptx::mbar_wait_warp(&tmem_full[acc], (j >> 1) & 1, dead);
      epi_bar_sync();
      ptx::tc_fence_after();
      if (et == 0) { SOD2_PAIR_TRACE(2, 100 + j) }
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
          // every column of this warp's share has left TMEM: tell the leader's MMA thread
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(empty_leader[acc]);
        }
        const float* bp = bias_t + ps * GEMM_PASS_COLS + half * 32;
        float v[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = apply_act<ACT>(__uint_as_float(r[ps & 1][i]) + bp[i]);
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
              const float2 f = __bfloat1622float2(h[i]);
              oh[i] = __floats2bfloat162_rn(v[g * 8 + 2 * i] + f.x, v[g * 8 + 2 * i + 1] + f.y);
            }
          }
        }
#pragma unroll
        for (int g = 0; g < 4; ++g) *reinterpret_cast<uint4*>(obase + (((half * 4 + g) ^ (row & 7)) << 4)) = pk[g];
        ptx::fence_proxy_async();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&buf_filled[bsel]);
      }
    }
  }
  if (threadIdx.x == 96) { SOD2_PAIR_TRACE(2, 999) }
  ptx::tc_fence_before();
  __syncthreads();
  cluster_sync_all();               // neither CTA leaves (or frees tensor memory) while the other can still reach it
  if (warp == 2) tmem_dealloc_pair(tmem, TMEM_COLS);
  if (threadIdx.x == 0 && *dead && ep.status) atomicExch(ep.status, 1);
}

}  // namespace k
}  // namespace sod2
