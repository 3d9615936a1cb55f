// 3x3 / stride 1 / pad 1 implicit-GEMM convolution, "row-halo" form (channels-last, bf16, tcgen05).
// An output tile is 128 consecutive pixels of ONE image row.  For each kernel row dy and 64-channel
// chunk, ONE TMA box {64 ch, 130 px} brings the input row segment [w0-1, w0+128] (zero-filled outside
// the image = the padding) into shared memory as 130 swizzled 128-byte rows; the three taps dx = 0,1,2
// are the same rows read through operand descriptors whose start address is shifted by dx rows (the
// tensor core applies the 128-byte swizzle to absolute shared-memory addresses, so a start that is not
// a multiple of 8 rows is fine).  Each input pixel therefore crosses L2 -> SM three times instead of
// nine, and a stage carries 12 MMAs.  With RES (Cin = 64 and the 9 weight taps fit in shared memory) the
// weights are loaded once per CTA and stay resident; otherwise they stream with the activations.
// Warps: 0 activation TMA, 1 weight TMA, 2 staging agent (residual prefetch + output stores), 3 and 12
// MMA issuers (one TMEM accumulator each, alternate tiles), 4..11 epilogue.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include "conv_tcgen05.cuh"

namespace sod2 {
namespace k {

constexpr int C3_A_SLOT = 17 * 1024;        // 130 rows x 128 B = 16640 B, rounded to the swizzle atom
constexpr int C3_A_BYTES = 130 * 128;
constexpr int CONV3_THREADS = 416;           // 13 warps, see the kernel's role list

// Up to C3_MAX_REQ requests of one layer in one launch: their tensor maps (extents differ per request)
// and the prefix of their pixel tiles.  One pool of tiles removes a launch ramp, a weight load and a
// drain per request and evens out the waves.
constexpr int C3_MAX_REQ = 8;
struct Conv3Batch {
  CUtensorMap tx[C3_MAX_REQ], to[C3_MAX_REQ], tr[C3_MAX_REQ];   // {C, W, H, N} maps: input (box 130 px), output, residual
  int n_req;
  int tile_start[C3_MAX_REQ + 1];   // prefix sum of ceil(Wo/128) * Ho * n_img (static image counts)
  int Ho[C3_MAX_REQ], Wo[C3_MAX_REQ];
};

template <int BN, bool RES, int STAGES>
struct Conv3Smem {
  static constexpr int B_STAGE = RES ? 0 : 3 * BN * 128;
  static constexpr int STAGE_BYTES = C3_A_SLOT + B_STAGE;
  static constexpr int W_RES = RES ? 9 * BN * 128 : 0;
  static constexpr int NSB = (BN == 128 && !RES) ? 1 : 2;   // staging buffers (what fits next to the ring)
  static constexpr int TOTAL = W_RES + STAGES * STAGE_BYTES + NSB * CONV_STAGE_OUT + 896 + 2048 + 128;
};

// B.tx: {Cin, W, H, N}, box {64, 130, 1, 1};  tmW: k-chunk view {64, Cout, K/64} of the weights in
// (dy, channel chunk, dx, ci) order, box {64, BN, 3};  B.to / B.tr: {Cout, W, H, N}, box {64, 128, 1, 1}.
// p.Ho / p.Wo / p.n_img are unused (per request in B); a run-time image count (p.n_img_ptr) is only
// honoured for single-request launches and then replaces B.tile_start[1].
template <int BN, bool RES, int STAGES, int ACT, bool HASRES>
__global__ void __launch_bounds__(CONV3_THREADS, 1)
conv3x3_rows_bf16_tcgen05(const __grid_constant__ Conv3Batch B, const __grid_constant__ CUtensorMap tmW, ConvParams p) {
  using S = Conv3Smem<BN, RES, STAGES>;
  constexpr int PASSES = BN / 64;
  constexpr int NSB = S::NSB;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* wres = base;
  uint8_t* tiles = base + S::W_RES;
  uint8_t* out_stage = tiles + STAGES * S::STAGE_BYTES;
  float* bias_s = reinterpret_cast<float*>(out_stage + NSB * CONV_STAGE_OUT);  // [2][256]
  uint64_t* full = reinterpret_cast<uint64_t*>(bias_s + 512);
  uint64_t* empty = full + STAGES;
  uint64_t* tmem_full = empty + STAGES;
  uint64_t* tmem_empty = tmem_full + 2;
  uint64_t* res_full = tmem_empty + 2;
  uint64_t* stage_ready = res_full + 2;
  uint64_t* w_full = stage_ready + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(w_full + 1);
  volatile int* dead = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr uint32_t TMEM_COLS = 2 * BN < 32 ? 32 : 2 * BN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { ptx::mbar_init(&full[s], RES ? 1 : 2); ptx::mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { ptx::mbar_init(&tmem_full[b], 1); ptx::mbar_init(&tmem_empty[b], 8); }
    for (int b = 0; b < 2; ++b) { ptx::mbar_init(&res_full[b], 1); ptx::mbar_init(&stage_ready[b], 8); }
    ptx::mbar_init(w_full, 1);
    *dead = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
    ptx::prefetch_tmap(&tmW);
    for (int r = 0; r < B.n_req; ++r) {
      ptx::prefetch_tmap(&B.tx[r]);
      ptx::prefetch_tmap(&B.to[r]);
      if (HASRES) ptx::prefetch_tmap(&B.tr[r]);
    }
  }
  if (warp == 3) { ptx::tmem_alloc(tmem_slot, TMEM_COLS); ptx::tmem_relinquish(); }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // the weights do not depend on the previous kernel: resident weights are fetched before the wait
  if (RES && warp == 1 && lane == 0) {
    ptx::mbar_expect_tx(w_full, 9 * BN * 128);
    for (int dy = 0; dy < 3; ++dy) ptx::tma_load_3d(wres + dy * 3 * BN * 128, &tmW, 0, 0, dy * 3, w_full);
  }
  ptx::pdl_wait();
  ptx::pdl_launch();
  int tiles_px = B.tile_start[B.n_req];
  if (p.n_img_ptr) {   // gated sub-batch (single request): the image count is on the device
    const int n_img = min(p.n_img, max(0, p.cnt_a + p.cnt_b * static_cast<int>(*p.n_img_ptr)));
    tiles_px = ((B.Wo[0] + 127) / 128) * B.Ho[0] * n_img;
  }
  const int num_tiles = tiles_px * ((p.Cout + BN - 1) / BN);
  const int cchunks = p.Cin / 64;
  const int kstages = 3 * cchunks;               // stage = (dy, channel chunk), dy outermost

  // tile index -> (channel tile, request, image, row, first pixel); pixel tiles vary fastest
  auto decode = [&](int t, int* n0, int* img, int* h0, int* w0) -> int {
    int tp = t % tiles_px;
    *n0 = (t / tiles_px) * BN;
    int r = 0;
    while (r + 1 < B.n_req && tp >= B.tile_start[r + 1]) ++r;
    tp -= B.tile_start[r];
    const int tiles_w = (B.Wo[r] + 127) / 128;
    const int per_img = tiles_w * B.Ho[r];
    *img = tp / per_img;
    const int rem = tp - *img * per_img;
    *h0 = rem / tiles_w;
    *w0 = (rem - *h0 * tiles_w) * 128;
    return r;
  };

  if (warp == 0) {
    if (lane == 0) {
      // ---- A producer: one halo row segment per stage
      int n = 0;
      for (int t = blockIdx.x; t < num_tiles; t += gridDim.x) {
        int n0, img, h0, w0;
        const int rq = decode(t, &n0, &img, &h0, &w0);
        if (p.in_ids) img = p.in_ids[img];
        for (int ks = 0; ks < kstages; ++ks, ++n) {
          const int s = n % STAGES;
          if (n >= STAGES) ptx::mbar_wait(&empty[s], ((n / STAGES) - 1) & 1, dead);
          const int dy = ks / cchunks, cc = ks % cchunks;
          SOD2_TRACE(0, 100 + ks)
          ptx::mbar_expect_tx(&full[s], C3_A_BYTES);
          ptx::tma_load_4d(tiles + s * S::STAGE_BYTES, &B.tx[rq], cc * 64, w0 - 1, h0 + dy - 1, img, &full[s]);
        }
      }
    }
  } else if (warp == 1) {
    if (!RES && lane == 0) {
      // ---- B producer (streaming weights): the three dx taps of (dy, chunk) are consecutive k-chunks
      int n = 0;
      for (int t = blockIdx.x; t < num_tiles; t += gridDim.x) {
        const int n0 = (t / tiles_px) * BN;
        for (int ks = 0; ks < kstages; ++ks, ++n) {
          const int s = n % STAGES;
          if (n >= STAGES) ptx::mbar_wait(&empty[s], ((n / STAGES) - 1) & 1, dead);
          ptx::mbar_expect_tx(&full[s], 3 * BN * 128);
          ptx::tma_load_3d(tiles + s * S::STAGE_BYTES + C3_A_SLOT, &tmW, 0, n0, ks * 3, &full[s]);
        }
      }
    }
  } else if (warp == 3 || warp == 12) {
    if (lane == 0) {
      // ---- two MMA issuers: warp 3 takes this CTA's even tiles (accumulator 0), warp 12 the odd ones
      // (accumulator 1).  A thread that waits on a barrier between MMAs leaves the tensor pipe idle for a
      // few hundred cycles; with two issuers one thread's wait is covered by the other's MMAs.  Both
      // consume the same ring, stage n = j * kstages + ks of tile j, and BOTH wait on every stage in
      // order, also on the other issuer's: a parity wait is only meaningful for a thread that has seen
      // the barrier's previous phase, and walking all stages keeps each issuer exactly in step (the
      // in-order producer cannot refill a slot twice while an issuer still owns an earlier stage).
      constexpr uint32_t idesc = ptx::idesc_bf16(128, BN);
      const int me = warp == 3 ? 0 : 1;
      if (RES) ptx::mbar_wait(w_full, 0, dead);
      int n = 0, j = 0;
      for (int t = blockIdx.x; t < num_tiles; t += gridDim.x, ++j) {
        const int acc = j & 1;
        const bool mine = acc == me;
        if (mine) {
          if (j >= 2) ptx::mbar_wait(&tmem_empty[acc], ((j >> 1) - 1) & 1, dead);
          ptx::tc_fence_after();
        }
        const uint32_t d = tmem + acc * BN;
        for (int ks = 0; ks < kstages; ++ks, ++n) {
          const int s = n % STAGES;
          ptx::mbar_wait(&full[s], (n / STAGES) & 1, dead);
          if (!mine) continue;
          ptx::tc_fence_after();
          if (me == 0) { SOD2_TRACE(1, 200 + ks) }
          const uint32_t a = ptx::smem_u32(tiles + s * S::STAGE_BYTES);
          const uint32_t b = RES ? ptx::smem_u32(wres) + ks * 3 * BN * 128 : a + C3_A_SLOT;
#pragma unroll
          for (int dx = 0; dx < 3; ++dx) {
            const uint64_t ad = ptx::smem_desc_sw128(a + dx * 128);     // rows shifted by dx pixels
            const uint64_t bd = ptx::smem_desc_sw128(b + dx * (BN * 128));
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) ptx::mma_bf16(d, ad + 2 * kk, bd + 2 * kk, idesc, (ks | dx | kk) != 0);
          }
          ptx::mma_commit(&empty[s]);
        }
        if (mine) ptx::mma_commit(&tmem_full[acc]);
        if (mine && me == 0) { SOD2_TRACE(1, 210) }
      }
    }
  } else if (warp == 2) {
    if (lane == 0) {
      // ---- staging agent: owns the staging buffers' traffic so that no epilogue thread waits on a TMA
      // round trip.  A unit is one 64-channel pass of one tile; unit u uses buffer u % NSB.  prepare(u)
      // hands the buffer to the epilogue warps: with a residual it is TMA-loaded into the buffer (the
      // epilogue updates it in place), otherwise a plain arrive.  After the epilogue warps have filled
      // the buffer the agent stores it and, once the store has read the buffer, prepares unit u + NSB.
      int my_tiles = 0;
      for (int t = blockIdx.x; t < num_tiles; t += gridDim.x) ++my_tiles;
      const int U = my_tiles * PASSES;
      auto prepare = [&](int u) {
        const int t = blockIdx.x + (u / PASSES) * gridDim.x;
        int n0, img, h0, w0;
        const int rq = decode(t, &n0, &img, &h0, &w0);
        const int np = n0 + (u % PASSES) * 64;
        const int bsel = u % NSB;
        if (HASRES && np < p.Cout) {
          ptx::mbar_expect_tx(&res_full[bsel], CONV_STAGE_OUT);
          ptx::tma_load_4d(out_stage + bsel * CONV_STAGE_OUT, &B.tr[rq], np, w0, h0, p.res_ids ? p.res_ids[img] : img, &res_full[bsel]);
        } else {
          ptx::mbar_arrive(&res_full[bsel]);
        }
      };
      for (int u = 0; u < NSB && u < U; ++u) prepare(u);
      for (int u = 0; u < U; ++u) {
        const int bsel = u % NSB;
        ptx::mbar_wait(&stage_ready[bsel], (u / NSB) & 1, dead);
        SOD2_TRACE(2, 300)
        const int t = blockIdx.x + (u / PASSES) * gridDim.x;
        int n0, img, h0, w0;
        const int rq = decode(t, &n0, &img, &h0, &w0);
        const int np = n0 + (u % PASSES) * 64;
        if (np < p.Cout) {
          tma_store_4d(&B.to[rq], out_stage + bsel * CONV_STAGE_OUT, np, w0, h0, p.out_ids ? p.out_ids[img] : img);
          bulk_commit();
        }
        if (u + NSB < U) {
          bulk_wait_read0();
          SOD2_TRACE(2, 310)
          prepare(u + NSB);
        }
      }
      bulk_wait0();
    }
  } else if (warp >= 4 && warp < 12) {
    // ---- epilogue warps 4..11: TMEM -> +bias -> act -> (+residual, act2) -> bf16 -> swizzled staging
    const int e = warp - 4;
    const int q = warp & 3;
    const int half = e >> 2;
    const int et = threadIdx.x - 128;
    const int row = q * 32 + lane;
    const float relu2_floor = p.act2 == ACT_RELU ? 0.0f : -INFINITY;
    int j = 0, u = 0;
    auto load_bias = [&](int t) -> float {
      const int idx = (t / max(tiles_px, 1)) * BN + et;
      return (p.bias && et < BN && t < num_tiles && idx < p.Cout) ? __bfloat162float(p.bias[idx]) : 0.0f;
    };
    float bias_next = load_bias(blockIdx.x);
    for (int t = blockIdx.x; t < num_tiles; t += gridDim.x, ++j) {
      const int acc = j & 1;
      const int n0 = (t / tiles_px) * BN;
      float* bias_t = bias_s + (j & 1) * 256;
      bias_t[et] = bias_next;
      bias_next = load_bias(t + gridDim.x);
      if (warp == 4) ptx::mbar_wait_warp(&tmem_full[acc], (j >> 1) & 1, dead);   // one polling warp, the others park at the barrier
      conv_epi_bar();
      ptx::tc_fence_after();
      if (et == 0) { SOD2_TRACE(3, 400) }
#pragma unroll 1
      for (int ps = 0; ps < PASSES; ++ps, ++u) {
        const int np = n0 + ps * 64;
        const bool live = np < p.Cout;
        const int bsel = u % NSB;
        uint8_t* obase = out_stage + bsel * CONV_STAGE_OUT + row * 128;
        uint32_t r[32];
        if (live) {
          ptx::tmem_ld32(tmem + (static_cast<uint32_t>(q * 32) << 16) + acc * BN + ps * 64 + half * 32, r);
          ptx::tmem_ld_wait();
        }
        if (ps == PASSES - 1) {
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&tmem_empty[acc]);
        }
        // bias and activation before the wait for the staging buffer; then the residual loads together, the
        // arithmetic, and the stores together (loads and stores of one buffer are not reordered by the compiler)
        const float* bp = bias_t + ps * 64 + half * 32;
        float v[32];
        if (live) {
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = apply_act<ACT>(__uint_as_float(r[i]) + bp[i]);
        }
        ptx::mbar_wait_warp(&res_full[bsel], (u / NSB) & 1, dead);
        if (et == 0) { SOD2_TRACE(3, 410) }
        if (live) {
          uint4 pk[4];
          if constexpr (HASRES) {
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
                oh[i] = __floats2bfloat162_rn(fmaxf(v[g * 8 + 2 * i] + f.x, relu2_floor), fmaxf(v[g * 8 + 2 * i + 1] + f.y, relu2_floor));
              }
            }
          } else {
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              __nv_bfloat162* oh = reinterpret_cast<__nv_bfloat162*>(&pk[g]);
#pragma unroll
              for (int i = 0; i < 4; ++i) oh[i] = __floats2bfloat162_rn(v[g * 8 + 2 * i], v[g * 8 + 2 * i + 1]);
            }
          }
#pragma unroll
          for (int g = 0; g < 4; ++g) *reinterpret_cast<uint4*>(obase + (((half * 4 + g) ^ (row & 7)) << 4)) = pk[g];
        }
        if (p.gap_sum) {
          conv_epi_bar();                               // every row of the tile is in the staging buffer
          if (live) {
            int n0g, img, h0, w0;
            const int rq = decode(t, &n0g, &img, &h0, &w0);
            const int img_o = p.out_ids ? p.out_ids[img] : img;
            const int wo = B.Wo[rq];
            gap_accumulate_tile(out_stage + bsel * CONV_STAGE_OUT, et, p.gap_sum + static_cast<long long>(img_o) * p.Cout + np,
                                [&](int px) { return w0 + px < wo; });
          }
        }
        ptx::fence_proxy_async();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&stage_ready[bsel]);
        if (et == 0) { SOD2_TRACE(3, 420) }
      }
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 3) ptx::tmem_dealloc(tmem, TMEM_COLS);
  if (threadIdx.x == 0 && *dead && p.status) atomicExch(p.status, 1);
}

// Conv weights [Cout, Cin, 3, 3] -> K-major [Cout, (dy, channel chunk, dx, ci)] for the row-halo kernel.
__global__ void __launch_bounds__(256) reorder_conv3x3_rows(const __nv_bfloat16* __restrict__ in, __nv_bfloat16* __restrict__ out,
                                                             int Cout, int Cin) {
  const int cch = Cin / 64;
  const long long total = static_cast<long long>(Cout) * Cin * 9;
  for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += static_cast<long long>(gridDim.x) * blockDim.x) {
    long long r = i;
    const int ci_in = static_cast<int>(r % 64); r /= 64;
    const int dx = static_cast<int>(r % 3); r /= 3;
    const int cc = static_cast<int>(r % cch); r /= cch;
    const int dy = static_cast<int>(r % 3);
    const int co = static_cast<int>(r / 3);
    out[i] = in[((static_cast<long long>(co) * Cin + cc * 64 + ci_in) * 3 + dy) * 3 + dx];
  }
}

}  // namespace k
}  // namespace sod2
