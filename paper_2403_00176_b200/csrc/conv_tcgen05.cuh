// Implicit-GEMM convolution on the tcgen05 main loop of the GEMM kernel, channels-last activations.
//   y[n,ho,wo,co] = act2( act( sum_{dy,dx,ci} x[n, ho*s+dy-p, wo*s+dx-p, ci] * w[co, (dy,dx), ci] + bias[co] ) + res[n,ho,wo,co] )
// bf16 in, fp32 accumulate (TMEM), bf16 out.  The "A operand" of output tile (128 pixels = TH x TW
// patch of one image) for tap (dy,dx) and 64 input channels is ONE 4-D TMA box {64 ch, TW, TH, 1} of
// the NHWC input at the shifted coordinate: every pixel is one 128-byte swizzled row, out-of-image
// coordinates are zero-filled by TMA, which is the zero padding; stride-2 convolutions use the
// tensor map's element stride.  The "B operand" is the prepacked weight matrix [Cout, taps*Cin]
// (K-major), loaded with the same k-chunk boxes as in the GEMM.  Extents H, W are per request and
// known only at run time: tensor maps are encoded per bound shape.
//
// Warp roles (384 threads, persistent, 1 CTA/SM):
//   warps 0,1   TMA producers for the A chunks of a stage (even / odd chunk: one thread sustains only
//               about one TMA instruction per 170 ns)
//   warp 2      TMA producer for B (one 3-D k-chunk box per stage)
//   warp 3      MMA issuer, two TMEM accumulators
//   warps 4..11 epilogue in passes of 64 output channels: TMEM -> +bias -> act -> +residual (TMA-loaded
//               into the staging tile, updated in place) -> act2 -> bf16 -> swizzled staging -> TMA store
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include "gemm_tcgen05.cuh"
#include "ptx.cuh"

namespace sod2 {
namespace k {

struct ConvParams {
  int n_img, Ho, Wo;         // output extents
  int Cin, Cout;
  int ksize, stride, pad;
  int TW, TH;                // pixel patch of a tile: TW * TH == 128
  int korder;                // 0: weight k-chunks in (dy, dx, chunk) order; 1: (dy, chunk, dx) order (3x3 only)
  // execution-determined image count (gated sub-batch): n_img = cnt_a + cnt_b * *n_img_ptr, read on the
  // device after the producing kernel has finished; n_img above is then only the static upper bound
  const long long* n_img_ptr;
  int cnt_a, cnt_b;
  // index-indirect operands (gated sub-batch without copies): image n of the operand is image ids[n] of
  // the tensor the map describes; nullptr = direct
  const int* in_ids;
  const int* res_ids;
  const int* out_ids;
  const __nv_bfloat16* bias; // [Cout] or nullptr
  // optional: per-(image, channel) sums of the stored (bf16) outputs, added with fp64 atomics to
  // gap_sum[image id][Cout] -- the global-average-pool numerators of the next gate, accumulated where the
  // tensor is produced instead of re-reading it (a decision scalar: the order of the fp64 additions moves
  // it by less than n * 2^-53, far inside the band in which decisions are compared)
  double* gap_sum;
  int has_residual;
  int act2;                  // ACT_NONE or ACT_RELU after the residual add
  int* status;
};

constexpr int CONV_THREADS = 384;
constexpr int CONV_STAGE_OUT = 128 * 128;   // 16 KB: 128 pixels x 64 channels bf16

template <int BN, int KCH, int STAGES>
struct ConvSmem {
  static constexpr int A_BYTES = KCH * 128 * 128;
  static constexpr int B_BYTES = KCH * BN * 128;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int TOTAL = STAGES * STAGE_BYTES + CONV_STAGE_OUT + 896 + 2048 + 128;
};

__device__ __forceinline__ void tma_store_4d(const void* tmap, const void* src, int c0, int c1, int c2, int c3) {
  asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
               ::"l"(tmap), "r"(ptx::smem_u32(src)), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void conv_epi_bar() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// Sum over the valid pixels of one staged [128 pixels x 64 channels] bf16 tile (128-byte rows, 16-byte
// granules XOR-ed with the row), by the 256 epilogue threads, in fp64 (a bf16 value is exact in fp64; masked
// pixels add +0.0).  valid(px) tells whether tile pixel px lies in the image.
template <typename Valid>
__device__ __forceinline__ void gap_accumulate_tile(const uint8_t* stage, int et, double* dst_row, Valid valid) {
  // thread (channel pair et & 31, pixel group et >> 5): 16 pixels x 2 channels, one 32-bit shared load per
  // pixel, four independent fp64 chains (even / odd pixels x two channels), then two atomics
  const int chp = et & 31, pg = et >> 5;
  double a0 = 0.0, a1 = 0.0, b0 = 0.0, b1 = 0.0;
#pragma unroll
  for (int i = 0; i < 16; i += 2) {
    const int px0 = pg * 16 + i, px1 = px0 + 1;
    const uint32_t w0 = valid(px0) ? *reinterpret_cast<const uint32_t*>(stage + px0 * 128 + ((((chp >> 2) ^ (px0 & 7)) << 4) + (chp & 3) * 4)) : 0u;
    const uint32_t w1 = valid(px1) ? *reinterpret_cast<const uint32_t*>(stage + px1 * 128 + ((((chp >> 2) ^ (px1 & 7)) << 4) + (chp & 3) * 4)) : 0u;
    a0 += static_cast<double>(__uint_as_float(w0 << 16)); a1 += static_cast<double>(__uint_as_float(w0 & 0xffff0000u));
    b0 += static_cast<double>(__uint_as_float(w1 << 16)); b1 += static_cast<double>(__uint_as_float(w1 & 0xffff0000u));
  }
  atomicAdd(dst_row + 2 * chp, a0 + b0);
  atomicAdd(dst_row + 2 * chp + 1, a1 + b1);
}

// tmX: {Cin, W, H, N} bf16, box {64, TW, TH, 1}, element strides {1, s, s, 1}
// tmW: {64, Cout, K/64} k-chunk view of [Cout, K], box {64, BN, KCH}
// tmOut / tmRes: {Cout, Wo, Ho, N}, box {64, TW, TH, 1}
template <int BN, int KCH, int STAGES, int ACT, bool HASRES>
__global__ void __launch_bounds__(CONV_THREADS, 1)
conv_igemm_bf16_tcgen05(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW,
                        const __grid_constant__ CUtensorMap tmOut, const __grid_constant__ CUtensorMap tmRes, ConvParams p) {
  using S = ConvSmem<BN, KCH, STAGES>;
  constexpr int PASSES = BN / 64;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* out_stage = tiles + STAGES * S::STAGE_BYTES;
  float* bias_s = reinterpret_cast<float*>(out_stage + CONV_STAGE_OUT);  // [2][256]
  uint64_t* full = reinterpret_cast<uint64_t*>(bias_s + 512);
  uint64_t* empty = full + STAGES;
  uint64_t* tmem_full = empty + STAGES;
  uint64_t* tmem_empty = tmem_full + 2;
  uint64_t* res_full = tmem_empty + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(res_full + 1);
  volatile int* dead = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr uint32_t TMEM_COLS = (2 * BN < 32) ? 32 : 2 * BN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { ptx::mbar_init(&full[s], 3); ptx::mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { ptx::mbar_init(&tmem_full[b], 1); ptx::mbar_init(&tmem_empty[b], 8); }
    ptx::mbar_init(res_full, 1);
    *dead = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
    ptx::prefetch_tmap(&tmX);
    ptx::prefetch_tmap(&tmW);
    ptx::prefetch_tmap(&tmOut);
    if (HASRES) ptx::prefetch_tmap(&tmRes);
  }
  if (warp == 3) { ptx::tmem_alloc(tmem_slot, TMEM_COLS); ptx::tmem_relinquish(); }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  ptx::pdl_wait();
  ptx::pdl_launch();
  int n_img = p.n_img;
  if (p.n_img_ptr) n_img = min(p.n_img, max(0, p.cnt_a + p.cnt_b * static_cast<int>(*p.n_img_ptr)));
  const int tiles_w = (p.Wo + p.TW - 1) / p.TW, tiles_h = (p.Ho + p.TH - 1) / p.TH;
  const int tiles_px = tiles_w * tiles_h * n_img;
  const int num_tiles = tiles_px * ((p.Cout + BN - 1) / BN);
  const int cchunks = p.Cin / 64;                         // 64-channel chunks per tap
  const int kchunks = p.ksize * p.ksize * cchunks;        // k-chunks in tap-major order
  const int kstages = (kchunks + KCH - 1) / KCH;

  // tile index -> (channel tile, image, patch origin); pixel tiles vary fastest so that CTAs running
  // together share the weight tile in L2
  auto decode = [&](int t, int* n0, int* img, int* ho0, int* wo0) {
    const int tp = t % tiles_px;
    *n0 = (t / tiles_px) * BN;
    *img = tp / (tiles_w * tiles_h);
    const int r = tp % (tiles_w * tiles_h);
    *ho0 = (r / tiles_w) * p.TH;
    *wo0 = (r % tiles_w) * p.TW;
  };

  if (warp < 2) {
    if (lane == 0) {
      // ---- A producers: warp 0 loads the even chunks of every stage, warp 1 the odd ones
      int n = 0;
      for (int t = blockIdx.x; t < num_tiles; t += gridDim.x) {
        int n0, img, ho0, wo0;
        decode(t, &n0, &img, &ho0, &wo0);
        if (p.in_ids) img = p.in_ids[img];
        for (int ks = 0; ks < kstages; ++ks, ++n) {
          const int s = n % STAGES;
          if (n >= STAGES) ptx::mbar_wait(&empty[s], ((n / STAGES) - 1) & 1, dead);
          int mine = 0;
          for (int c = warp; c < KCH; c += 2) ++mine;
          ptx::mbar_expect_tx(&full[s], mine * 128 * 128);
          for (int c = warp; c < KCH; c += 2) {
            const int q = ks * KCH + c;          // k-chunk: tap-major, then 64-channel chunk
            int dy, dx, cc;
            if (p.korder) { dy = q / (3 * cchunks); cc = (q / 3) % cchunks; dx = q % 3; }
            else { const int tap = q / cchunks; cc = q % cchunks; dy = tap / p.ksize; dx = tap % p.ksize; }
            // chunks past the end (K tail of the last stage) are loaded far out of range: zero fill
            const int hi = q < kchunks ? ho0 * p.stride + dy - p.pad : -100000;
            ptx::tma_load_4d(tiles + s * S::STAGE_BYTES + c * (128 * 128), &tmX, cc * 64, wo0 * p.stride + dx - p.pad, hi, img, &full[s]);
          }
        }
      }
    }
  } else if (warp == 2) {
    if (lane == 0) {
      // ---- B producer
      int n = 0;
      for (int t = blockIdx.x; t < num_tiles; t += gridDim.x) {
        const int n0 = (t / tiles_px) * BN;
        for (int ks = 0; ks < kstages; ++ks, ++n) {
          const int s = n % STAGES;
          if (n >= STAGES) ptx::mbar_wait(&empty[s], ((n / STAGES) - 1) & 1, dead);
          ptx::mbar_expect_tx(&full[s], S::B_BYTES);
          ptx::tma_load_3d(tiles + s * S::STAGE_BYTES + S::A_BYTES, &tmW, 0, n0, ks * KCH, &full[s]);
        }
      }
    }
  } else if (warp == 3) {
    if (lane == 0) {
      // ---- MMA issuer
      constexpr uint32_t idesc = ptx::idesc_bf16(128, BN);
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
              const uint64_t ad = ptx::smem_desc_sw128(a + c * (128 * 128));
              const uint64_t bd = ptx::smem_desc_sw128(a + S::A_BYTES + c * (BN * 128));
#pragma unroll
              for (int kk = 0; kk < 4; ++kk) ptx::mma_bf16(d, ad + 2 * kk, bd + 2 * kk, idesc, (ks | c | kk) != 0);
            }
          }
          ptx::mma_commit(&empty[s]);
        }
        ptx::mma_commit(&tmem_full[acc]);
      }
    }
  } else {
    // ---- epilogue warps 4..11
    const int e = warp - 4;
    const int q = warp & 3;
    const int half = e >> 2;          // which 32-channel half of the 64-channel pass
    const int et = threadIdx.x - 128; // 0..255
    const int row = q * 32 + lane;    // pixel inside the tile
    const float relu2_floor = p.act2 == ACT_RELU ? 0.0f : -INFINITY;
    int j = 0, rp = 0;
    auto load_bias = [&](int t) -> float {
      const int idx = (t / tiles_px) * BN + et;
      return (p.bias && et < BN && t < num_tiles && idx < p.Cout) ? __bfloat162float(p.bias[idx]) : 0.0f;
    };
    float bias_next = load_bias(blockIdx.x);
    for (int t = blockIdx.x; t < num_tiles; t += gridDim.x, ++j) {
      const int acc = j & 1;
      int n0, img, ho0, wo0;
      decode(t, &n0, &img, &ho0, &wo0);
      const int img_r = p.res_ids ? p.res_ids[img] : img, img_o = p.out_ids ? p.out_ids[img] : img;
      float* bias_t = bias_s + (j & 1) * 256;
      bias_t[et] = bias_next;
      bias_next = load_bias(t + gridDim.x);
      if (warp == 4) ptx::mbar_wait_warp(&tmem_full[acc], (j >> 1) & 1, dead);   // one polling warp, the others park at the barrier
      conv_epi_bar();
      ptx::tc_fence_after();
#pragma unroll 1
      for (int ps = 0; ps < PASSES; ++ps) {
        const int np = n0 + ps * 64;
        const bool live = np < p.Cout;
        constexpr bool res_t = HASRES;
        const bool res = res_t && live;
        if (res) {
          if (et == 0) {
            bulk_wait_read0();
            ptx::mbar_expect_tx(res_full, CONV_STAGE_OUT);
            ptx::tma_load_4d(out_stage, &tmRes, np, wo0, ho0, img_r, res_full);
          }
          ptx::mbar_wait_warp(res_full, rp & 1, dead);
          ++rp;
        }
        uint8_t* obase = out_stage + row * 128;
        uint4 pk[4];
        if (live) {
          uint32_t r[32];
          ptx::tmem_ld32(tmem + (static_cast<uint32_t>(q * 32) << 16) + acc * BN + ps * 64 + half * 32, r);
          ptx::tmem_ld_wait();
          const float* bp = bias_t + ps * 64 + half * 32;
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            float v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = apply_act<ACT>(__uint_as_float(r[g * 8 + i]) + bp[g * 8 + i]);
            if constexpr (HASRES) {
              const uint4 rv = *reinterpret_cast<const uint4*>(obase + (((half * 4 + g) ^ (row & 7)) << 4));
              const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&rv);
#pragma unroll
              for (int i = 0; i < 4; ++i) { const float2 f = __bfloat1622float2(h[i]); v[2 * i] += f.x; v[2 * i + 1] += f.y; }
#pragma unroll
              for (int i = 0; i < 8; ++i) v[i] = fmaxf(v[i], relu2_floor);
            }
            __nv_bfloat162* oh = reinterpret_cast<__nv_bfloat162*>(&pk[g]);
#pragma unroll
            for (int i = 0; i < 4; ++i) oh[i] = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
          }
        }
        if (!res) {
          if (et == 0) bulk_wait_read0();
          conv_epi_bar();
        }
        if (live) {
#pragma unroll
          for (int g = 0; g < 4; ++g) *reinterpret_cast<uint4*>(obase + (((half * 4 + g) ^ (row & 7)) << 4)) = pk[g];
        }
        ptx::tc_fence_before();
        ptx::fence_proxy_async();
        __syncwarp();
        if (ps == PASSES - 1 && lane == 0) ptx::mbar_arrive(&tmem_empty[acc]);
        conv_epi_bar();
        if (et == 0 && live) {
          tma_store_4d(&tmOut, out_stage, np, wo0, ho0, img_o);
          bulk_commit();
        }
        if (p.gap_sum && live) {
          const int tw_shift = __ffs(p.TW) - 1;      // TW * TH == 128: a power of two
          gap_accumulate_tile(out_stage, et, p.gap_sum + static_cast<long long>(img_o) * p.Cout + np, [&](int px) {
            return ho0 + (px >> tw_shift) < p.Ho && wo0 + (px & (p.TW - 1)) < p.Wo;
          });
        }
      }
    }
    if (et == 0) bulk_wait0();
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 3) ptx::tmem_dealloc(tmem, TMEM_COLS);
  if (threadIdx.x == 0 && *dead && p.status) atomicExch(p.status, 1);
}

// ---------------------------------------------------------------------------------------------
// Layout changes between the graph's NCHW tensors and the channels-last layout the convolution
// groups use internally: [N, C, H*W] <-> [N, H*W, C], 32x32 tiles through shared memory.
__global__ void __launch_bounds__(256) nchw_to_nhwc_bf16(const __nv_bfloat16* __restrict__ in, __nv_bfloat16* __restrict__ out,
                                                          int C, long long HW) {
  // tile: 64 channels x 64 pixels; reads are 128-byte pixel runs per channel, writes 128-byte channel runs per pixel
  __shared__ __nv_bfloat16 tile[64][66];
  const long long img = blockIdx.z;
  const long long p0 = static_cast<long long>(blockIdx.x) * 64;
  const int c0 = blockIdx.y * 64;
  for (int i = threadIdx.x; i < 64 * 32; i += 256) {       // 64 channels x 32 pixel pairs
    const int c = i >> 5, pp = (i & 31) * 2;
    const long long px = p0 + pp;
    if (c0 + c < C) {
      const __nv_bfloat16* src = in + (img * C + c0 + c) * HW + px;
      if (px + 1 < HW && ((reinterpret_cast<uintptr_t>(src) & 3) == 0)) {
        const __nv_bfloat162 v = *reinterpret_cast<const __nv_bfloat162*>(src);
        tile[c][pp] = v.x; tile[c][pp + 1] = v.y;
      } else {
        if (px < HW) tile[c][pp] = src[0];
        if (px + 1 < HW) tile[c][pp + 1] = src[1];
      }
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < 64 * 32; i += 256) {       // 64 pixels x 32 channel pairs
    const int pxl = i >> 5, cp = (i & 31) * 2;
    const long long px = p0 + pxl;
    if (px < HW && c0 + cp < C) {
      __nv_bfloat16* dst = out + (img * HW + px) * C + c0 + cp;
      if (c0 + cp + 1 < C && ((reinterpret_cast<uintptr_t>(dst) & 3) == 0)) *reinterpret_cast<__nv_bfloat162*>(dst) = __nv_bfloat162(tile[cp][pxl], tile[cp + 1][pxl]);
      else { dst[0] = tile[cp][pxl]; if (c0 + cp + 1 < C) dst[1] = tile[cp + 1][pxl]; }
    }
  }
}
__global__ void __launch_bounds__(256) nhwc_to_nchw_bf16(const __nv_bfloat16* __restrict__ in, __nv_bfloat16* __restrict__ out,
                                                          int C, long long HW) {
  __shared__ __nv_bfloat16 tile[64][66];   // [pixel][channel]
  const long long img = blockIdx.z;
  const long long p0 = static_cast<long long>(blockIdx.x) * 64;
  const int c0 = blockIdx.y * 64;
  for (int i = threadIdx.x; i < 64 * 32; i += 256) {
    const int pxl = i >> 5, cp = (i & 31) * 2;
    const long long px = p0 + pxl;
    if (px < HW && c0 + cp < C) {
      const __nv_bfloat16* src = in + (img * HW + px) * C + c0 + cp;
      if (c0 + cp + 1 < C && ((reinterpret_cast<uintptr_t>(src) & 3) == 0)) {
        const __nv_bfloat162 v = *reinterpret_cast<const __nv_bfloat162*>(src);
        tile[pxl][cp] = v.x; tile[pxl][cp + 1] = v.y;
      } else { tile[pxl][cp] = src[0]; if (c0 + cp + 1 < C) tile[pxl][cp + 1] = src[1]; }
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < 64 * 32; i += 256) {
    const int c = i >> 5, pp = (i & 31) * 2;
    const long long px = p0 + pp;
    if (c0 + c < C) {
      __nv_bfloat16* dst = out + (img * C + c0 + c) * HW + px;
      if (px + 1 < HW && ((reinterpret_cast<uintptr_t>(dst) & 3) == 0)) *reinterpret_cast<__nv_bfloat162*>(dst) = __nv_bfloat162(tile[pp][c], tile[pp + 1][c]);
      else { if (px < HW) dst[0] = tile[pp][c]; if (px + 1 < HW) dst[1] = tile[pp + 1][c]; }
    }
  }
}

// The same two layout changes with 16-byte global accesses on both sides (C % 8 == 0, HW % 8 == 0): a
// 64 x 64 tile goes through shared memory as rows of eight-element vectors whose position inside the row
// is XOR-ed with the row's group of eight, so that the strided 2-byte gathers of the transposed read hit
// distinct banks.
// Up to LAYOUT_MAX_SEG tensors (the requests of a batch, each with its own image size) per launch: blockIdx.x
// walks the 64-pixel tiles of all images of all segments.
constexpr int LAYOUT_MAX_SEG = 8;
struct LayoutBatch {
  int n_seg, C;
  int tile_start[LAYOUT_MAX_SEG + 1];        // prefix sum of images * ceil(HW / 64)
  const __nv_bfloat16* in[LAYOUT_MAX_SEG];
  __nv_bfloat16* out[LAYOUT_MAX_SEG];
  long long HW[LAYOUT_MAX_SEG];
};
__device__ __forceinline__ int layout_locate(const LayoutBatch& B, long long* img, long long* p0) {
  int si = 0;
  while (si + 1 < B.n_seg && static_cast<int>(blockIdx.x) >= B.tile_start[si + 1]) ++si;
  const int tl = static_cast<int>(blockIdx.x) - B.tile_start[si];
  const int per_img = static_cast<int>((B.HW[si] + 63) / 64);
  *img = tl / per_img;
  *p0 = static_cast<long long>(tl - static_cast<int>(*img) * per_img) * 64;
  return si;
}
__global__ void __launch_bounds__(256) nchw_to_nhwc_bf16_v8(const __grid_constant__ LayoutBatch B) {
  __shared__ __align__(16) __nv_bfloat16 tile[64][72];   // [channel][pixel vectors, permuted]
  long long img, p0;
  const int si = layout_locate(B, &img, &p0);
  const __nv_bfloat16* __restrict__ in = B.in[si];
  __nv_bfloat16* __restrict__ out = B.out[si];
  const int C = B.C;
  const long long HW = B.HW[si];
  const int c0 = blockIdx.y * 64;
#pragma unroll
  for (int it = 0; it < 2; ++it) {
    const int i = threadIdx.x + it * 256;
    const int c = i >> 3, v = i & 7;
    if (c0 + c < C && p0 + v * 8 < HW)
      *reinterpret_cast<uint4*>(&tile[c][(v ^ ((c >> 3) & 7)) * 8]) = *reinterpret_cast<const uint4*>(in + (img * C + c0 + c) * HW + p0 + v * 8);
  }
  __syncthreads();
#pragma unroll
  for (int it = 0; it < 2; ++it) {
    const int i = threadIdx.x + it * 256;
    const int px = i >> 3, cv = i & 7;
    if (p0 + px < HW && c0 + cv * 8 < C) {
      __align__(16) __nv_bfloat16 o[8];
      const int col = (((px >> 3) ^ cv) * 8) + (px & 7);
#pragma unroll
      for (int k8 = 0; k8 < 8; ++k8) o[k8] = tile[cv * 8 + k8][col];
      *reinterpret_cast<uint4*>(out + (img * HW + p0 + px) * C + c0 + cv * 8) = *reinterpret_cast<const uint4*>(o);
    }
  }
}
__global__ void __launch_bounds__(256) nhwc_to_nchw_bf16_v8(const __grid_constant__ LayoutBatch B) {
  __shared__ __align__(16) __nv_bfloat16 tile[64][72];   // [pixel][channel vectors, permuted]
  long long img, p0;
  const int si = layout_locate(B, &img, &p0);
  const __nv_bfloat16* __restrict__ in = B.in[si];
  __nv_bfloat16* __restrict__ out = B.out[si];
  const int C = B.C;
  const long long HW = B.HW[si];
  const int c0 = blockIdx.y * 64;
#pragma unroll
  for (int it = 0; it < 2; ++it) {
    const int i = threadIdx.x + it * 256;
    const int px = i >> 3, cv = i & 7;
    if (p0 + px < HW && c0 + cv * 8 < C)
      *reinterpret_cast<uint4*>(&tile[px][(cv ^ ((px >> 3) & 7)) * 8]) = *reinterpret_cast<const uint4*>(in + (img * HW + p0 + px) * C + c0 + cv * 8);
  }
  __syncthreads();
#pragma unroll
  for (int it = 0; it < 2; ++it) {
    const int i = threadIdx.x + it * 256;
    const int c = i >> 3, v = i & 7;
    if (c0 + c < C && p0 + v * 8 < HW) {
      __align__(16) __nv_bfloat16 o[8];
      const int col = (((c >> 3) ^ v) * 8) + (c & 7);
#pragma unroll
      for (int k8 = 0; k8 < 8; ++k8) o[k8] = tile[v * 8 + k8][col];
      *reinterpret_cast<uint4*>(out + (img * C + c0 + c) * HW + p0 + v * 8) = *reinterpret_cast<const uint4*>(o);
    }
  }
}

// Global average pool of a channels-last tensor with fp64 accumulation (decision scalar / final
// feature): p[n,c] = mean_{h,w} x[n,h,w,c].  Two kernels with a fixed summation order, so the result
// is deterministic: pixel slabs -> partial sums in scratch, then a serial sum over the slabs.
struct GapParams {
  const __nv_bfloat16* x;   // [N, HW, C]
  double* partial;          // scratch [N, slabs, C]
  void* out;                // [N, C] bf16 or f32 (or nullptr when only the fp64 means are wanted)
  double* out_f64;          // optional [N, C] fp64 means
  int out_bf16;
  int C, slabs;
  long long HW;
};
// Up to GAP_MAX_SEG tensors (the requests of a batch) pooled by one launch: blockIdx.z walks the images of
// all segments, blockIdx.y the pixel slabs (CTAs past a segment's slab count exit).
constexpr int GAP_MAX_SEG = 8;
struct GapBatch {
  int n_seg;
  int img_start[GAP_MAX_SEG + 1];
  GapParams seg[GAP_MAX_SEG];
};
__global__ void __launch_bounds__(256) gap_partial_f64(const __grid_constant__ GapBatch B) {
  // every thread owns 8 channels (one 16-byte load) of a pixel; C/8 threads cover a pixel, the
  // remaining factor of the CTA walks pixels; fp64 partial sums, fixed-order reduction in shared memory
  __shared__ double part[256][8];
  ptx::pdl_wait();
  ptx::pdl_launch();
  int si = 0;
  while (si + 1 < B.n_seg && static_cast<int>(blockIdx.z) >= B.img_start[si + 1]) ++si;
  const GapParams& p = B.seg[si];
  if (static_cast<int>(blockIdx.y) >= p.slabs) return;
  const long long img = static_cast<int>(blockIdx.z) - B.img_start[si];
  const int tpp = (p.C + 7) >> 3;                 // threads per pixel (C <= 2048)
  const int ppi = 256 / tpp;                      // pixels per CTA iteration
  const int cg = threadIdx.x % tpp, pg = threadIdx.x / tpp;
  const long long per = (p.HW + p.slabs - 1) / p.slabs;
  const long long p0 = blockIdx.y * per, p1 = min(p.HW, p0 + per);
  double acc[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i] = 0.0;
  if (pg < ppi && (p.C & 7) == 0) {
    // eight loads in flight per thread, added in pixel order (the summation order does not change)
    const __nv_bfloat16* base = p.x + img * p.HW * p.C + cg * 8;
    long long px = p0 + pg;
    for (; px + 7LL * ppi < p1; px += 8LL * ppi) {
      uint4 u[8];
#pragma unroll
      for (int k8 = 0; k8 < 8; ++k8) u[k8] = *reinterpret_cast<const uint4*>(base + (px + static_cast<long long>(k8) * ppi) * p.C);
#pragma unroll
      for (int k8 = 0; k8 < 8; ++k8) {
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u[k8]);
#pragma unroll
        for (int i = 0; i < 4; ++i) { const float2 f = __bfloat1622float2(h[i]); acc[2 * i] += static_cast<double>(f.x); acc[2 * i + 1] += static_cast<double>(f.y); }
      }
    }
    for (; px < p1; px += ppi) {
      const uint4 u = *reinterpret_cast<const uint4*>(base + px * p.C);
      const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
      for (int i = 0; i < 4; ++i) { const float2 f = __bfloat1622float2(h[i]); acc[2 * i] += static_cast<double>(f.x); acc[2 * i + 1] += static_cast<double>(f.y); }
    }
  } else if (pg < ppi) {
    for (long long px = p0 + pg; px < p1; px += ppi)
      for (int i = 0; i < 8 && cg * 8 + i < p.C; ++i) acc[i] += static_cast<double>(__bfloat162float(p.x[(img * p.HW + px) * p.C + cg * 8 + i]));
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) part[threadIdx.x][i] = acc[i];
  __syncthreads();
  // fixed-order reduction over the CTA's pixel groups, spread over all threads: thread (cg, i) with
  // i = channel inside the group of eight adds its column of `part` in group order
  for (int o = threadIdx.x; o < tpp * 8; o += 256) {
    const int cg2 = o >> 3, i = o & 7;
    double s = 0.0;
    for (int g2 = 0; g2 < ppi; ++g2) s += part[g2 * tpp + cg2][i];
    if (cg2 * 8 + i < p.C) p.partial[(img * p.slabs + blockIdx.y) * p.C + cg2 * 8 + i] = s;
  }
}
__global__ void __launch_bounds__(256) gap_final_f64(const __grid_constant__ GapBatch B) {
  // 8 channels x 32 slab lanes per CTA (blockIdx.y = segment): lane g sums slabs g, g+32, ... in order,
  // then the 32 lane sums are added in order: a fixed summation tree, so the result is deterministic
  __shared__ double part[32][8];
  ptx::pdl_wait();
  ptx::pdl_launch();
  const GapParams& p = B.seg[blockIdx.y];
  const int n_img = B.img_start[blockIdx.y + 1] - B.img_start[blockIdx.y];
  const int cl = threadIdx.x & 7, g = threadIdx.x >> 3;
  const long long i = static_cast<long long>(blockIdx.x) * 8 + cl;     // flat (img, c)
  if (static_cast<long long>(blockIdx.x) * 8 >= static_cast<long long>(n_img) * p.C) return;
  const bool ok = i < static_cast<long long>(n_img) * p.C;
  const long long img = ok ? i / p.C : 0;
  const int c = ok ? static_cast<int>(i % p.C) : 0;
  double acc = 0.0;
  if (ok) {
#pragma unroll 4
    for (int s = g; s < p.slabs; s += 32) acc += p.partial[(img * p.slabs + s) * p.C + c];
  }
  part[g][cl] = acc;
  __syncthreads();
  if (g == 0 && ok) {
    double t = 0.0;
#pragma unroll
    for (int k2 = 0; k2 < 32; ++k2) t += part[k2][cl];
    const double mean = t / static_cast<double>(p.HW);
    if (p.out_f64) p.out_f64[i] = mean;
    if (p.out) {
      if (p.out_bf16) reinterpret_cast<__nv_bfloat16*>(p.out)[i] = __double2bfloat16(mean);
      else reinterpret_cast<float*>(p.out)[i] = static_cast<float>(mean);
    }
  }
}

// [rows, K] -> [rows, Kp] with zero padding (weights of thin-channel convolutions).
__global__ void __launch_bounds__(256) pad_rows_bf16(const __nv_bfloat16* __restrict__ in, __nv_bfloat16* __restrict__ out, int rows, int K, int Kp) {
  const long long total = static_cast<long long>(rows) * Kp;
  for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += static_cast<long long>(gridDim.x) * blockDim.x) {
    const int kk = static_cast<int>(i % Kp);
    out[i] = kk < K ? in[(i / Kp) * K + kk] : __float2bfloat16(0.0f);
  }
}

// Patch gathering for a thin-channel convolution (e.g. the RGB stem): A[pixel, (ci, dy, dx)] from an
// NCHW image, zero outside the image and in the K padding.  One thread per (pixel, 8-wide k group).
struct Im2colParams {
  const __nv_bfloat16* x;   // [N, C, H, W]
  __nv_bfloat16* a;         // [N*Ho*Wo, Kp]
  int N, C, H, W, Ho, Wo, ks, stride, pad, K, Kp;
};
__global__ void __launch_bounds__(256) im2col_nchw_bf16(Im2colParams p) {
  // CTA = 64 consecutive output pixels of one output row.  The input window (C x ks rows x span
  // columns) is staged in shared memory with coalesced reads; every thread then writes 16-byte
  // groups of the K-major patch rows (coalesced: a pixel's row is Kp*2 contiguous bytes).
  extern __shared__ __nv_bfloat16 win[];          // [C][ks][span], then int koff[Kp]
  const int segs = (p.Wo + 63) / 64;
  const int seg = blockIdx.x % segs;
  const int ho = (blockIdx.x / segs) % p.Ho;
  const int n = blockIdx.x / (segs * p.Ho);
  const int wo0 = seg * 64;
  const int span = 63 * p.stride + p.ks;          // input columns needed by 64 output pixels
  const int w_in0 = wo0 * p.stride - p.pad, h_in0 = ho * p.stride - p.pad;
  const int total = p.C * p.ks * span;
  // window offset of every k = (ci, dy, dx), computed once per CTA: the gather loop below would otherwise
  // spend most of its instructions on the divisions
  int* koff = reinterpret_cast<int*>(win + ((total + 7) & ~7));
  for (int kk = threadIdx.x; kk < p.Kp; kk += 256) {
    const int dx = kk % p.ks, dy = (kk / p.ks) % p.ks, ci = kk / (p.ks * p.ks);
    koff[kk] = kk < p.K ? (ci * p.ks + dy) * span + dx : -1;
  }
  // window rows (one per (channel, kernel row)) by warps, columns by lanes: coalesced, no divisions per element
  for (int r = threadIdx.x >> 5; r < p.C * p.ks; r += 8) {
    const int ci = r / p.ks, row = r - ci * p.ks;
    const int h = h_in0 + row;
    const bool hok = h >= 0 && h < p.H;
    const __nv_bfloat16* src = p.x + ((static_cast<long long>(n) * p.C + ci) * p.H + (hok ? h : 0)) * p.W;
    for (int col = threadIdx.x & 31; col < span; col += 32) {
      const int w = w_in0 + col;
      win[r * span + col] = (hok && w >= 0 && w < p.W) ? src[w] : __float2bfloat16(0.0f);
    }
  }
  __syncthreads();
  const int groups = p.Kp >> 3;
  for (int i = threadIdx.x; i < 64 * groups; i += 256) {
    const int gq = i % groups, px = i / groups;
    const int wo = wo0 + px;
    if (wo >= p.Wo) continue;
    __align__(16) __nv_bfloat16 v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int o = koff[gq * 8 + j];
      v[j] = o >= 0 ? win[o + px * p.stride] : __float2bfloat16(0.0f);
    }
    const long long pix = (static_cast<long long>(n) * p.Ho + ho) * p.Wo + wo;
    *reinterpret_cast<uint4*>(p.a + pix * p.Kp + gq * 8) = *reinterpret_cast<const uint4*>(v);
  }
}

// Per-sample regrouping (Switch): stable partition of the sample ids by the gate.  One warp-sized CTA:
// ballot + prefix popcount per chunk of 32 samples.  *count_exec = executed (the run-time symbol's
// slot in the arena header), *count_skip = skipped; idx_exec / idx_skip = original sample ids.
struct PartitionParams {
  const unsigned char* gate;
  int n;
  int* idx_exec; int* idx_skip;    // scratch [n] each
  long long* count_exec;           // the run-time symbol's slot in the arena header
  long long* count_skip;
};
__device__ __forceinline__ int partition_by_gate(const PartitionParams& p, int lane) {
  int ne = 0, ns = 0;
  for (int base = 0; base < p.n; base += 32) {
    const int i = base + lane;
    const bool in = i < p.n;
    const bool g = in && __ldcg(p.gate + i) != 0;
    const unsigned be = __ballot_sync(0xffffffffu, g), bs = __ballot_sync(0xffffffffu, in && !g);
    const unsigned lower = (1u << lane) - 1;
    if (g) p.idx_exec[ne + __popc(be & lower)] = i;
    else if (in) p.idx_skip[ns + __popc(bs & lower)] = i;
    ne += __popc(be);
    ns += __popc(bs);
  }
  if (lane == 0) { *p.count_exec = ne; *p.count_skip = ns; }
  return ne;
}

// Gate of a skip block (decision scalar): z[n] = sum_c w[c] * mean_hw x[n,:,:,c] + b, gate[n] = z[n] > 0,
// all in fp64 from the bf16 values, so the decision does not depend on the summation order beyond 2^-53.
// Runs after gap_partial_f64 (slab sums in scratch); one CTA per image.
struct GateParams {
  const double* partial;        // [N, slabs, C]
  const __nv_bfloat16* w;       // [C]
  const __nv_bfloat16* b;       // [1]
  unsigned char* gate;          // [N] bytes (0/1)
  void* z_out;                  // optional logits [N] (bf16 or f32), may be nullptr
  int z_bf16;
  int C, slabs;
  long long HW;
  // ticket != nullptr: the CTA that finishes last also partitions the sample ids by the gate bits (the
  // Switch that consumes this gate then launches nothing for it).  *ticket is zero on entry (the run
  // clears the arena header) and is left at zero.
  int* ticket;
  PartitionParams part;
  // zero_rows != nullptr: the last CTA also clears the rows of the executed samples in the [N, C] table of
  // per-sample channel sums, which the block's last convolution then accumulates anew (ConvParams::gap_sum)
  double* zero_rows;
};
__global__ void __launch_bounds__(256) gate_logit_f64(GateParams p) {
  __shared__ double red[256];
  __shared__ int last_cta, n_exec;
  ptx::pdl_wait();
  ptx::pdl_launch();
  const int img = blockIdx.x;
  // item (q, c): slabs q, q+8, ... of channel c added in order (independent loads, unrolled), times w[c];
  // a thread adds its items in index order and the 256 thread sums go through a fixed tree, so the
  // decision does not depend on scheduling
  double acc = 0.0;
  for (int idx = threadIdx.x; idx < 8 * p.C; idx += 256) {
    const int q8 = idx / p.C, c = idx - q8 * p.C;
    const double* pp = p.partial + static_cast<long long>(img) * p.slabs * p.C + c;
    double s = 0.0;
#pragma unroll 4
    for (int k = q8; k < p.slabs; k += 8) s += pp[static_cast<long long>(k) * p.C];
    acc += s * static_cast<double>(__bfloat162float(p.w[c]));
  }
  acc /= static_cast<double>(p.HW);
  red[threadIdx.x] = acc;
  __syncthreads();
  for (int o = 128; o; o >>= 1) { if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o]; __syncthreads(); }
  if (threadIdx.x == 0) {
    const double z = red[0] + static_cast<double>(__bfloat162float(p.b[0]));
    p.gate[img] = z > 0.0 ? 1 : 0;
    if (p.z_out) {
      if (p.z_bf16) reinterpret_cast<__nv_bfloat16*>(p.z_out)[img] = __double2bfloat16(z);
      else reinterpret_cast<float*>(p.z_out)[img] = static_cast<float>(z);
    }
    if (p.ticket) {
      __threadfence();
      last_cta = atomicAdd(p.ticket, 1) == static_cast<int>(gridDim.x) - 1;
    }
  }
  if (p.ticket) {
    __syncthreads();
    if (last_cta) {
      if (threadIdx.x < 32) {
        __threadfence();
        const int ne = partition_by_gate(p.part, threadIdx.x);
        if (threadIdx.x == 0) { *p.ticket = 0; n_exec = ne; }
      }
      if (p.zero_rows) {
        __syncthreads();                                  // uniform over the CTA: last_cta is shared
        // a warp per executed sample: the id is read once, the lanes clear the row
        for (int k2 = threadIdx.x >> 5; k2 < n_exec; k2 += 8) {
          double* rowp = p.zero_rows + static_cast<long long>(p.part.idx_exec[k2]) * p.C;
          for (int cc = threadIdx.x & 31; cc < p.C; cc += 32) rowp[cc] = 0.0;
        }
      }
    }
  }
}

// The same gate as ONE CTA: a warp per image (lane-strided channels in order, fixed shuffle tree), then warp 0
// partitions the ids and all warps clear the executed rows.  No ticket, no second trip through global memory
// for the gate bits and the id list: what the grid form above spends on its chain of dependent round trips
// (ticket atomic, gate bytes, id list) this form does behind one CTA barrier.  For the table form of the sums
// (a few slabs per image at most), where one SM can read all of them in about a microsecond.
__global__ void __launch_bounds__(1024) gate_logit_block_f64(GateParams p, int N) {
  __shared__ int n_exec;
  ptx::pdl_wait();
  ptx::pdl_launch();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const double bias = static_cast<double>(__bfloat162float(p.b[0]));
  for (int img = warp; img < N; img += 32) {
    const double* pp = p.partial + static_cast<long long>(img) * p.slabs * p.C;
    double acc = 0.0;
    if (p.slabs == 1) {
      for (int c0 = lane; c0 < p.C; c0 += 128) {       // four loads in flight per lane, added in channel order
        double v[4], w[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int c = c0 + 32 * q;
          v[q] = c < p.C ? pp[c] : 0.0;
          w[q] = c < p.C ? static_cast<double>(__bfloat162float(p.w[c])) : 0.0;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) acc += v[q] * w[q];
      }
    } else {
      for (int c = lane; c < p.C; c += 32) {
        double sl = 0.0;
        for (int k = 0; k < p.slabs; ++k) sl += pp[static_cast<long long>(k) * p.C + c];
        acc += sl * static_cast<double>(__bfloat162float(p.w[c]));
      }
    }
    acc /= static_cast<double>(p.HW);
#pragma unroll
    for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) {
      const double z = acc + bias;
      p.gate[img] = z > 0.0 ? 1 : 0;
      if (p.z_out) {
        if (p.z_bf16) reinterpret_cast<__nv_bfloat16*>(p.z_out)[img] = __double2bfloat16(z);
        else reinterpret_cast<float*>(p.z_out)[img] = static_cast<float>(z);
      }
    }
  }
  if (p.ticket) {          // here only a flag: partition the ids too
    __syncthreads();       // the gate bytes written above are visible to warp 0
    if (warp == 0) {
      const int ne = partition_by_gate(p.part, lane);
      if (lane == 0) n_exec = ne;
    }
    if (p.zero_rows) {
      __syncthreads();     // the id list written by warp 0 is visible to the CTA
      for (int k2 = warp; k2 < n_exec; k2 += 32) {
        double* rowp = p.zero_rows + static_cast<long long>(p.part.idx_exec[k2]) * p.C;
        for (int cc = lane; cc < p.C; cc += 32) rowp[cc] = 0.0;
      }
    }
  }
}

__global__ void __launch_bounds__(32) gate_partition(PartitionParams p) {
  ptx::pdl_wait();
  ptx::pdl_launch();
  partition_by_gate(p, threadIdx.x);
}

// Sample gather / scatter for Switch and Combine: whole per-sample blocks (channels-last, contiguous)
// copied with 128-bit accesses.  dst[j] = src[idx[j]] (gather) or dst[idx[j]] = src[j] (scatter) for
// j < *count; grid.y walks the samples, tail blocks exit on the device-side count.
struct SampleCopyParams {
  const uint4* src; uint4* dst;
  const int* idx;
  const long long* count;
  long long vec_per_sample;   // 16-byte units per sample
  int scatter;                // 0: dst[j] = src[idx[j]];  1: dst[idx[j]] = src[j];  2: dst[idx[j]] = src[idx[j]]
};
__global__ void __launch_bounds__(256) sample_copy(SampleCopyParams p) {
  ptx::pdl_wait();
  ptx::pdl_launch();
  const int j = blockIdx.y;
  const long long cnt = *p.count;
  const long long s = p.idx[j];      // requested together with the count (the list has an entry for every j of the grid)
  if (j >= cnt) return;
  const uint4* src = p.src + (p.scatter == 1 ? static_cast<long long>(j) : s) * p.vec_per_sample;
  uint4* dst = p.dst + (p.scatter != 0 ? s : static_cast<long long>(j)) * p.vec_per_sample;
  for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < p.vec_per_sample; i += static_cast<long long>(gridDim.x) * blockDim.x) dst[i] = src[i];
}

// Conv weights [Cout, Cin, kh, kw] -> K-major [Cout, (dy, dx, ci)] for the implicit-GEMM B operand.
__global__ void __launch_bounds__(256) reorder_conv_weights(const __nv_bfloat16* __restrict__ in, __nv_bfloat16* __restrict__ out,
                                                             int Cout, int Cin, int kh, int kw) {
  const long long total = static_cast<long long>(Cout) * Cin * kh * kw;
  for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += static_cast<long long>(gridDim.x) * blockDim.x) {
    long long r = i;
    const int ci = static_cast<int>(r % Cin); r /= Cin;
    const int dx = static_cast<int>(r % kw); r /= kw;
    const int dy = static_cast<int>(r % kh);
    const int co = static_cast<int>(r / kh);
    out[i] = in[((static_cast<long long>(co) * Cin + ci) * kh + dy) * kw + dx];
  }
}

}  // namespace k
}  // namespace sod2
