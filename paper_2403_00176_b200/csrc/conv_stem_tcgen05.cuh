// Fused RGB stem: 7x7 convolution, stride 2, padding 3, 3 -> 64 channels, + bias + activation, as an
// implicit GEMM on tcgen05 whose A operand is assembled in shared memory.
//   in : x [N, 3, H, W] bf16, NCHW contiguous (the graph input)
//   out: y [N, Ho, Wo, 64] bf16, channels-last
// With three input channels neither TMA im2col nor a channels-last box applies (a pixel is 6 bytes), and
// materialising the [pixels, 147 -> 192] patch matrix costs 16 x the input in traffic.  Here a CTA
// owns a segment of up to 128 pixels of one output row.  The 7 input rows x 3 channels the segment
// needs are copied into shared memory (six TMA boxes of 7 rows x 144 columns per tile: three channels x
// two overlapping column halves, zero filled outside the image; for images whose width is not a multiple
// of 8 the builder warps copy them instead), and the
// A tile [128 pixels x 192] is built from them in the 128-byte-swizzled K-major layout: K is ordered
// (dy, ci, dx') with dx' = dx + 1 in 0..7, so that one 16-byte unit of a pixel's row of A is eight
// consecutive input columns starting at the even column 2*ox - 4 -- four aligned 32-bit shared loads.
// dx' = 0 carries a zero weight (and is zeroed in A), units 21..23 are zero padding: K = 24 x 8.
//   warp 0       weights (24 KB, resident) and the input patches (three-deep ring) by TMA
//   warps 1..8   builders: A tile (double buffered) from the patch
//   warps 9..12  epilogue: TMEM -> +bias -> activation -> bf16 -> swizzled staging -> TMA store
//   warp 13      MMA issuer: 12 x tcgen05.mma (M=128, N=64, K=16) per tile into one of two accumulators
// Persistent, one CTA per SM.  Every wait is bounded (ptx.cuh).
#pragma once
#include "conv_tcgen05.cuh"

namespace sod2 {
namespace k {

struct StemParams {
  const __nv_bfloat16* x;      // [N, 3, H, W]
  const __nv_bfloat16* bias;   // [64] or nullptr
  int N, H, W, Ho, Wo;
  int vec_ok;                  // x is 16-byte aligned and W % 8 == 0: 16-byte copies
  int* status;
};

constexpr int STEM_THREADS = 448;
constexpr int STEM_PITCH = 272;                       // patch columns: 2 * 128 + 16
constexpr int STEM_ROWS = 21;                         // (dy, ci)
constexpr int STEM_PATCH_BYTES = 12288;               // 21 rows x 272 columns (11424 B), or six TMA boxes 2048 B apart
constexpr int STEM_A_BYTES = 3 * 128 * 128;           // three k-chunks of [128 x 64]
constexpr int STEM_W_BYTES = 3 * 64 * 128;
constexpr int STEM_OUT_BYTES = 128 * 128;
constexpr int STEM_BOX_W = 144;                       // columns of a TMA box: two of them, 128 apart, cover the 272 patch columns
constexpr int STEM_BOX_BYTES = 7 * STEM_BOX_W * 2;    // one TMA box: 7 input rows (2016 B)
constexpr int STEM_BOX_STRIDE = 2048;                 // boxes 2048 B apart: a TMA destination is 128-byte aligned
constexpr int STEM_SMEM = STEM_W_BYTES + 2 * STEM_A_BYTES + 2 * STEM_OUT_BYTES + 3 * STEM_PATCH_BYTES + 256 /*bias*/ + 128 /*barriers*/ + 1024 /*align*/;

// Weights [64, 3, 7, 7] -> [64, 192] in the (dy, ci, dx') order of the kernel, zero where dx' = 0 or unit >= 21.
__global__ void reorder_stem_weights(const __nv_bfloat16* __restrict__ w, __nv_bfloat16* __restrict__ out) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < 64 * 192; i += gridDim.x * blockDim.x) {
    const int co = i / 192, k = i % 192, u = k >> 3, dxp = k & 7;
    float v = 0.f;
    if (u < 21 && dxp >= 1) {
      const int dy = u / 3, ci = u % 3;
      v = __bfloat162float(w[((co * 3 + ci) * 7 + dy) * 7 + (dxp - 1)]);
    }
    out[i] = __float2bfloat16(v);
  }
}

// TMA_PATCH: tmX is a map {W, H, N * 3} of the input with boxes {144, 7, 1} (W % 8 == 0); otherwise tmX is unused.
template <int ACT, bool TMA_PATCH>
__global__ void __launch_bounds__(STEM_THREADS, 1)
conv_stem_bf16_tcgen05(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmOut,
                       const __grid_constant__ CUtensorMap tmX, const StemParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sW = base;
  uint8_t* sA = sW + STEM_W_BYTES;             // [2]
  uint8_t* sOut = sA + 2 * STEM_A_BYTES;       // [2]
  uint8_t* sPatch = sOut + 2 * STEM_OUT_BYTES; // [3]
  float* bias_s = reinterpret_cast<float*>(sPatch + 3 * STEM_PATCH_BYTES);   // [64]
  uint64_t* bars = reinterpret_cast<uint64_t*>(bias_s + 64);
  uint64_t* w_full = bars;            // 1
  uint64_t* a_full = bars + 1;        // [2] builders have written A[b]
  uint64_t* a_free = bars + 3;        // [2] the MMAs that read A[b] have completed
  uint64_t* acc_full = bars + 5;      // [2]
  uint64_t* acc_free = bars + 7;      // [2] the epilogue warps have drained accumulator b
  uint64_t* patch_full = bars + 9;    // [3] the tile's six boxes have landed
  uint64_t* patch_free = bars + 12;   // [3] the builder warps have read the patch
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 15);
  volatile int* dead = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nseg = (p.Wo + 127) >> 7;
  const int n_tiles = p.N * p.Ho * nseg;   // the host keeps it below 2^31 (64-bit divisions in the tile loop cost more than the tile)

  if (threadIdx.x == 0) {
    ptx::mbar_init(w_full, 1);
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(&a_full[b], 8); ptx::mbar_init(&a_free[b], 1);
      ptx::mbar_init(&acc_full[b], 1); ptx::mbar_init(&acc_free[b], 4);
    }
    for (int b = 0; b < 3; ++b) { ptx::mbar_init(&patch_full[b], 1); ptx::mbar_init(&patch_free[b], 8); }
    *dead = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
    ptx::prefetch_tmap(&tmW);
    ptx::prefetch_tmap(&tmOut);
    if (TMA_PATCH) ptx::prefetch_tmap(&tmX);
  }
  if (threadIdx.x < 64) bias_s[threadIdx.x] = p.bias ? __bfloat162float(p.bias[threadIdx.x]) : 0.0f;   // a constant of the graph
  if (warp == 13) { ptx::tmem_alloc(tmem_slot, 128); ptx::tmem_relinquish(); }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  ptx::pdl_launch();

  if (warp == 0) {
    if (lane == 0) {
      ptx::mbar_expect_tx(w_full, STEM_W_BYTES);
      ptx::tma_load_3d(sW, &tmW, 0, 0, 0, w_full);
      if constexpr (TMA_PATCH) {
        // ---- patch producer: box (ci, half) of tile t = input rows 2*oy-3 .. 2*oy+3 of channel ci, columns
        // 2*ox0 - 8 + 128*half .. +143 (the halves overlap by 16, so a pixel's 8 columns always lie inside one box)
        ptx::pdl_wait();
        int it = 0;
        for (int t = blockIdx.x; t < n_tiles; t += gridDim.x, ++it) {
          const int s = it % 3;
          if (it >= 3) ptx::mbar_wait(&patch_free[s], ((it / 3) - 1) & 1, dead);
          const int rowi = t / nseg, seg = t - rowi * nseg;
          const int n = rowi / p.Ho, oy = rowi - n * p.Ho;
          ptx::mbar_expect_tx(&patch_full[s], 6 * STEM_BOX_BYTES);
#pragma unroll
          for (int bx = 0; bx < 6; ++bx)
            ptx::tma_load_3d(sPatch + s * STEM_PATCH_BYTES + bx * STEM_BOX_STRIDE, &tmX, 256 * seg - 8 + 128 * (bx & 1), 2 * oy - 3,
                             n * 3 + (bx >> 1), &patch_full[s]);
        }
      }
    }
  } else if (warp <= 8) {
    // ---- builders
    const int tb = threadIdx.x - 32;        // 0..255
    const int m = tb & 127, ug = tb >> 7;
    ptx::pdl_wait();
    // copy of the patch of tile t into ring slot s: rows (dy, ci), columns 2*ox0 - 8 .. 2*ox0 + 263
    // warp wb copies patch rows wb, wb + 8, wb + 16; a lane copies the 16-byte chunks lane and lane + 32
    // of a row (34 chunks).  What does not depend on the tile is computed once.
    const int wb = tb >> 5;
    int row_dy[3], row_ci[3];
    uint32_t row_dst[3];
#pragma unroll
    for (int j = 0; j < 3; ++j) {
      const int r = wb + 8 * j;
      row_dy[j] = r / 3;
      row_ci[j] = r - row_dy[j] * 3;
      row_dst[j] = static_cast<uint32_t>((r * STEM_PITCH + lane * 8) * 2);
    }
    const long long plane = static_cast<long long>(p.H) * p.W;
    auto load_patch = [&](int t, int s) {
      const int rowi = t / nseg, seg = t - rowi * nseg;
      const int n = rowi / p.Ho, oy = rowi - n * p.Ho;
      const int c0a = 2 * (seg * 128) - 8 + lane * 8, c0b = c0a + 256;
      const uint32_t dst = ptx::smem_u32(sPatch + s * STEM_PATCH_BYTES);
      const __nv_bfloat16* img = p.x + static_cast<long long>(n) * 3 * plane;
#pragma unroll
      for (int j = 0; j < 3; ++j) {
        if (wb + 8 * j >= STEM_ROWS) break;
        const int iy = 2 * oy + row_dy[j] - 3;
        const bool row_in = iy >= 0 && iy < p.H;
        const __nv_bfloat16* src = img + row_ci[j] * plane + static_cast<long long>(row_in ? iy : 0) * p.W;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (h == 1 && lane >= STEM_PITCH / 8 - 32) break;
          const int c0 = h ? c0b : c0a;
          const uint32_t d = dst + row_dst[j] + h * 512;
          if (p.vec_ok) {
            if (row_in && c0 >= 0 && c0 + 8 <= p.W) {
              asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(src + c0));
            } else {
              asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(d), "r"(0u));
            }
          } else {
            uint32_t wv[4];
#pragma unroll
            for (int q2 = 0; q2 < 4; ++q2) {
              const int ca = c0 + 2 * q2, cb = ca + 1;
              const uint32_t lo = (row_in && ca >= 0 && ca < p.W) ? static_cast<uint32_t>(__bfloat16_as_ushort(src[ca])) : 0u;
              const uint32_t hi = (row_in && cb >= 0 && cb < p.W) ? static_cast<uint32_t>(__bfloat16_as_ushort(src[cb])) : 0u;
              wv[q2] = lo | (hi << 16);
            }
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(d), "r"(wv[0]), "r"(wv[1]), "r"(wv[2]), "r"(wv[3]));
          }
        }
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    const int t0 = blockIdx.x, step = gridDim.x;
    // source offset of unit i of this thread inside a patch, per layout
    uint32_t uoff[12];
#pragma unroll
    for (int i = 0; i < 12; ++i) {
      const int u = ug + 2 * i;
      const int dy = u / 3, ci = u - dy * 3;
      if constexpr (TMA_PATCH) {
        const int half = m >= 64 ? 1 : 0;   // columns 2m+4 .. 2m+11: inside box 0 (0..143) for m <= 66, box 1 (128..271) for m >= 62
        uoff[i] = static_cast<uint32_t>((ci * 2 + half) * STEM_BOX_STRIDE + dy * (STEM_BOX_W * 2) + (2 * m + 4 - 128 * half) * 2);
      } else {
        uoff[i] = static_cast<uint32_t>((u * STEM_PITCH + 2 * m + 4) * 2);
      }
    }
    if constexpr (!TMA_PATCH) {
      if (t0 < n_tiles) load_patch(t0, 0); else asm volatile("cp.async.commit_group;" ::: "memory");
      if (t0 + step < n_tiles) load_patch(t0 + step, 1); else asm volatile("cp.async.commit_group;" ::: "memory");
    }
    int it = 0;
    for (int t = t0; t < n_tiles; t += step, ++it) {
      if constexpr (TMA_PATCH) {
        ptx::mbar_wait_warp(&patch_full[it % 3], (it / 3) & 1, dead);
      } else {
        // this thread's copies for tile `it` have landed (one newer group may be in flight); after the
        // barrier so have everyone's, and every builder has finished reading the slot of tile it - 1
        asm volatile("cp.async.wait_group 1;" ::: "memory");
        asm volatile("bar.sync 2, 256;" ::: "memory");
        if (t + 2 * step < n_tiles) load_patch(t + 2 * step, (it + 2) % 3); else asm volatile("cp.async.commit_group;" ::: "memory");
      }
      if (tb == 0) { SOD2_TRACE(0, 10) }
      const int buf = it & 1;
      if (it >= 2) ptx::mbar_wait_warp(&a_free[buf], ((it >> 1) - 1) & 1, dead);
      if (tb == 0) { SOD2_TRACE(0, 20) }
      const uint32_t patch = ptx::smem_u32(sPatch + (it % 3) * STEM_PATCH_BYTES);
      uint8_t* arow = sA + buf * STEM_A_BYTES + m * 128;
      // all loads first, then the stores: patch and A live in the same array, so the compiler would keep
      // every store ahead of the next unit's loads
      uint4 v[12];
#pragma unroll
      for (int i = 0; i < 12; ++i) {
        const int u = ug + 2 * i;                       // unit = patch row (dy, ci); 21..23 are padding
        v[i] = make_uint4(0u, 0u, 0u, 0u);
        if (u < STEM_ROWS) {
          const uint32_t sa = patch + uoff[i];
          asm volatile("ld.shared.b32 %0, [%4];\n\tld.shared.b32 %1, [%4+4];\n\tld.shared.b32 %2, [%4+8];\n\tld.shared.b32 %3, [%4+12];"
                       : "=r"(v[i].x), "=r"(v[i].y), "=r"(v[i].z), "=r"(v[i].w) : "r"(sa));
          v[i].x &= 0xffff0000u;                        // dx' = 0 has no tap
        }
      }
#pragma unroll
      for (int i = 0; i < 12; ++i) {
        const int u = ug + 2 * i;
        *reinterpret_cast<uint4*>(arow + (u >> 3) * (128 * 128) + (((u & 7) ^ (m & 7)) << 4)) = v[i];
      }
      ptx::fence_proxy_async();
      __syncwarp();
      if (lane == 0) {
        ptx::mbar_arrive(&a_full[buf]);
        if (TMA_PATCH) ptx::mbar_arrive(&patch_free[it % 3]);   // the stores above depend on every value read from the patch
      }
      if (tb == 0) { SOD2_TRACE(0, 30) }
    }
    if constexpr (!TMA_PATCH) asm volatile("cp.async.wait_group 0;" ::: "memory");
  } else if (warp == 13) {
    if (lane == 0) {
      // ---- MMA issuer
      constexpr uint32_t idesc = ptx::idesc_bf16(128, 64);
      ptx::mbar_wait(w_full, 0, dead);
      const uint32_t aW = ptx::smem_u32(sW);
      int it = 0;
      for (int t = blockIdx.x; t < n_tiles; t += gridDim.x, ++it) {
        const int b = it & 1;
        ptx::mbar_wait(&a_full[b], (it >> 1) & 1, dead);
        SOD2_TRACE(1, 40)
        if (it >= 2) ptx::mbar_wait(&acc_free[b], ((it >> 1) - 1) & 1, dead);
        SOD2_TRACE(1, 41)
        ptx::tc_fence_after();
        const uint32_t aA = ptx::smem_u32(sA + b * STEM_A_BYTES);
#pragma unroll
        for (int c = 0; c < 3; ++c) {
          const uint64_t ad = ptx::smem_desc_sw128(aA + c * (128 * 128)), bd = ptx::smem_desc_sw128(aW + c * (64 * 128));
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) ptx::mma_bf16(tmem + b * 64, ad + 2 * kk, bd + 2 * kk, idesc, (c | kk) != 0);
        }
        ptx::mma_commit(&a_free[b]);
        ptx::mma_commit(&acc_full[b]);
        SOD2_TRACE(1, 42)
      }
    }
  } else {
    // ---- epilogue warps 9..12: warp w drains TMEM lane quarter w % 4; a thread holds one pixel
    const int q = warp & 3;
    const int row = q * 32 + lane;
    const bool leader = threadIdx.x == 9 * 32;
    ptx::pdl_wait();
    int it = 0;
    for (int t = blockIdx.x; t < n_tiles; t += gridDim.x, ++it) {
      const int b = it & 1;
      const int rowi = t / nseg, seg = t - rowi * nseg;
      const int n = rowi / p.Ho, oy = rowi - n * p.Ho;
      ptx::mbar_wait_warp(&acc_full[b], (it >> 1) & 1, dead);
      ptx::tc_fence_after();
      if (leader) { SOD2_TRACE(2, 50) }
      uint32_t r[2][32];
      const uint32_t taddr = tmem + (static_cast<uint32_t>(q * 32) << 16) + b * 64;
      ptx::tmem_ld32(taddr, r[0]);
      ptx::tmem_ld32(taddr + 32, r[1]);
      ptx::tmem_ld_wait();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&acc_free[b]);
      if (leader) { SOD2_TRACE(2, 51) }
      uint4 pk[8];
#pragma unroll
      for (int g = 0; g < 8; ++g) {
        __nv_bfloat162* oh = reinterpret_cast<__nv_bfloat162*>(&pk[g]);
        const float4 b0 = *reinterpret_cast<const float4*>(bias_s + g * 8), b1 = *reinterpret_cast<const float4*>(bias_s + g * 8 + 4);
        const float bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int cch = g * 8 + 2 * i;
          const float v0 = apply_act<ACT>(__uint_as_float(r[cch >> 5][cch & 31]) + bb[2 * i]);
          const float v1 = apply_act<ACT>(__uint_as_float(r[(cch + 1) >> 5][(cch + 1) & 31]) + bb[2 * i + 1]);
          oh[i] = __floats2bfloat162_rn(v0, v1);
        }
      }
      // the store that read this staging buffer two tiles ago must have finished reading it
      if (leader) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
      asm volatile("bar.sync 3, 128;" ::: "memory");
      uint8_t* orow = sOut + b * STEM_OUT_BYTES + row * 128;
#pragma unroll
      for (int g = 0; g < 8; ++g) *reinterpret_cast<uint4*>(orow + ((g ^ (row & 7)) << 4)) = pk[g];
      ptx::fence_proxy_async();
      asm volatile("bar.sync 3, 128;" ::: "memory");
      if (leader) {
        tma_store_4d(&tmOut, sOut + b * STEM_OUT_BYTES, 0, seg * 128, oy, n);
        bulk_commit();
        SOD2_TRACE(2, 52)
      }
    }
    if (leader) bulk_wait_read0();
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 13) ptx::tmem_dealloc(tmem, 128);
  if (threadIdx.x == 0 && *dead && p.status) atomicExch(p.status, 1);
}

}  // namespace k
}  // namespace sod2
