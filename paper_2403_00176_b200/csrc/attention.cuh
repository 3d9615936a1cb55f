// Fused attention group for packed variable-length requests:
//   O = softmax(Q K^T * scale) V  per (request, head), head dim 64, bf16 in / fp32 accumulate / bf16 out.
// The score and probability tensors never reach global memory (the fusion argument of Section 4.2:
// no materialised intermediates). Rows and columns at or beyond a request's length are never read as
// data (zero-filled in shared memory, masked to -inf before the softmax) and never written.
// Q, K, V, O are strided views (token stride, head stride) of the producing / consuming GEMM
// buffers, so the Slice / Reshape / Transpose operators around attention cost nothing.
// Online-softmax tiling: 64 query rows per CTA (4 warps x 16 rows), 64 keys per step, K/V tiles
// double-buffered with cp.async, mma.sync m16n8k16.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <cstdint>

#include "ptx.cuh"

namespace sod2 {
namespace k {

constexpr int ATTN_MAX_REQ = 32;
struct AttnReq {
  long long q_off, k_off, v_off, o_off;  // element offsets of this request's views
  int L;
  int q_ts, k_ts, v_ts, o_ts;            // token strides (elements)
  int q_hs, k_hs, v_hs, o_hs;            // head strides
};
struct AttnParams {
  const __nv_bfloat16* q; const __nv_bfloat16* k; const __nv_bfloat16* v; __nv_bfloat16* o;
  int n_req, H;
  float scale_log2e;
  int tile_start[ATTN_MAX_REQ + 1];      // prefix sum of ceil(L/64)
  AttnReq r[ATTN_MAX_REQ];
};

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem, bool valid) {
  const uint32_t s = static_cast<uint32_t>(__cvta_generic_to_shared(smem));
  const int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(s), "l"(gmem), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, const void* p) {
  const uint32_t s = static_cast<uint32_t>(__cvta_generic_to_shared(p));
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(s));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, const void* p) {
  const uint32_t s = static_cast<uint32_t>(__cvta_generic_to_shared(p));
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(s));
}
__device__ __forceinline__ void mma_16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}

// tile of 64 rows x 64 bf16 (128 B per row), 16-byte chunks XOR-swizzled by the row
__device__ __forceinline__ __nv_bfloat16* tile_ptr(__nv_bfloat16* t, int row, int chunk) {
  return t + row * 64 + ((chunk ^ (row & 7)) << 3);
}

__device__ __forceinline__ void load_tile(__nv_bfloat16* dst, const __nv_bfloat16* src, int ts, int row0, int L, int tid) {
  // 64 rows x 8 chunks = 512 chunks, 128 threads -> 4 each
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int idx = tid + i * 128;
    const int row = idx >> 3, ch = idx & 7;
    const bool ok = row0 + row < L;
    const __nv_bfloat16* g = src + static_cast<long long>(ok ? row0 + row : 0) * ts + ch * 8;
    cp_async16(tile_ptr(dst, row, ch), g, ok);
  }
}

__global__ void __launch_bounds__(128) attention_fwd_bf16(const __grid_constant__ AttnParams p) {
  __shared__ __align__(128) __nv_bfloat16 sQ[64 * 64];
  __shared__ __align__(128) __nv_bfloat16 sK[2][64 * 64];
  __shared__ __align__(128) __nv_bfloat16 sV[2][64 * 64];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int head = blockIdx.y;
  int ri = 0;
  while (ri + 1 < p.n_req && static_cast<int>(blockIdx.x) >= p.tile_start[ri + 1]) ++ri;
  const AttnReq& R = p.r[ri];
  const int L = R.L;
  const int q0 = (blockIdx.x - p.tile_start[ri]) * 64;
  const __nv_bfloat16* qg = p.q + R.q_off + static_cast<long long>(head) * R.q_hs;
  const __nv_bfloat16* kg = p.k + R.k_off + static_cast<long long>(head) * R.k_hs;
  const __nv_bfloat16* vg = p.v + R.v_off + static_cast<long long>(head) * R.v_hs;
  const int nkv = (L + 63) >> 6;
  ptx::pdl_wait();
  ptx::pdl_launch();

  load_tile(sQ, qg, R.q_ts, q0, L, tid);
  load_tile(sK[0], kg, R.k_ts, 0, L, tid);
  load_tile(sV[0], vg, R.v_ts, 0, L, tid);
  cp_async_commit();

  float o[8][4];
#pragma unroll
  for (int j = 0; j < 8; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }
  float mrow[2] = {-INFINITY, -INFINITY}, lrow[2] = {0.f, 0.f};
  uint32_t qf[4][4];

  for (int t = 0; t < nkv; ++t) {
    const int buf = t & 1;
    if (t + 1 < nkv) {
      load_tile(sK[buf ^ 1], kg, R.k_ts, (t + 1) * 64, L, tid);
      load_tile(sV[buf ^ 1], vg, R.v_ts, (t + 1) * 64, L, tid);
      cp_async_commit();
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    if (t == 0) {
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
        const int row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
        ldsm_x4(qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], tile_ptr(sQ, row, ks * 2 + (lane >> 4)));
      }
    }
    // S = Q K^T for this warp's 16 rows x 64 keys
    float s[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j) { s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f; }
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
      for (int jp = 0; jp < 4; ++jp) {
        uint32_t b0, b1, b2, b3;
        const int row = jp * 16 + (lane & 7) + (lane >> 4) * 8;
        ldsm_x4(b0, b1, b2, b3, tile_ptr(sK[buf], row, ks * 2 + ((lane >> 3) & 1)));
        mma_16816(s[2 * jp], qf[ks], b0, b1);
        mma_16816(s[2 * jp + 1], qf[ks], b2, b3);
      }
    }
    // mask keys beyond the request's length, scale, online softmax
    const int kv0 = t * 64;
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int c = kv0 + j * 8 + (lane & 3) * 2;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const bool ok = (c + (e & 1)) < L;
        s[j][e] = ok ? s[j][e] * p.scale_log2e : -INFINITY;
        mx[e >> 1] = fmaxf(mx[e >> 1], s[j][e]);
      }
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
      mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
    }
    float corr[2], mnew[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      mnew[h] = fmaxf(mrow[h], mx[h]);
      corr[h] = exp2f(mrow[h] - mnew[h]);
      mrow[h] = mnew[h];
      lrow[h] *= corr[h];
    }
    float ps[2] = {0.f, 0.f};
#pragma unroll
    for (int j = 0; j < 8; ++j) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float pv = exp2f(s[j][e] - mnew[e >> 1]);
        s[j][e] = pv;
        ps[e >> 1] += pv;
      }
      o[j][0] *= corr[0]; o[j][1] *= corr[0]; o[j][2] *= corr[1]; o[j][3] *= corr[1];
    }
    lrow[0] += ps[0];
    lrow[1] += ps[1];
    // O += P V
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      uint32_t a[4];
      a[0] = pack_bf16(s[2 * kk][0], s[2 * kk][1]);
      a[1] = pack_bf16(s[2 * kk][2], s[2 * kk][3]);
      a[2] = pack_bf16(s[2 * kk + 1][0], s[2 * kk + 1][1]);
      a[3] = pack_bf16(s[2 * kk + 1][2], s[2 * kk + 1][3]);
#pragma unroll
      for (int jp = 0; jp < 4; ++jp) {
        uint32_t b0, b1, b2, b3;
        const int row = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
        ldsm_x4_t(b0, b1, b2, b3, tile_ptr(sV[buf], row, jp * 2 + (lane >> 4)));
        mma_16816(o[2 * jp], a, b0, b1);
        mma_16816(o[2 * jp + 1], a, b2, b3);
      }
    }
    __syncthreads();
  }
  // finish: divide by the row sums (summed over the quad), store rows < L
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    lrow[h] += __shfl_xor_sync(0xffffffffu, lrow[h], 1);
    lrow[h] += __shfl_xor_sync(0xffffffffu, lrow[h], 2);
  }
  __nv_bfloat16* og = p.o + R.o_off + static_cast<long long>(head) * R.o_hs;
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int row = q0 + warp * 16 + (lane >> 2) + h * 8;
    if (row < L) {
      const float inv = 1.0f / lrow[h];
      __nv_bfloat16* orow = og + static_cast<long long>(row) * R.o_ts + (lane & 3) * 2;
#pragma unroll
      for (int j = 0; j < 8; ++j)
        *reinterpret_cast<__nv_bfloat162*>(orow + j * 8) = __floats2bfloat162_rn(o[j][2 * h] * inv, o[j][2 * h + 1] * inv);
    }
  }
}

}  // namespace k
}  // namespace sod2
