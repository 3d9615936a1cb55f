// Scan-based compaction for execution-determined operators (Section 3, "Execution Determined
// Output"; Fig. 1(c) TopK): top-k token keeping, NonZero.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <cstdint>

#include "ptx.cuh"

namespace sod2 {
namespace k {

constexpr int COMPACT_MAX_REQ = 32;

// ---------------------------------------------------------------------------------------------
// Token scores: s_i = sum_d y[i,d]^2 accumulated in fp64 (squares of bf16 values are exact in fp64,
// so the score depends on the summation order only at the 2^-53 level; decisions are then taken on
// these fp64 scores). One warp per row, fixed lane-strided order + fixed shuffle tree: deterministic.
struct ScoreParams {
  const __nv_bfloat16* y;   // packed rows of all requests, [rows, D]
  double* score;            // [rows]
  long long rows;
  int D;
};
__global__ void __launch_bounds__(256) row_sumsq_f64(ScoreParams p) {
  ptx::pdl_wait();
  ptx::pdl_launch();
  const int lane = threadIdx.x & 31;
  const long long row = static_cast<long long>(blockIdx.x) * 8 + (threadIdx.x >> 5);
  if (row >= p.rows) return;
  const __nv_bfloat16* yr = p.y + row * p.D;
  double acc = 0.0;
  if ((p.D & 7) == 0) {
    const uint4* v = reinterpret_cast<const uint4*>(yr);
    for (int i = lane; i < (p.D >> 3); i += 32) {
      uint4 u = v[i];
      const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        float2 f = __bfloat1622float2(h[t]);
        acc += static_cast<double>(f.x) * f.x;
        acc += static_cast<double>(f.y) * f.y;
      }
    }
  } else {
    for (int i = lane; i < p.D; i += 32) { const double f = __bfloat162float(yr[i]); acc += f * f; }
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) p.score[row] = acc;
}

// ---------------------------------------------------------------------------------------------
// Keep the k highest-scoring tokens of each request in ascending index order.
//   rank_i = #{j : s_j > s_i} + #{j < i : s_j == s_i};  keep_i = rank_i < k
//   pos_i  = exclusive scan of keep;  idx[pos_i] = i;  out[pos_i, :] = y[i, :]
// One CTA per request: ranks by counting against the scores staged in shared memory, block-wide
// scan of the flags, then warp-per-row gather with 128-bit copies.
struct TopkReq {
  long long row0;      // first packed input row of the request
  long long out_row0;  // first packed output row
  long long idx0;      // first packed index entry
  int n, k;
};
struct TopkParams {
  const __nv_bfloat16* y;
  const double* score;
  __nv_bfloat16* out;
  long long* idx;      // packed [sum k] int64, per request k entries
  int D;
  int n_req;
  TopkReq r[COMPACT_MAX_REQ];
};

__global__ void __launch_bounds__(1024) topk_keep(const __grid_constant__ TopkParams p) {
  extern __shared__ double s_score[];                  // [n]
  int* s_pos = reinterpret_cast<int*>(s_score + ((p.r[blockIdx.x].n + 1) & ~1));  // [n] kept position or -1
  __shared__ int warp_tot[32];
  const TopkReq R = p.r[blockIdx.x];
  ptx::pdl_wait();
  ptx::pdl_launch();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int i = tid; i < R.n; i += blockDim.x) s_score[i] = p.score[R.row0 + i];
  __syncthreads();
  int carry = 0;  // kept count of earlier chunks (same in every thread)
  for (int base = 0; base < R.n; base += blockDim.x) {
    const int i = base + tid;
    int keep = 0;
    if (i < R.n) {
      const double si = s_score[i];
      int rank = 0;
      for (int j = 0; j < R.n; ++j) {
        const double sj = s_score[j];
        rank += (sj > si) || (sj == si && j < i);
      }
      keep = rank < R.k;
    }
    // block exclusive scan of keep
    const unsigned bal = __ballot_sync(0xffffffffu, keep);
    const int wpre = __popc(bal & ((1u << lane) - 1));
    if (lane == 0) warp_tot[warp] = __popc(bal);
    __syncthreads();
    int woff = 0, tot = 0;
    for (int w = 0; w < 32; ++w) { const int c = warp_tot[w]; if (w < warp) woff += c; tot += c; }
    if (i < R.n) s_pos[i] = keep ? carry + woff + wpre : -1;
    carry += tot;
    __syncthreads();
  }
  // gather: one warp per source row
  const int vec = (p.D * 2) >> 4;  // 16-byte chunks per row (D % 8 == 0 checked on the host)
  for (int i = warp; i < R.n; i += 32) {
    const int pos = s_pos[i];
    if (pos < 0) continue;
    if (lane == 0) p.idx[R.idx0 + pos] = i;
    const uint4* src = reinterpret_cast<const uint4*>(p.y + (R.row0 + i) * p.D);
    uint4* dst = reinterpret_cast<uint4*>(p.out + (R.out_row0 + pos) * p.D);
    for (int c = lane; c < vec; c += 32) dst[c] = src[c];
  }
}

// ---------------------------------------------------------------------------------------------
// NonZero: int64 coordinates [rank, nnz] of the non-zero elements in row-major order.
// Pass 1: per-block counts into scratch; pass 2 (one CTA): exclusive scan of the counts + total;
// pass 3: each block rescans its flags and writes coordinates at its offset. nnz is known only
// after pass 2, so the row pitch of the output (= nnz) is read from device memory in pass 3.
constexpr int NZ_BLOCK = 1024;
struct NonZeroParams {
  const void* x; int is_bf16;
  long long numel;
  int rank;
  long long dims[4];
  int* block_count;       // scratch [nblocks + 1]; after pass 2: exclusive offsets, [nblocks] = total
  long long* out;         // [rank, nnz]
  long long* count_out;   // device word: nnz
  int nblocks;
};
__device__ __forceinline__ bool nz_flag(const NonZeroParams& p, long long i) {
  if (i >= p.numel) return false;
  return p.is_bf16 ? (__bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p.x)[i]) != 0.0f)
                   : (reinterpret_cast<const float*>(p.x)[i] != 0.0f);
}
__global__ void __launch_bounds__(NZ_BLOCK) nonzero_count(NonZeroParams p) {
  __shared__ int wc[32];
  const long long i = static_cast<long long>(blockIdx.x) * NZ_BLOCK + threadIdx.x;
  const unsigned bal = __ballot_sync(0xffffffffu, nz_flag(p, i));
  if ((threadIdx.x & 31) == 0) wc[threadIdx.x >> 5] = __popc(bal);
  __syncthreads();
  if (threadIdx.x == 0) {
    int t = 0;
    for (int w = 0; w < 32; ++w) t += wc[w];
    p.block_count[blockIdx.x] = t;
  }
}
__global__ void __launch_bounds__(1024) nonzero_scan(NonZeroParams p) {
  // single CTA, sequential over chunks of 1024 block counts
  __shared__ int wt[32];
  __shared__ int carry_s;
  if (threadIdx.x == 0) carry_s = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int base = 0; base < p.nblocks; base += 1024) {
    const int i = base + threadIdx.x;
    const int v = i < p.nblocks ? p.block_count[i] : 0;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += t; }
    if (lane == 31) wt[warp] = inc;
    __syncthreads();
    int woff = 0;
    for (int w = 0; w < warp; ++w) woff += wt[w];
    const int carry = carry_s;
    if (i < p.nblocks) p.block_count[i] = carry + woff + inc - v;
    __syncthreads();
    if (threadIdx.x == 1023) carry_s = carry + woff + inc;
    __syncthreads();
  }
  if (threadIdx.x == 0) { p.block_count[p.nblocks] = carry_s; *p.count_out = carry_s; }
}
__global__ void __launch_bounds__(NZ_BLOCK) nonzero_write(NonZeroParams p) {
  __shared__ int wc[32];
  const long long i = static_cast<long long>(blockIdx.x) * NZ_BLOCK + threadIdx.x;
  const bool f = nz_flag(p, i);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned bal = __ballot_sync(0xffffffffu, f);
  if (lane == 0) wc[warp] = __popc(bal);
  __syncthreads();
  if (!f) return;
  int off = p.block_count[blockIdx.x] + __popc(bal & ((1u << lane) - 1));
  for (int w = 0; w < warp; ++w) off += wc[w];
  const long long nnz = p.block_count[p.nblocks];
  long long r = i;
  for (int d = p.rank - 1; d >= 0; --d) {
    p.out[static_cast<long long>(d) * nnz + off] = r % p.dims[d];
    r /= p.dims[d];
  }
}

}  // namespace k
}  // namespace sod2
