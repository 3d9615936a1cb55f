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
// Two kernels over the same grid, one CTA per chunk of 64 tokens of a request (so a batch of 16
// requests spreads over about a hundred SMs instead of 16):
//   topk_flags   the request's fp64 scores staged in shared memory; four threads share a token's
//                ranking (a quarter of the comparisons each); writes keep_i as a byte
//   topk_gather  counts the kept tokens before the chunk, scans the chunk's 64 flags with two ballots,
//                writes the indices and copies the kept rows, one warp per row, 128-bit accesses
constexpr int TOPK_CHUNK = 64;
struct TopkReq {
  long long row0;      // first packed input row of the request
  long long out_row0;  // first packed output row
  long long idx0;      // first packed index entry
  int n, k;
};
struct TopkParams {
  const __nv_bfloat16* y;
  const double* score;       // packed [rows] relative to the first request's row0
  unsigned char* keep;       // packed [rows], same indexing as score
  __nv_bfloat16* out;
  long long* idx;            // packed [sum k] int64, per request k entries
  int D;
  int n_req;
  long long first_row;       // row0 of the first request (score / keep are indexed from it)
  int chunk_start[COMPACT_MAX_REQ + 1];   // prefix sum of ceil(n / 64)
  TopkReq r[COMPACT_MAX_REQ];
};

__device__ __forceinline__ int topk_locate(const TopkParams& p, int cta, int* chunk) {
  int ri = 0;
  while (ri + 1 < p.n_req && cta >= p.chunk_start[ri + 1]) ++ri;
  *chunk = cta - p.chunk_start[ri];
  return ri;
}

__global__ void __launch_bounds__(256) topk_flags(const __grid_constant__ TopkParams p) {
  extern __shared__ double s_score[];                  // [n]
  int chunk;
  const TopkReq R = p.r[topk_locate(p, blockIdx.x, &chunk)];
  ptx::pdl_wait();
  ptx::pdl_launch();
  const int tid = threadIdx.x;
  const double* sc = p.score + (R.row0 - p.first_row);
  // a NaN score (an overflow upstream) compares false with everything and would be kept by every chunk: it ranks
  // last instead, ties among NaNs by index, so that exactly k tokens are kept whatever the data
  for (int i = tid; i < R.n; i += 256) { const double v = sc[i]; s_score[i] = v == v ? v : -INFINITY; }
  __syncthreads();
  const int i = chunk * TOPK_CHUNK + (tid >> 2), part = tid & 3;
  int rank = 0;
  if (i < R.n) {
    const double si = s_score[i];
    const int per = (R.n + 3) >> 2, j0 = part * per, j1 = min(R.n, j0 + per);
    for (int j = j0; j < j1; ++j) {
      const double sj = s_score[j];
      rank += (sj > si) || (sj == si && j < i);
    }
  }
  rank += __shfl_xor_sync(0xffffffffu, rank, 1);
  rank += __shfl_xor_sync(0xffffffffu, rank, 2);
  if (i < R.n && part == 0) p.keep[R.row0 - p.first_row + i] = rank < R.k;
}

__global__ void __launch_bounds__(256) topk_gather(const __grid_constant__ TopkParams p) {
  __shared__ int warp_cnt[8];
  __shared__ int s_pos[TOPK_CHUNK];
  int chunk;
  const TopkReq R = p.r[topk_locate(p, blockIdx.x, &chunk)];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int base = chunk * TOPK_CHUNK;
  // The rows of the chunk are fetched before the dependency wait: they were written by the kernel before the
  // score kernel, which had completed before the flag kernel (the one waited for here) let this one start, so
  // only the flags are still in flight.  Whether a row is kept is not known yet: all rows of the chunk are read.
  const int vec = (p.D * 2) >> 4;  // 16-byte pieces per row (D % 8 == 0 checked on the host)
  const uint4* src = reinterpret_cast<const uint4*>(p.y + (R.row0 + base) * p.D);
  const int items = min(TOPK_CHUNK, R.n - base) * vec;
  constexpr int PRE = 12;
  uint4 pre[PRE];
#pragma unroll
  for (int u = 0; u < PRE; ++u) {
    const int it = tid + u * 256;
    if (it < items) pre[u] = src[it];
  }
  ptx::pdl_wait();
  ptx::pdl_launch();
  const unsigned char* kp = p.keep + (R.row0 - p.first_row);
  // kept tokens before this chunk
  int c = 0;
  for (int j = tid; j < base; j += 256) c += kp[j];
#pragma unroll
  for (int o = 16; o; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
  if (lane == 0) warp_cnt[warp] = c;
  __syncthreads();
  int carry = 0;
#pragma unroll
  for (int w = 0; w < 8; ++w) carry += warp_cnt[w];
  // the chunk's own 64 flags: warps 0 and 1 take 32 each
  if (warp < 2) {
    const int i = base + tid;
    const int keep = i < R.n ? kp[i] : 0;
    const unsigned bal = __ballot_sync(0xffffffffu, keep);
    const int pre = __popc(bal & ((1u << lane) - 1));
    if (lane == 0) warp_cnt[warp] = __popc(bal);
    __syncwarp();
    s_pos[tid] = keep ? pre : -1;
  }
  __syncthreads();
  if (tid < TOPK_CHUNK && s_pos[tid] >= 0) {
    s_pos[tid] += carry + (tid >= 32 ? warp_cnt[0] : 0);
    p.idx[R.idx0 + s_pos[tid]] = base + tid;
  }
  __syncthreads();
  // write the kept rows: (row, 16-byte piece) items spread over the whole CTA; the first PRE per thread are
  // already in registers, wider rows load the rest now
  uint4* dst = reinterpret_cast<uint4*>(p.out + R.out_row0 * p.D);
#pragma unroll
  for (int u = 0; u < PRE; ++u) {
    const int it = tid + u * 256;
    if (it < items) {
      const int t = it / vec, c4 = it - t * vec;
      const int pos = s_pos[t];
      if (pos >= 0) dst[static_cast<long long>(pos) * vec + c4] = pre[u];
    }
  }
#pragma unroll 4
  for (int it = tid + PRE * 256; it < items; it += 256) {
    const int t = it / vec, c4 = it - t * vec;
    const int pos = s_pos[t];
    if (pos >= 0) dst[static_cast<long long>(pos) * vec + c4] = src[it];
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
