// Stand-alone kernels of the unfused execution mode (SOD2_OPT_NO_FUSION) for the operators that otherwise only run
// inside fused groups: MatMul of two activations (attention's QK^T and PV), ReduceSumSquare, TopK and Gather.  The
// mode exists to show that fusion equals unfused execution (Section 4.2), so these are plain SIMT kernels: every
// intermediate is materialised in the graph's storage type, one kernel per operator and request.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <cstdint>

namespace sod2 {
namespace k {

__device__ __forceinline__ float uf_load(const void* p, long long i, int is_bf16) {
  return is_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[i]) : reinterpret_cast<const float*>(p)[i];
}
__device__ __forceinline__ void uf_store(void* p, long long i, float v, int is_bf16) {
  if (is_bf16) reinterpret_cast<__nv_bfloat16*>(p)[i] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(p)[i] = v;
}

// C[b0,b1,m,n] = sum_k A[b0,b1,m,k] * B[b0,b1,k,n]; element strides per operand (0 = broadcast batch dim), fp32
// accumulation in k order inside 16 x 16 tiles staged through shared memory.
struct BmmParams {
  const void* a; const void* b; void* c;
  int is_bf16;
  int B0, B1, M, N, K;
  long long as[4], bs[4], cs[4];     // strides of (b0, b1, row, col)
};
__global__ void __launch_bounds__(256) bmm_strided(BmmParams p) {
  __shared__ float sa[16][17], sb[16][17];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int b1 = blockIdx.z % p.B1, b0 = blockIdx.z / p.B1;
  const int m = blockIdx.y * 16 + ty, n = blockIdx.x * 16 + tx;
  const long long ao = b0 * p.as[0] + b1 * p.as[1], bo = b0 * p.bs[0] + b1 * p.bs[1];
  float acc = 0.f;
  for (int k0 = 0; k0 < p.K; k0 += 16) {
    sa[ty][tx] = (m < p.M && k0 + tx < p.K) ? uf_load(p.a, ao + m * p.as[2] + (k0 + tx) * p.as[3], p.is_bf16) : 0.f;
    sb[ty][tx] = (k0 + ty < p.K && n < p.N) ? uf_load(p.b, bo + (k0 + ty) * p.bs[2] + n * p.bs[3], p.is_bf16) : 0.f;
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) acc = fmaf(sa[ty][kk], sb[kk][tx], acc);
    __syncthreads();
  }
  if (m < p.M && n < p.N) uf_store(p.c, b0 * p.cs[0] + b1 * p.cs[1] + m * p.cs[2] + n * p.cs[3], acc, p.is_bf16);
}

// out[row] = sum_d x[row, d]^2 over a contiguous last dim, fp64 accumulation (fixed lane-strided order + shuffle
// tree), stored in the graph's type.  One warp per row.
struct SumSqParams { const void* x; void* out; long long rows; int D; int in_bf16, out_bf16; };
__global__ void __launch_bounds__(256) reduce_sumsq_rows(SumSqParams p) {
  const int lane = threadIdx.x & 31;
  const long long row = static_cast<long long>(blockIdx.x) * 8 + (threadIdx.x >> 5);
  if (row >= p.rows) return;
  double acc = 0.0;
  for (int i = lane; i < p.D; i += 32) { const double f = uf_load(p.x, row * p.D + i, p.in_bf16); acc += f * f; }
#pragma unroll
  for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) uf_store(p.out, row, static_cast<float>(acc), p.out_bf16);
}

// TopK over a contiguous last dim of n scores (n * 4 bytes of shared memory): rank_i = #{j : s_j better than s_i} +
// #{j < i : s_j == s_i}; element i is kept iff rank_i < k; order = 0: kept positions ascending ("index"),
// 1: by rank ("value").  One CTA per row; values in the graph's type, indices int64.
struct TopkRowsParams { const void* s; void* vals; long long* idx; long long rows; int n, k, largest, by_value, is_bf16; };
__global__ void __launch_bounds__(256) topk_rows(TopkRowsParams p) {
  extern __shared__ float sc[];            // [n] scores, then [n] ints: keep flags / positions
  int* pos = reinterpret_cast<int*>(sc + p.n);
  __shared__ int warp_tot[8];
  for (long long row = blockIdx.x; row < p.rows; row += gridDim.x) {
    for (int i = threadIdx.x; i < p.n; i += 256) {
      const float v = uf_load(p.s, row * p.n + i, p.is_bf16);
      sc[i] = v == v ? v : (p.largest ? -INFINITY : INFINITY);       // NaN ranks last
    }
    __syncthreads();
    for (int i = threadIdx.x; i < p.n; i += 256) {
      const float si = sc[i];
      int rank = 0;
      for (int j = 0; j < p.n; ++j) {
        const float sj = sc[j];
        rank += (p.largest ? sj > si : sj < si) || (sj == si && j < i);
      }
      pos[i] = rank < p.k ? (p.by_value ? rank : -2) : -1;            // -2: kept, position still to be scanned
    }
    __syncthreads();
    if (!p.by_value) {
      // exclusive scan of the keep flags in index order, 256 elements per sweep
      int carry = 0;
      for (int base = 0; base < p.n; base += 256) {
        const int i = base + threadIdx.x;
        const int keep = i < p.n && pos[i] == -2;
        const unsigned bal = __ballot_sync(0xffffffffu, keep);
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        if (lane == 0) warp_tot[warp] = __popc(bal);
        __syncthreads();
        int off = carry + __popc(bal & ((1u << lane) - 1));
        for (int w = 0; w < warp; ++w) off += warp_tot[w];
        int tot = 0;
        for (int w = 0; w < 8; ++w) tot += warp_tot[w];
        if (keep) pos[i] = off;
        carry += tot;
        __syncthreads();
      }
    }
    for (int i = threadIdx.x; i < p.n; i += 256)
      if (pos[i] >= 0) {
        if (p.idx) p.idx[row * p.k + pos[i]] = i;
        if (p.vals) uf_store(p.vals, row * p.k + pos[i], uf_load(p.s, row * p.n + i, p.is_bf16), p.is_bf16);
      }
    __syncthreads();
  }
}

// out[o, j, i] = x[o, idx[j], i]: Gather along one axis with int64 indices; outer = product of the dims before the
// axis, inner = product of those after it (contiguous).  One thread per output element, grid-stride.
struct GatherParams { const void* x; const long long* idx; void* out; long long outer, n_in, n_idx, inner; int esz; };
__global__ void __launch_bounds__(256) gather_axis(GatherParams p) {
  const long long total = p.outer * p.n_idx * p.inner;
  for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += static_cast<long long>(gridDim.x) * blockDim.x) {
    const long long in = i % p.inner, j = (i / p.inner) % p.n_idx, o = i / (p.inner * p.n_idx);
    long long src = p.idx[j];
    if (src < 0) src += p.n_in;
    const long long s = (o * p.n_in + src) * p.inner + in;
    if (p.esz == 2) reinterpret_cast<uint16_t*>(p.out)[i] = reinterpret_cast<const uint16_t*>(p.x)[s];
    else if (p.esz == 4) reinterpret_cast<uint32_t*>(p.out)[i] = reinterpret_cast<const uint32_t*>(p.x)[s];
    else reinterpret_cast<uint64_t*>(p.out)[i] = reinterpret_cast<const uint64_t*>(p.x)[s];
  }
}

// Resize / Upsample, nearest neighbour (Table 2: input shape & value determined output shape): along every axis the
// source index of output index o is floor(o * in / out), the "asymmetric" coordinate rule with the index rounded down;
// for integer scales this repeats every element `scale` times.  Operands are addressed through their strides (element
// units), so packed and channels-last storage both work; one thread per output element in the output's storage
// order (`order[k]` = k-th fastest axis of the output), so stores coalesce.
struct ResizeParams {
  const void* x; void* out;
  long long in_dim[6], out_dim[6], in_stride[6], out_stride[6];
  int order[6];
  int rank, esz;
  long long total;
};
__global__ void __launch_bounds__(256) resize_nearest(ResizeParams p) {
  for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < p.total; i += static_cast<long long>(gridDim.x) * blockDim.x) {
    long long rem = i, so = 0, si = 0;
    for (int k = 0; k < p.rank; ++k) {
      const int ax = p.order[k];
      const long long o = rem % p.out_dim[ax];
      rem /= p.out_dim[ax];
      long long src = o * p.in_dim[ax] / p.out_dim[ax];
      if (src > p.in_dim[ax] - 1) src = p.in_dim[ax] - 1;
      so += o * p.out_stride[ax];
      si += src * p.in_stride[ax];
    }
    if (p.esz == 2) reinterpret_cast<uint16_t*>(p.out)[so] = reinterpret_cast<const uint16_t*>(p.x)[si];
    else if (p.esz == 4) reinterpret_cast<uint32_t*>(p.out)[so] = reinterpret_cast<const uint32_t*>(p.x)[si];
    else reinterpret_cast<uint64_t*>(p.out)[so] = reinterpret_cast<const uint64_t*>(p.x)[si];
  }
}

// out[i] = start + i * step for i < n: Range (int64) and ConstantOfShape (step 0; fp32, bf16 or int64).
struct FillParams { void* out; long long n; double start, step; int dtype; /* 0 f32, 1 bf16, 2 i64 */ };
__global__ void __launch_bounds__(256) fill_linear(FillParams p) {
  for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < p.n; i += static_cast<long long>(gridDim.x) * blockDim.x) {
    const double v = p.start + static_cast<double>(i) * p.step;
    if (p.dtype == 2) reinterpret_cast<long long*>(p.out)[i] = static_cast<long long>(v);
    else if (p.dtype == 1) reinterpret_cast<__nv_bfloat16*>(p.out)[i] = __float2bfloat16_rn(static_cast<float>(v));
    else reinterpret_cast<float*>(p.out)[i] = static_cast<float>(v);
  }
}

}  // namespace k
}  // namespace sod2
