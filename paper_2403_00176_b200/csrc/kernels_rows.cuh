// HBM-bound row kernels: the fp32 fused group (MatMul + bias + GELU + residual + LayerNorm in one
// kernel), LayerNorm / softmax over a run-time number of rows, and the generic fused
// broadcast-elementwise chain with an optional trailing row reduction (Section 4.2 of the paper:
// once RDP resolves every broadcast dim to "1" or "same", one fused loop nest suffices).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <cstdint>

#include "ptx.cuh"

namespace sod2 {
namespace k {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float act_apply(int act, float x) {
  if (act == 1) return 0.5f * x * (1.0f + erff(x * 0.70710678118654752f));
  if (act == 2) return fmaxf(x, 0.0f);
  if (act == 3) return 1.0f / (1.0f + __expf(-x));
  return x;
}

// ---------------------------------------------------------------------------------------------
// Y[M,N] = LN( act(X[M,K] W[K,N] + bias) + R ) in fp32 on CUDA cores; K, N <= 128, N % 32 == 0.
// W sits in shared memory, one warp per row, lane j owns columns j, j+32, ...; LayerNorm by warp
// shuffles. fp32 has to stay on FFMA: TF32 tensor cores cannot meet a 1e-5 tolerance.
struct MlpLnParams {
  const float* X; const float* W; const float* bias; const float* R; const float* gamma; const float* beta;
  float* Y;
  int M, K, N;
  int act;       // 0 none, 1 gelu(erf), 2 relu
  int has_ln;
  float eps;
};

template <int NC>  // NC = N / 32
__global__ void __launch_bounds__(256) fused_mlp_ln_f32(MlpLnParams p) {
  extern __shared__ float smem_f[];
  float* Ws = smem_f;                 // [K][N]
  float* Xs = smem_f + p.K * p.N;     // [8 warps][K]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // The group is a few thousand elements per request, so its time is its chain of round trips to memory:
  // everything the warp's first row needs (the row, the per-column constants, its residual) is requested
  // together with W, before the first wait.
  const int row0 = blockIdx.x * 8 + warp;
  float xpre[4];                      // K <= 128
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int kk = lane + 32 * q;
    xpre[q] = (row0 < p.M && kk < p.K) ? p.X[static_cast<long long>(row0) * p.K + kk] : 0.f;
  }
  float bias_r[NC], gam[NC], bet[NC], res[NC];
#pragma unroll
  for (int c = 0; c < NC; ++c) {
    const int col = c * 32 + lane;
    bias_r[c] = p.bias ? p.bias[col] : 0.f;
    gam[c] = p.has_ln ? p.gamma[col] : 1.f;
    bet[c] = p.has_ln ? p.beta[col] : 0.f;
    res[c] = (p.R && row0 < p.M) ? p.R[static_cast<long long>(row0) * p.N + col] : 0.f;
  }
  if ((reinterpret_cast<uintptr_t>(p.W) & 15) == 0) {      // K * N is a multiple of 32
    const float4* W4 = reinterpret_cast<const float4*>(p.W);
    float4* Ws4 = reinterpret_cast<float4*>(Ws);
#pragma unroll 4
    for (int i = threadIdx.x; i < (p.K * p.N) >> 2; i += 256) Ws4[i] = W4[i];
  } else {
    for (int i = threadIdx.x; i < p.K * p.N; i += 256) Ws[i] = p.W[i];
  }
  __syncthreads();
  float* xs = Xs + warp * p.K;
  for (int row = row0; row < p.M; row += gridDim.x * 8) {
    if (row == row0) {
#pragma unroll
      for (int q = 0; q < 4; ++q) { const int kk = lane + 32 * q; if (kk < p.K) xs[kk] = xpre[q]; }
    } else {
      for (int kk = lane; kk < p.K; kk += 32) xs[kk] = p.X[static_cast<long long>(row) * p.K + kk];
      if (p.R) {
#pragma unroll
        for (int c = 0; c < NC; ++c) res[c] = p.R[static_cast<long long>(row) * p.N + c * 32 + lane];
      }
    }
    __syncwarp();
    float acc[NC];
#pragma unroll
    for (int c = 0; c < NC; ++c) acc[c] = 0.f;
    for (int kk = 0; kk < p.K; ++kk) {
      const float x = xs[kk];
#pragma unroll
      for (int c = 0; c < NC; ++c) acc[c] = fmaf(x, Ws[kk * p.N + c * 32 + lane], acc[c]);
    }
    float s = 0.f;
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      float v = acc[c];
      if (p.bias) v += bias_r[c];
      v = act_apply(p.act, v);
      if (p.R) v += res[c];
      acc[c] = v;
      s += v;
    }
    if (p.has_ln) {
      const float mu = warp_sum(s) / p.N;
      float q = 0.f;
#pragma unroll
      for (int c = 0; c < NC; ++c) { const float d = acc[c] - mu; q += d * d; }
      const float rstd = rsqrtf(warp_sum(q) / p.N + p.eps);
#pragma unroll
      for (int c = 0; c < NC; ++c) acc[c] = (acc[c] - mu) * rstd * gam[c] + bet[c];
    }
#pragma unroll
    for (int c = 0; c < NC; ++c) p.Y[static_cast<long long>(row) * p.N + c * 32 + lane] = acc[c];
    __syncwarp();
  }
}

// ---------------------------------------------------------------------------------------------
// LayerNorm over the last dim of a packed [rows, D] bf16 matrix, rows known only at run time.
// One warp per row, 128-bit loads, the row lives in registers (D <= 256 * CH), fp32 math.
// FULL: D == CH * 256, every lane owns CH full vectors: no guards, so the loads of a row are issued
// back to back (a guard per vector puts every load into a basic block of its own and serialises their
// latencies).
template <int CH, bool FULL>
__global__ void __launch_bounds__(256) layernorm_bf16(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ gamma,
                                                       const __nv_bfloat16* __restrict__ beta, __nv_bfloat16* __restrict__ y,
                                                       long long rows, int D, float eps) {
  // gamma and beta are constants of the graph: fetch them before waiting for the previous kernel
  const int lane = threadIdx.x & 31;
  const long long row = static_cast<long long>(blockIdx.x) * 8 + (threadIdx.x >> 5);
  const int nvec = D >> 3;
  uint4 g4[CH], b4[CH];
#pragma unroll
  for (int c = 0; c < CH; ++c) {
    const int i = FULL ? c * 32 + lane : min(c * 32 + lane, nvec - 1);
    g4[c] = reinterpret_cast<const uint4*>(gamma)[i];
    b4[c] = reinterpret_cast<const uint4*>(beta)[i];
  }
  ptx::pdl_launch();
  ptx::pdl_wait();
  if (row >= rows) return;
  const uint4* xr = reinterpret_cast<const uint4*>(x + row * D);
  float v[CH][8];
  float s = 0.f;
#pragma unroll
  // all loads of the row first, unconditionally (a lane past the row's end re-reads the last vector and
  // discards it): guarded loads would sit in basic blocks of their own and wait for one another
  uint4 u4[CH];
#pragma unroll
  for (int c = 0; c < CH; ++c) u4[c] = xr[FULL ? c * 32 + lane : min(c * 32 + lane, nvec - 1)];
#pragma unroll
  for (int c = 0; c < CH; ++c) {
    const bool in = FULL || c * 32 + lane < nvec;
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u4[c]);
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const float2 f = __bfloat1622float2(h[t]);
      v[c][2 * t] = in ? f.x : 0.f;
      v[c][2 * t + 1] = in ? f.y : 0.f;
      s += in ? f.x + f.y : 0.f;
    }
  }
  const float mu = warp_sum(s) / D;
  float q = 0.f;
#pragma unroll
  for (int c = 0; c < CH; ++c)
    if (FULL || c * 32 + lane < nvec) {
#pragma unroll
      for (int t = 0; t < 8; ++t) { const float d = v[c][t] - mu; q += d * d; }
    }
  const float rstd = rsqrtf(warp_sum(q) / D + eps);
  uint4* yr = reinterpret_cast<uint4*>(y + row * D);
#pragma unroll
  for (int c = 0; c < CH; ++c) {
    const int i = c * 32 + lane;
    if (FULL || i < nvec) {
      uint4 o;
      const __nv_bfloat162* gh = reinterpret_cast<const __nv_bfloat162*>(&g4[c]);
      const __nv_bfloat162* bh = reinterpret_cast<const __nv_bfloat162*>(&b4[c]);
      __nv_bfloat162* oh = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        float2 gf = __bfloat1622float2(gh[t]), bf = __bfloat1622float2(bh[t]);
        oh[t] = __floats2bfloat162_rn((v[c][2 * t] - mu) * rstd * gf.x + bf.x, (v[c][2 * t + 1] - mu) * rstd * gf.y + bf.y);
      }
      yr[i] = o;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Finish of a split-K GEMM whose group ends in LayerNorm:
//   y = LayerNorm(sum_s acc[s] + bias + residual) * gamma + beta,  acc = fp32 [splits, rows, D] workspace
// holding the K ranges' partial products, added in slab order (deterministic).  The pre-normalisation
// row never exists in bf16.
template <int CH>
__global__ void __launch_bounds__(256) splitk_ln_finish(const float* __restrict__ acc, int splits, const __nv_bfloat16* __restrict__ bias,
                                                         const __nv_bfloat16* __restrict__ res, long long ldr,
                                                         const __nv_bfloat16* __restrict__ gamma, const __nv_bfloat16* __restrict__ beta,
                                                         __nv_bfloat16* __restrict__ y, long long rows, int D, float eps) {
  const int lane = threadIdx.x & 31;
  const long long row = static_cast<long long>(blockIdx.x) * 8 + (threadIdx.x >> 5);
  const int nvec = D >> 3;
  uint4 g4[CH], b4[CH], c4[CH];
#pragma unroll
  for (int c = 0; c < CH; ++c) {
    const int i = c * 32 + lane;
    if (i < nvec) {
      g4[c] = reinterpret_cast<const uint4*>(gamma)[i]; b4[c] = reinterpret_cast<const uint4*>(beta)[i];
      c4[c] = bias ? reinterpret_cast<const uint4*>(bias)[i] : make_uint4(0, 0, 0, 0);
    }
  }
  ptx::pdl_launch();
  ptx::pdl_wait();
  if (row >= rows) return;
  const float4* ar = reinterpret_cast<const float4*>(acc + row * D);
  const long long slab4 = rows * D / 4;      // float4 per slab
  const uint4* rr = res ? reinterpret_cast<const uint4*>(res + row * ldr) : nullptr;
  float v[CH][8];
  float s = 0.f;
#pragma unroll
  for (int c = 0; c < CH; ++c) {
    const int i = c * 32 + lane;
    if (i < nvec) {
      float4 a0 = ar[2 * i], a1 = ar[2 * i + 1];
      for (int sp = 1; sp < splits; ++sp) {
        const float4 b0 = ar[sp * slab4 + 2 * i], b1 = ar[sp * slab4 + 2 * i + 1];
        a0.x += b0.x; a0.y += b0.y; a0.z += b0.z; a0.w += b0.w;
        a1.x += b1.x; a1.y += b1.y; a1.z += b1.z; a1.w += b1.w;
      }
      const uint4 ru = rr ? rr[i] : make_uint4(0, 0, 0, 0);
      const __nv_bfloat162* rh = reinterpret_cast<const __nv_bfloat162*>(&ru);
      const __nv_bfloat162* ch = reinterpret_cast<const __nv_bfloat162*>(&c4[c]);
      const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const float2 rf = __bfloat1622float2(rh[t]), cf = __bfloat1622float2(ch[t]);
        v[c][2 * t] = a[2 * t] + cf.x + rf.x;
        v[c][2 * t + 1] = a[2 * t + 1] + cf.y + rf.y;
        s += v[c][2 * t] + v[c][2 * t + 1];
      }
    } else {
#pragma unroll
      for (int t = 0; t < 8; ++t) v[c][t] = 0.f;
    }
  }
  const float mu = warp_sum(s) / D;
  float q = 0.f;
#pragma unroll
  for (int c = 0; c < CH; ++c)
    if (c * 32 + lane < nvec) {
#pragma unroll
      for (int t = 0; t < 8; ++t) { const float d = v[c][t] - mu; q += d * d; }
    }
  const float rstd = rsqrtf(warp_sum(q) / D + eps);
  uint4* yr = reinterpret_cast<uint4*>(y + row * D);
#pragma unroll
  for (int c = 0; c < CH; ++c) {
    const int i = c * 32 + lane;
    if (i < nvec) {
      uint4 o;
      const __nv_bfloat162* gh = reinterpret_cast<const __nv_bfloat162*>(&g4[c]);
      const __nv_bfloat162* bh = reinterpret_cast<const __nv_bfloat162*>(&b4[c]);
      __nv_bfloat162* oh = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        float2 gf = __bfloat1622float2(gh[t]), bf = __bfloat1622float2(bh[t]);
        oh[t] = __floats2bfloat162_rn((v[c][2 * t] - mu) * rstd * gf.x + bf.x, (v[c][2 * t + 1] - mu) * rstd * gf.y + bf.y);
      }
      yr[i] = o;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Generic fused chain: v = load(in0); v = op_i(v [, operand_i]) ...; optional softmax / LayerNorm
// over the last dim; store. Index space = the group's output [d0..d3] (rank <= 4 after
// right-alignment); every operand is read through its own strides, 0 on broadcast dims.
constexpr int CHAIN_MAX_OPS = 8;
enum ChainOp : int { C_ADD = 0, C_SUB, C_RSUB, C_MUL, C_DIV, C_RDIV, C_RELU, C_GELU, C_SIGMOID };
enum ChainRed : int { RED_NONE = 0, RED_SOFTMAX = 1, RED_LAYERNORM = 2 };

struct ChainOperand {
  const void* ptr;      // nullptr: use `scalar`
  long long stride[4];  // elements
  float scalar;
  int is_bf16;
};
struct ChainParams {
  ChainOperand in0;
  ChainOperand operand[CHAIN_MAX_OPS];
  int op[CHAIN_MAX_OPS];
  int n_ops;
  long long dim[4];
  void* out;            // contiguous
  int out_bf16;
  int red;
  const void* gamma; const void* beta; int gb_bf16; float eps;
};

__device__ __forceinline__ float chain_load(const ChainOperand& o, long long i0, long long i1, long long i2, long long i3) {
  if (!o.ptr) return o.scalar;
  const long long off = i0 * o.stride[0] + i1 * o.stride[1] + i2 * o.stride[2] + i3 * o.stride[3];
  return o.is_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(o.ptr)[off]) : reinterpret_cast<const float*>(o.ptr)[off];
}
__device__ __forceinline__ float chain_eval(const ChainParams& p, long long i0, long long i1, long long i2, long long i3) {
  float v = chain_load(p.in0, i0, i1, i2, i3);
  for (int k = 0; k < p.n_ops; ++k) {
    const int op = p.op[k];
    if (op >= C_RELU) { v = act_apply(op == C_RELU ? 2 : op == C_GELU ? 1 : 3, v); continue; }
    const float w = chain_load(p.operand[k], i0, i1, i2, i3);
    switch (op) {
      case C_ADD: v = v + w; break;
      case C_SUB: v = v - w; break;
      case C_RSUB: v = w - v; break;
      case C_MUL: v = v * w; break;
      case C_DIV: v = v / w; break;
      default: v = w / v; break;
    }
  }
  return v;
}
__device__ __forceinline__ void chain_store(const ChainParams& p, long long lin, float v) {
  if (p.out_bf16) reinterpret_cast<__nv_bfloat16*>(p.out)[lin] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(p.out)[lin] = v;
}

// no reduction: one thread per output element, grid-stride
__global__ void __launch_bounds__(256) chain_elementwise(ChainParams p) {
  const long long total = p.dim[0] * p.dim[1] * p.dim[2] * p.dim[3];
  for (long long lin = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; lin < total;
       lin += static_cast<long long>(gridDim.x) * blockDim.x) {
    long long r = lin;
    const long long i3 = r % p.dim[3]; r /= p.dim[3];
    const long long i2 = r % p.dim[2]; r /= p.dim[2];
    const long long i1 = r % p.dim[1];
    const long long i0 = r / p.dim[1];
    chain_store(p, lin, chain_eval(p, i0, i1, i2, i3));
  }
}

// trailing row reduction: one CTA per row of the last dim, the row is staged in shared memory
__global__ void __launch_bounds__(256) chain_rowreduce(ChainParams p) {
  extern __shared__ float rowbuf[];
  __shared__ float red[8];
  __shared__ float bc[2];
  const long long cols = p.dim[3];
  const long long rows = p.dim[0] * p.dim[1] * p.dim[2];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (long long row = blockIdx.x; row < rows; row += gridDim.x) {
    long long r = row;
    const long long i2 = r % p.dim[2]; r /= p.dim[2];
    const long long i1 = r % p.dim[1];
    const long long i0 = r / p.dim[1];
    float m = -INFINITY, s = 0.f;
    for (long long c = threadIdx.x; c < cols; c += blockDim.x) {
      const float v = chain_eval(p, i0, i1, i2, c);
      rowbuf[c] = v;
      m = fmaxf(m, v);
      s += v;
    }
    // first statistic: max (softmax) or mean (LayerNorm)
    float a = p.red == RED_SOFTMAX ? warp_max(m) : warp_sum(s);
    if (lane == 0) red[warp] = a;
    __syncthreads();
    if (threadIdx.x == 0) {
      float t = red[0];
      for (int w = 1; w < 8; ++w) t = p.red == RED_SOFTMAX ? fmaxf(t, red[w]) : t + red[w];
      bc[0] = p.red == RED_SOFTMAX ? t : t / cols;
    }
    __syncthreads();
    const float st0 = bc[0];
    float q = 0.f;
    for (long long c = threadIdx.x; c < cols; c += blockDim.x) {
      if (p.red == RED_SOFTMAX) { const float e = __expf(rowbuf[c] - st0); rowbuf[c] = e; q += e; }
      else { const float d = rowbuf[c] - st0; q += d * d; }
    }
    q = warp_sum(q);
    __syncthreads();
    if (lane == 0) red[warp] = q;
    __syncthreads();
    if (threadIdx.x == 0) {
      float t = 0.f;
      for (int w = 0; w < 8; ++w) t += red[w];
      bc[1] = p.red == RED_SOFTMAX ? 1.0f / t : rsqrtf(t / cols + p.eps);
    }
    __syncthreads();
    const float st1 = bc[1];
    for (long long c = threadIdx.x; c < cols; c += blockDim.x) {
      float v;
      if (p.red == RED_SOFTMAX) v = rowbuf[c] * st1;
      else {
        const float g = p.gb_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p.gamma)[c]) : reinterpret_cast<const float*>(p.gamma)[c];
        const float b = p.gb_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p.beta)[c]) : reinterpret_cast<const float*>(p.beta)[c];
        v = (rowbuf[c] - st0) * st1 * g + b;
      }
      chain_store(p, row * cols + c, v);
    }
    __syncthreads();
  }
}

}  // namespace k
}  // namespace sod2
