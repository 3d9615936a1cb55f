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
// Generic fused chain (the paper's Fig. 4 form): v = load(in0); v = op_i(v [, operand_i]) ...; optional softmax /
// LayerNorm over the last dim; store.  Index space = the group's output [d0..d3] (rank <= 4 after
// right-alignment); every operand is read through its own strides, 0 on the dims RDP resolved to "broadcast".
// All requests of a batch run in ONE launch through a request table (up to CHAIN_MAX_REQ entries): the operands of
// the requests live in the same packed buffers, so an entry is extents, element offsets and strides.
//   chain_elementwise_vec   work item = 8 or 16 consecutive outputs along the last dim: 128-bit loads / stores, operands
//                           broadcast along the last dim fetched once per item; (row, column) decomposition in 32-bit
//                           arithmetic, one division chain per item instead of per element
//   chain_elementwise       work item = one output (any strides, any extents): the fallback
//   chain_rowreduce_warp    a warp per row (rows up to ROWRED_WARP_COLS), the row staged in the warp's slice of shared
//                           memory, statistics by shuffles: no CTA barrier, eight rows in flight per CTA
//   chain_rowreduce         a CTA per row for longer rows
constexpr int CHAIN_MAX_OPS = 8;
constexpr int CHAIN_MAX_REQ = 8;
constexpr int ROWRED_WARP_COLS = 2048;
enum ChainOp : int { C_ADD = 0, C_SUB, C_RSUB, C_MUL, C_DIV, C_RDIV, C_RELU, C_GELU, C_SIGMOID };
enum ChainRed : int { RED_NONE = 0, RED_SOFTMAX = 1, RED_LAYERNORM = 2 };

struct ChainReq {
  int dim[4];                               // output extents
  long long first;                          // first work item of this request in the launch
  long long out_off;                        // elements from `out`
  long long off[1 + CHAIN_MAX_OPS];         // elements from base[k]; k = 0 is in0, k = 1 + i operand i
  int stride[1 + CHAIN_MAX_OPS][4];         // elements
};
struct ChainBatch {
  const void* base[1 + CHAIN_MAX_OPS];      // nullptr: use scalar[k]
  float scalar[1 + CHAIN_MAX_OPS];
  int is_bf16[1 + CHAIN_MAX_OPS];
  int op[CHAIN_MAX_OPS];
  int n_ops;
  void* out;                                // every request's output instance is contiguous
  int out_bf16;
  int red;
  const void* gamma; const void* beta; int gb_bf16; float eps;
  int n_req;
  long long total;                          // work items of all requests
  ChainReq r[CHAIN_MAX_REQ];
};

__device__ __forceinline__ int chain_find_req(const ChainBatch& p, long long item) {
  int ri = 0;
  while (ri + 1 < p.n_req && item >= p.r[ri + 1].first) ++ri;
  return ri;
}
__device__ __forceinline__ float chain_apply(int op, float v, float w) {
  switch (op) {
    case C_ADD: return v + w;
    case C_SUB: return v - w;
    case C_RSUB: return w - v;
    case C_MUL: return v * w;
    case C_DIV: return v / w;
    case C_RDIV: return w / v;
    case C_RELU: return fmaxf(v, 0.f);
    case C_GELU: return act_apply(1, v);
    default: return act_apply(3, v);
  }
}
__device__ __forceinline__ float chain_load1(const ChainBatch& p, const ChainReq& R, int k, int i0, int i1, int i2, int i3) {
  if (!p.base[k]) return p.scalar[k];
  const long long off = R.off[k] + static_cast<long long>(i0) * R.stride[k][0] + static_cast<long long>(i1) * R.stride[k][1] +
                        static_cast<long long>(i2) * R.stride[k][2] + static_cast<long long>(i3) * R.stride[k][3];
  return p.is_bf16[k] ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p.base[k])[off]) : reinterpret_cast<const float*>(p.base[k])[off];
}
__device__ __forceinline__ float chain_eval(const ChainBatch& p, const ChainReq& R, int i0, int i1, int i2, int i3) {
  float v = chain_load1(p, R, 0, i0, i1, i2, i3);
  for (int k = 0; k < p.n_ops; ++k) {
    const int op = p.op[k];
    v = chain_apply(op, v, op >= C_RELU ? 0.f : chain_load1(p, R, 1 + k, i0, i1, i2, i3));
  }
  return v;
}
__device__ __forceinline__ void chain_store1(const ChainBatch& p, long long lin, float v) {
  if (p.out_bf16) reinterpret_cast<__nv_bfloat16*>(p.out)[lin] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(p.out)[lin] = v;
}

// eight consecutive elements of operand k along the last dim (stride 1, 16-byte aligned), or one broadcast value
__device__ __forceinline__ void chain_load8(const ChainBatch& p, const ChainReq& R, int k, int i0, int i1, int i2, int i3, float* w) {
  if (!p.base[k]) {
#pragma unroll
    for (int t = 0; t < 8; ++t) w[t] = p.scalar[k];
    return;
  }
  const long long off = R.off[k] + static_cast<long long>(i0) * R.stride[k][0] + static_cast<long long>(i1) * R.stride[k][1] +
                        static_cast<long long>(i2) * R.stride[k][2] + static_cast<long long>(i3) * R.stride[k][3];
  if (R.stride[k][3] == 0) {
    const float x = p.is_bf16[k] ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p.base[k])[off]) : reinterpret_cast<const float*>(p.base[k])[off];
#pragma unroll
    for (int t = 0; t < 8; ++t) w[t] = x;
  } else if (p.is_bf16[k]) {
    const uint4 u = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p.base[k]) + off);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
    for (int t = 0; t < 4; ++t) { const float2 f = __bfloat1622float2(h[t]); w[2 * t] = f.x; w[2 * t + 1] = f.y; }
  } else {
    const float4 a = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(p.base[k]) + off);
    const float4 c = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(p.base[k]) + off + 4);
    w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w; w[4] = c.x; w[5] = c.y; w[6] = c.z; w[7] = c.w;
  }
}

// The host selects this kernel only if, for every request, dim[3] % (8 * NV) == 0, every operand's last-dim stride is
// 0 or 1, and all offsets and leading strides of stride-1 operands (and the output offset) are multiples of 8
// elements.  NV = 8-element vectors per work item (1 or 2): the index arithmetic is paid once per item.
template <int NV>
__global__ void __launch_bounds__(256) chain_elementwise_vec(const __grid_constant__ ChainBatch p) {
  for (long long item = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; item < p.total;
       item += static_cast<long long>(gridDim.x) * blockDim.x) {
    const ChainReq& R = p.r[chain_find_req(p, item)];
    const unsigned li = static_cast<unsigned>(item - R.first);      // the host keeps a request below 2^31 items
    const unsigned cv = static_cast<unsigned>(R.dim[3]) / (8 * NV);
    unsigned row = li / cv;
    const int i3 = static_cast<int>(li - row * cv) * (8 * NV);
    const unsigned d2 = R.dim[2], d1 = R.dim[1];
    const unsigned t2 = row / d2;
    const int i2 = static_cast<int>(row - t2 * d2);
    const unsigned t1 = t2 / d1;
    const int i1 = static_cast<int>(t2 - t1 * d1), i0 = static_cast<int>(t1);
    // While every operand so far is broadcast along the last dim the values of an item are one value: that prefix
    // of the chain (Fig. 4: Sigmoid of the [I,1,1] operand) is evaluated once per item, not once per element.
    float v[NV][8], w[NV][8];
    int k0 = 0;
    if (!p.base[0] || R.stride[0][3] == 0) {
      float u = chain_load1(p, R, 0, i0, i1, i2, i3);
      for (; k0 < p.n_ops; ++k0) {
        const int op = p.op[k0];
        if (op < C_RELU && p.base[1 + k0] && R.stride[1 + k0][3] != 0) break;
        u = chain_apply(op, u, op >= C_RELU ? 0.f : chain_load1(p, R, 1 + k0, i0, i1, i2, i3));
      }
#pragma unroll
      for (int n = 0; n < NV; ++n)
#pragma unroll
        for (int t = 0; t < 8; ++t) v[n][t] = u;
    } else {
#pragma unroll
      for (int n = 0; n < NV; ++n) chain_load8(p, R, 0, i0, i1, i2, i3 + 8 * n, v[n]);
    }
    for (int k = k0; k < p.n_ops; ++k) {
      const int op = p.op[k];
      if (op < C_RELU) {
#pragma unroll
        for (int n = 0; n < NV; ++n) chain_load8(p, R, 1 + k, i0, i1, i2, i3 + 8 * n, w[n]);
      }
      // the operator is chosen once per item; the elements run through straight-line code
      switch (op) {
#define SOD2_CHAIN_CASE(OP_)                                                                                   \
        case OP_:                                                                                              \
          _Pragma("unroll") for (int n = 0; n < NV; ++n)                                                       \
            _Pragma("unroll") for (int t = 0; t < 8; ++t) v[n][t] = chain_apply(OP_, v[n][t], w[n][t]);        \
          break;
        SOD2_CHAIN_CASE(C_ADD)
        SOD2_CHAIN_CASE(C_SUB)
        SOD2_CHAIN_CASE(C_RSUB)
        SOD2_CHAIN_CASE(C_MUL)
        SOD2_CHAIN_CASE(C_DIV)
        SOD2_CHAIN_CASE(C_RDIV)
        SOD2_CHAIN_CASE(C_RELU)
        SOD2_CHAIN_CASE(C_GELU)
        default:
        SOD2_CHAIN_CASE(C_SIGMOID)
#undef SOD2_CHAIN_CASE
      }
    }
    const long long lin = R.out_off + static_cast<long long>(li) * (8 * NV);
#pragma unroll
    for (int n = 0; n < NV; ++n) {
      if (p.out_bf16) {
        uint4 o;
        __nv_bfloat162* oh = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
        for (int t = 0; t < 4; ++t) oh[t] = __floats2bfloat162_rn(v[n][2 * t], v[n][2 * t + 1]);
        *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.out) + lin + 8 * n) = o;
      } else {
        float* o = reinterpret_cast<float*>(p.out) + lin + 8 * n;
        *reinterpret_cast<float4*>(o) = make_float4(v[n][0], v[n][1], v[n][2], v[n][3]);
        *reinterpret_cast<float4*>(o + 4) = make_float4(v[n][4], v[n][5], v[n][6], v[n][7]);
      }
    }
  }
}

// fallback: one thread per output element, grid-stride
__global__ void __launch_bounds__(256) chain_elementwise(const __grid_constant__ ChainBatch p) {
  for (long long item = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; item < p.total;
       item += static_cast<long long>(gridDim.x) * blockDim.x) {
    const ChainReq& R = p.r[chain_find_req(p, item)];
    long long r = item - R.first;
    const int i3 = static_cast<int>(r % R.dim[3]); r /= R.dim[3];
    const int i2 = static_cast<int>(r % R.dim[2]); r /= R.dim[2];
    const int i1 = static_cast<int>(r % R.dim[1]);
    const int i0 = static_cast<int>(r / R.dim[1]);
    chain_store1(p, R.out_off + (item - R.first), chain_eval(p, R, i0, i1, i2, i3));
  }
}

__device__ __forceinline__ void chain_row_index(const ChainReq& R, long long row, int* i0, int* i1, int* i2) {
  *i2 = static_cast<int>(row % R.dim[2]); row /= R.dim[2];
  *i1 = static_cast<int>(row % R.dim[1]);
  *i0 = static_cast<int>(row / R.dim[1]);
}
__device__ __forceinline__ float chain_gb(const ChainBatch& p, const void* v, int c) {
  return p.gb_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(v)[c]) : reinterpret_cast<const float*>(v)[c];
}

// trailing row reduction, a warp per row: work item = row; dynamic shared memory = 8 rows of `max_cols` floats
__global__ void __launch_bounds__(256) chain_rowreduce_warp(const __grid_constant__ ChainBatch p, int max_cols) {
  extern __shared__ float rowbuf_all[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float* rowbuf = rowbuf_all + static_cast<size_t>(warp) * max_cols;
  for (long long item = static_cast<long long>(blockIdx.x) * 8 + warp; item < p.total; item += static_cast<long long>(gridDim.x) * 8) {
    const ChainReq& R = p.r[chain_find_req(p, item)];
    const long long row = item - R.first;
    const int cols = R.dim[3];
    int i0, i1, i2;
    chain_row_index(R, row, &i0, &i1, &i2);
    float m = -INFINITY, s = 0.f;
    for (int c = lane; c < cols; c += 32) {
      const float v = chain_eval(p, R, i0, i1, i2, c);
      rowbuf[c] = v;
      m = fmaxf(m, v);
      s += v;
    }
    const float st0 = p.red == RED_SOFTMAX ? warp_max(m) : warp_sum(s) / cols;
    float q = 0.f;
    for (int c = lane; c < cols; c += 32) {
      if (p.red == RED_SOFTMAX) { const float e = __expf(rowbuf[c] - st0); rowbuf[c] = e; q += e; }
      else { const float d = rowbuf[c] - st0; q += d * d; }
    }
    q = warp_sum(q);
    const float st1 = p.red == RED_SOFTMAX ? 1.0f / q : rsqrtf(q / cols + p.eps);
    const long long obase = R.out_off + row * cols;
    for (int c = lane; c < cols; c += 32) {
      const float v = p.red == RED_SOFTMAX ? rowbuf[c] * st1 : (rowbuf[c] - st0) * st1 * chain_gb(p, p.gamma, c) + chain_gb(p, p.beta, c);
      chain_store1(p, obase + c, v);
    }
    __syncwarp();
  }
}

// trailing row reduction, a CTA per row (long rows): dynamic shared memory = one row
__global__ void __launch_bounds__(256) chain_rowreduce(const __grid_constant__ ChainBatch p) {
  extern __shared__ float rowbuf[];
  __shared__ float red[8];
  __shared__ float bc[2];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (long long item = blockIdx.x; item < p.total; item += gridDim.x) {
    const ChainReq& R = p.r[chain_find_req(p, item)];
    const long long row = item - R.first;
    const int cols = R.dim[3];
    int i0, i1, i2;
    chain_row_index(R, row, &i0, &i1, &i2);
    float m = -INFINITY, s = 0.f;
    for (int c = threadIdx.x; c < cols; c += blockDim.x) {
      const float v = chain_eval(p, R, i0, i1, i2, c);
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
    for (int c = threadIdx.x; c < cols; c += blockDim.x) {
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
    const long long obase = R.out_off + row * cols;
    for (int c = threadIdx.x; c < cols; c += blockDim.x) {
      const float v = p.red == RED_SOFTMAX ? rowbuf[c] * st1 : (rowbuf[c] - st0) * st1 * chain_gb(p, p.gamma, c) + chain_gb(p, p.beta, c);
      chain_store1(p, obase + c, v);
    }
    __syncthreads();
  }
}

}  // namespace k
}  // namespace sod2
