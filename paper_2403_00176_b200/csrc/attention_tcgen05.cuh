// Fused attention group on tcgen05 / TMEM for packed variable-length requests, head dim 64:
//   O = softmax(Q K^T * scale) V  per (request, head), bf16 in / fp32 accumulate / bf16 out.
// The score and probability tensors never reach global memory (the fusion argument of Section 4.2).
// One CTA owns 128 query rows of one (request, head) and walks the request's keys in blocks of 128:
//   S_j = Q K_j^T          tcgen05.mma, M=128, N=128, K=64; Q and K_j are K-major TMA tiles
//   P_j = exp2(S_j*c - m)  softmax threads: two threads per query row, each owns 64 of the block's 128
//                          score columns and reads them from TMEM in two 32-column halves, twice: once for
//                          the row maximum, once for the exponentials (a TMEM read is cheaper than holding
//                          64 scores in registers at two CTAs per SM); P_j goes as packed bf16 pairs into 64
//                          columns of TMEM (tcgen05.st: each thread its own row)
//   O  += P_j V_j          tcgen05.mma with the A operand in TMEM, M=128, N=64, K=128; V_j is the natural
//                          [key, d] tile, used as an MN-major B operand
//   (O *= corr)            only when a block's maximum moves the exponent reference by more than 2^8
// A block of 128 keys halves the number of hand-overs per key (barrier round trips, the row-maximum
// exchange, the P hand-over cost about as much as the exponentials of 64 keys).  S (128 columns), O (64) and P (64)
// live in TMEM -- handing P over through shared memory (32 KB of stores per block, a proxy fence) took 680-750 cycles
// of a 3300-cycle block, through TMEM 180 --; S is single buffered: the softmax threads release it after their last read,
// about half way through the block, and the next S = Q K^T runs under the second half of the
// exponentials (tried: half of them as a cubic on the FMA pipe -- slower, the block is bound by issue slots and
// latencies at 80 registers, not by the special-function pipe).  K and P are single buffered, V double buffered; two
// CTAs share an SM.
// Q, K, V are 2-D tensor maps over the packed [tokens, row stride] buffers; a tile that runs past a
// request's rows reads the next request's rows (finite data) or zeros past the end of the buffer, and
// those keys are masked to -inf before the softmax; query rows past the request are never written.
// Warps: 0 TMA, 1 issues S = Q K^T, 10 issues O = P V, 2..9 softmax (warp w reads TMEM lane quarter
// w % 4; two threads per row).
// Every wait is bounded (ptx.cuh).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include "ptx.cuh"

namespace sod2 {
namespace k {

constexpr int ATC_MAX_REQ = 32;
constexpr int ATC_THREADS = 352;
struct AtcReq {
  int L;                       // tokens of this request
  int q_row, k_row, v_row;     // first row of the request in the Q / K / V tensor maps
  long long o_off;             // element offset of the request's output view
};
struct AtcParams {
  __nv_bfloat16* o;
  int n_req, H;
  int q_col, k_col, v_col;     // column of head 0 in the Q / K / V tensor maps
  int q_hs, k_hs, v_hs;        // head strides in columns
  int o_ts, o_hs;              // output token / head strides in elements (multiples of 8)
  float scale_log2e;
  int* status;
  int tile_start[ATC_MAX_REQ + 1];   // prefix sum of ceil(L / 128); requests in descending L
  AtcReq r[ATC_MAX_REQ];
};

constexpr int ATC_KB = 128;               // keys per block
constexpr int ATC_Q_BYTES = 128 * 128;    // 128 rows x 64 bf16
constexpr int ATC_KV_BYTES = ATC_KB * 128;   // 128 keys x 64 bf16
constexpr int ATC_O_BYTES = 128 * 128;       // output staging: 128 rows x 64 bf16
constexpr int ATC_SMEM = ATC_Q_BYTES + 3 * ATC_KV_BYTES + ATC_O_BYTES + 2048 /*row maxima*/ + 1024 /*align*/ + 256 /*barriers*/;
constexpr uint32_t ATC_TMEM_S = 0, ATC_TMEM_O = 128, ATC_TMEM_P = 192;   // columns: scores, output, probabilities (packed bf16 pairs)

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__global__ void __launch_bounds__(ATC_THREADS, 2)
attention_tcgen05_bf16(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                       const __grid_constant__ CUtensorMap tmV, const __grid_constant__ AtcParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = base;
  uint8_t* sK = sQ + ATC_Q_BYTES;
  uint8_t* sV = sK + ATC_KV_BYTES;          // [2]
  uint8_t* sO = sV + 2 * ATC_KV_BYTES;
  float* xmax = reinterpret_cast<float*>(sO + ATC_O_BYTES);   // [block parity][column half][row]
  uint64_t* bars = reinterpret_cast<uint64_t*>(xmax + 512);
  uint64_t* q_full = bars;            // 1
  uint64_t* k_full = bars + 1;        // K_j landed (one phase per block)
  uint64_t* v_full = bars + 2;        // [2] V_j landed
  uint64_t* s_full = bars + 4;        // S_j done (also: the K buffer is free)
  uint64_t* s_free = bars + 5;        // softmax warps have read S_j for the last time
  uint64_t* p_full = bars + 6;        // softmax warps have written P_j
  uint64_t* o_full = bars + 7;        // [2] O_j done (also: V stage j & 1 and the P buffer are free)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 9);
  volatile int* dead = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // work item: blockIdx.x = tile * H + head, tiles ordered by descending request length
  const int tile = blockIdx.x / p.H, head = blockIdx.x % p.H;
  int ri = 0;
  while (ri + 1 < p.n_req && tile >= p.tile_start[ri + 1]) ++ri;
  const AtcReq& R = p.r[ri];
  const int L = R.L;
  const int q0 = (tile - p.tile_start[ri]) * 128;
  const int nkv = (L + ATC_KB - 1) / ATC_KB;

  if (threadIdx.x == 0) {
    ptx::mbar_init(q_full, 1);
    ptx::mbar_init(k_full, 1); ptx::mbar_init(s_full, 1); ptx::mbar_init(s_free, 8); ptx::mbar_init(p_full, 8);
    for (int b = 0; b < 2; ++b) { ptx::mbar_init(&v_full[b], 1); ptx::mbar_init(&o_full[b], 1); }
    *dead = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
    ptx::prefetch_tmap(&tmQ);
    ptx::prefetch_tmap(&tmK);
    ptx::prefetch_tmap(&tmV);
  }
  if (warp == 1) { ptx::tmem_alloc(tmem_slot, 256); ptx::tmem_relinquish(); }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  ptx::pdl_launch();
  if (threadIdx.x == 0) { SOD2_TRACE(0, 1) }

  if (warp == 0) {
    if (lane == 0) {
      // ---- TMA producer
      ptx::pdl_wait();
      ptx::mbar_expect_tx(q_full, ATC_Q_BYTES);
      ptx::tma_load_2d(sQ, &tmQ, p.q_col + head * p.q_hs, R.q_row + q0, q_full);
      for (int j = 0; j < nkv; ++j) {
        const int b = j & 1;
        if (j >= 1) ptx::mbar_wait(s_full, (j - 1) & 1, dead);               // S_{j-1} done: the K buffer is free
        ptx::mbar_expect_tx(k_full, ATC_KV_BYTES);
        ptx::tma_load_2d(sK, &tmK, p.k_col + head * p.k_hs, R.k_row + j * ATC_KB, k_full);
        if (j >= 2) ptx::mbar_wait(&o_full[b], ((j >> 1) - 1) & 1, dead);    // O_{j-2} done: V stage free
        ptx::mbar_expect_tx(&v_full[b], ATC_KV_BYTES);
        ptx::tma_load_2d(sV + b * ATC_KV_BYTES, &tmV, p.v_col + head * p.v_hs, R.v_row + j * ATC_KB, &v_full[b]);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---- S issuer: S_j = Q K_j^T.  A thread that waits on a barrier between MMAs stalls for a few
      // hundred cycles, so the two products get a thread each and one commit per block: "S_j done"
      // both publishes S_j and frees the K buffer.
      constexpr uint32_t idesc_qk = ptx::idesc_bf16(128, ATC_KB);
      const uint64_t dQ = ptx::smem_desc_sw128(ptx::smem_u32(sQ)), dK = ptx::smem_desc_sw128(ptx::smem_u32(sK));
      ptx::mbar_wait(q_full, 0, dead);
      for (int j = 0; j < nkv; ++j) {
        ptx::mbar_wait(k_full, j & 1, dead);
        if (j >= 1) ptx::mbar_wait(s_free, (j - 1) & 1, dead);
        ptx::tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) ptx::mma_bf16(tmem, dQ + 2 * kk, dK + 2 * kk, idesc_qk, kk != 0);
        ptx::mma_commit(s_full);
        SOD2_TRACE(1, 10 + j)
      }
    }
  } else if (warp == 10) {
    if (lane == 0) {
      // ---- O issuer: O += P_j V_j, accumulated in TMEM over the request's key blocks.  "O_j done" frees
      // the V stage and the P buffer.  The softmax warps rescale O (rarely) before they hand over P_j,
      // so the accumulator needs no barrier of its own.
      constexpr uint32_t idesc_pv = ptx::idesc_bf16(128, 64) | (1u << 16);   // B (= V tile) is MN-major
      for (int i = 0; i < nkv; ++i) {
        const int b = i & 1;
        ptx::mbar_wait(&v_full[b], (i >> 1) & 1, dead);
        ptx::mbar_wait(p_full, i & 1, dead);
        ptx::tc_fence_after();
        const uint32_t aV = ptx::smem_u32(sV + b * ATC_KV_BYTES);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)   // 16 keys per step: 8 packed columns of P in tensor memory, 16 rows (2048 B) down V
          ptx::mma_bf16_a_tmem(tmem + ATC_TMEM_O, tmem + ATC_TMEM_P + kk * 8, ptx::smem_desc_sw128(aV + kk * 2048), idesc_pv, (i | kk) != 0);
        ptx::mma_commit(&o_full[b]);
        SOD2_TRACE(1, 20 + i)
      }
    }
  } else {
    // ---- softmax warps 2..9: two threads per query row.  Warp w reads TMEM lane quarter w % 4; warps
    // 2..5 own score columns 0..31 of a block (and output columns 0..31), warps 6..9 the other half.
    // The two threads of a row exchange their partial row maximum through shared memory once per
    // block; the row sum stays split until the end.
    const int q = warp & 3;
    const int hh = (warp - 2) >> 2;
    const int row = q * 32 + lane;
    const bool warp_live = q0 + q * 32 < L;        // a warp whose 32 rows are all past the request only keeps the barriers moving
    const uint32_t lane_base = static_cast<uint32_t>(q * 32) << 16;
    const bool tracer = threadIdx.x == 64;
    ptx::pdl_wait();
    // Online softmax with a lazily updated reference: the exponent reference m only moves when a block's
    // row maximum exceeds it by more than 2^8 after scaling, so p stays <= 256 (exact enough in bf16 and
    // fp32) and the accumulator O in TMEM is rescaled only then -- for almost every block nothing is read
    // back from TMEM.  l and O always refer to the same m, so O / l at the end is the softmax average.
    float m = -INFINITY, l = 0.f;
    const float c = p.scale_log2e;
    const uint32_t o_addr = tmem + lane_base + ATC_TMEM_O + hh * 32;
    const uint32_t s_addr = tmem + lane_base + ATC_TMEM_S + hh * 64;      // this thread's 64 score columns of the block
    const uint32_t p_addr = tmem + lane_base + ATC_TMEM_P + hh * 32;      // ... and its 32 packed probability columns
    for (int j = 0; j < nkv; ++j) {
      const int b = j & 1;
      ptx::mbar_wait_warp(s_full, j & 1, dead);
      ptx::tc_fence_after();
      if (tracer) { SOD2_TRACE(2, 30 + j) }
      const int valid = L - j * ATC_KB - hh * 64;     // keys of this thread's 64 columns inside the request
      // ---- pass 1: partial row maximum on the raw scores (the scale is positive), both 32-column halves
      // (a 32-column half that lies entirely past the request is skipped in both passes: `valid` is uniform
      // over the warp)
      float mx = -INFINITY;
#pragma unroll
      for (int h2 = 0; h2 < 2; ++h2) {
        const int v2 = valid - h2 * 32;
        if (v2 > 0) {
          uint32_t s[32];
          ptx::tmem_ld32(s_addr + h2 * 32, s);
          ptx::tmem_ld_wait();
          if (v2 < 32) {
#pragma unroll
            for (int e = 0; e < 32; ++e) if (e >= v2) s[e] = 0xff800000u;
          }
          float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
          for (int e = 0; e < 32; e += 4) {
            mx0 = fmaxf(mx0, __uint_as_float(s[e])); mx1 = fmaxf(mx1, __uint_as_float(s[e + 1]));
            mx2 = fmaxf(mx2, __uint_as_float(s[e + 2])); mx3 = fmaxf(mx3, __uint_as_float(s[e + 3]));
          }
          mx = fmaxf(mx, fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)));
        }
      }
      xmax[(b * 2 + hh) * 128 + row] = mx;
      asm volatile("bar.sync 1, 256;" ::: "memory");
      const float mrow = fmaxf(mx, xmax[(b * 2 + (hh ^ 1)) * 128 + row]);
      if (tracer) { SOD2_TRACE(2, 60 + j) }
      // move the reference?  (both threads of a row, and both warps of a row group, decide alike)
      const bool move = warp_live && (mrow - m) * c > 8.0f;
      float corr = 1.f;
      if (move) { corr = ex2_approx((m - mrow) * c); m = mrow; l *= corr; }
      if (j > 0 && __any_sync(0xffffffffu, move)) {
        // all products issued so far must have landed in O before it is scaled
        ptx::mbar_wait_warp(&o_full[(j - 1) & 1], ((j - 1) >> 1) & 1, dead);
        ptx::tc_fence_after();
        uint32_t r[32];
        ptx::tmem_ld32(o_addr, r);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * corr);
        ptx::tmem_st32(o_addr, r);
        ptx::tmem_st_wait();
        ptx::tc_fence_before();
      }
      // ---- pass 2: p = 2^(s*c - m*c), 32 columns at a time: the scale rides in the FMA that feeds ex2.  The
      // special-function pipe (16 results per clock per SM) bounds this loop.
      const float mc = -m * c;
      float sum0 = 0.f, sum1 = 0.f;
      uint32_t pk[2][16];
#pragma unroll
      for (int h2 = 0; h2 < 2; ++h2) {
        const int v2 = valid - h2 * 32;
        uint32_t s[32];
        if (v2 > 0) {
          ptx::tmem_ld32(s_addr + h2 * 32, s);
          ptx::tmem_ld_wait();
        }
        if (h2 == 1) {
          // last read of S_j: the next S = Q K^T may overwrite it
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(s_free);
        }
        if (v2 > 0) {
          if (v2 < 32) {
#pragma unroll
            for (int e = 0; e < 32; ++e) if (e >= v2) s[e] = 0xff800000u;   // -inf
          }
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            const float p0 = ex2_approx(fmaf(__uint_as_float(s[e]), c, mc)), p1 = ex2_approx(fmaf(__uint_as_float(s[e + 1]), c, mc));
            sum0 += p0; sum1 += p1;
            const __nv_bfloat162 pb = __floats2bfloat162_rn(p0, p1);
            pk[h2][e >> 1] = warp_live ? *reinterpret_cast<const uint32_t*>(&pb) : 0u;
          }
        } else {
#pragma unroll
          for (int e = 0; e < 16; ++e) pk[h2][e] = 0u;
        }
      }
      l += sum0 + sum1;
      if (tracer) { SOD2_TRACE(2, 40 + j) }
      // P_j into tensor memory (32 columns of packed bf16 pairs per thread: its 64 keys) once the MMA that read the
      // P columns for the last block has finished; the product reads it from there as its A operand
      if (j >= 1) ptx::mbar_wait_warp(&o_full[(j - 1) & 1], ((j - 1) >> 1) & 1, dead);    // O_{j-1} done: the P columns are free
      ptx::tc_fence_after();
      ptx::tmem_st32(p_addr, &pk[0][0]);
      ptx::tmem_st_wait();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(p_full);
      if (tracer) { SOD2_TRACE(2, 50 + j) }
    }
    // ---- output: O / l.  The row sums of the two halves are added through shared memory, the scaled rows
    // are staged (swizzled) in shared memory and written four full 128-byte rows per instruction.
    {
      ptx::mbar_wait_warp(&o_full[(nkv - 1) & 1], ((nkv - 1) >> 1) & 1, dead);   // every product has landed
      ptx::tc_fence_after();
      uint32_t r[32];
      ptx::tmem_ld32(o_addr, r);
      ptx::tmem_ld_wait();
      ptx::tc_fence_before();
      if (tracer) { SOD2_TRACE(2, 70) }
      xmax[hh * 128 + row] = l;
      asm volatile("bar.sync 1, 256;" ::: "memory");
      const float lt = l + xmax[(hh ^ 1) * 128 + row];
      const float inv = warp_live ? 1.0f / lt : 0.f;
      uint8_t* prow = sO + row * 128;
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        uint4 v;
        __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
        for (int i = 0; i < 4; ++i) h2[i] = __floats2bfloat162_rn(__uint_as_float(r[g * 8 + 2 * i]) * inv, __uint_as_float(r[g * 8 + 2 * i + 1]) * inv);
        *reinterpret_cast<uint4*>(prow + (((hh * 4 + g) ^ (row & 7)) << 4)) = v;
      }
      asm volatile("bar.sync 1, 256;" ::: "memory");
      __nv_bfloat16* og = p.o + R.o_off + static_cast<long long>(head) * p.o_hs;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int rr = q * 32 + hh * 16 + i * 4 + (lane >> 3), ch = lane & 7;
        const uint4 v = *reinterpret_cast<const uint4*>(sO + rr * 128 + ((ch ^ (rr & 7)) << 4));
        if (q0 + rr < L) *reinterpret_cast<uint4*>(og + static_cast<long long>(q0 + rr) * p.o_ts + ch * 8) = v;
      }
    }
  }
  if (threadIdx.x == 64) { SOD2_TRACE(2, 80) }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) ptx::tmem_dealloc(tmem, 256);
  if (threadIdx.x == 0 && *dead && p.status) atomicExch(p.status, 1);
  SOD2_TRACE_DUMP()
}

}  // namespace k
}  // namespace sod2
