// Self-test / measurement entry point: the issue rate of tcgen05.mma, for one CTA and for a CTA pair.
// One thread per CTA (or per pair) issues `iters` bf16 MMAs of shape 128 x N x 16 (256 x N x 16 for a pair) on
// operands that sit in shared memory for the whole run; nothing is loaded, the data is irrelevant.  Three issue
// patterns: MMAs only; a tcgen05.commit after every stage of `per_stage` instructions; the full / empty barrier
// handshake of the GEMM main loops (the issuing thread waits for `full`, commits to `empty`, a second thread waits
// for `empty` and arrives on `full`), whose waits are always satisfied at once.  The result says how much of the
// issuing thread's own work the tensor pipe overlaps: none of it (a stage costs its MMA cycles plus the wait, the
// fence and the commit), identically for both forms.  The paper has no counterpart of this call: it documents the
// machine facts the kernels were shaped by, and lets a test pin them.
// Every wait is bounded; a wait that runs out makes the call return SOD2_E_TIMEOUT.
#include <cuda_runtime.h>

#include <string>

#include "../../include/sod2.h"
#include "engine.h"
#include "gemm_pair_tcgen05.cuh"

namespace sod2 {
namespace {

constexpr int MR_SLOTS = 4;
constexpr int MR_SLOT_BYTES = 49152;       // A: 128 rows x 128 B, B: up to 256 rows x 128 B
constexpr int MR_SMEM = MR_SLOTS * MR_SLOT_BYTES + 1024 + 256;

template <int PAIR, int N, int HS>
__global__ void __launch_bounds__(128, 1) mma_rate_kernel(long long* out, int iters, int per_stage) {
  extern __shared__ uint8_t raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bar = reinterpret_cast<uint64_t*>(base + MR_SLOTS * MR_SLOT_BYTES);   // [0] done, [1] unobserved, [2..5] full, [6..9] empty
  uint32_t* slot = reinterpret_cast<uint32_t*>(bar + 10);
  volatile int* dead = reinterpret_cast<volatile int*>(slot + 1);
  for (int i = threadIdx.x; i < MR_SLOTS * MR_SLOT_BYTES / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(base)[i] = 0x3c003c00u;
  const uint32_t rank = k::cluster_ctarank();
  if (threadIdx.x == 0) {
    for (int q = 0; q < 10; ++q) ptx::mbar_init(bar + q, 1);
    *dead = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
  }
  if (threadIdx.x < 32) {
    if (PAIR) { k::tmem_alloc_pair(slot, 512); k::tmem_relinquish_pair(); }
    else { ptx::tmem_alloc(slot, 512); ptx::tmem_relinquish(); }
  }
  ptx::tc_fence_before();
  __syncthreads();
  k::cluster_sync_all();
  ptx::tc_fence_after();
  const uint32_t tmem = *slot;
  const bool issuer = threadIdx.x == 0 && (!PAIR || rank == 0);
  if (issuer) {
    constexpr uint32_t idesc = ptx::idesc_bf16(PAIR ? 256 : 128, N);
    const uint64_t ad0 = ptx::smem_desc_sw128(ptx::smem_u32(base)), bd0 = ptx::smem_desc_sw128(ptx::smem_u32(base + 16384));
    int sl = 0;
    uint32_t par = 0;
    const long long t0 = clock64();
    for (int it = 0; it < iters; it += per_stage) {
      const uint64_t off = static_cast<uint64_t>((sl * MR_SLOT_BYTES) >> 4);
      const int cur = sl;
      if (HS == 2) {
        ptx::mbar_wait(bar + 2 + cur, par, dead);
        ptx::tc_fence_after();
      }
      if (cur + 1 == MR_SLOTS) par ^= 1;
      sl = cur + 1 == MR_SLOTS ? 0 : cur + 1;
#pragma unroll 8
      for (int g = 0; g < per_stage; ++g) {
        if (PAIR) k::mma_bf16_pair(tmem, ad0 + off + 2 * (g & 3), bd0 + off + 2 * (g & 3), idesc, 1);
        else ptx::mma_bf16(tmem, ad0 + off + 2 * (g & 3), bd0 + off + 2 * (g & 3), idesc, 1);
      }
      if (HS == 1) { if (PAIR) k::mma_commit_pair(bar + 1); else ptx::mma_commit(bar + 1); }
      if (HS == 2) { if (PAIR) k::mma_commit_pair(bar + 6 + cur); else ptx::mma_commit(bar + 6 + cur); }
    }
    if (PAIR) k::mma_commit_pair(bar); else ptx::mma_commit(bar);
    ptx::mbar_wait(bar, 0, dead);
    const long long t1 = clock64();
    out[blockIdx.x * 2] = t1 - t0;
  } else if (threadIdx.x == 0) {
    ptx::mbar_wait(bar, 0, dead);          // the odd CTA of a pair: the last commit reaches both CTAs
  } else if (threadIdx.x == 32 && HS == 2) {
    // the "producer": waits for a slot to be free and declares it full (the odd CTA of a pair only waits, as in the GEMM)
    int n = 0;
    for (int it = 0; it < iters; it += per_stage, ++n) {
      const int s = n % MR_SLOTS;
      if (n >= MR_SLOTS) ptx::mbar_wait(bar + 6 + s, ((n / MR_SLOTS) - 1) & 1, dead);
      if (!PAIR || rank == 0) ptx::mbar_arrive(bar + 2 + s);
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) out[blockIdx.x * 2 + 1] = *dead;
  k::cluster_sync_all();
  if (threadIdx.x < 32) { if (PAIR) k::tmem_dealloc_pair(tmem, 512); else ptx::tmem_dealloc(tmem, 512); }
}

template <int PAIR, int N, int HS>
cudaError_t launch_rate(long long* out, int iters, int per_stage, int clusters, cudaStream_t st) {
  auto kern = mma_rate_kernel<PAIR, N, HS>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, MR_SMEM);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * clusters);
  cfg.blockDim = dim3(128);
  cfg.dynamicSmemBytes = MR_SMEM;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, out, iters, per_stage);
}

template <int PAIR, int N>
cudaError_t launch_rate_hs(int hs, long long* out, int iters, int per_stage, int clusters, cudaStream_t st) {
  switch (hs) {
    case 0: return launch_rate<PAIR, N, 0>(out, iters, per_stage, clusters, st);
    case 1: return launch_rate<PAIR, N, 1>(out, iters, per_stage, clusters, st);
    default: return launch_rate<PAIR, N, 2>(out, iters, per_stage, clusters, st);
  }
}

}  // namespace
}  // namespace sod2

extern "C" sod2_status sod2_selftest_mma_rate(int pair, int n_cols, int per_stage, int handshake, int iters, int clusters,
                                              void* cuda_stream, double* cycles_per_mma) {
  using namespace sod2;
  auto fail = [&](sod2_status s, const std::string& m) { set_thread_error(m); return s; };
  if (!cycles_per_mma) return fail(SOD2_E_INVALID_ARG, "sod2_selftest_mma_rate: null result pointer");
  if (n_cols != 64 && n_cols != 128 && n_cols != 256) return fail(SOD2_E_INVALID_ARG, "sod2_selftest_mma_rate: n_cols must be 64, 128 or 256");
  if (per_stage < 1 || per_stage > 64 || iters < per_stage || iters > (1 << 16) || iters % per_stage || handshake < 0 || handshake > 2 ||
      clusters < 1 || clusters > 74)
    return fail(SOD2_E_INVALID_ARG, "sod2_selftest_mma_rate: per_stage in 1..64 dividing iters <= 65536, handshake in 0..2, clusters in 1..74");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  long long* out = nullptr;
  const size_t bytes = static_cast<size_t>(2 * clusters) * 2 * sizeof(long long);
  if (cudaMalloc(&out, bytes) != cudaSuccess) return fail(SOD2_E_CUDA, "sod2_selftest_mma_rate: cudaMalloc failed");
  cudaMemsetAsync(out, 0, bytes, st);
  cudaError_t e = cudaSuccess;
  for (int rep = 0; rep < 2 && e == cudaSuccess; ++rep) {      // the second launch is the measured one (warm instruction cache)
    if (pair) {
      e = n_cols == 256 ? launch_rate_hs<1, 256>(handshake, out, iters, per_stage, clusters, st)
        : n_cols == 128 ? launch_rate_hs<1, 128>(handshake, out, iters, per_stage, clusters, st)
                        : launch_rate_hs<1, 64>(handshake, out, iters, per_stage, clusters, st);
    } else {
      e = n_cols == 256 ? launch_rate_hs<0, 256>(handshake, out, iters, per_stage, clusters, st)
        : n_cols == 128 ? launch_rate_hs<0, 128>(handshake, out, iters, per_stage, clusters, st)
                        : launch_rate_hs<0, 64>(handshake, out, iters, per_stage, clusters, st);
    }
  }
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  long long h[4] = {0, 0, 0, 0};
  if (e == cudaSuccess) e = cudaMemcpy(h, out, sizeof(h), cudaMemcpyDeviceToHost);
  cudaFree(out);
  if (e != cudaSuccess) return fail(SOD2_E_CUDA, std::string("sod2_selftest_mma_rate: ") + cudaGetErrorString(e));
  if (h[1] || h[3]) return fail(SOD2_E_TIMEOUT, "sod2_selftest_mma_rate: a bounded wait ran out");
  *cycles_per_mma = static_cast<double>(h[0]) / iters;
  return SOD2_OK;
}
