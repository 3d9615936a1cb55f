// NonZero for callers that cannot allocate device memory.
//
// Some callers of this library are not allowed to call cudaMalloc at all: code that runs inside a
// CUDA-graph capture or a latency-critical serving loop where an allocation would synchronise the
// device, plug-ins whose host framework owns every byte of device memory and hands out only the
// input and output buffers, and processes running under a fixed memory budget.  The regular path
// takes its scratch from the caller's arena; this entry point needs no arena: the per-block counters
// of the compaction live in a fixed array inside the library's device image.
//
// Consequences of that design, all of which the header repeats:
//  - the input is limited to SOD2_NONZERO_STATIC_MAX_ELEMS elements (larger inputs are rejected);
//  - every GPU that loads the library holds the array (about 65 KB) until the process exits;
//  - all calls share the array, which keeps the previous call's contents.  Nothing in it has to
//    start at zero: each call overwrites every counter it later reads.  Two calls that overlap on
//    the GPU (different streams, or two host threads) race on it;
//  - the first call on each device looks up the array's device address (cudaGetSymbolAddress);
//    make that first call outside of any stream capture.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include "ptx.cuh"

#include <cstdint>
#include <string>

#include "../../include/sod2.h"
#include "engine.h"

namespace {

constexpr int NZS_BLOCK = 1024;
constexpr long long NZS_MAX_ELEMS = SOD2_NONZERO_STATIC_MAX_ELEMS;
constexpr int NZS_MAX_BLOCKS = static_cast<int>((NZS_MAX_ELEMS + NZS_BLOCK - 1) / NZS_BLOCK);

// Scratch: one counter per block of 1024 elements plus the total.  In host code this name is only a
// stand-in for the symbol, never a device address; the address comes from cudaGetSymbolAddress.
static __device__ __align__(256) int g_nzs_counters[NZS_MAX_BLOCKS + 64];

struct NzsParams {
  const void* x;
  int is_bf16;
  long long numel;
  int rank;
  long long dims[4];
  int* counters;        // device address of g_nzs_counters
  long long* out;       // [rank, nnz]
  long long* count_out;
  int nblocks;
};

__device__ __forceinline__ bool nzs_flag(const NzsParams& p, long long i) {
  if (i >= p.numel) return false;
  return p.is_bf16 ? (__bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p.x)[i]) != 0.0f)
                   : (reinterpret_cast<const float*>(p.x)[i] != 0.0f);
}

__global__ void __launch_bounds__(NZS_BLOCK) nzs_count(NzsParams p) {
  __shared__ int wc[32];
  const long long i = static_cast<long long>(blockIdx.x) * NZS_BLOCK + threadIdx.x;
  const unsigned bal = __ballot_sync(0xffffffffu, nzs_flag(p, i));
  if ((threadIdx.x & 31) == 0) wc[threadIdx.x >> 5] = __popc(bal);
  __syncthreads();
  if (threadIdx.x == 0) {
    int t = 0;
    for (int w = 0; w < 32; ++w) t += wc[w];
    p.counters[blockIdx.x] = t;
  }
}

// one CTA: exclusive scan of the block counters in place, total into counters[nblocks] and *count_out
__global__ void __launch_bounds__(1024) nzs_scan(NzsParams p) {
  __shared__ int wt[32];
  __shared__ int carry_s;
  if (threadIdx.x == 0) carry_s = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int base = 0; base < p.nblocks; base += 1024) {
    const int i = base + threadIdx.x;
    const int v = i < p.nblocks ? p.counters[i] : 0;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += t; }
    if (lane == 31) wt[warp] = inc;
    __syncthreads();
    int woff = 0;
    for (int w = 0; w < warp; ++w) woff += wt[w];
    const int carry = carry_s;
    if (i < p.nblocks) p.counters[i] = carry + woff + inc - v;
    __syncthreads();
    if (threadIdx.x == 1023) carry_s = carry + woff + inc;
    __syncthreads();
  }
  if (threadIdx.x == 0) { p.counters[p.nblocks] = carry_s; *p.count_out = carry_s; }
}

__global__ void __launch_bounds__(NZS_BLOCK) nzs_write(NzsParams p) {
  __shared__ int wc[32];
  const long long i = static_cast<long long>(blockIdx.x) * NZS_BLOCK + threadIdx.x;
  const bool f = nzs_flag(p, i);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned bal = __ballot_sync(0xffffffffu, f);
  if (lane == 0) wc[warp] = __popc(bal);
  __syncthreads();
  if (!f) return;
  int off = p.counters[blockIdx.x] + __popc(bal & ((1u << lane) - 1));
  for (int w = 0; w < warp; ++w) off += wc[w];
  const long long nnz = p.counters[p.nblocks];
  long long r = i;
  for (int d = p.rank - 1; d >= 0; --d) {
    p.out[static_cast<long long>(d) * nnz + off] = r % p.dims[d];
    r /= p.dims[d];
  }
}

// device address of the scratch array, per device; looked up once per device with that device current
int* g_nzs_addr[64] = {nullptr};

sod2_status nzs_fail(sod2_status s, const std::string& msg) {
  sod2::set_thread_error(msg);
  return s;
}

}  // namespace

extern "C" sod2_status sod2_nonzero_static(const void* dev_x, int dtype, int rank, const int64_t* dims, int64_t* dev_out,
                                           int64_t* dev_count, void* cuda_stream) {
  if (!dev_x || !dims || !dev_out || !dev_count) return nzs_fail(SOD2_E_INVALID_ARG, "sod2_nonzero_static: null pointer");
  if (dtype != 0 && dtype != 1) return nzs_fail(SOD2_E_INVALID_ARG, "sod2_nonzero_static: dtype must be 0 (f32) or 1 (bf16)");
  if (rank < 1 || rank > 4) return nzs_fail(SOD2_E_RANK_MISMATCH, "sod2_nonzero_static: rank must be 1..4");
  long long numel = 1;
  for (int i = 0; i < rank; ++i) {
    if (dims[i] < 0) return nzs_fail(SOD2_E_BAD_DIM, "sod2_nonzero_static: negative extent");
    // compared before multiplying: the product of two large extents would wrap around the 64-bit range and
    // pass as a small (or empty) input.  An extent of 0 anywhere makes the input empty, whatever the others are.
    if (numel > 0 && dims[i] > NZS_MAX_ELEMS / numel)
      return nzs_fail(SOD2_E_BAD_DIM, "sod2_nonzero_static: input has more than " + std::to_string(NZS_MAX_ELEMS) +
                                          " elements, the limit of the built-in scratch; use the arena-based path");
    numel *= dims[i];
  }
  // every extent is checked even when an earlier one is 0 (an empty input must still have sane extents)
  for (int i = 0; i < rank; ++i)
    if (dims[i] > NZS_MAX_ELEMS)
      return nzs_fail(SOD2_E_BAD_DIM, "sod2_nonzero_static: an extent exceeds " + std::to_string(NZS_MAX_ELEMS));
  // the scratch array of the device that owns the input (the stream must belong to the same device)
  int dev = 0;
  {
    cudaPointerAttributes at{};
    if (cudaPointerGetAttributes(&at, dev_x) == cudaSuccess && at.type == cudaMemoryTypeDevice) dev = at.device;
    else { cudaGetLastError(); if (cudaGetDevice(&dev) != cudaSuccess) return nzs_fail(SOD2_E_CUDA, "sod2_nonzero_static: no current device"); }
  }
  if (dev < 0 || dev >= 64) return nzs_fail(SOD2_E_CUDA, "sod2_nonzero_static: device index out of range");
  int cur = 0;
  if (cudaGetDevice(&cur) != cudaSuccess) return nzs_fail(SOD2_E_CUDA, "sod2_nonzero_static: no current device");
  if (cur != dev) return nzs_fail(SOD2_E_INVALID_ARG, "sod2_nonzero_static: the device that holds dev_x must be the current device");
  if (!g_nzs_addr[dev]) {
    int* ptr = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_nzs_counters);
    if (e != cudaSuccess || !ptr) return nzs_fail(SOD2_E_CUDA, std::string("sod2_nonzero_static: cudaGetSymbolAddress failed: ") + cudaGetErrorString(e));
    g_nzs_addr[dev] = ptr;
  }
  NzsParams p{};
  p.x = dev_x;
  p.is_bf16 = dtype;
  p.numel = numel;
  p.rank = rank;
  for (int i = 0; i < rank; ++i) p.dims[i] = dims[i];
  p.counters = g_nzs_addr[dev];
  p.out = reinterpret_cast<long long*>(dev_out);
  p.count_out = reinterpret_cast<long long*>(dev_count);
  p.nblocks = static_cast<int>((numel + NZS_BLOCK - 1) / NZS_BLOCK);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (p.nblocks) nzs_count<<<p.nblocks, NZS_BLOCK, 0, st>>>(p);
  nzs_scan<<<1, 1024, 0, st>>>(p);   // also writes the count when the input is empty
  if (p.nblocks) nzs_write<<<p.nblocks, NZS_BLOCK, 0, st>>>(p);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return nzs_fail(SOD2_E_CUDA, std::string("sod2_nonzero_static: launch failed: ") + cudaGetErrorString(e));
  return SOD2_OK;
}

namespace {
__global__ void empty_kernel() {}

// One warp waits, with the library's bounded wait and a limit of a few thousand polls, on a barrier that
// nothing ever arrives on; the wait runs out, raises the CTA's flag and the kernel records it in the status
// word exactly as the tensor-core kernels do, then returns.
__global__ void bounded_wait_selftest(int* status) {
  __shared__ uint64_t bar;
  __shared__ int dead;
  if (threadIdx.x == 0) {
    dead = 0;
    sod2::ptx::mbar_init(&bar, 1);
    sod2::ptx::fence_barrier_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) sod2::ptx::mbar_wait_limited(&bar, 0, &dead, 4096u);
  __syncthreads();
  if (threadIdx.x == 0 && dead && status) atomicExch(status, 1);
}
}  // namespace

extern "C" sod2_status sod2_selftest_bounded_wait(void* dev_status_word, void* cuda_stream) {
  if (!dev_status_word) return nzs_fail(SOD2_E_INVALID_ARG, "sod2_selftest_bounded_wait: null status word");
  bounded_wait_selftest<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(static_cast<int*>(dev_status_word));
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return nzs_fail(SOD2_E_CUDA, std::string("sod2_selftest_bounded_wait: launch failed: ") + cudaGetErrorString(e));
  return SOD2_OK;
}

extern "C" sod2_status sod2_launch_empty(void* cuda_stream) {
  empty_kernel<<<1, 1, 0, static_cast<cudaStream_t>(cuda_stream)>>>();
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return nzs_fail(SOD2_E_CUDA, std::string("sod2_launch_empty: launch failed: ") + cudaGetErrorString(e));
  return SOD2_OK;
}
