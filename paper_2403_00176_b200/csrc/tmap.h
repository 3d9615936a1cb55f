// Host-side TMA tensor-map encoding. The driver entry point is looked up at run time
// through the CUDA runtime, so the library links against cudart only and still loads on a
// machine without a driver.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>

namespace sod2 {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// Row-major bf16 matrix [rows, cols] with row pitch ld elements; box = [box_rows, 64 cols], 128-B swizzle.
// Requirements: base 16-B aligned, ld*2 a multiple of 16. Returns false on failure.
inline bool encode_bf16_2d(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint64_t ld,
                           uint32_t box_rows, uint32_t box_cols = 64) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {ld * 2};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// `slabs` row-major fp32 matrices [rows, cols] back to back, as {cols, rows, slabs}; box = {32 cols
// (128-byte rows), box_rows, 1}, 128-B swizzle.  Rows past `rows` are clipped per slab.
inline bool encode_f32_slabs(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint64_t slabs, uint32_t box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {cols, rows, slabs};
  cuuint64_t strides[2] = {cols * 4, rows * cols * 4};
  cuuint32_t box[3] = {32, box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Row-major bf16 matrix [rows, K] (K % 64 == 0) viewed as {64, rows, K/64}: the third coordinate
// walks the 64-element k-chunks of a row, so one box {64, box_rows, kch} fills kch consecutive
// swizzled [box_rows x 64] chunk tiles in shared memory.
inline bool encode_bf16_kchunks(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t K, uint64_t ld,
                                uint32_t box_rows, uint32_t kch) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn || K % 64) return false;
  cuuint64_t dims[3] = {64, rows, K / 64};
  cuuint64_t strides[2] = {ld * 2, 128};
  cuuint32_t box[3] = {64, box_rows, kch};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Channels-last activation [N, H, W, C] bf16 viewed as {C, W, H, N}; box = 64 channels x (box_w x box_h)
// pixels of one image, 128-byte swizzle; `stride` is the traversal stride along W and H (strided
// convolutions): the box spans box_w*stride x box_h*stride source pixels and loads every stride-th.
inline bool encode_bf16_nhwc(CUtensorMap* tm, const void* base, uint64_t N, uint64_t H, uint64_t W, uint64_t C,
                             uint32_t box_w, uint32_t box_h, uint32_t stride) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn || C % 8) return false;
  cuuint64_t dims[4] = {C, W, H, N};
  cuuint64_t strides[3] = {C * 2, W * C * 2, H * W * C * 2};
  cuuint32_t box[4] = {64, box_w * stride, box_h * stride, 1};
  cuuint32_t estr[4] = {1, stride, stride, 1};
  if (box[1] > 256 || box[2] > 256) return false;
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Planes of rows: bf16 [planes, H, W] (e.g. an NCHW tensor with planes = N * C) viewed as {W, H, planes};
// box = {box_w columns, box_h rows, 1 plane}, no swizzle.  Requirements: W % 8 == 0, box_w % 8 == 0.
inline bool encode_bf16_planes(CUtensorMap* tm, const void* base, uint64_t planes, uint64_t H, uint64_t W, uint32_t box_w, uint32_t box_h) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn || W % 8 || box_w % 8 || box_w > 256 || box_h > 256) return false;
  cuuint64_t dims[3] = {W, H, planes};
  cuuint64_t strides[2] = {W * 2, H * W * 2};
  cuuint32_t box[3] = {box_w, box_h, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace sod2
