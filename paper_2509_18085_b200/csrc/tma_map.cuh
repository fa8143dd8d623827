// Host side of the TMA tile loads: the tensor-map encoder (a driver entry point
// fetched through the runtime, so that the library does not link the driver
// library) and the one tensor shape every tensor-core kernel of this library
// reads.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

namespace spiffy {
namespace {

constexpr int kMapInner = 128;  // bf16 elements of the innermost rows (a head row; 128 columns of a matrix)

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess)
      f = nullptr;
    return reinterpret_cast<EncodeTiledFn>(f);
  }();
  return fn;
}

// Tensor [outer][rows][heads][128] of bf16 (equally: a [rows][heads * 128] matrix) seen as a
// 4-D TMA tensor with the 64-element half of a head row innermost; box = 64 x box_heads x
// box_rows x 1.
// `outer_stride_rows`: rows between consecutive outer slices (0 = densely packed, i.e. `rows`);
// larger when the tensor is a window of `rows` rows into a longer one.
bool make_map(CUtensorMap* m, const void* base, int heads, int64_t rows, int outer, int box_heads,
              int box_rows, int64_t outer_stride_rows = 0) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return false;
  if (outer_stride_rows <= 0) outer_stride_rows = rows;
  const cuuint64_t dims[4] = {(cuuint64_t)kMapInner, (cuuint64_t)heads, (cuuint64_t)rows, (cuuint64_t)outer};
  const cuuint64_t strides[3] = {(cuuint64_t)kMapInner * 2, (cuuint64_t)heads * kMapInner * 2,
                                 (cuuint64_t)outer_stride_rows * heads * kMapInner * 2};
  const cuuint32_t box[4] = {64, (cuuint32_t)box_heads, (cuuint32_t)box_rows, 1};
  const cuuint32_t es[4] = {1, 1, 1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box,
             es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace
}  // namespace spiffy
