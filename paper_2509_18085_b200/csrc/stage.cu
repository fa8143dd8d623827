// Staging of logits rows: copies, from memory the device can read (pinned host
// memory mapped into the device's address space, or device memory), only the
// rows whose position is still masked -- the rows the decision step will read.
// One kernel instead of one copy per run of rows: over the bus a copy command
// costs about as much as a whole row of a 126k-entry vocabulary.
#include "common.cuh"

namespace spiffy {
namespace {

constexpr int kStageThreads = 256;
constexpr int kStageUnroll = 8;  // 16-byte loads in flight per thread

// grid = (chunks per row, rows); a CTA copies kStageThreads * kStageUnroll vectors of its row
__global__ void __launch_bounds__(kStageThreads)
stage_masked_rows_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, int64_t row_vecs,
                         const int32_t* __restrict__ tokens, int mask_id) {
#if __CUDA_ARCH__ >= 900
  cudaGridDependencySynchronize();  // the destination may still be read by an earlier kernel
#endif
  const int64_t row = blockIdx.y;
  if (tokens[row] != mask_id) return;
  const uint4* s = src + row * row_vecs;
  uint4* d = dst + row * row_vecs;
  const int64_t base = (int64_t)blockIdx.x * kStageThreads * kStageUnroll + threadIdx.x;
  uint4 v[kStageUnroll];
#pragma unroll
  for (int u = 0; u < kStageUnroll; ++u) {
    const int64_t i = base + (int64_t)u * kStageThreads;
    if (i < row_vecs)
      asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                   : "=r"(v[u].x), "=r"(v[u].y), "=r"(v[u].z), "=r"(v[u].w)
                   : "l"(s + i));
  }
#pragma unroll
  for (int u = 0; u < kStageUnroll; ++u) {
    const int64_t i = base + (int64_t)u * kStageThreads;
    if (i < row_vecs) d[i] = v[u];
  }
}

}  // namespace

spiffy_status launch_stage_masked_rows(const void* src, void* dst, int64_t row_bytes,
                                       const int32_t* tokens, int32_t mask_id, int64_t n_rows,
                                       cudaStream_t stream) {
  const int64_t row_vecs = row_bytes / 16;
  const int64_t per_cta = (int64_t)kStageThreads * kStageUnroll;
  const dim3 grid((unsigned)((row_vecs + per_cta - 1) / per_cta), (unsigned)n_rows);
  const cudaError_t e = launch_pdl(stage_masked_rows_kernel, grid, dim3(kStageThreads), (size_t)0, stream,
                                   static_cast<const uint4*>(src), static_cast<uint4*>(dst), row_vecs,
                                   tokens, (int)mask_id);
  count_launch();
  return e == cudaSuccess ? SPIFFY_OK : SPIFFY_ECUDA;
}

}  // namespace spiffy
