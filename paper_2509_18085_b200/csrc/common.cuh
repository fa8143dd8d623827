// Internal helpers shared by the kernels of libspiffy (not part of the ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "spiffy.h"

namespace spiffy {

constexpr float kLog2e = 1.4426950408889634f;

// 2^x on the special-function unit (approximate, denormals flushed).
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Two fp32 lanes in one 64-bit register: Blackwell issues their multiply-add and
// their add as one instruction each (for loops bound by instruction issue).
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
// 128-bit streaming load: read-only path, no L1 allocation (data used once).
__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// Every launch of the library goes through this counter (spiffy_launch_count).
void count_launch(int n = 1);

// Poll limits of the bounded device-side waits, read at launch.  The defaults
// (about a fraction of a second) change only through spiffy_set_wait_limits,
// which exists so that the give-up paths can be exercised.
uint32_t mbar_poll_limit();   // polls of one mbarrier wait (tensor-core kernels)
uint32_t flag_poll_limit();   // polls of one wait on a global-memory word (lazy call)
int32_t lazy_extra_arrivals();  // arrivals sequence 0's tail expects beyond those that can come

// Entry points implemented in the kernel files; all validated by the caller.
spiffy_status launch_decide(const spiffy_decide_desc& d, const void* logits,
                            const int32_t* block_tokens, float* conf,
                            int32_t* top_tok, uint64_t* unmask_bits,
                            int32_t* n_unmask, int32_t* dev_status, void* ws,
                            cudaStream_t stream);
size_t decide_workspace_bytes(const spiffy_decide_desc& d);
int decide_splits(const spiffy_decide_desc& d, int64_t* chunk_elems);

spiffy_status launch_walk(const spiffy_decide_desc& d,
                          const int32_t* block_tokens,
                          const int32_t* parent_off, const int32_t* parent_idx,
                          int32_t parent_cap, const int32_t* top_tok,
                          const uint64_t* unmask_bits, int32_t* accepted_node,
                          int32_t* n_accepted, int32_t* path,
                          int32_t* next_block, int32_t* dev_status,
                          cudaStream_t stream);

spiffy_status launch_decide_walk(const spiffy_decide_desc& d, const void* logits,
                                 const int32_t* block_tokens, float* conf, int32_t* top_tok,
                                 uint64_t* unmask_bits, int32_t* n_unmask,
                                 int32_t* decide_status, const int32_t* parent_off,
                                 const int32_t* parent_idx, int32_t parent_cap,
                                 int32_t* accepted_node, int32_t* n_accepted, int32_t* path,
                                 int32_t* next_block, int32_t* walk_status, void* ws,
                                 cudaStream_t stream);

size_t decide_lazy_workspace_bytes(const spiffy_decide_desc& d);
spiffy_status launch_decide_walk_lazy(const spiffy_decide_desc& d, const void* logits,
                                      const int32_t* block_tokens, float* conf, int32_t* top_tok,
                                      uint64_t* unmask_bits, int32_t* n_unmask,
                                      int32_t* decide_status, const int32_t* parent_off,
                                      const int32_t* parent_idx, int32_t parent_cap,
                                      int32_t* accepted_node, int32_t* n_accepted, int32_t* path,
                                      int32_t* next_block, int32_t* walk_status, void* ws,
                                      cudaStream_t stream);

spiffy_status launch_stage_masked_rows(const void* src, void* dst, int64_t row_bytes,
                                       const int32_t* tokens, int32_t mask_id, int64_t n_rows,
                                       cudaStream_t stream);

size_t decide_sampled_workspace_bytes(const spiffy_decide_desc& d);
spiffy_status launch_decide_sampled(const spiffy_decide_desc& d, float temperature, uint64_t seed,
                                    const void* logits, const int32_t* block_tokens, float* conf,
                                    int32_t* top_tok, uint64_t* unmask_bits, int32_t* n_unmask,
                                    int32_t* dev_status, void* ws, cudaStream_t stream);

spiffy_status launch_decide_finalize(const spiffy_decide_desc& d, const void* partials, int splits,
                                     const int32_t* block_tokens, float* conf, int32_t* top_tok,
                                     uint64_t* unmask_bits, int32_t* n_unmask, int32_t* dev_status,
                                     cudaStream_t stream);
int lmhead_grid(const spiffy_decide_desc& d);
size_t lmhead_workspace_bytes(const spiffy_decide_desc& d, int grid);
spiffy_status launch_lmhead_decide(const spiffy_decide_desc& d, int hidden, const void* hstates,
                                   const void* weight, const int32_t* block_tokens, float* conf,
                                   int32_t* top_tok, uint64_t* unmask_bits, int32_t* n_unmask,
                                   int32_t* dev_status, void* ws, cudaStream_t stream);

spiffy_status launch_attention_simt(const spiffy_attn_desc& d, const void* q,
                                    const void* kp, const void* vp,
                                    const void* kb, const void* vb, void* out,
                                    cudaStream_t stream);

size_t draft_workspace_bytes(const spiffy_draft_desc& d);
spiffy_status launch_draft(const spiffy_draft_desc& d, const void* logits, const int32_t* state,
                           const int32_t* formula_off, const int32_t* formula_i,
                           const int32_t* formula_j, const int32_t* child_off,
                           const int32_t* child_idx, int32_t* tokens, int32_t* kept, float* score,
                           int32_t* parent_off, int32_t* parent_idx, int32_t* dev_status, void* ws,
                           cudaStream_t stream);

// tcgen05 path: shape support query, workspace and launch.  The cached context
// comes as up to two segments of keys/values, [B][len][Hkv][d] each, whose
// sequences may lie `batch_stride_rows` rows apart (0: densely packed).
struct AttnContext {
  const void* k;
  const void* v;
  int len;
  int64_t batch_stride_rows;
};
bool attention_tc_supported(const spiffy_attn_desc& d);
size_t attention_tc_workspace_bytes(const spiffy_attn_desc& d, int ctx2_len);
spiffy_status launch_attention_tc(const spiffy_attn_desc& d, const void* q, const AttnContext& ctx,
                                  const AttnContext& ctx2, const void* kb, const void* vb, void* out,
                                  int32_t* dev_status, void* ws, cudaStream_t stream);

// Launch with programmatic stream serialisation: the kernel may be scheduled
// while its predecessor in the stream is still draining.  Every kernel launched
// this way calls cudaGridDependencySynchronize() before it writes global memory
// or reads what the calls of one step hand to each other (logits, partial
// results, top tokens, unmask sets).  The walk, tail and draft-build kernels
// fetch the graph arrays (block states, parent lists, draft formulas) ahead of
// that wait: those must be complete before the predecessor can trigger its
// dependents, which the library's own kernels guarantee (each waits for its
// predecessor before it triggers) and the header states for callers.
template <typename... Args>
cudaError_t launch_pdl(void (*kern)(Args...), dim3 grid, dim3 block, size_t smem,
                       cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, args...);
}

// The next kernel in the stream may be launched from here on (it still waits
// in cudaGridDependencySynchronize() for this one to finish), which takes its
// launch latency off the critical path.  Used by the small kernels only: behind
// the attention and the decision reduce it measured slower, their successors'
// many CTAs crowding the SMs early.
__device__ __forceinline__ void pdl_launch_dependents() {
#if defined(__CUDA_ARCH__) && __CUDA_ARCH__ >= 900
  cudaTriggerProgrammaticLaunchCompletion();
#endif
}

inline spiffy_status check_launch() {
  return cudaGetLastError() == cudaSuccess ? SPIFFY_OK : SPIFFY_ECUDA;
}

}  // namespace spiffy
