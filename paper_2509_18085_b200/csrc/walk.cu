// Acceptance walk: step 5 of Algorithm 1 over the draft graph of Sec. 4.4.1.
// One CTA per sequence: its warps link every child to the parents it follows,
// then warp 0 chases the links from the true block.
#include "common.cuh"
#include "walk_core.cuh"

namespace spiffy {
namespace {

constexpr int kWalkThreads = 256;

__global__ void __launch_bounds__(kWalkThreads)
accept_walk_kernel(int N, int L, const int32_t* __restrict__ block_tokens,
                   const int32_t* __restrict__ parent_off,
                   const int32_t* __restrict__ parent_idx, int parent_cap,
                   const int32_t* __restrict__ top_tok,
                   const uint64_t* __restrict__ unmask_bits,
                   int32_t* __restrict__ accepted_node,
                   int32_t* __restrict__ n_accepted, int32_t* __restrict__ path,
                   int32_t* __restrict__ next_block,
                   int32_t* __restrict__ dev_status, int stage_in_smem, int link_in_smem) {
  const int b = blockIdx.x;
  const int tid = threadIdx.x;
  const int32_t* state = block_tokens + (int64_t)b * N * L;
  const int32_t* top = top_tok + (int64_t)b * N * L;
  const int32_t* off = parent_off + (int64_t)b * (N + 1);
  const int32_t* idx = parent_idx + (int64_t)b * parent_cap;
  const uint64_t* ubits = unmask_bits + (int64_t)b * N;
  int32_t* pth = path + (int64_t)b * N;
  // When the sequence's graph fits, it is copied to shared memory first (all
  // loads in flight at once): [bits | state | top | off | idx | link].  The
  // links of a graph too large for that live in the path output, which the
  // chase overwrites only behind itself (hop h is written at index h <= node).
  extern __shared__ __align__(8) unsigned char walk_smem[];
  uint64_t* s_bits = reinterpret_cast<uint64_t*>(walk_smem);
  int32_t* s_state = reinterpret_cast<int32_t*>(s_bits + (stage_in_smem ? N : 0));
  int32_t* s_top = s_state + (stage_in_smem ? N * L : 0);
  int32_t* s_off = s_top + (stage_in_smem ? N * L : 0);
  int32_t* s_idx = s_off + (stage_in_smem ? N + 1 : 0);
  int* link = link_in_smem ? s_idx + (stage_in_smem ? parent_cap : 0) : pth;
  auto copy4 = [](void* dst, const void* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(
                     (uint32_t)__cvta_generic_to_shared(dst)),
                 "l"(src)
                 : "memory");
  };
  // the graph itself does not depend on the decision kernel: fetch it before waiting
  if (stage_in_smem) {
    for (int i = tid; i < N * L; i += kWalkThreads) copy4(s_state + i, state + i);
    for (int i = tid; i <= N; i += kWalkThreads) copy4(s_off + i, off + i);
    for (int i = tid; i < parent_cap; i += kWalkThreads) copy4(s_idx + i, idx + i);
  }
#if __CUDA_ARCH__ >= 900
  pdl_launch_dependents();
  cudaGridDependencySynchronize();  // the decision kernel's outputs are visible
#endif
  for (int i = tid; i < N; i += kWalkThreads) link[i] = kNoLink;
  if (stage_in_smem) {
    for (int i = tid; i < N * L; i += kWalkThreads) copy4(s_top + i, top + i);
    for (int i = tid; i < 2 * N; i += kWalkThreads)
      copy4(reinterpret_cast<int32_t*>(s_bits) + i, reinterpret_cast<const int32_t*>(ubits) + i);
    asm volatile("cp.async.wait_all;" ::: "memory");
    state = s_state; top = s_top; off = s_off; idx = s_idx; ubits = s_bits;
  }
  __syncthreads();
  const int warp = tid >> 5, lane = tid & 31;
  const bool bad = walk_link_children(N, L, parent_cap, state, top, off, idx, ubits, link, warp,
                                      kWalkThreads / 32, lane);
  if (bad && lane == 0 && dev_status) atomicOr(dev_status + b, SPIFFY_DEV_BADGRAPH);
  __syncthreads();
  if (warp == 0)
    walk_chase(N, L, state, top, ubits, link, pth, next_block + (int64_t)b * L, accepted_node + b,
               n_accepted + b, lane);
}

}  // namespace

spiffy_status launch_walk(const spiffy_decide_desc& d,
                          const int32_t* block_tokens,
                          const int32_t* parent_off, const int32_t* parent_idx,
                          int32_t parent_cap, const int32_t* top_tok,
                          const uint64_t* unmask_bits, int32_t* accepted_node,
                          int32_t* n_accepted, int32_t* path,
                          int32_t* next_block, int32_t* dev_status,
                          cudaStream_t stream) {
  const size_t graph = (size_t)d.n_nodes * 8 +
                       ((size_t)2 * d.n_nodes * d.block_len + d.n_nodes + 1 + parent_cap) * 4;
  const size_t links = (size_t)d.n_nodes * 4;
  const int stage_in_smem = graph + links <= 40 * 1024;
  const int link_in_smem = stage_in_smem || links <= 40 * 1024;
  const size_t smem = (stage_in_smem ? graph : 0) + (link_in_smem ? links : 0);
  const cudaError_t e = launch_pdl(
      accept_walk_kernel, dim3(d.batch), dim3(kWalkThreads), smem, stream,
      (int)d.n_nodes, (int)d.block_len, block_tokens, parent_off, parent_idx, (int)parent_cap,
      top_tok, unmask_bits, accepted_node, n_accepted, path, next_block, dev_status,
      stage_in_smem, link_in_smem);
  count_launch();
  return e == cudaSuccess ? SPIFFY_OK : SPIFFY_ECUDA;
}

}  // namespace spiffy
