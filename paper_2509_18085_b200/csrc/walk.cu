// Acceptance walk: step 5 of Algorithm 1 over the draft graph of Sec. 4.4.1.
// One warp per sequence; lane k owns block positions k and k + 32.
#include "common.cuh"

namespace spiffy {
namespace {

__global__ void __launch_bounds__(32)
accept_walk_kernel(int N, int L, const int32_t* __restrict__ block_tokens,
                   const int32_t* __restrict__ parent_off,
                   const int32_t* __restrict__ parent_idx, int parent_cap,
                   const int32_t* __restrict__ top_tok,
                   const uint64_t* __restrict__ unmask_bits,
                   int32_t* __restrict__ accepted_node,
                   int32_t* __restrict__ n_accepted, int32_t* __restrict__ path,
                   int32_t* __restrict__ next_block,
                   int32_t* __restrict__ dev_status, int stage_in_smem) {
#if __CUDA_ARCH__ >= 900
  pdl_launch_dependents();
  cudaGridDependencySynchronize();  // the decision kernel's outputs are visible
#endif
  const int b = blockIdx.x;
  const int lane = threadIdx.x;
  const unsigned full = 0xffffffffu;
  const int32_t* state = block_tokens + (int64_t)b * N * L;
  const int32_t* top = top_tok + (int64_t)b * N * L;
  const int32_t* off = parent_off + (int64_t)b * (N + 1);
  const int32_t* idx = parent_idx + (int64_t)b * parent_cap;
  const uint64_t* ubits = unmask_bits + (int64_t)b * N;
  // The walk is a chain of dependent reads: when the sequence's graph fits,
  // copy it to shared memory first (all loads in flight at once) and walk there.
  extern __shared__ __align__(8) unsigned char walk_smem[];
  if (stage_in_smem) {
    uint64_t* s_bits = reinterpret_cast<uint64_t*>(walk_smem);
    int32_t* s_state = reinterpret_cast<int32_t*>(s_bits + N);
    int32_t* s_top = s_state + N * L;
    int32_t* s_off = s_top + N * L;
    int32_t* s_idx = s_off + (N + 1);
    // asynchronous copies: every load is in flight before the first one is waited for
    auto copy4 = [](void* dst, const void* src) {
      asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(
                       (uint32_t)__cvta_generic_to_shared(dst)),
                   "l"(src)
                   : "memory");
    };
    for (int i = lane; i < N * L; i += 32) { copy4(s_state + i, state + i); copy4(s_top + i, top + i); }
    for (int i = lane; i <= N; i += 32) copy4(s_off + i, off + i);
    for (int i = lane; i < parent_cap; i += 32) copy4(s_idx + i, idx + i);
    for (int i = lane; i < 2 * N; i += 32)
      copy4(reinterpret_cast<int32_t*>(s_bits) + i, reinterpret_cast<const int32_t*>(ubits) + i);
    asm volatile("cp.async.wait_all;" ::: "memory");
    __syncwarp();
    state = s_state; top = s_top; off = s_off; idx = s_idx; ubits = s_bits;
  }
  int32_t* pth = path + (int64_t)b * N;
  for (int i = lane; i < N; i += 32) pth[i] = i == 0 ? 0 : -1;
  const int l0 = lane, l1 = lane + 32;
  bool bad = false;
  int cur = 0, hops = 0;
  // next(cur) on this lane's two positions
  auto next_of = [&](int node, uint64_t bits, int l) -> int32_t {
    if (l >= L) return 0;
    return ((bits >> l) & 1ull) ? top[node * L + l] : state[node * L + l];
  };
  uint64_t bits = ubits[0];
  int32_t nx0 = next_of(0, bits, l0), nx1 = next_of(0, bits, l1);
  while (hops < N - 1 && bits != 0) {
    int found = -1;
    // children have larger indices than their parents (topological order)
    for (int m = cur + 1; m < N && found < 0; ++m) {
      int e0 = off[m], e1 = off[m + 1];
      if (e0 < 0 || e1 < e0 || e1 > parent_cap) {  // malformed offsets
        bad = true;
        continue;
      }
      bool is_child = false;
      for (int e = e0 + lane; e < e1; e += 32) {
        const int p = idx[e];
        if (p < 0 || p >= m) bad = true;  // ignored entry
        is_child |= p == cur;
      }
      if (!__any_sync(full, is_child)) continue;
      bool eq = true;
      if (l0 < L) eq &= state[m * L + l0] == nx0;
      if (l1 < L) eq &= state[m * L + l1] == nx1;
      if (__all_sync(full, eq)) found = m;
    }
    if (found < 0) break;
    cur = found;  // accepted: its distribution replaces the target's
    ++hops;
    if (lane == 0) pth[hops] = cur;
    bits = ubits[cur];
    nx0 = next_of(cur, bits, l0);
    nx1 = next_of(cur, bits, l1);
  }
  if (l0 < L) next_block[(int64_t)b * L + l0] = nx0;
  if (l1 < L) next_block[(int64_t)b * L + l1] = nx1;
  if (lane == 0) {
    accepted_node[b] = cur;
    n_accepted[b] = hops;
  }
  if (__any_sync(full, bad) && lane == 0 && dev_status)
    atomicOr(dev_status + b, SPIFFY_DEV_BADGRAPH);
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
  const size_t need = (size_t)d.n_nodes * 8 +
                      ((size_t)2 * d.n_nodes * d.block_len + d.n_nodes + 1 + parent_cap) * 4;
  const int stage_in_smem = need <= 40 * 1024;
  const cudaError_t e = launch_pdl(
      accept_walk_kernel, dim3(d.batch), dim3(32), stage_in_smem ? need : (size_t)0, stream,
      (int)d.n_nodes, (int)d.block_len, block_tokens, parent_off, parent_idx, (int)parent_cap,
      top_tok, unmask_bits, accepted_node, n_accepted, path, next_block, dev_status,
      stage_in_smem);
  count_launch();
  return e == cudaSuccess ? SPIFFY_OK : SPIFFY_ECUDA;
}

}  // namespace spiffy
