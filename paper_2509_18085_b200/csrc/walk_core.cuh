// Step 5 of Algorithm 1 for one sequence.  The walk starts at the true block
// (node 0) and moves to the first node (ascending index) that lists the current
// one as a parent and whose state equals the current node's next state; it stops
// when there is none, or at a node with nothing left to unmask.
//
// Whether node m follows node p depends on p and m alone, not on the path, so
// the links are found for all (parent, child) entries at once -- one warp per
// child, lane k owning block positions k and k + 32 -- and the walk itself is a
// chase through at most N-1 links.  The graph arrays may live in shared or
// global memory; `link` is N ints of shared memory.
#pragma once
#include "common.cuh"

namespace spiffy {

constexpr int kNoLink = 0x7fffffff;

__device__ __forceinline__ int32_t walk_next_token(const int32_t* state, const int32_t* top,
                                                   uint64_t bits, int node, int L, int l) {
  return ((bits >> l) & 1ull) ? top[node * L + l] : state[node * L + l];
}

// Called by `n_warps` warps together (warp index `warp`); `link` must hold
// kNoLink everywhere beforehand and is complete after the next block-wide sync.
// Returns true on every lane of a warp that met a malformed offset or entry
// (such entries are ignored).
__device__ __forceinline__ bool walk_link_children(int N, int L, int parent_cap,
                                                   const int32_t* state, const int32_t* top,
                                                   const int32_t* off, const int32_t* idx,
                                                   const uint64_t* ubits, int* link, int warp,
                                                   int n_warps, int lane) {
  const unsigned full = 0xffffffffu;
  const int l0 = lane, l1 = lane + 32;
  bool bad = false;
  for (int m = 1 + warp; m < N; m += n_warps) {
    const int e0 = off[m], e1 = off[m + 1];
    if (e0 < 0 || e1 < e0 || e1 > parent_cap) {  // malformed offsets
      bad = true;
      continue;
    }
    const int32_t s0 = l0 < L ? state[m * L + l0] : 0;
    const int32_t s1 = l1 < L ? state[m * L + l1] : 0;
    for (int e = e0; e < e1; ++e) {
      const int p = idx[e];
      if (p < 0 || p >= m) {  // ignored entry
        bad = true;
        continue;
      }
      const uint64_t bits = ubits[p];
      if (bits == 0) continue;  // a node with nothing to unmask ends the walk
      bool eq = true;
      if (l0 < L) eq &= s0 == walk_next_token(state, top, bits, p, L, l0);
      if (l1 < L) eq &= s1 == walk_next_token(state, top, bits, p, L, l1);
      if (__all_sync(full, eq) && lane == 0) atomicMin(link + p, m);
    }
  }
  return __any_sync(full, bad);
}

// Called by one warp after the links are complete (a block-wide sync after
// walk_link_children).
__device__ __forceinline__ void walk_chase(int N, int L, const int32_t* state, const int32_t* top,
                                           const uint64_t* ubits, const int* link, int32_t* pth,
                                           int32_t* next_block, int32_t* accepted_node,
                                           int32_t* n_accepted, int lane) {
  int cur = 0, hops = 0;
  if (lane == 0) {
    // `link` may be the path array itself: a link is read before the slot at or
    // below its node is reused for the path (hop h is stored at index h <= node)
    int m = link[0];
    pth[0] = 0;
    while (hops < N - 1 && m != kNoLink) {
      cur = m;  // accepted: its distribution replaces the target's
      m = link[cur];
      pth[++hops] = cur;
    }
    *accepted_node = cur;
    *n_accepted = hops;
  }
  cur = __shfl_sync(0xffffffffu, cur, 0);
  hops = __shfl_sync(0xffffffffu, hops, 0);
  for (int i = hops + 1 + lane; i < N; i += 32) pth[i] = -1;
  const uint64_t bits = ubits[cur];
  if (lane < L) next_block[lane] = walk_next_token(state, top, bits, cur, L, lane);
  if (lane + 32 < L) next_block[lane + 32] = walk_next_token(state, top, bits, cur, L, lane + 32);
}

}  // namespace spiffy
