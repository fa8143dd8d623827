// Lazy chain evaluation of Algorithm 1: the decision (steps 1-4) is computed
// only for the nodes the walk (step 5) actually reaches.
//
// The eager path reduces the logits of every node of the draft graph; only the
// 1 + n_accepted nodes on the accepted path are ever used.  Here one
// cooperative kernel works level by level.  For every sequence b that is still
// walking:
//   R  the CTAs that own the (position, vocabulary slice) items of b reduce the
//      rows of b's current node (the HBM-bound part, 1/N of the eager traffic
//      per level) and count themselves in on arrivals[b];
//   T  CTA b waits for those arrivals, merges the slices, applies the unmasking
//      rule, forms the next state, looks for the child that equals it (the graph
//      of b sits in its shared memory) and publishes the new current node with
//      epoch[b] = level + 1, for which the reducers of b wait.
// Sequences never wait for one another.  The arithmetic is the code the eager
// kernels use (decide_core.cuh), so the results on the path have the same bits.
//
// Waiting: a wait for level k of sequence b depends only on work of levels
// < k, or of level k's R phase, so there is no cycle; the launch is cooperative
// (all CTAs resident); every wait is bounded, and when one runs out the kernel
// sets SPIFFY_DEV_TIMEOUT, tells the others through the header and returns.
// The host zeroes header, arrivals and epoch before the launch.
#include "common.cuh"
#include "decide_core.cuh"
#include "walk_core.cuh"

namespace spiffy {
namespace {

struct LazyHeader {
  int timeout;  // a bounded wait ran out somewhere
  int pad[3];
};

struct LazyParams {
  const void* logits;
  int64_t row_stride, chunk;
  int B, N, L, V, splits, mask_id, rule, top_s;
  float tau;
  const int32_t* block_tokens;
  const int32_t* parent_off;
  const int32_t* parent_idx;
  int parent_cap;
  float* conf;
  int32_t* top_tok;
  uint64_t* unmask_bits;
  int32_t* n_unmask;
  int32_t* decide_status;
  int32_t* accepted_node;
  int32_t* n_accepted;
  int32_t* path;
  int32_t* next_block;
  int32_t* walk_status;
  Partial* partials;   // [B][L][splits]
  LazyHeader* header;
  unsigned* arrivals;  // [B] slices of b reduced so far, over all levels
  int32_t* epoch;      // [B] levels of b whose tail has finished
  int32_t* cur;        // [B] node b stands on at level epoch[b], -1 once its walk has ended
  int stage_graph;     // the sequence's states and parent lists fit shared memory
  unsigned wait_spins;   // polls of one wait before it gives up
  unsigned extra_arrivals;  // test hook: sequence 0 expects this many arrivals that never come
};


__device__ __forceinline__ unsigned ld_acquire_u32(const void* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// Thread 0 waits until the word at `p` has reached `target`; every thread of
// the CTA gets the verdict (false: the wait ran out, here or elsewhere).
__device__ __forceinline__ bool wait_reached(const void* p, unsigned target, LazyHeader* h,
                                             unsigned limit) {
  __shared__ int ok_flag;
  if (threadIdx.x == 0) {
    unsigned spins = 0;
    bool ok = true;
    while (ld_acquire_u32(p) < target) {
      if (++spins > limit || *reinterpret_cast<volatile int*>(&h->timeout)) {
        ok = false;
        h->timeout = 1;
        break;
      }
      __nanosleep(100);
    }
    ok_flag = ok;
  }
  __syncthreads();
  const bool ok = ok_flag != 0;
  __syncthreads();  // ok_flag may be rewritten by the next wait
  return ok;
}

template <typename T>
__global__ void __launch_bounds__(kReduceThreads, 6)  // 80 registers, no spills: six CTAs per SM
decide_walk_lazy_kernel(const LazyParams p) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int b_own = blockIdx.x < p.B ? (int)blockIdx.x : -1;  // the sequence whose tail this CTA runs
  const int N = p.N, L = p.L;
  __shared__ float s_conf[64];
  __shared__ int32_t s_top[64], s_next[64];
  __shared__ uint64_t s_bits;
  __shared__ int s_found, s_node, s_bad;
  extern __shared__ __align__(8) unsigned char lazy_smem[];
  // the graph of the own sequence: [states N*L | off N+1 | idx cap], staged when it fits
  const int32_t* g_state = nullptr;
  const int32_t* g_off = nullptr;
  const int32_t* g_idx = nullptr;
  if (b_own >= 0) {
    g_state = p.block_tokens + (int64_t)b_own * N * L;
    g_off = p.parent_off + (int64_t)b_own * (N + 1);
    g_idx = p.parent_idx + (int64_t)b_own * p.parent_cap;
    if (p.stage_graph) {
      int32_t* s_state = reinterpret_cast<int32_t*>(lazy_smem);
      int32_t* s_off = s_state + N * L;
      int32_t* s_idx = s_off + (N + 1);
      auto copy4 = [](void* dst, const void* src) {
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(
                         (uint32_t)__cvta_generic_to_shared(dst)),
                     "l"(src)
                     : "memory");
      };
      for (int i = tid; i < N * L; i += kReduceThreads) copy4(s_state + i, g_state + i);
      for (int i = tid; i <= N; i += kReduceThreads) copy4(s_off + i, g_off + i);
      for (int i = tid; i < p.parent_cap; i += kReduceThreads) copy4(s_idx + i, g_idx + i);
      g_state = s_state;
      g_off = s_off;
      g_idx = s_idx;  // waited for before the first tail phase
    }
    for (int i = tid; i < N; i += kReduceThreads) {
      p.path[(int64_t)b_own * N + i] = i == 0 ? 0 : -1;
      p.n_unmask[(int64_t)b_own * N + i] = -1;  // not evaluated (yet)
    }
  }
  if (tid == 0) s_bad = 0;
  int own_node = b_own >= 0 ? 0 : -1;  // uniform over the CTA
  int own_hops = 0;
  // arrivals[b_own] once the current level is reduced
  unsigned own_expected = b_own == 0 ? p.extra_arrivals : 0u;
  bool failed = false;
  const int items = p.B * L * p.splits;
  for (int level = 0; level < N && !failed; ++level) {
    bool alive = false;
    // R: this CTA's slices of the current nodes
    for (int item = blockIdx.x; item < items; item += gridDim.x) {
      const int b = item / (L * p.splits);
      const int l = (item / p.splits) % L;
      const int split = item % p.splits;
      int node = 0;
      if (level > 0) {
        if (b == b_own) {
          node = own_node;
        } else {
          if (!wait_reached(p.epoch + b, (unsigned)level, p.header, p.wait_spins)) {
            failed = true;
            break;
          }
          if (tid == 0) s_node = __ldcg(p.cur + b);
          __syncthreads();
          node = s_node;
          __syncthreads();
        }
      }
      if (node < 0) continue;  // this sequence's walk has ended
      alive = true;
      const int64_t row = ((int64_t)b * N + node) * L + l;
      if (p.block_tokens[row] != p.mask_id) continue;  // already unmasked: never read, never counted
      reduce_slice(static_cast<const T*>(p.logits) + row * p.row_stride, p.V, p.chunk, split,
                   p.partials + ((int64_t)b * L + l) * p.splits + split);
      if (tid == 0) {  // the thread that stored the result counts it in
        __threadfence();
        atomicAdd(p.arrivals + b, 1u);
      }
      __syncthreads();  // the reduce's shared scratch is reused by the next item
    }
    if (failed) break;
    // T: the own sequence
    if (own_node >= 0) {
      alive = true;
      const int b = b_own, node = own_node;
      if (level == 0) {
        asm volatile("cp.async.wait_all;" ::: "memory");
        __syncthreads();
      }
      const int32_t* state = g_state + node * L;
      {  // slices of this level: every still-masked row of the node, `splits` each
        int masked = 0;
        for (int l = lane; l < L; l += 32) masked += state[l] == p.mask_id;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) masked += __shfl_xor_sync(0xffffffffu, masked, off);
        own_expected += (unsigned)masked * (unsigned)p.splits;
      }
      if (!wait_reached(p.arrivals + b, own_expected, p.header, p.wait_spins)) {
        failed = true;
        break;
      }
      {
        const int r = tid >> 1, sub = tid & 1, l = min(r, L - 1);
        const int32_t st = state[l];
        float conf;
        int32_t tok;
        const bool ok = finalize_row<2>(p.partials + ((int64_t)b * L + l) * p.splits, p.splits, sub, st,
                                        p.mask_id, conf, tok);
        if (sub == 0 && r < L) {
          const int64_t row = ((int64_t)b * N + node) * L + l;
          p.conf[row] = conf;
          p.top_tok[row] = tok;
          s_conf[l] = conf;
          s_top[l] = tok;
          if (!ok && p.decide_status) atomicOr(p.decide_status + b, SPIFFY_DEV_NONFINITE);
        }
      }
      __syncthreads();
      if (warp == 0) {
        const uint64_t bits = unmask_rule(s_conf, state, L, p.mask_id, p.rule, p.top_s, p.tau, lane);
        if (lane == 0) {
          p.unmask_bits[(int64_t)b * N + node] = bits;
          p.n_unmask[(int64_t)b * N + node] = __popcll(bits);
          s_bits = bits;
          s_found = kNoLink;
        }
      }
      __syncthreads();
      const uint64_t bits = s_bits;
      if (tid < L) s_next[tid] = ((bits >> tid) & 1ull) ? s_top[tid] : state[tid];
      __syncthreads();
      const bool may_go_on = bits != 0 && own_hops < N - 1;
      if (may_go_on) {
        // the first node (ascending) that lists `node` as a parent and equals its next state
        bool bad = false;
        for (int m = node + 1 + warp; m < N; m += kReduceThreads / 32) {
          const int e0 = g_off[m], e1 = g_off[m + 1];
          if (e0 < 0 || e1 < e0 || e1 > p.parent_cap) {  // malformed offsets
            bad = true;
            continue;
          }
          bool is_child = false;
          for (int e = e0 + lane; e < e1; e += 32) {
            const int q = g_idx[e];
            if (q < 0 || q >= m) bad = true;  // ignored entry
            is_child |= q == node;
          }
          if (!__any_sync(0xffffffffu, is_child)) continue;
          const int32_t* sm = g_state + m * L;
          bool eq = true;
          if (lane < L) eq &= sm[lane] == s_next[lane];
          if (lane + 32 < L) eq &= sm[lane + 32] == s_next[lane + 32];
          if (__all_sync(0xffffffffu, eq) && lane == 0) atomicMin(&s_found, m);
        }
        if (__any_sync(0xffffffffu, bad) && lane == 0) s_bad = 1;
      }
      __syncthreads();
      const int found = may_go_on ? s_found : kNoLink;
      if (found != kNoLink) {  // accepted: its distribution replaces the target's
        own_hops += 1;
        own_node = found;
        if (tid == 0) p.path[(int64_t)b * N + own_hops] = found;
      } else {  // the walk ends on `node`
        if (tid < L) p.next_block[(int64_t)b * L + tid] = s_next[tid];
        if (tid == 0) {
          p.accepted_node[b] = node;
          p.n_accepted[b] = own_hops;
          if (s_bad && p.walk_status) atomicOr(p.walk_status + b, SPIFFY_DEV_BADGRAPH);
        }
        own_node = -1;
      }
      if (tid == 0) {  // publish: the reducers of b wait for epoch[b] > level, then read cur[b]
        p.cur[b] = own_node;
        __threadfence();
        atomicExch(p.epoch + b, own_node < 0 ? 0x7fffffff : level + 1);
      }
      __syncthreads();
    }
    if (!alive) return;  // every sequence this CTA works for has ended
  }
  // a bounded wait ran out (here or in another CTA): say so on the sequence this CTA owns
  if (*reinterpret_cast<volatile int*>(&p.header->timeout) && b_own >= 0 && tid == 0) {
    if (p.decide_status) atomicOr(p.decide_status + b_own, SPIFFY_DEV_TIMEOUT);
    if (p.walk_status) atomicOr(p.walk_status + b_own, SPIFFY_DEV_TIMEOUT);
  }
}

size_t lazy_graph_bytes(const spiffy_decide_desc& d, int parent_cap) {
  return ((size_t)d.n_nodes * d.block_len + d.n_nodes + 1 + parent_cap) * 4;
}

// CTAs that can be resident at once on `device` (cooperative launch limit).
template <typename T>
int resident_ctas(int device, size_t smem) {
  static int sm_count[64];
  if (device < 0 || device >= 64) return 0;
  if (sm_count[device] == 0 &&
      cudaDeviceGetAttribute(&sm_count[device], cudaDevAttrMultiProcessorCount, device) != cudaSuccess)
    return 0;
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decide_walk_lazy_kernel<T>,
                                                    kReduceThreads, smem) != cudaSuccess)
    return 0;
  return per_sm * sm_count[device];
}

}  // namespace

size_t decide_lazy_workspace_bytes(const spiffy_decide_desc& d) {
  const size_t partials = (size_t)d.batch * d.block_len * decide_splits(d, nullptr) * sizeof(Partial);
  // header | arrivals[B] | epoch[B] | cur[B], the first three zeroed by every call
  return partials + sizeof(LazyHeader) + (((size_t)d.batch * 12 + 15) / 16) * 16;
}

spiffy_status launch_decide_walk_lazy(const spiffy_decide_desc& d, const void* logits,
                                      const int32_t* block_tokens, float* conf, int32_t* top_tok,
                                      uint64_t* unmask_bits, int32_t* n_unmask,
                                      int32_t* decide_status, const int32_t* parent_off,
                                      const int32_t* parent_idx, int32_t parent_cap,
                                      int32_t* accepted_node, int32_t* n_accepted, int32_t* path,
                                      int32_t* next_block, int32_t* walk_status, void* ws,
                                      cudaStream_t stream) {
  int device = 0;
  if (cudaGetDevice(&device) != cudaSuccess) return SPIFFY_ECUDA;
  const bool bf16 = d.logits_dtype == SPIFFY_BF16;
  const size_t graph = lazy_graph_bytes(d, parent_cap);
  const int stage_graph = graph <= 16 * 1024;  // beyond that it would cost resident CTAs
  const size_t smem = stage_graph ? graph : 0;
  const int resident = bf16 ? resident_ctas<__nv_bfloat16>(device, smem) : resident_ctas<float>(device, smem);
  if (resident <= 0) return SPIFFY_ECUDA;
  if (d.batch > resident) return SPIFFY_EUNSUPPORTED;  // one resident CTA per sequence runs its tail
  LazyParams p;
  p.logits = logits;
  p.row_stride = d.row_stride;
  p.splits = decide_splits(d, &p.chunk);
  p.B = d.batch;
  p.N = d.n_nodes;
  p.L = d.block_len;
  p.V = d.vocab;
  p.mask_id = d.mask_token_id;
  p.rule = d.rule;
  p.top_s = d.top_s;
  p.tau = d.threshold;
  p.block_tokens = block_tokens;
  p.parent_off = parent_off;
  p.parent_idx = parent_idx;
  p.parent_cap = parent_cap;
  p.conf = conf;
  p.top_tok = top_tok;
  p.unmask_bits = unmask_bits;
  p.n_unmask = n_unmask;
  p.decide_status = decide_status;
  p.accepted_node = accepted_node;
  p.n_accepted = n_accepted;
  p.path = path;
  p.next_block = next_block;
  p.walk_status = walk_status;
  const size_t partial_bytes = (size_t)d.batch * d.block_len * p.splits * sizeof(Partial);
  p.partials = static_cast<Partial*>(ws);
  p.header = reinterpret_cast<LazyHeader*>(static_cast<char*>(ws) + partial_bytes);
  p.arrivals = reinterpret_cast<unsigned*>(p.header + 1);
  p.epoch = reinterpret_cast<int32_t*>(p.arrivals + d.batch);
  p.cur = p.epoch + d.batch;
  p.stage_graph = stage_graph;
  p.wait_spins = flag_poll_limit();
  p.extra_arrivals = (unsigned)lazy_extra_arrivals();
  const int64_t items = (int64_t)d.batch * d.block_len * p.splits;
  int grid = (int)(items < resident ? items : resident);
  if (grid < d.batch) grid = d.batch;
  if (cudaMemsetAsync(p.header, 0, sizeof(LazyHeader) + (size_t)d.batch * 8, stream) != cudaSuccess)
    return SPIFFY_ECUDA;
  void* args[] = {&p};
  const void* fn = bf16 ? (const void*)decide_walk_lazy_kernel<__nv_bfloat16>
                        : (const void*)decide_walk_lazy_kernel<float>;
  const cudaError_t e =
      cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(kReduceThreads), args, smem, stream);
  count_launch();
  return e == cudaSuccess ? SPIFFY_OK : SPIFFY_ECUDA;
}

}  // namespace spiffy
