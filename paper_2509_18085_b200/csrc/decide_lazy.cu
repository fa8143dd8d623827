// Lazy chain evaluation of Algorithm 1: the decision (steps 1-4) is computed
// only for the nodes the walk (step 5) actually reaches.
//
// The eager path reduces the logits of every node of the draft graph; only the
// 1 + n_accepted nodes on the accepted path are ever used.  Here one
// cooperative kernel alternates, level by level, between
//   R  all CTAs: the vocabulary-slice reduce of the current node of every
//      sequence that is still walking (the HBM-bound part, 1/N of the eager
//      traffic per level), and
//   T  CTA b: for sequence b the slice merge, the unmasking rule, the next
//      state and the search for the child that equals it,
// separated by grid-wide barriers.  The arithmetic is the code the eager kernels
// use (decide_core.cuh), so the results on the path have the same bits.
//
// The grid barrier counts arrivals in global memory; the host zeroes the
// counter before the launch, the launch is cooperative (all CTAs resident), and
// every wait is bounded: when it runs out the kernel sets SPIFFY_DEV_TIMEOUT and
// returns.
#include "common.cuh"
#include "decide_core.cuh"
#include "walk_core.cuh"

namespace spiffy {
namespace {

struct LazyHeader {
  unsigned int arrivals;  // grid barrier: total arrivals so far
  int done;               // sequences whose walk has ended
  int timeout;            // a barrier wait ran out
  int pad;
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
  Partial* partials;  // [B][L][splits]
  LazyHeader* header;
  int32_t* cur;       // [B] node each sequence stands on, -1 once its walk has ended
};

constexpr unsigned kBarrierSpins = 1u << 21;  // x ~100 ns: gives up after a fraction of a second

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// All CTAs of the (cooperative) grid call this the same number of times;
// `target` is gridDim.x times the number of barriers so far.  Returns false on
// every thread of the CTA when the wait ran out.
__device__ __forceinline__ bool grid_barrier(LazyHeader* h, unsigned target) {
  __shared__ int ok_flag;
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    atomicAdd(&h->arrivals, 1u);
    unsigned spins = 0;
    bool ok = true;
    while (ld_acquire_u32(&h->arrivals) < target) {
      if (++spins > kBarrierSpins || *reinterpret_cast<volatile int*>(&h->timeout)) {
        ok = false;
        h->timeout = 1;
        break;
      }
      __nanosleep(100);
    }
    __threadfence();
    ok_flag = ok;
  }
  __syncthreads();
  return ok_flag != 0;
}

template <typename T>
__global__ void __launch_bounds__(kReduceThreads)
decide_walk_lazy_kernel(const LazyParams p) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int b_own = blockIdx.x < p.B ? (int)blockIdx.x : -1;  // the sequence whose tail this CTA runs
  const int N = p.N, L = p.L;
  __shared__ float s_conf[64];
  __shared__ int32_t s_top[64], s_state[64], s_next[64];
  __shared__ uint64_t s_bits;
  __shared__ int s_found, s_cur, s_hops, s_bad;
  if (tid == 0) {
    s_cur = 0;
    s_hops = 0;
    s_bad = 0;
  }
  if (b_own >= 0) {
    for (int i = tid; i < N; i += kReduceThreads) {
      p.path[(int64_t)b_own * N + i] = i == 0 ? 0 : -1;
      p.n_unmask[(int64_t)b_own * N + i] = -1;  // not evaluated (yet)
    }
  }
  unsigned barriers = 0;
  const int items = p.B * L * p.splits;
  for (int level = 0; level < N; ++level) {
    // R: slices of the rows of every walking sequence's current node
    for (int item = blockIdx.x; item < items; item += gridDim.x) {
      const int b = item / (L * p.splits);
      const int l = (item / p.splits) % L;
      const int split = item % p.splits;
      const int node = level == 0 ? 0 : __ldcg(p.cur + b);
      if (node < 0) continue;
      const int64_t row = ((int64_t)b * N + node) * L + l;
      if (p.block_tokens[row] != p.mask_id) continue;  // already unmasked: never read
      reduce_slice(static_cast<const T*>(p.logits) + row * p.row_stride, p.V, p.chunk, split,
                   p.partials + ((int64_t)b * L + l) * p.splits + split);
      __syncthreads();  // the reduce's shared scratch is reused by the next item
    }
    if (!grid_barrier(p.header, gridDim.x * ++barriers)) break;
    // T: sequence b_own
    if (b_own >= 0 && s_cur >= 0) {
      const int b = b_own, node = s_cur;
      const int32_t* state = p.block_tokens + ((int64_t)b * N + node) * L;
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
          s_state[l] = st;
          if (!ok && p.decide_status) atomicOr(p.decide_status + b, SPIFFY_DEV_NONFINITE);
        }
      }
      __syncthreads();
      if (warp == 0) {
        const uint64_t bits = unmask_rule(s_conf, s_state, L, p.mask_id, p.rule, p.top_s, p.tau, lane);
        if (lane == 0) {
          p.unmask_bits[(int64_t)b * N + node] = bits;
          p.n_unmask[(int64_t)b * N + node] = __popcll(bits);
          s_bits = bits;
          s_found = kNoLink;
        }
      }
      __syncthreads();
      const uint64_t bits = s_bits;
      if (tid < L) s_next[tid] = ((bits >> tid) & 1ull) ? s_top[tid] : s_state[tid];
      __syncthreads();
      if (bits != 0 && s_hops < N - 1) {
        // the first node (ascending) that lists `node` as a parent and equals its next state
        const int32_t* off = p.parent_off + (int64_t)b * (N + 1);
        const int32_t* idx = p.parent_idx + (int64_t)b * p.parent_cap;
        bool bad = false;
        for (int m = node + 1 + warp; m < N; m += kReduceThreads / 32) {
          const int e0 = off[m], e1 = off[m + 1];
          if (e0 < 0 || e1 < e0 || e1 > p.parent_cap) {  // malformed offsets
            bad = true;
            continue;
          }
          bool is_child = false;
          for (int e = e0 + lane; e < e1; e += 32) {
            const int q = idx[e];
            if (q < 0 || q >= m) bad = true;  // ignored entry
            is_child |= q == node;
          }
          if (!__any_sync(0xffffffffu, is_child)) continue;
          const int32_t* sm = p.block_tokens + ((int64_t)b * N + m) * L;
          bool eq = true;
          if (lane < L) eq &= sm[lane] == s_next[lane];
          if (lane + 32 < L) eq &= sm[lane + 32] == s_next[lane + 32];
          if (__all_sync(0xffffffffu, eq) && lane == 0) atomicMin(&s_found, m);
        }
        if (__any_sync(0xffffffffu, bad) && lane == 0) s_bad = 1;
      }
      __syncthreads();
      const int found = (bits != 0 && s_hops < N - 1) ? s_found : kNoLink;
      if (found == kNoLink) {  // the walk ends on `node`
        if (tid < L) p.next_block[(int64_t)b * L + tid] = s_next[tid];
      }
      __syncthreads();
      if (tid == 0) {
        if (found != kNoLink) {  // accepted: its distribution replaces the target's
          s_hops += 1;
          p.path[(int64_t)b * N + s_hops] = found;
          s_cur = found;
          p.cur[b] = found;
        } else {
          p.accepted_node[b] = node;
          p.n_accepted[b] = s_hops;
          if (s_bad && p.walk_status) atomicOr(p.walk_status + b, SPIFFY_DEV_BADGRAPH);
          s_cur = -1;
          p.cur[b] = -1;
          __threadfence();
          atomicAdd(&p.header->done, 1);
        }
      }
    }
    if (!grid_barrier(p.header, gridDim.x * ++barriers)) break;
    if (__ldcg(&p.header->done) >= p.B) return;
  }
  // a barrier wait ran out: say so on the sequence this CTA owns
  if (*reinterpret_cast<volatile int*>(&p.header->timeout) && b_own >= 0 && tid == 0) {
    if (p.decide_status) atomicOr(p.decide_status + b_own, SPIFFY_DEV_TIMEOUT);
    if (p.walk_status) atomicOr(p.walk_status + b_own, SPIFFY_DEV_TIMEOUT);
  }
}

// CTAs that can be resident at once on `device` (cooperative launch limit).
template <typename T>
int resident_ctas(int device) {
  static int cached[64];
  if (device < 0 || device >= 64) return 0;
  if (cached[device] == 0) {
    int per_sm = 0, sms = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decide_walk_lazy_kernel<T>,
                                                      kReduceThreads, 0) != cudaSuccess)
      return 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) return 0;
    cached[device] = per_sm * sms;
  }
  return cached[device];
}

}  // namespace

size_t decide_lazy_workspace_bytes(const spiffy_decide_desc& d) {
  const size_t partials = (size_t)d.batch * d.block_len * decide_splits(d, nullptr) * sizeof(Partial);
  return partials + sizeof(LazyHeader) + (((size_t)d.batch * 4 + 15) / 16) * 16;
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
  const int resident = bf16 ? resident_ctas<__nv_bfloat16>(device) : resident_ctas<float>(device);
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
  p.cur = reinterpret_cast<int32_t*>(p.header + 1);
  const int64_t items = (int64_t)d.batch * d.block_len * p.splits;
  int grid = (int)(items < resident ? items : resident);
  if (grid < d.batch) grid = d.batch;
  if (cudaMemsetAsync(p.header, 0, sizeof(LazyHeader), stream) != cudaSuccess) return SPIFFY_ECUDA;
  void* args[] = {&p};
  const void* fn = bf16 ? (const void*)decide_walk_lazy_kernel<__nv_bfloat16>
                        : (const void*)decide_walk_lazy_kernel<float>;
  const cudaError_t e =
      cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(kReduceThreads), args, (size_t)0, stream);
  count_launch();
  return e == cudaSuccess ? SPIFFY_OK : SPIFFY_ECUDA;
}

}  // namespace spiffy
