// Decision kernels: steps 1-4 of Algorithm 1 (the function Next() of App. A)
// evaluated for every node of the draft graph, and their fusion with step 5.
//
//   decide_reduce_kernel    streams the logits rows of still-masked positions
//                           once (the HBM-bound part): per (row, vocabulary
//                           slice) the maximum, the sum of exponentials and the
//                           lowest index that attains the maximum
//   decide_finalize_kernel  per node: merges the slices in a fixed order, turns
//                           them into (confidence, top token) and applies the
//                           unmasking rule of Sec. 3.1
//   decide_tail_kernel      per sequence, for small graphs: the finalize step
//                           of all its nodes and the acceptance walk (step 5)
//                           in one CTA, resident before the reduce ends
//
// The arithmetic shared with the other decision kernels is in decide_core.cuh,
// the walk in walk_core.cuh.
#include "common.cuh"
#include "decide_core.cuh"
#include "walk_core.cuh"

namespace spiffy {
namespace {

// grid = (splits, B*N*L); one CTA reduces one vocabulary slice of one row.
template <typename T>
__global__ void __launch_bounds__(kReduceThreads, 8)  // 64 registers: eight CTAs per SM
decide_reduce_kernel(const T* __restrict__ logits, int64_t row_stride, int V,
                     int64_t chunk, int splits,
                     const int32_t* __restrict__ block_tokens, int mask_id,
                     Partial* __restrict__ partials, int early_trigger) {
#if __CUDA_ARCH__ >= 900
  cudaGridDependencySynchronize();  // inputs written by earlier kernels are visible
  // The one-CTA-per-sequence tail kernel may take its SM while this grid still
  // runs (it waits there for this grid to finish): its launch latency is hidden.
  if (early_trigger) pdl_launch_dependents();
#endif
  const int row = blockIdx.y;
  if (block_tokens[row] != mask_id) return;  // already unmasked: never read
  reduce_slice(logits + (int64_t)row * row_stride, V, chunk, (int)blockIdx.x,
               partials + (int64_t)row * splits + blockIdx.x);
}

// grid = B*N nodes, 512 threads: eight threads per position merge the slices of
// its row, then warp 0 applies the rule.
constexpr int kFinalizeThreads = 512;
__global__ void __launch_bounds__(kFinalizeThreads)
decide_finalize_kernel(const Partial* __restrict__ partials, int splits, int N,
                       int L, const int32_t* __restrict__ block_tokens,
                       int mask_id, int rule, int top_s, float tau,
                       float* __restrict__ conf_out, int32_t* __restrict__ tok_out,
                       uint64_t* __restrict__ bits_out,
                       int32_t* __restrict__ n_unmask_out,
                       int32_t* __restrict__ dev_status) {
#if __CUDA_ARCH__ >= 900
  pdl_launch_dependents();
  cudaGridDependencySynchronize();  // the reduce kernel's partials are visible
#endif
  const int node = blockIdx.x;
  const int pos = threadIdx.x >> 3, sub = threadIdx.x & 7;
  __shared__ float sconf[64];
  {
    const int row = node * L + min(pos, L - 1);
    // the token and the partials are read together (one trip to memory); the
    // partials of an unmasked row were never written and are ignored
    const int32_t state = block_tokens[row];
    float conf;
    int32_t tok;
    const bool ok = finalize_row<8>(partials + (int64_t)row * splits, splits, sub, state, mask_id, conf, tok);
    if (sub == 0 && pos < L) {
      conf_out[row] = conf;
      tok_out[row] = tok;
      sconf[pos] = conf;
      if (!ok && dev_status) atomicOr(dev_status + node / N, SPIFFY_DEV_NONFINITE);
    }
  }
  __syncthreads();
  if (threadIdx.x >= 32) return;
  const uint64_t bits = unmask_rule(sconf, block_tokens + (int64_t)node * L, L, mask_id, rule, top_s,
                                    tau, threadIdx.x);
  if (threadIdx.x == 0) {
    bits_out[node] = bits;
    n_unmask_out[node] = __popcll(bits);
  }
}

// Decision tail and acceptance walk of one sequence in one CTA (Algorithm 1,
// steps 1-5 after the vocabulary reduce): eight threads per row merge the
// slices, one warp per node applies the rule, warp 0 walks the draft graph with
// every array it needs already in shared memory.  The graph (states, parent
// lists) does not depend on the reduce kernel and is fetched before the wait on
// it.  grid = B, kTailThreads threads, dynamic shared memory tail_smem_bytes().
constexpr int kTailThreads = 1024;
template <int kLanes>  // threads per row: all N * L rows are merged in one pass when kLanes * N * L <= 1024
__global__ void __launch_bounds__(kTailThreads)
decide_tail_kernel(const Partial* __restrict__ partials, int splits, int N, int L,
                   const int32_t* __restrict__ block_tokens, int mask_id, int rule, int top_s,
                   float tau, float* __restrict__ conf_out, int32_t* __restrict__ tok_out,
                   uint64_t* __restrict__ bits_out, int32_t* __restrict__ n_unmask_out,
                   int32_t* __restrict__ decide_status,
                   const int32_t* __restrict__ parent_off, const int32_t* __restrict__ parent_idx,
                   int parent_cap, int32_t* __restrict__ accepted_node,
                   int32_t* __restrict__ n_accepted, int32_t* __restrict__ path,
                   int32_t* __restrict__ next_block, int32_t* __restrict__ walk_status) {
  extern __shared__ __align__(8) unsigned char tail_smem[];
  const int b = blockIdx.x;
  const int rows = N * L;
  uint64_t* s_bits = reinterpret_cast<uint64_t*>(tail_smem);
  int32_t* s_state = reinterpret_cast<int32_t*>(s_bits + N);
  int32_t* s_top = s_state + rows;
  float* s_conf = reinterpret_cast<float*>(s_top + rows);
  int32_t* s_off = reinterpret_cast<int32_t*>(s_conf + rows);
  int32_t* s_idx = s_off + (N + 1);
  int* s_link = s_idx + parent_cap;
  const int32_t* state = block_tokens + (int64_t)b * rows;
  {
    auto copy4 = [](void* dst, const void* src) {
      asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(
                       (uint32_t)__cvta_generic_to_shared(dst)),
                   "l"(src)
                   : "memory");
    };
    const int32_t* off = parent_off + (int64_t)b * (N + 1);
    const int32_t* idx = parent_idx + (int64_t)b * parent_cap;
    for (int i = threadIdx.x; i < rows; i += kTailThreads) copy4(s_state + i, state + i);
    for (int i = threadIdx.x; i <= N; i += kTailThreads) copy4(s_off + i, off + i);
    for (int i = threadIdx.x; i < parent_cap; i += kTailThreads) copy4(s_idx + i, idx + i);
    for (int i = threadIdx.x; i < N; i += kTailThreads) s_link[i] = kNoLink;
  }
#if __CUDA_ARCH__ >= 900
  cudaGridDependencySynchronize();  // the reduce kernel's partials are visible
  pdl_launch_dependents();          // only now: this CTA was resident during the reduce, the next kernel's need not be
#endif
  const int sub = threadIdx.x & (kLanes - 1);
  for (int base = 0; base < rows; base += kTailThreads / kLanes) {
    const int r = base + threadIdx.x / kLanes;
    const int row = min(r, rows - 1);
    const int32_t st = state[row];
    float conf;
    int32_t tok;
    const bool ok = finalize_row<kLanes>(partials + ((int64_t)b * rows + row) * splits, splits, sub,
                                         st, mask_id, conf, tok);
    if (sub == 0 && r < rows) {
      conf_out[(int64_t)b * rows + row] = conf;
      tok_out[(int64_t)b * rows + row] = tok;
      s_conf[row] = conf;
      s_top[row] = tok;
      if (!ok && decide_status) atomicOr(decide_status + b, SPIFFY_DEV_NONFINITE);
    }
  }
  asm volatile("cp.async.wait_all;" ::: "memory");
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int node = warp; node < N; node += kTailThreads / 32) {
    const uint64_t bits = unmask_rule(s_conf + node * L, s_state + node * L, L, mask_id, rule, top_s,
                                      tau, lane);
    if (lane == 0) {
      bits_out[(int64_t)b * N + node] = bits;
      n_unmask_out[(int64_t)b * N + node] = __popcll(bits);
      s_bits[node] = bits;
    }
  }
  __syncthreads();
  const bool bad = walk_link_children(N, L, parent_cap, s_state, s_top, s_off, s_idx, s_bits, s_link,
                                      warp, kTailThreads / 32, lane);
  if (bad && lane == 0 && walk_status) atomicOr(walk_status + b, SPIFFY_DEV_BADGRAPH);
  __syncthreads();
  if (warp == 0)
    walk_chase(N, L, s_state, s_top, s_bits, s_link, path + (int64_t)b * N,
               next_block + (int64_t)b * L, accepted_node + b, n_accepted + b, lane);
}

size_t tail_smem_bytes(const spiffy_decide_desc& d, int parent_cap) {
  return (size_t)d.n_nodes * 8 +
         ((size_t)3 * d.n_nodes * d.block_len + 2 * d.n_nodes + 1 + parent_cap) * 4;
}

}  // namespace

int decide_splits(const spiffy_decide_desc& d, int64_t* chunk_elems) {
  // A slice is at most what one CTA holds in registers: kReduceThreads * kUnroll
  // vectors of 16 bytes (8192 bf16 or 4096 fp32 logits); slices start on
  // 16-byte boundaries.
  const int64_t epv = d.logits_dtype == SPIFFY_BF16 ? 8 : 4;
  const int64_t most = (int64_t)kReduceThreads * kUnroll * epv;
  const int64_t splits = (d.vocab + most - 1) / most;
  // equal slices, rounded up to whole vectors
  int64_t chunk = (d.vocab + splits - 1) / splits;
  chunk = (chunk + epv - 1) / epv * epv;
  if (chunk_elems) *chunk_elems = chunk;
  return (int)(splits < 1 ? 1 : splits);
}

size_t decide_workspace_bytes(const spiffy_decide_desc& d) {
  const int64_t rows = (int64_t)d.batch * d.n_nodes * d.block_len;
  return (size_t)rows * decide_splits(d, nullptr) * sizeof(Partial);
}

namespace {

spiffy_status launch_reduce(const spiffy_decide_desc& d, const void* logits,
                            const int32_t* block_tokens, Partial* partials, int splits,
                            int64_t chunk, int early_trigger, cudaStream_t stream) {
  const int rows = d.batch * d.n_nodes * d.block_len;
  const dim3 grid(splits, rows);
  cudaError_t e;
  if (d.logits_dtype == SPIFFY_BF16)
    e = launch_pdl(decide_reduce_kernel<__nv_bfloat16>, grid, dim3(kReduceThreads), (size_t)0, stream,
                   static_cast<const __nv_bfloat16*>(logits), (int64_t)d.row_stride, (int)d.vocab,
                   chunk, splits, block_tokens, (int)d.mask_token_id, partials, early_trigger);
  else
    e = launch_pdl(decide_reduce_kernel<float>, grid, dim3(kReduceThreads), (size_t)0, stream,
                   static_cast<const float*>(logits), (int64_t)d.row_stride, (int)d.vocab, chunk,
                   splits, block_tokens, (int)d.mask_token_id, partials, early_trigger);
  count_launch();
  return e == cudaSuccess ? SPIFFY_OK : SPIFFY_ECUDA;
}

}  // namespace

spiffy_status launch_decide(const spiffy_decide_desc& d, const void* logits,
                            const int32_t* block_tokens, float* conf,
                            int32_t* top_tok, uint64_t* unmask_bits,
                            int32_t* n_unmask, int32_t* dev_status, void* ws,
                            cudaStream_t stream) {
  int64_t chunk = 0;
  const int splits = decide_splits(d, &chunk);
  Partial* partials = static_cast<Partial*>(ws);
  const spiffy_status st = launch_reduce(d, logits, block_tokens, partials, splits, chunk, 0, stream);
  if (st != SPIFFY_OK) return st;
  // The finalize kernel's launch overlaps the tail of the reduce kernel; it
  // waits on the device (cudaGridDependencySynchronize) for the partials.
  const Partial* cpart = partials;
  const cudaError_t e =
      launch_pdl(decide_finalize_kernel, dim3(d.batch * d.n_nodes), dim3(kFinalizeThreads), (size_t)0,
                 stream, cpart, splits, (int)d.n_nodes, (int)d.block_len, block_tokens,
                 (int)d.mask_token_id, (int)d.rule, (int)d.top_s, d.threshold, conf, top_tok,
                 unmask_bits, n_unmask, dev_status);
  count_launch();
  return e == cudaSuccess ? SPIFFY_OK : SPIFFY_ECUDA;
}

// The finalize kernel alone, on partial results another kernel produced
// (`splits` per row, in the layout of this file's reduce kernel).
spiffy_status launch_decide_finalize(const spiffy_decide_desc& d, const void* partials, int splits,
                                     const int32_t* block_tokens, float* conf, int32_t* top_tok,
                                     uint64_t* unmask_bits, int32_t* n_unmask, int32_t* dev_status,
                                     cudaStream_t stream) {
  const Partial* cpart = static_cast<const Partial*>(partials);
  const cudaError_t e =
      launch_pdl(decide_finalize_kernel, dim3(d.batch * d.n_nodes), dim3(kFinalizeThreads), (size_t)0,
                 stream, cpart, splits, (int)d.n_nodes, (int)d.block_len, block_tokens,
                 (int)d.mask_token_id, (int)d.rule, (int)d.top_s, d.threshold, conf, top_tok,
                 unmask_bits, n_unmask, dev_status);
  count_launch();
  return e == cudaSuccess ? SPIFFY_OK : SPIFFY_ECUDA;
}

// Decision and walk in one call.  Small graphs (at most kTailRows rows per
// sequence, arrays within the default shared-memory limit) take the fused tail:
// two launches instead of three.  Larger ones keep one finalize CTA per node,
// which spreads the merging over more SMs.
constexpr int kTailRows = 512;
spiffy_status launch_decide_walk(const spiffy_decide_desc& d, const void* logits,
                                 const int32_t* block_tokens, float* conf, int32_t* top_tok,
                                 uint64_t* unmask_bits, int32_t* n_unmask,
                                 int32_t* decide_status, const int32_t* parent_off,
                                 const int32_t* parent_idx, int32_t parent_cap,
                                 int32_t* accepted_node, int32_t* n_accepted, int32_t* path,
                                 int32_t* next_block, int32_t* walk_status, void* ws,
                                 cudaStream_t stream) {
  const size_t smem = tail_smem_bytes(d, parent_cap);
  if ((int64_t)d.n_nodes * d.block_len > kTailRows || smem > 48 * 1024) {
    const spiffy_status st = launch_decide(d, logits, block_tokens, conf, top_tok, unmask_bits,
                                           n_unmask, decide_status, ws, stream);
    if (st != SPIFFY_OK) return st;
    return launch_walk(d, block_tokens, parent_off, parent_idx, parent_cap, top_tok, unmask_bits,
                       accepted_node, n_accepted, path, next_block, walk_status, stream);
  }
  int64_t chunk = 0;
  const int splits = decide_splits(d, &chunk);
  Partial* partials = static_cast<Partial*>(ws);
  const spiffy_status st = launch_reduce(d, logits, block_tokens, partials, splits, chunk, 1, stream);
  if (st != SPIFFY_OK) return st;
  const Partial* cpart = partials;
  const int rows = d.n_nodes * d.block_len;
  auto launch = [&](auto kernel) {
    return launch_pdl(kernel, dim3(d.batch), dim3(kTailThreads), smem, stream, cpart, splits,
                      (int)d.n_nodes, (int)d.block_len, block_tokens, (int)d.mask_token_id,
                      (int)d.rule, (int)d.top_s, d.threshold, conf, top_tok, unmask_bits, n_unmask,
                      decide_status, parent_off, parent_idx, (int)parent_cap, accepted_node,
                      n_accepted, path, next_block, walk_status);
  };
  const cudaError_t e = rows <= kTailThreads / 8   ? launch(decide_tail_kernel<8>)
                        : rows <= kTailThreads / 4 ? launch(decide_tail_kernel<4>)
                                                   : launch(decide_tail_kernel<2>);
  count_launch();
  return e == cudaSuccess ? SPIFFY_OK : SPIFFY_ECUDA;
}

}  // namespace spiffy
