// Decision kernels: steps 1-4 of Algorithm 1 (the function Next() of App. A)
// evaluated for every node of the draft graph.
//
//   decide_reduce_kernel    streams the logits rows of still-masked positions
//                           once (the HBM-bound part): per (row, vocabulary
//                           slice) the maximum, the sum of exponentials and the
//                           lowest index that attains the maximum
//   decide_finalize_kernel  per node: merges the slices in a fixed order, turns
//                           them into (confidence, top token) and applies the
//                           unmasking rule of Sec. 3.1
//
// The argmax compares logit values exactly ((value desc, index asc) order);
// probabilities only enter the confidence.  All merges run in a fixed order, so
// repeated calls give identical bits.
#include <math.h>

#include "common.cuh"

namespace spiffy {
namespace {

// 128 threads holding 8 vectors each measured best among 64..512 threads and
// 2..16 vectors (smaller slices pay more per CTA, larger ones leave too few
// CTAs in flight per SM).
constexpr int kReduceThreads = 128;
constexpr int kUnroll = 8;  // 128-bit vectors per thread, all loaded at once

struct __align__(16) Partial {
  float m;    // slice maximum (-inf for an empty slice)
  float s;    // sum over the slice of exp(x - m)
  int idx;    // lowest index attaining m
  int pad;
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// (value desc, index asc) merge of two partial results.
__device__ __forceinline__ void merge(float& m, float& s, int& idx, float m2,
                                      float s2, int idx2) {
  if (m2 > m || (m2 == m && idx2 < idx)) idx = idx2;
  const float M = fmaxf(m, m2);
  const float f1 = (m == M) ? 1.f : ex2((m - M) * kLog2e);
  const float f2 = (m2 == M) ? 1.f : ex2((m2 - M) * kLog2e);
  s = s * f1 + s2 * f2;
  m = M;
}

template <typename T>
struct Elem;

template <>
struct Elem<__nv_bfloat16> {
  static constexpr int kPerVec = 8;
  static constexpr uint32_t kNegInf = 0xff80ff80u;  // two bf16 -inf
  static __device__ __forceinline__ float lo(uint32_t w) { return __uint_as_float(w << 16); }
  static __device__ __forceinline__ float hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
  static __device__ __forceinline__ __nv_bfloat162 pk(uint32_t w) {
    return *reinterpret_cast<const __nv_bfloat162*>(&w);
  }
  // exact maximum of one vector / of a group of vectors, on the packed bf16 pipe
  static __device__ __forceinline__ float vmax(uint4 v) {
    const __nv_bfloat162 p = __hmax2(__hmax2(pk(v.x), pk(v.y)), __hmax2(pk(v.z), pk(v.w)));
    return fmaxf(__low2float(p), __high2float(p));
  }
  static __device__ __forceinline__ float gmax(const uint4 (&v)[kUnroll]) {
    __nv_bfloat162 p = __hmax2(__hmax2(pk(v[0].x), pk(v[0].y)), __hmax2(pk(v[0].z), pk(v[0].w)));
#pragma unroll
    for (int k = 1; k < kUnroll; ++k)
      p = __hmax2(p, __hmax2(__hmax2(pk(v[k].x), pk(v[k].y)), __hmax2(pk(v[k].z), pk(v[k].w))));
    return fmaxf(__low2float(p), __high2float(p));
  }
  // sum over the vector of 2^(x * log2e - ml)
  static __device__ __forceinline__ float sum_terms(uint4 v, float ml) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    float t = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i)
      t += ex2(fmaf(lo(w[i]), kLog2e, -ml)) + ex2(fmaf(hi(w[i]), kLog2e, -ml));
    return t;
  }
  // position of the first element equal to x, kPerVec if there is none
  static __device__ __forceinline__ int first_equal(uint4 v, float x) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    int j = kPerVec;
#pragma unroll
    for (int i = 3; i >= 0; --i) {
      j = (hi(w[i]) == x) ? 2 * i + 1 : j;
      j = (lo(w[i]) == x) ? 2 * i : j;
    }
    return j;
  }
  static __device__ __forceinline__ float load1(const __nv_bfloat16* p) {
    return __bfloat162float(*p);
  }
};

template <>
struct Elem<float> {
  static constexpr int kPerVec = 4;
  static constexpr uint32_t kNegInf = 0xff800000u;
  static __device__ __forceinline__ float vmax(uint4 v) {
    return fmaxf(fmaxf(__uint_as_float(v.x), __uint_as_float(v.y)),
                 fmaxf(__uint_as_float(v.z), __uint_as_float(v.w)));
  }
  static __device__ __forceinline__ float gmax(const uint4 (&v)[kUnroll]) {
    float g = -INFINITY;
#pragma unroll
    for (int k = 0; k < kUnroll; ++k)
      g = fmaxf(g, fmaxf(fmaxf(__uint_as_float(v[k].x), __uint_as_float(v[k].y)),
                         fmaxf(__uint_as_float(v[k].z), __uint_as_float(v[k].w))));
    return g;
  }
  static __device__ __forceinline__ float sum_terms(uint4 v, float ml) {
    return (ex2(fmaf(__uint_as_float(v.x), kLog2e, -ml)) + ex2(fmaf(__uint_as_float(v.y), kLog2e, -ml))) +
           (ex2(fmaf(__uint_as_float(v.z), kLog2e, -ml)) + ex2(fmaf(__uint_as_float(v.w), kLog2e, -ml)));
  }
  static __device__ __forceinline__ int first_equal(uint4 v, float x) {
    int j = kPerVec;
    j = (__uint_as_float(v.w) == x) ? 3 : j;
    j = (__uint_as_float(v.z) == x) ? 2 : j;
    j = (__uint_as_float(v.y) == x) ? 1 : j;
    j = (__uint_as_float(v.x) == x) ? 0 : j;
    return j;
  }
  static __device__ __forceinline__ float load1(const float* p) { return *p; }
};

// grid = (splits, B*N*L); one CTA reduces one vocabulary slice of one row.  A
// slice is at most kReduceThreads * kUnroll vectors, so that every thread holds
// its whole share in registers: all loads go out at once, the slice maximum is
// found first and the exponentials are then taken against it directly.
template <typename T>
__global__ void __launch_bounds__(kReduceThreads)
decide_reduce_kernel(const T* __restrict__ logits, int64_t row_stride, int V,
                     int64_t chunk, int splits,
                     const int32_t* __restrict__ block_tokens, int mask_id,
                     Partial* __restrict__ partials) {
#if __CUDA_ARCH__ >= 900
  cudaGridDependencySynchronize();  // inputs written by earlier kernels are visible
#endif
  const int row = blockIdx.y;
  if (block_tokens[row] != mask_id) return;  // already unmasked: never read
  const int split = blockIdx.x;
  const int64_t begin = (int64_t)split * chunk;
  const int64_t end = min((int64_t)V, begin + chunk);
  constexpr int EPV = Elem<T>::kPerVec;
  constexpr uint32_t NI = Elem<T>::kNegInf;
  const T* base = logits + (int64_t)row * row_stride;
  const int nvec = begin < end ? (int)((end - begin) / EPV) : 0;  // <= kReduceThreads * kUnroll
  const int ntail = begin < end ? (int)(end - begin) - nvec * EPV : 0;  // < EPV, last slice only
  const uint4* p = reinterpret_cast<const uint4*>(base + begin);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // 1. the thread's vectors t, t + kReduceThreads, ...; thread 0 also takes the ragged tail
  uint4 v[kUnroll];
#pragma unroll
  for (int u = 0; u < kUnroll; ++u)
    v[u] = (tid + u * kReduceThreads < nvec) ? ld_stream(p + tid + u * kReduceThreads)
                                             : make_uint4(NI, NI, NI, NI);
  float tail[EPV];
#pragma unroll
  for (int e = 0; e < EPV; ++e)
    tail[e] = (tid == 0 && e < ntail) ? Elem<T>::load1(base + begin + (int64_t)nvec * EPV + e) : -INFINITY;
  // 2. slice maximum: lanes, warps
  float m = Elem<T>::gmax(v);
#pragma unroll
  for (int e = 0; e < EPV; ++e) m = fmaxf(m, tail[e]);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
  __shared__ float warp_m[kReduceThreads / 32], warp_s[kReduceThreads / 32];
  __shared__ int slice_idx;
  if (lane == 0) warp_m[warp] = m;
  if (tid == 0) slice_idx = 0x7fffffff;
  __syncthreads();
  m = warp_m[0];
#pragma unroll
  for (int w = 1; w < kReduceThreads / 32; ++w) m = fmaxf(m, warp_m[w]);
  // 3. sum of exp(x - m) and the lowest index that attains m
  const float ml = (m == -INFINITY) ? 0.f : m * kLog2e;  // an all -inf slice sums to 0
  float s = 0.f;
  int idx = 0x7fffffff;
#pragma unroll
  for (int u = kUnroll - 1; u >= 0; --u) {
    s += Elem<T>::sum_terms(v[u], ml);
    if (Elem<T>::vmax(v[u]) == m)  // rare: only the vectors that hold the slice maximum are searched
      idx = (int)begin + (tid + u * kReduceThreads) * EPV + Elem<T>::first_equal(v[u], m);
  }
  if (ntail > 0 && tid == 0) {
    int tidx = 0x7fffffff;
#pragma unroll
    for (int e = EPV - 1; e >= 0; --e) {
      s += ex2(fmaf(tail[e], kLog2e, -ml));  // -inf beyond the tail: adds 0
      if (e < ntail && tail[e] == m) tidx = (int)begin + nvec * EPV + e;
    }
    idx = min(idx, tidx);
  }
  if (m == -INFINITY) idx = 0x7fffffff;
  // fixed order: lanes (butterfly), then warps
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    s += __shfl_xor_sync(0xffffffffu, s, off);
    idx = min(idx, __shfl_xor_sync(0xffffffffu, idx, off));
  }
  if (lane == 0) {
    warp_s[warp] = s;
    if (idx != 0x7fffffff) atomicMin(&slice_idx, idx);
  }
  __syncthreads();
  if (tid == 0) {
    s = warp_s[0];
    for (int w = 1; w < kReduceThreads / 32; ++w) s += warp_s[w];
    partials[(int64_t)row * splits + split] = Partial{m, s, slice_idx, 0};
  }
}

// grid = B*N nodes, 512 threads: eight threads per position merge the slices of
// its row, then threads 0..63 apply the rule (thread l owns position l).
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
  __shared__ uint32_t sballot[2];
  if (threadIdx.x < 64) sconf[threadIdx.x] = -INFINITY;
  __syncthreads();
  {
    const int row = node * L + min(pos, L - 1);
    // the token and the partials are read together (one trip to memory); the
    // partials of an unmasked row were never written and are ignored below
    const int32_t state = block_tokens[row];
    float m = -INFINITY, s = 0.f;
    int idx = 0x7fffffff;
    const Partial* p = partials + (int64_t)row * splits;
    for (int k = sub; k < splits; k += 8) {
      const Partial q = p[k];
      merge(m, s, idx, q.m, q.s, q.idx);
    }
#pragma unroll
    for (int off = 4; off > 0; off >>= 1) {  // fixed order inside the group of eight
      const float m2 = __shfl_xor_sync(0xffffffffu, m, off);
      const float s2 = __shfl_xor_sync(0xffffffffu, s, off);
      const int i2 = __shfl_xor_sync(0xffffffffu, idx, off);
      merge(m, s, idx, m2, s2, i2);
    }
    if (sub == 0 && pos < L) {
      const bool masked = state == mask_id;
      const float conf = masked ? fminf(1.0f, 1.0f / s) : -INFINITY;  // the sum can round just below one
      conf_out[row] = conf;
      tok_out[row] = masked ? idx : state;
      sconf[pos] = conf;
      // a usable row has a finite maximum and a finite, positive sum (the sum is one or more up to rounding)
      if (masked && (!(fabsf(m) < INFINITY) || !(s > 0.f) || !(s < INFINITY))) {
        if (dev_status) atomicOr(dev_status + node / N, SPIFFY_DEV_NONFINITE);
      }
    }
  }
  __syncthreads();
  if (threadIdx.x >= 64) return;
  const int l = threadIdx.x;
  const bool masked = l < L && block_tokens[node * L + min(l, L - 1)] == mask_id;
  const float conf = masked ? sconf[l] : -INFINITY;
  // rank among the masked positions by (confidence desc, position asc); the
  // confidence of an unmasked position is -inf and a masked one's is not
  int rank = 0;
  if (masked) {
    for (int j = 0; j < L; ++j) {
      const float c = sconf[j];
      rank += (c > conf || (c == conf && j < l)) ? 1 : 0;
    }
  }
  bool take;
  if (rule == SPIFFY_RULE_TOPS) {
    take = masked && rank < top_s;
  } else {
    const bool pass = masked && conf > tau;  // strict, Sec. 3.1
    const uint32_t any0 = __ballot_sync(0xffffffffu, pass);
    if ((l & 31) == 0) sballot[l >> 5] = any0;
    asm volatile("bar.sync 1, 64;" ::: "memory");
    const bool any = (sballot[0] | sballot[1]) != 0u;
    asm volatile("bar.sync 1, 64;" ::: "memory");
    take = any ? pass : (masked && rank == 0);
  }
  const uint32_t bal = __ballot_sync(0xffffffffu, take);
  if ((l & 31) == 0) sballot[l >> 5] = bal;
  asm volatile("bar.sync 1, 64;" ::: "memory");
  if (l == 0) {
    const uint64_t bits = (uint64_t)sballot[0] | ((uint64_t)sballot[1] << 32);
    bits_out[node] = bits;
    n_unmask_out[node] = __popcll(bits);
  }
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

spiffy_status launch_decide(const spiffy_decide_desc& d, const void* logits,
                            const int32_t* block_tokens, float* conf,
                            int32_t* top_tok, uint64_t* unmask_bits,
                            int32_t* n_unmask, int32_t* dev_status, void* ws,
                            cudaStream_t stream) {
  int64_t chunk = 0;
  const int splits = decide_splits(d, &chunk);
  const int rows = d.batch * d.n_nodes * d.block_len;
  Partial* partials = static_cast<Partial*>(ws);
  const dim3 grid(splits, rows);
  cudaError_t e;
  if (d.logits_dtype == SPIFFY_BF16)
    e = launch_pdl(decide_reduce_kernel<__nv_bfloat16>, grid, dim3(kReduceThreads), (size_t)0, stream,
                   static_cast<const __nv_bfloat16*>(logits), (int64_t)d.row_stride, (int)d.vocab,
                   chunk, splits, block_tokens, (int)d.mask_token_id, partials);
  else
    e = launch_pdl(decide_reduce_kernel<float>, grid, dim3(kReduceThreads), (size_t)0, stream,
                   static_cast<const float*>(logits), (int64_t)d.row_stride, (int)d.vocab, chunk,
                   splits, block_tokens, (int)d.mask_token_id, partials);
  count_launch();
  if (e != cudaSuccess) return SPIFFY_ECUDA;

  // The finalize kernel's launch overlaps the tail of the reduce kernel; it
  // waits on the device (cudaGridDependencySynchronize) for the partials.
  const Partial* cpart = partials;
  e = launch_pdl(decide_finalize_kernel, dim3(d.batch * d.n_nodes), dim3(kFinalizeThreads), (size_t)0, stream,
                 cpart, splits, (int)d.n_nodes, (int)d.block_len, block_tokens,
                 (int)d.mask_token_id, (int)d.rule, (int)d.top_s, d.threshold, conf, top_tok,
                 unmask_bits, n_unmask, dev_status);
  count_launch();
  return e == cudaSuccess ? SPIFFY_OK : SPIFFY_ECUDA;
}

}  // namespace spiffy
