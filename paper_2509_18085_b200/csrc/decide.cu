// Decision kernels: steps 1-4 of Algorithm 1 (the function Next() of App. A)
// evaluated for every node of the draft graph.
//
//   decide_reduce_kernel    streams the logits rows of still-masked positions
//                           once (the HBM-bound part): per (row, vocabulary
//                           slice) an online (max, argmax, sum of exponentials)
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

constexpr int kReduceThreads = 256;
constexpr int kUnroll = 4;

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

// Running state of one thread (or of a merged group of threads).
struct Acc {
  float m = -INFINITY;  // running maximum
  float ml = 0.f;       // m * log2(e), 0 while m is still -inf
  float s = 0.f;        // sum of exp(x - m)
  int idx = 0x7fffffff;
};

__device__ __forceinline__ void raise_max(Acc& a, float vm, int idx) {
  const float nl = vm * kLog2e;
  a.s *= ex2(a.ml - nl);
  a.m = vm;
  a.ml = nl;
  a.idx = idx;
}

__device__ __forceinline__ float term(const Acc& a, float x) {
  return ex2(fmaf(x, kLog2e, -a.ml));
}

// (value desc, index asc) merge of two accumulators.
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
  static __device__ __forceinline__ void consume(Acc& a, uint4 v, int base) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    float f[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
    // exact maximum of the eight inputs on the packed bf16 pipe
    __nv_bfloat162 p0 = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&w[0]),
                                *reinterpret_cast<const __nv_bfloat162*>(&w[1]));
    __nv_bfloat162 p1 = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&w[2]),
                                *reinterpret_cast<const __nv_bfloat162*>(&w[3]));
    p0 = __hmax2(p0, p1);
    const float vm = fmaxf(__low2float(p0), __high2float(p0));
    if (vm > a.m) {
      int j = 7;
#pragma unroll
      for (int i = 6; i >= 0; --i) j = (f[i] == vm) ? i : j;
      raise_max(a, vm, base + j);
    }
    float t[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) t[i] = term(a, f[i]);
    a.s += ((t[0] + t[1]) + (t[2] + t[3])) + ((t[4] + t[5]) + (t[6] + t[7]));
  }
  static __device__ __forceinline__ float load1(const __nv_bfloat16* p) {
    return __bfloat162float(*p);
  }
};

template <>
struct Elem<float> {
  static constexpr int kPerVec = 4;
  static __device__ __forceinline__ void consume(Acc& a, uint4 v, int base) {
    const float f[4] = {__uint_as_float(v.x), __uint_as_float(v.y),
                        __uint_as_float(v.z), __uint_as_float(v.w)};
    const float vm = fmaxf(fmaxf(f[0], f[1]), fmaxf(f[2], f[3]));
    if (vm > a.m) {
      int j = 3;
#pragma unroll
      for (int i = 2; i >= 0; --i) j = (f[i] == vm) ? i : j;
      raise_max(a, vm, base + j);
    }
    a.s += (term(a, f[0]) + term(a, f[1])) + (term(a, f[2]) + term(a, f[3]));
  }
  static __device__ __forceinline__ float load1(const float* p) { return *p; }
};

// grid = (splits, B*N*L); one CTA reduces one vocabulary slice of one row.
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
  const T* base = logits + (int64_t)row * row_stride;
  Acc a;
  if (begin < end) {
    const int nvec = (int)((end - begin) / EPV);
    const uint4* p = reinterpret_cast<const uint4*>(base + begin);
    for (int i = threadIdx.x; i < nvec; i += kReduceThreads * kUnroll) {
      uint4 v[kUnroll];
#pragma unroll
      for (int k = 0; k < kUnroll; ++k)
        if (i + k * kReduceThreads < nvec) v[k] = ld_stream(p + i + k * kReduceThreads);
#pragma unroll
      for (int k = 0; k < kUnroll; ++k)
        if (i + k * kReduceThreads < nvec)
          Elem<T>::consume(a, v[k], (int)begin + (i + k * kReduceThreads) * EPV);
    }
    // ragged tail of the slice (fewer than one vector)
    const int64_t tail = begin + (int64_t)nvec * EPV;
    if (threadIdx.x == 0) {
      for (int64_t e = tail; e < end; ++e) {
        const float x = Elem<T>::load1(base + e);
        if (x > a.m) raise_max(a, x, (int)e);
        a.s += term(a, x);
      }
    }
  }
  // CTA-wide merge in a fixed order: lanes, then warps
  float m = a.m, s = a.s;
  int idx = a.idx;
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const float m2 = __shfl_down_sync(0xffffffffu, m, off);
    const float s2 = __shfl_down_sync(0xffffffffu, s, off);
    const int i2 = __shfl_down_sync(0xffffffffu, idx, off);
    merge(m, s, idx, m2, s2, i2);
  }
  __shared__ Partial warp_part[kReduceThreads / 32];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) warp_part[warp] = Partial{m, s, idx, 0};
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < kReduceThreads / 32; ++w)
      merge(m, s, idx, warp_part[w].m, warp_part[w].s, warp_part[w].idx);
    partials[(int64_t)row * splits + split] = Partial{m, s, idx, 0};
  }
}

// grid = B*N nodes, 64 threads: thread l owns position l of the node.
__global__ void __launch_bounds__(64)
decide_finalize_kernel(const Partial* __restrict__ partials, int splits, int N,
                       int L, const int32_t* __restrict__ block_tokens,
                       int mask_id, int rule, int top_s, float tau,
                       float* __restrict__ conf_out, int32_t* __restrict__ tok_out,
                       uint64_t* __restrict__ bits_out,
                       int32_t* __restrict__ n_unmask_out,
                       int32_t* __restrict__ dev_status) {
#if __CUDA_ARCH__ >= 900
  cudaGridDependencySynchronize();  // the reduce kernel's partials are visible
#endif
  const int node = blockIdx.x;
  const int l = threadIdx.x;
  __shared__ float sconf[64];
  __shared__ uint32_t sballot[2];
  bool masked = false;
  float conf = -INFINITY;
  if (l < L) {
    const int row = node * L + l;
    const int32_t state = block_tokens[row];
    int tok = state;
    masked = state == mask_id;
    if (masked) {
      const Partial* p = partials + (int64_t)row * splits;
      float m = p[0].m, s = p[0].s;
      int idx = p[0].idx;
      for (int k = 1; k < splits; ++k) merge(m, s, idx, p[k].m, p[k].s, p[k].idx);
      conf = 1.0f / s;
      tok = idx;
      // a usable row has a finite maximum and a finite, positive sum
      if (!(fabsf(m) < INFINITY) || !(s >= 1.0f) || !(s < INFINITY)) {
        if (dev_status) atomicOr(dev_status + node / N, SPIFFY_DEV_NONFINITE);
      }
    }
    conf_out[row] = conf;
    tok_out[row] = tok;
  }
  sconf[l] = masked ? conf : -INFINITY;
  __syncthreads();
  // rank among the masked positions by (confidence desc, position asc)
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
    const int any = __syncthreads_or(pass ? 1 : 0);
    take = any ? pass : (masked && rank == 0);
  }
  const uint32_t b = __ballot_sync(0xffffffffu, take);
  if ((l & 31) == 0) sballot[l >> 5] = b;
  __syncthreads();
  if (l == 0) {
    const uint64_t bits = (uint64_t)sballot[0] | ((uint64_t)sballot[1] << 32);
    bits_out[node] = bits;
    n_unmask_out[node] = __popcll(bits);
  }
}

}  // namespace

int decide_splits(const spiffy_decide_desc& d, int64_t* chunk_elems) {
  // Enough CTAs to keep every SM streaming (about 8 CTAs of 256 threads per
  // SM over 148 SMs), slices never shorter than 4096 elements and cut on
  // 2048-element boundaries so that every slice starts on a 16-byte boundary.
  const int64_t rows = (int64_t)d.batch * d.n_nodes * d.block_len;
  int64_t want = (148 * 8 + rows - 1) / rows;
  const int64_t max_by_len = (d.vocab + 4095) / 4096;
  if (want > max_by_len) want = max_by_len;
  if (want < 1) want = 1;
  if (want > 64) want = 64;
  int64_t chunk = (d.vocab + want - 1) / want;
  chunk = (chunk + 2047) / 2048 * 2048;
  const int splits = (int)((d.vocab + chunk - 1) / chunk);
  if (chunk_elems) *chunk_elems = chunk;
  return splits < 1 ? 1 : splits;
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
  e = launch_pdl(decide_finalize_kernel, dim3(d.batch * d.n_nodes), dim3(64), (size_t)0, stream,
                 cpart, splits, (int)d.n_nodes, (int)d.block_len, block_tokens,
                 (int)d.mask_token_id, (int)d.rule, (int)d.top_s, d.threshold, conf, top_tok,
                 unmask_bits, n_unmask, dev_status);
  count_launch();
  return e == cudaSuccess ? SPIFFY_OK : SPIFFY_ECUDA;
}

}  // namespace spiffy
