// Device code of the decision step shared by its kernels: the vocabulary-slice
// reduce (Algorithm 1, steps 1-2: per position the top token and its softmax
// probability), the fixed-order merge of slices, and the unmasking rule of
// Sec. 3.1 (step 3).
//
// The argmax compares logit values exactly ((value desc, index asc) order);
// probabilities only enter the confidence.  All merges run in a fixed order, so
// repeated calls -- and the different kernels that use this code -- give
// identical bits.
#pragma once
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

// acc += {2^(x0 * log2e - ml), 2^(x1 * log2e - ml)}; k2 = {log2e, log2e}, nml2 = {-ml, -ml}
__device__ __forceinline__ uint64_t add_exp2(uint64_t acc, float x0, float x1, uint64_t k2,
                                             uint64_t nml2) {
  float a0, a1;
  unpack2(fma2(pack2(x0, x1), k2, nml2), a0, a1);
  return add2(acc, pack2(ex2(a0), ex2(a1)));
}

// (value desc, index asc) merge of two partial results.
__device__ __forceinline__ void merge(float& m, float& s, int& idx, float m2,
                                      float s2, int idx2) {
  if (m2 > m || (m2 == m && idx2 < idx)) idx = idx2;
  const float M = fmaxf(m, m2);
  const float f1 = (m == M) ? 1.f : ex2((m - M) * kLog2e);
  const float f2 = (m2 == M) ? 1.f : ex2((m2 - M) * kLog2e);
  s = __fmaf_rn(s, f1, __fmul_rn(s2, f2));  // spelled out: every instance rounds the same way
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
  // true when some element of the vector equals x (x is one of the inputs, hence a bf16 value)
  static __device__ __forceinline__ bool holds(uint4 v, float x) {
    const __nv_bfloat162 xx = __float2bfloat162_rn(x);
    return (__heq2_mask(pk(v.x), xx) | __heq2_mask(pk(v.y), xx) | __heq2_mask(pk(v.z), xx) |
            __heq2_mask(pk(v.w), xx)) != 0u;
  }
  static __device__ __forceinline__ float gmax(const uint4 (&v)[kUnroll]) {
    __nv_bfloat162 p = __hmax2(__hmax2(pk(v[0].x), pk(v[0].y)), __hmax2(pk(v[0].z), pk(v[0].w)));
#pragma unroll
    for (int k = 1; k < kUnroll; ++k)
      p = __hmax2(p, __hmax2(__hmax2(pk(v[k].x), pk(v[k].y)), __hmax2(pk(v[k].z), pk(v[k].w))));
    return fmaxf(__low2float(p), __high2float(p));
  }
  // acc (two running sums) += 2^(x * log2e - ml) over the vector, even elements into the
  // low lane, odd ones into the high lane
  static __device__ __forceinline__ uint64_t sum_terms(uint4 v, uint64_t k2, uint64_t nml2,
                                                       uint64_t acc) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) acc = add_exp2(acc, lo(w[i]), hi(w[i]), k2, nml2);
    return acc;
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
  static __device__ __forceinline__ bool holds(uint4 v, float x) { return vmax(v) == x; }
  static __device__ __forceinline__ float gmax(const uint4 (&v)[kUnroll]) {
    float g = -INFINITY;
#pragma unroll
    for (int k = 0; k < kUnroll; ++k)
      g = fmaxf(g, fmaxf(fmaxf(__uint_as_float(v[k].x), __uint_as_float(v[k].y)),
                         fmaxf(__uint_as_float(v[k].z), __uint_as_float(v[k].w))));
    return g;
  }
  static __device__ __forceinline__ uint64_t sum_terms(uint4 v, uint64_t k2, uint64_t nml2,
                                                       uint64_t acc) {
    acc = add_exp2(acc, __uint_as_float(v.x), __uint_as_float(v.y), k2, nml2);
    return add_exp2(acc, __uint_as_float(v.z), __uint_as_float(v.w), k2, nml2);
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

// One CTA of kReduceThreads threads reduces one vocabulary slice
// [split * chunk, min(V, (split + 1) * chunk)) of the logits row at `base` to
// (maximum, sum of exp(x - maximum), lowest index attaining the maximum).  A
// slice is at most kReduceThreads * kUnroll vectors, so that every thread holds
// its whole share in registers: all loads go out at once, the slice maximum is
// found first and the exponentials are then taken against it directly.  All
// threads of the CTA call it together; thread 0 stores the result.  `k` is
// log2(e) for the plain softmax; the sampled decision passes log2(e) / T and
// gets the sum of exp((x - maximum) / T).
template <typename T>
__device__ __forceinline__ void reduce_slice(const T* __restrict__ base, int V, int64_t chunk,
                                             int split, Partial* __restrict__ out,
                                             const float k = kLog2e) {
  const int64_t begin = (int64_t)split * chunk;
  const int64_t end = min((int64_t)V, begin + chunk);
  constexpr int EPV = Elem<T>::kPerVec;
  constexpr uint32_t NI = Elem<T>::kNegInf;
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
  const float ml = (m == -INFINITY) ? 0.f : m * k;  // an all -inf slice sums to 0
  const uint64_t k2 = pack2(k, k), nml2 = pack2(-ml, -ml);
  uint64_t acc = pack2(0.f, 0.f);
  int idx = 0x7fffffff;
#pragma unroll
  for (int u = kUnroll - 1; u >= 0; --u) {
    acc = Elem<T>::sum_terms(v[u], k2, nml2, acc);
    if (Elem<T>::holds(v[u], m))  // rare: only the vectors that hold the slice maximum are searched
      idx = (int)begin + (tid + u * kReduceThreads) * EPV + Elem<T>::first_equal(v[u], m);
  }
  float s;
  {
    float s0, s1;
    unpack2(acc, s0, s1);
    s = s0 + s1;
  }
  if (ntail > 0 && tid == 0) {
    int tidx = 0x7fffffff;
#pragma unroll
    for (int e = EPV - 1; e >= 0; --e) {
      s += ex2(fmaf(tail[e], k, -ml));  // -inf beyond the tail: adds 0
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
    *out = Partial{m, s, slice_idx, 0};
  }
}

// kLanes (8, 4, 2 or 1) neighbouring lanes merge the slices of one row and lane
// 0 of the group gets the row's confidence and top token (Algorithm 1, steps
// 1-2).  The order is fixed and the same for every kLanes: eight accumulators
// (accumulator j takes slices j, j + 8, ...) are combined by the butterfly
// 4, 2, 1 with the lower index first; a lane holds the accumulators j = sub,
// sub + kLanes, ... and does the butterfly steps that stay inside it locally.
// Returns false on lane 0 when the row is masked and not usable.
template <int kLanes>
__device__ __forceinline__ bool finalize_row(const Partial* __restrict__ p, int splits, int sub,
                                             int32_t state, int mask_id, float& conf, int32_t& tok) {
  constexpr int kAcc = 8 / kLanes;
  float m[kAcc], s[kAcc];
  int idx[kAcc];
#pragma unroll
  for (int a = 0; a < kAcc; ++a) {
    m[a] = -INFINITY;
    s[a] = 0.f;
    idx[a] = 0x7fffffff;
  }
  // this lane's slices are sub, sub + kLanes, sub + 2 kLanes, ...; slice number t
  // goes to accumulator t mod kAcc.  They are fetched kBatch at a time, all
  // loads of a batch in flight together; a missing slice merges as the identity.
  constexpr int kBatch = kAcc > 4 ? kAcc : 4;
  for (int t0 = 0; sub + kLanes * t0 < splits; t0 += kBatch) {
    Partial q[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const int k = sub + kLanes * (t0 + u);
      q[u] = Partial{-INFINITY, 0.f, 0x7fffffff, 0};
      if (k < splits && state == mask_id) {  // read at L2: another grid wrote these while this CTA may already have been resident; the slices of an unmasked row were never written
        const int4 w = __ldcg(reinterpret_cast<const int4*>(p + k));
        q[u] = Partial{__int_as_float(w.x), __int_as_float(w.y), w.z, w.w};
      }
    }
#pragma unroll
    for (int u = 0; u < kBatch; ++u)
      merge(m[u % kAcc], s[u % kAcc], idx[u % kAcc], q[u].m, q[u].s, q[u].idx);
  }
#pragma unroll
  for (int oa = kAcc / 2; oa > 0; oa >>= 1) {  // butterfly steps 4.. down to kLanes
#pragma unroll
    for (int a = 0; a < kAcc; ++a)
      if (a < oa) merge(m[a], s[a], idx[a], m[a + oa], s[a + oa], idx[a + oa]);
  }
#pragma unroll
  for (int off = kLanes / 2; off > 0; off >>= 1) {  // the remaining steps cross lanes
    const float m2 = __shfl_xor_sync(0xffffffffu, m[0], off);
    const float s2 = __shfl_xor_sync(0xffffffffu, s[0], off);
    const int i2 = __shfl_xor_sync(0xffffffffu, idx[0], off);
    merge(m[0], s[0], idx[0], m2, s2, i2);
  }
  const bool masked = state == mask_id;
  conf = masked ? fminf(1.0f, 1.0f / s[0]) : -INFINITY;  // the sum can round just below one
  tok = masked ? idx[0] : state;
  // a usable row has a finite maximum and a finite, positive sum (the sum is one or more up to rounding)
  return !(masked && (!(fabsf(m[0]) < INFINITY) || !(s[0] > 0.f) || !(s[0] < INFINITY)));
}

// One warp applies the unmasking rule of Sec. 3.1 (Algorithm 1, step 3) to one
// node; lane k owns positions k and k + 32.  conf: the node's L confidences,
// -inf at unmasked positions.  Returns the bit mask of positions to unmask.
__device__ __forceinline__ uint64_t unmask_rule(const float* conf, const int32_t* state, int L,
                                                int mask_id, int rule, int top_s, float tau,
                                                int lane) {
  const unsigned full = 0xffffffffu;
  bool masked[2], take[2];
  float c[2];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int l = lane + 32 * h;
    masked[h] = l < L && state[min(l, L - 1)] == mask_id;
    c[h] = masked[h] ? conf[l] : -INFINITY;
  }
  if (rule == SPIFFY_RULE_TOPS && top_s > 1) {
    // rank among the masked positions by (confidence desc, position asc); the
    // confidence of an unmasked position is -inf and a masked one's is not
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int l = lane + 32 * h;
      int rank = 0;
      if (masked[h]) {
        for (int j = 0; j < L; ++j) {
          const float cj = conf[j];
          rank += (cj > c[h] || (cj == c[h] && j < l)) ? 1 : 0;
        }
      }
      take[h] = masked[h] && rank < top_s;
    }
  } else {
    // only the single most confident masked position matters (top-1, or the
    // fallback of the threshold rule): a warp arg-max, ties to the lower position
    float bc = (c[0] == c[0]) ? c[0] : -INFINITY;  // an unusable row never wins
    int bp = lane;
    if (c[1] > bc) {
      bc = c[1];
      bp = lane + 32;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const float c2 = __shfl_xor_sync(full, bc, off);
      const int p2 = __shfl_xor_sync(full, bp, off);
      if (c2 > bc || (c2 == bc && p2 < bp)) {
        bc = c2;
        bp = p2;
      }
    }
    const bool any_masked = __any_sync(full, masked[0] || masked[1]);
    bool pass0 = false, pass1 = false;
    if (rule != SPIFFY_RULE_TOPS) {
      pass0 = masked[0] && c[0] > tau;  // strict, Sec. 3.1
      pass1 = masked[1] && c[1] > tau;
    }
    const bool any_pass = __any_sync(full, pass0 || pass1);
    take[0] = any_pass ? pass0 : (any_masked && masked[0] && bp == lane);
    take[1] = any_pass ? pass1 : (any_masked && masked[1] && bp == lane + 32);
  }
  return (uint64_t)__ballot_sync(full, take[0]) | ((uint64_t)__ballot_sync(full, take[1]) << 32);
}

}  // namespace
}  // namespace spiffy
