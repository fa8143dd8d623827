// Decision step at sampling temperature T > 0 (Sec. 5.3 evaluates Spiffy at
// T > 0; the paper does not spell the sampler out).
//
// Per still-masked position the token is drawn from softmax(x / T) by the
// Gumbel-max construction, token = argmax_v (x_v / T + g_v), g_v = -ln(-ln u_v),
// and its confidence is softmax(x / T)[token]; the unmasking rule of Sec. 3.1
// then runs on the confidences exactly as at T = 0 (decide_core.cuh).
//
// Losslessness (App. A) needs a draft block and the true block that equals it
// to draw the same token.  The uniforms therefore come from a counter-based
// generator, Philox4x32-10 (Salmon et al., SC 2011), with
//   counter = (v / 4, position l, sequence b, still-masked positions of the node)
//   key     = the two halves of the caller's 64-bit seed
// vocabulary entry v taking output word v % 4 and u = (word + 0.5) / 2^32: the
// noise follows the state of the block, never the node's index.
//
// Same two-kernel shape as the greedy decision: a register-resident reduce per
// (row, vocabulary slice) and a finalize per node.  The reduce is bound by
// integer and special-function arithmetic (about 50 instructions per logit),
// not by HBM.
#include "common.cuh"
#include "decide_core.cuh"

namespace spiffy {
namespace {

struct __align__(16) SampledPartial {
  float m;    // slice maximum of z = x / T (-inf for an empty slice)
  float s;    // sum over the slice of exp(z - m)
  float y;    // best noisy score z + g of the slice (-inf for an empty slice)
  int idx;    // its token (lowest on ties)
  float z;    // z of that token
  int pad[3];
};

struct Philox {
  uint32_t k0, k1;  // key
  uint32_t c1, c2, c3;  // the fixed counter words: position, sequence, masked count
  // the four output words of counter (block, c1, c2, c3)
  __device__ __forceinline__ void draw(uint32_t block, uint32_t (&w)[4]) const {
    uint32_t a = block, b = c1, c = c2, d = c3, x0 = k0, x1 = k1;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
      const uint32_t hi0 = __umulhi(0xD2511F53u, a), lo0 = 0xD2511F53u * a;
      const uint32_t hi1 = __umulhi(0xCD9E8D57u, c), lo1 = 0xCD9E8D57u * c;
      a = hi1 ^ b ^ x0;
      b = lo1;
      c = hi0 ^ d ^ x1;
      d = lo0;
      x0 += 0x9E3779B9u;
      x1 += 0xBB67AE85u;
    }
    w[0] = a; w[1] = b; w[2] = c; w[3] = d;
  }
};

__device__ __forceinline__ float lg2(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// g = -ln(-ln u), u = (word + 0.5) / 2^32, accurate in both tails: near u = 1,
// where the largest draws live, -ln u is taken from 1 - u = (~word + 0.5) / 2^32.
__device__ __forceinline__ float gumbel(uint32_t word) {
  constexpr float kLn2 = 0.6931471805599453f;
  float w;  // -ln u
  if (word < 0x80000000u) {
    w = kLn2 * (32.0f - lg2(__uint2float_rn(word) + 0.5f));
  } else {
    const float d = (__uint2float_rn(~word) + 0.5f) * 2.3283064365386963e-10f;  // 1 - u, in (0, 0.5]
    w = d > 0.015625f ? -kLn2 * lg2(1.0f - d)
                      : d * (1.0f + d * (0.5f + d * (0.33333334f + d * 0.25f)));
  }
  return -kLn2 * lg2(w);
}

// running best of (noisy score desc, token asc)
struct Best {
  float y, z;
  int idx;
  __device__ __forceinline__ void take(float y2, float z2, int i2) {
    if (y2 > y || (y2 == y && i2 < idx)) {
      y = y2;
      z = z2;
      idx = i2;
    }
  }
};

template <typename T>
struct Lanes;
template <>
struct Lanes<__nv_bfloat16> {
  static __device__ __forceinline__ void get(uint4 v, float (&f)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = Elem<__nv_bfloat16>::lo(w[i]);
      f[2 * i + 1] = Elem<__nv_bfloat16>::hi(w[i]);
    }
  }
};
template <>
struct Lanes<float> {
  static __device__ __forceinline__ void get(uint4 v, float (&f)[4]) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
    f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
  }
};

// grid = (splits, B*N*L); one CTA reduces one vocabulary slice of one row
template <typename T>
__global__ void __launch_bounds__(kReduceThreads)
decide_sampled_reduce_kernel(const T* __restrict__ logits, int64_t row_stride, int V, int64_t chunk,
                             int splits, int N, int L, const int32_t* __restrict__ block_tokens,
                             int mask_id, float inv_t, uint32_t seed_lo, uint32_t seed_hi,
                             SampledPartial* __restrict__ partials) {
#if __CUDA_ARCH__ >= 900
  cudaGridDependencySynchronize();
#endif
  const int row = blockIdx.y;
  if (block_tokens[row] != mask_id) return;  // already unmasked: never read
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int node = row / L, l = row - node * L, b = node / N;
  int masked_count;  // how far the node has been denoised: part of the noise's counter
  {
    const int32_t* st = block_tokens + (int64_t)node * L;
    const bool m0 = lane < L && st[min(lane, L - 1)] == mask_id;
    const bool m1 = lane + 32 < L && st[min(lane + 32, L - 1)] == mask_id;
    masked_count = __popc(__ballot_sync(0xffffffffu, m0)) + __popc(__ballot_sync(0xffffffffu, m1));
  }
  const Philox rng{seed_lo, seed_hi, (uint32_t)l, (uint32_t)b, (uint32_t)masked_count};
  const int split = blockIdx.x;
  const int64_t begin = (int64_t)split * chunk;
  const int64_t end = min((int64_t)V, begin + chunk);
  constexpr int EPV = Elem<T>::kPerVec;
  constexpr uint32_t NI = Elem<T>::kNegInf;
  const T* base = logits + (int64_t)row * row_stride;
  const int nvec = begin < end ? (int)((end - begin) / EPV) : 0;
  const int ntail = begin < end ? (int)(end - begin) - nvec * EPV : 0;
  const uint4* p = reinterpret_cast<const uint4*>(base + begin);

  uint4 v[kUnroll];
#pragma unroll
  for (int u = 0; u < kUnroll; ++u)
    v[u] = (tid + u * kReduceThreads < nvec) ? ld_stream(p + tid + u * kReduceThreads)
                                             : make_uint4(NI, NI, NI, NI);
  float tail[EPV];
#pragma unroll
  for (int e = 0; e < EPV; ++e)
    tail[e] = (tid == 0 && e < ntail) ? Elem<T>::load1(base + begin + (int64_t)nvec * EPV + e) : -INFINITY;
  // slice maximum of x; the maximum of z = x / T is its image (T > 0)
  float mx = Elem<T>::gmax(v);
#pragma unroll
  for (int e = 0; e < EPV; ++e) mx = fmaxf(mx, tail[e]);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
  __shared__ float warp_m[kReduceThreads / 32], warp_s[kReduceThreads / 32];
  __shared__ float warp_y[kReduceThreads / 32], warp_z[kReduceThreads / 32];
  __shared__ int warp_i[kReduceThreads / 32];
  if (lane == 0) warp_m[warp] = mx;
  __syncthreads();
  mx = warp_m[0];
#pragma unroll
  for (int w = 1; w < kReduceThreads / 32; ++w) mx = fmaxf(mx, warp_m[w]);
  const float m = mx * inv_t;
  const float k = inv_t * kLog2e;
  const float ml = (mx == -INFINITY) ? 0.f : m * kLog2e;  // an all -inf slice sums to 0

  float s = 0.f;
  Best best{-INFINITY, -INFINITY, 0x7fffffff};
#pragma unroll
  for (int u = 0; u < kUnroll; ++u) {
    if (tid + u * kReduceThreads < nvec) {
      float x[EPV];
      Lanes<T>::get(v[u], x);
      const int v0 = (int)begin + (tid + u * kReduceThreads) * EPV;  // a multiple of 4
#pragma unroll
      for (int q = 0; q < EPV / 4; ++q) {
        uint32_t w[4];
        rng.draw((uint32_t)(v0 >> 2) + q, w);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float xe = x[4 * q + e];
          s += ex2(fmaf(xe, k, -ml));
          const float z = xe * inv_t;
          if (xe != -INFINITY) best.take(z + gumbel(w[e]), z, v0 + 4 * q + e);
        }
      }
    }
  }
  if (ntail > 0 && tid == 0) {
    const int v0 = (int)begin + nvec * EPV;  // a multiple of 4
#pragma unroll
    for (int q = 0; q < (EPV + 3) / 4; ++q) {
      if (4 * q < ntail) {
        uint32_t w[4];
        rng.draw((uint32_t)(v0 >> 2) + q, w);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (4 * q + e < ntail) {
            const float xe = tail[4 * q + e];
            s += ex2(fmaf(xe, k, -ml));
            const float z = xe * inv_t;
            if (xe != -INFINITY) best.take(z + gumbel(w[e]), z, v0 + 4 * q + e);
          }
        }
      }
    }
  }
  // fixed order: lanes (butterfly), then warps
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    s += __shfl_xor_sync(0xffffffffu, s, off);
    const float y2 = __shfl_xor_sync(0xffffffffu, best.y, off);
    const float z2 = __shfl_xor_sync(0xffffffffu, best.z, off);
    const int i2 = __shfl_xor_sync(0xffffffffu, best.idx, off);
    best.take(y2, z2, i2);
  }
  if (lane == 0) {
    warp_s[warp] = s;
    warp_y[warp] = best.y;
    warp_z[warp] = best.z;
    warp_i[warp] = best.idx;
  }
  __syncthreads();
  if (tid == 0) {
    s = warp_s[0];
    best = Best{warp_y[0], warp_z[0], warp_i[0]};
    for (int w = 1; w < kReduceThreads / 32; ++w) {
      s += warp_s[w];
      best.take(warp_y[w], warp_z[w], warp_i[w]);
    }
    partials[(int64_t)row * splits + split] = SampledPartial{m, s, best.y, best.idx, best.z, {0, 0, 0}};
  }
}

// grid = B*N nodes, 512 threads: eight threads per position merge the slices of
// its row, then warp 0 applies the rule.
constexpr int kThreads = 512;
__global__ void __launch_bounds__(kThreads)
decide_sampled_finalize_kernel(const SampledPartial* __restrict__ partials, int splits, int N, int L,
                               const int32_t* __restrict__ block_tokens, int mask_id, int rule,
                               int top_s, float tau, float* __restrict__ conf_out,
                               int32_t* __restrict__ tok_out, uint64_t* __restrict__ bits_out,
                               int32_t* __restrict__ n_unmask_out, int32_t* __restrict__ dev_status) {
#if __CUDA_ARCH__ >= 900
  pdl_launch_dependents();
  cudaGridDependencySynchronize();  // the reduce kernel's partials are visible
#endif
  const int node = blockIdx.x;
  const int pos = threadIdx.x >> 3, sub = threadIdx.x & 7;
  __shared__ float sconf[64];
  {
    const int row = node * L + min(pos, L - 1);
    const int32_t state = block_tokens[row];
    float m = -INFINITY, s = 0.f;
    int unused = 0x7fffffff;
    Best best{-INFINITY, -INFINITY, 0x7fffffff};
    const SampledPartial* p = partials + (int64_t)row * splits;
    for (int k0 = sub; k0 < splits; k0 += 8) {
      const SampledPartial q = p[k0];
      merge(m, s, unused, q.m, q.s, 0x7fffffff);
      best.take(q.y, q.z, q.idx);
    }
#pragma unroll
    for (int off = 4; off > 0; off >>= 1) {  // fixed order inside the group of eight
      const float m2 = __shfl_xor_sync(0xffffffffu, m, off);
      const float s2 = __shfl_xor_sync(0xffffffffu, s, off);
      merge(m, s, unused, m2, s2, 0x7fffffff);
      const float y2 = __shfl_xor_sync(0xffffffffu, best.y, off);
      const float z2 = __shfl_xor_sync(0xffffffffu, best.z, off);
      const int i2 = __shfl_xor_sync(0xffffffffu, best.idx, off);
      best.take(y2, z2, i2);
    }
    if (sub == 0 && pos < L) {
      const bool masked = state == mask_id;
      // probability of the drawn token under softmax(x / T)
      const float conf = masked ? fminf(1.0f, ex2((best.z - m) * kLog2e) / s) : -INFINITY;
      conf_out[row] = conf;
      tok_out[row] = masked ? best.idx : state;
      sconf[pos] = conf;
      if (masked && (!(fabsf(m) < INFINITY) || !(s > 0.f) || !(s < INFINITY) || best.idx == 0x7fffffff)) {
        if (dev_status) atomicOr(dev_status + node / N, SPIFFY_DEV_NONFINITE);
      }
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

}  // namespace

size_t decide_sampled_workspace_bytes(const spiffy_decide_desc& d) {
  const int64_t rows = (int64_t)d.batch * d.n_nodes * d.block_len;
  return (size_t)rows * decide_splits(d, nullptr) * sizeof(SampledPartial);
}

spiffy_status launch_decide_sampled(const spiffy_decide_desc& d, float temperature, uint64_t seed,
                                    const void* logits, const int32_t* block_tokens, float* conf,
                                    int32_t* top_tok, uint64_t* unmask_bits, int32_t* n_unmask,
                                    int32_t* dev_status, void* ws, cudaStream_t stream) {
  int64_t chunk = 0;
  const int splits = decide_splits(d, &chunk);
  const int rows = d.batch * d.n_nodes * d.block_len;
  SampledPartial* partials = static_cast<SampledPartial*>(ws);
  const dim3 grid(splits, rows);
  const float inv_t = 1.0f / temperature;
  const uint32_t lo = (uint32_t)(seed & 0xffffffffu), hi = (uint32_t)(seed >> 32);
  cudaError_t e;
  if (d.logits_dtype == SPIFFY_BF16)
    e = launch_pdl(decide_sampled_reduce_kernel<__nv_bfloat16>, grid, dim3(kReduceThreads), (size_t)0,
                   stream, static_cast<const __nv_bfloat16*>(logits), (int64_t)d.row_stride,
                   (int)d.vocab, chunk, splits, (int)d.n_nodes, (int)d.block_len, block_tokens,
                   (int)d.mask_token_id, inv_t, lo, hi, partials);
  else
    e = launch_pdl(decide_sampled_reduce_kernel<float>, grid, dim3(kReduceThreads), (size_t)0, stream,
                   static_cast<const float*>(logits), (int64_t)d.row_stride, (int)d.vocab, chunk,
                   splits, (int)d.n_nodes, (int)d.block_len, block_tokens, (int)d.mask_token_id,
                   inv_t, lo, hi, partials);
  count_launch();
  if (e != cudaSuccess) return SPIFFY_ECUDA;
  const SampledPartial* cpart = partials;
  e = launch_pdl(decide_sampled_finalize_kernel, dim3(d.batch * d.n_nodes), dim3(kThreads), (size_t)0,
                 stream, cpart, splits, (int)d.n_nodes, (int)d.block_len, block_tokens,
                 (int)d.mask_token_id, (int)d.rule, (int)d.top_s, d.threshold, conf, top_tok,
                 unmask_bits, n_unmask, dev_status);
  count_launch();
  return e == cudaSuccess ? SPIFFY_OK : SPIFFY_ECUDA;
}

}  // namespace spiffy
