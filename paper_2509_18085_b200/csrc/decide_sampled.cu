// Decision step at sampling temperature T > 0 (Sec. 5.3 evaluates Spiffy at
// T > 0; the paper does not spell the sampler out).
//
// Per still-masked position the token is drawn from softmax(z), z = x / T, in
// two levels over the vocabulary slices of the reduce kernel (width
// spiffy_sampled_slice_width):
//   1. the slice: s* = argmax_s (ln Z_s + g_s), Z_s = sum of exp(z) over the
//      slice, g_s = -ln(-ln u_s)  (Gumbel-max on the slices' total weights);
//   2. the entry: the first v of slice s* whose running sum of exp(z) reaches
//      u' * Z_s*  (inversion of the cumulative distribution inside the slice).
// Its confidence is softmax(z)[token]; the unmasking rule of Sec. 3.1 then runs
// on the confidences exactly as at T = 0 (decide_core.cuh).
//
// Losslessness (App. A) needs a draft block and the true block that equals it
// to draw the same token.  The uniforms therefore come from a counter-based
// generator, Philox4x32-10 (Salmon et al., SC 2011), with
//   counter = (slice s, position l, sequence b, still-masked positions of the node)
//   key     = the two halves of the caller's 64-bit seed
// output word 0 giving u_s, word 1 giving u' and u = (word + 0.5) / 2^32: the
// noise follows the state of the block, never the node's index.
//
// Two kernels.  The reduce is the greedy decision's (one pass over the logits,
// HBM-bound) with the exponent scaled by 1 / T.  The select kernel, one CTA per
// row, picks the slice from the partial results (one generator call per slice),
// re-reads that one slice (16 KB, mostly still in L2), inverts its running sum,
// and the last CTA of a node to finish applies the rule.
#include <type_traits>

#include "common.cuh"
#include "decide_core.cuh"

namespace spiffy {
namespace {

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

// (maximum of x, sum of exp((x - maximum) / T)) of two slices merged; k = log2(e) / T
__device__ __forceinline__ void merge_t(float& m, float& s, float m2, float s2, float k) {
  const float M = fmaxf(m, m2);
  const float f1 = (m == M) ? 1.f : ex2((m - M) * k);
  const float f2 = (m2 == M) ? 1.f : ex2((m2 - M) * k);
  s = __fmaf_rn(s, f1, __fmul_rn(s2, f2));
  m = M;
}

// grid = (splits, B*N*L); one CTA reduces one vocabulary slice of one row and
// the first CTA of a node clears the node's arrival counter for the select kernel.
template <typename T>
__global__ void __launch_bounds__(kReduceThreads, 8)
decide_sampled_reduce_kernel(const T* __restrict__ logits, int64_t row_stride, int V, int64_t chunk,
                             int splits, int L, const int32_t* __restrict__ block_tokens, int mask_id,
                             float k, Partial* __restrict__ partials, int* __restrict__ node_count) {
#if __CUDA_ARCH__ >= 900
  cudaGridDependencySynchronize();
#endif
  const int row = blockIdx.y;
  if (blockIdx.x == 0 && threadIdx.x == 0 && row % L == 0) node_count[row / L] = 0;
  if (block_tokens[row] != mask_id) return;  // already unmasked: never read
  reduce_slice(logits + (int64_t)row * row_stride, V, chunk, (int)blockIdx.x,
               partials + (int64_t)row * splits + blockIdx.x, k);
}

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

// What warp 0 of the select kernel finds for its row and leaves in shared memory.
struct SliceChoice {
  int slice;       // the chosen slice, 0x7fffffff when no slice has any weight
  uint32_t word;   // generator word behind u'
  float m, z;      // the slice's maximum of x and its sum of exp((x - m) / T)
  float row_m, row_s;  // the same for the whole row
};

// grid = B*N*L rows; kReduceThreads threads; thread t holds the vectors
// 8 t ... 8 t + 7 of the chosen slice, i.e. a contiguous run of entries.
template <typename T>
__global__ void __launch_bounds__(kReduceThreads)
decide_sampled_select_kernel(const T* __restrict__ logits, int64_t row_stride, int V, int64_t chunk,
                             int splits, int N, int L, const int32_t* __restrict__ block_tokens,
                             int mask_id, int rule, int top_s, float tau, float inv_t,
                             uint32_t seed_lo, uint32_t seed_hi, const Partial* __restrict__ partials,
                             int* __restrict__ node_count, float* __restrict__ conf_out,
                             int32_t* __restrict__ tok_out, uint64_t* __restrict__ bits_out,
                             int32_t* __restrict__ n_unmask_out, int32_t* __restrict__ dev_status) {
  constexpr int EPV = Elem<T>::kPerVec;
  constexpr uint32_t NI = Elem<T>::kNegInf;
  const int row = blockIdx.x;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int node = row / L, l = row - node * L, b = node / N;
  // The block's tokens were there before the reduce kernel started: they are read, and the
  // node's masked positions counted, ahead of the wait for that kernel.
  const int32_t state = block_tokens[row];
  int masked_count = 0;  // how far the node has been denoised: part of the noise's counter
  if (warp == 0) {
    const int32_t* st = block_tokens + (int64_t)node * L;
    const bool m0 = lane < L && st[min(lane, L - 1)] == mask_id;
    const bool m1 = lane + 32 < L && st[min(lane + 32, L - 1)] == mask_id;
    masked_count = __popc(__ballot_sync(0xffffffffu, m0)) + __popc(__ballot_sync(0xffffffffu, m1));
  }
#if __CUDA_ARCH__ >= 900
  pdl_launch_dependents();
  cudaGridDependencySynchronize();  // the reduce kernel's partials and cleared counters are visible
#endif
  const float k = inv_t * kLog2e;
  __shared__ SliceChoice choice;
  __shared__ double warp_total[kReduceThreads / 32];
  __shared__ int is_last;
  __shared__ float sconf[64];
  if (state == mask_id) {  // the whole CTA takes the same branch
    if (warp == 0) {
      // level 1: lanes over slices
      const Philox rng{seed_lo, seed_hi, (uint32_t)l, (uint32_t)b, (uint32_t)masked_count};
      float rm = -INFINITY, rs = 0.f;      // row maximum of x and sum of exp((x - rm) / T)
      float best = -INFINITY, bm = 0.f, bz = 0.f;
      int bs = 0x7fffffff;
      uint32_t bw = 0;
      const Partial* p = partials + (int64_t)row * splits;
      for (int s = lane; s < splits; s += 32) {
        const int4 raw = __ldcg(reinterpret_cast<const int4*>(p + s));
        const float m = __int_as_float(raw.x), z = __int_as_float(raw.y);
        merge_t(rm, rs, m, z, k);
        if (z > 0.f && m > -INFINITY) {
          uint32_t w[4];
          rng.draw((uint32_t)s, w);
          const float score = fmaf(m, inv_t, 0.6931471805599453f * lg2(z)) + gumbel(w[0]);
          if (score > best || (score == best && s < bs)) {
            best = score; bs = s; bw = w[1]; bm = m; bz = z;
          }
        }
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {  // fixed order
        merge_t(rm, rs, __shfl_xor_sync(0xffffffffu, rm, off), __shfl_xor_sync(0xffffffffu, rs, off), k);
        const float s2 = __shfl_xor_sync(0xffffffffu, best, off);
        const int i2 = __shfl_xor_sync(0xffffffffu, bs, off);
        const uint32_t w2 = __shfl_xor_sync(0xffffffffu, bw, off);
        const float m2 = __shfl_xor_sync(0xffffffffu, bm, off);
        const float z2 = __shfl_xor_sync(0xffffffffu, bz, off);
        if (i2 != 0x7fffffff && (bs == 0x7fffffff || s2 > best || (s2 == best && i2 < bs))) {
          best = s2; bs = i2; bw = w2; bm = m2; bz = z2;
        }
      }
      if (lane == 0) choice = SliceChoice{bs, bw, bm, bz, rm, rs};
    }
    __syncthreads();
    const SliceChoice c = choice;
    const bool usable = c.slice != 0x7fffffff && fabsf(c.row_m) < INFINITY && c.row_s > 0.f && c.row_s < INFINITY;
    if (!usable) {
      if (tid == 0) {
        conf_out[row] = __int_as_float(0x7fc00000);  // NaN: never wins the rule
        tok_out[row] = 0;
        if (dev_status) atomicOr(dev_status + b, SPIFFY_DEV_NONFINITE);
        __threadfence();
      }
    } else {
      // level 2: the chosen slice, entries in ascending order over (thread, vector, element)
      const int64_t begin = (int64_t)c.slice * chunk;
      const int64_t end = min((int64_t)V, begin + chunk);
      const int nvec = (int)((end - begin) / EPV);
      const int ntail = (int)(end - begin) - nvec * EPV;
      const T* base = logits + (int64_t)row * row_stride + begin;
      const uint4* p = reinterpret_cast<const uint4*>(base);
      uint4 v[kUnroll];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int j = tid * kUnroll + u;
        v[u] = j < nvec ? ld_stream(p + j) : make_uint4(NI, NI, NI, NI);
      }
      const float nml = -c.m * k;
      // the ragged end of the last slice sits in the vector slot after the last whole vector
      const bool has_tail = ntail > 0 && tid == nvec / kUnroll;
      const int tail_u = nvec % kUnroll;
      float tail[EPV];
#pragma unroll
      for (int e = 0; e < EPV; ++e)
        tail[e] = (has_tail && e < ntail) ? Elem<T>::load1(base + (int64_t)nvec * EPV + e) : -INFINITY;
      auto slot = [&](int u, float (&x)[EPV]) {  // the logits of vector slot u
        Lanes<T>::get(v[u], x);
        if (has_tail && u == tail_u) {
#pragma unroll
          for (int e = 0; e < EPV; ++e) x[e] = tail[e];
        }
      };
      float local = 0.f;  // weight of this thread's entries, summed in ascending order
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        float x[EPV];
        slot(u, x);
#pragma unroll
        for (int e = 0; e < EPV; ++e) local += ex2(fmaf(x[e], k, nml));
      }
      // running sums across threads, in double: thread t's exclusive sum is thread t - 1's inclusive one, bit for bit
      double in_warp = (double)local;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const double up = __shfl_up_sync(0xffffffffu, in_warp, off);
        if (lane >= off) in_warp += up;
      }
      const double before = __shfl_up_sync(0xffffffffu, in_warp, 1);
      if (lane == 31) warp_total[warp] = in_warp;
      __syncthreads();
      double warps_before = 0.0, total = 0.0;
      for (int w = 0; w < kReduceThreads / 32; ++w) {
        if (w == warp) warps_before = total;
        total += warp_total[w];  // the last thread's inclusive sum, bit for bit
      }
      const double incl = warps_before + in_warp;
      const double excl = lane > 0 ? warps_before + before : warps_before;
      // u' times the slice's weight as summed here, so that the running sums and their total agree
      const double target = ((double)c.word + 0.5) * 2.3283064365386963e-10 * total;
      const bool mine = incl >= target && excl < target;  // exactly one thread: u' < 1
      if (mine) {
        // excl + run >= target for a float run is run >= (target - excl) rounded up to a float
        const float need = __double2float_ru(target - excl);
        int first_reach = -1, last_weight = -1;
        float x_reach = 0.f, x_weight = 0.f, run = 0.f;
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
          float x[EPV];
          slot(u, x);
#pragma unroll
          for (int e = 0; e < EPV; ++e) {
            const float w = ex2(fmaf(x[e], k, nml));
            run += w;  // the order of `local`
            if (first_reach < 0 && w > 0.f && run >= need) {
              first_reach = (tid * kUnroll + u) * EPV + e;
              x_reach = x[e];
            }
            if (w > 0.f) {
              last_weight = (tid * kUnroll + u) * EPV + e;
              x_weight = x[e];
            }
          }
        }
        // the thread's own partial sums end at `local`, which can miss incl by a rounding of the scan
        const bool reach = first_reach >= 0;
        const int pick = reach ? first_reach : max(last_weight, 0);
        const float x_pick = reach ? x_reach : x_weight;
        conf_out[row] = fminf(1.0f, ex2((x_pick - c.row_m) * k) / c.row_s);
        tok_out[row] = (int32_t)begin + pick;
        __threadfence();
      }
    }
  } else if (tid == 0) {
    conf_out[row] = -INFINITY;
    tok_out[row] = state;
    __threadfence();
  }
  // the last row of a node to arrive applies the rule to the node
  __syncthreads();
  if (tid == 0) is_last = atomicAdd(node_count + node, 1) == L - 1;
  __syncthreads();
  if (!is_last || warp != 0) return;
  __threadfence();
  for (int i = lane; i < L; i += 32) sconf[i] = __ldcg(conf_out + (int64_t)node * L + i);
  __syncwarp();
  const uint64_t bits = unmask_rule(sconf, block_tokens + (int64_t)node * L, L, mask_id, rule, top_s, tau, lane);
  if (lane == 0) {
    bits_out[node] = bits;
    n_unmask_out[node] = __popcll(bits);
  }
}

size_t partial_bytes(const spiffy_decide_desc& d) {
  const int64_t rows = (int64_t)d.batch * d.n_nodes * d.block_len;
  return ((size_t)rows * decide_splits(d, nullptr) * sizeof(Partial) + 255) / 256 * 256;
}

}  // namespace

size_t decide_sampled_workspace_bytes(const spiffy_decide_desc& d) {
  return partial_bytes(d) + (size_t)d.batch * d.n_nodes * sizeof(int);
}

spiffy_status launch_decide_sampled(const spiffy_decide_desc& d, float temperature, uint64_t seed,
                                    const void* logits, const int32_t* block_tokens, float* conf,
                                    int32_t* top_tok, uint64_t* unmask_bits, int32_t* n_unmask,
                                    int32_t* dev_status, void* ws, cudaStream_t stream) {
  int64_t chunk = 0;
  const int splits = decide_splits(d, &chunk);
  const int rows = d.batch * d.n_nodes * d.block_len;
  Partial* partials = static_cast<Partial*>(ws);
  int* node_count = reinterpret_cast<int*>(static_cast<char*>(ws) + partial_bytes(d));
  const float inv_t = 1.0f / temperature;
  const uint32_t lo = (uint32_t)(seed & 0xffffffffu), hi = (uint32_t)(seed >> 32);
  const Partial* cpart = partials;
  cudaError_t e;
  auto run = [&](auto* typed) -> cudaError_t {
    using T = std::remove_cv_t<std::remove_pointer_t<decltype(typed)>>;
    cudaError_t r = launch_pdl(decide_sampled_reduce_kernel<T>, dim3(splits, rows), dim3(kReduceThreads),
                               (size_t)0, stream, typed, (int64_t)d.row_stride, (int)d.vocab, chunk, splits,
                               (int)d.block_len, block_tokens, (int)d.mask_token_id, inv_t * kLog2e, partials,
                               node_count);
    count_launch();
    if (r != cudaSuccess) return r;
    r = launch_pdl(decide_sampled_select_kernel<T>, dim3(rows), dim3(kReduceThreads), (size_t)0, stream,
                   typed, (int64_t)d.row_stride, (int)d.vocab, chunk, splits, (int)d.n_nodes,
                   (int)d.block_len, block_tokens, (int)d.mask_token_id, (int)d.rule, (int)d.top_s,
                   d.threshold, inv_t, lo, hi, cpart, node_count, conf, top_tok, unmask_bits, n_unmask,
                   dev_status);
    count_launch();
    return r;
  };
  if (d.logits_dtype == SPIFFY_BF16)
    e = run(static_cast<const __nv_bfloat16*>(logits));
  else
    e = run(static_cast<const float*>(logits));
  return e == cudaSuccess ? SPIFFY_OK : SPIFFY_ECUDA;
}

}  // namespace spiffy
