// Drafting and pruning (Sec. 4.4.2 "Drafting Source", Sec. 4.4.4 "Draft Graph
// Pruning"): from the target distribution of the current block build the draft
// blocks that the next verification step will score.
//
//   draft_topk_kernel   per (row, vocabulary slice) of a still-masked position:
//                       the K largest logits with their token ids (value desc,
//                       id asc), the slice maximum and sum of exponentials.  A
//                       slice is held in registers, like in the decision step.
//   draft_build_kernel  one CTA per sequence: merges the slices into the K
//                       candidates c_ij and probabilities of every position,
//                       ranks the positions (Eq. token-position-sort), builds
//                       every draft formula, scores it by geometric means,
//                       keeps the D* best and writes their blocks and parent
//                       lists.
#include <math.h>

#include "common.cuh"

namespace spiffy {
namespace {

constexpr int kThreads = 128;  // top-k kernel
constexpr int kVecs = 8;       // 128-bit vectors per thread
constexpr int kMaxK = 4;       // vocabulary ranks
constexpr int kBuildThreads = 1024;  // a warp per block position
constexpr int kGraphInts = 6144;     // shared-memory copy of the draft graph (24 KB)

struct __align__(16) TopPartial {
  float m, s;          // slice maximum, sum of exp(x - m)
  float val[kMaxK];    // the K largest values, -inf when the slice has fewer
  int idx[kMaxK];      // their token ids
  int pad[2];
};

// (value desc, id asc): is (v2, i2) ahead of (v1, i1)?
__device__ __forceinline__ bool ahead(float v2, int i2, float v1, int i1) {
  return v2 > v1 || (v2 == v1 && i2 < i1);
}

template <typename T>
struct Unpack;
template <>
struct Unpack<__nv_bfloat16> {
  static constexpr int kPerVec = 8;
  static __device__ __forceinline__ void get(uint4 v, float (&f)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  static __device__ __forceinline__ float load1(const __nv_bfloat16* p) { return __bfloat162float(*p); }
};
template <>
struct Unpack<float> {
  static constexpr int kPerVec = 4;
  static __device__ __forceinline__ void get(uint4 v, float (&f)[4]) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
    f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
  }
  static __device__ __forceinline__ float load1(const float* p) { return *p; }
};

// grid = (slices, B*L rows), 128 threads.
template <typename T>
__global__ void __launch_bounds__(kThreads)
draft_topk_kernel(const T* __restrict__ logits, int64_t row_stride, int V, int64_t chunk,
                  int splits, int K, const int32_t* __restrict__ state, int mask_id,
                  TopPartial* __restrict__ partials) {
#if __CUDA_ARCH__ >= 900
  cudaGridDependencySynchronize();
  pdl_launch_dependents();  // the build kernel (one CTA per sequence) may take its SM and stage the graph
#endif
  const int row = blockIdx.y;
  if (state[row] != mask_id) return;
  const int split = blockIdx.x;
  const int64_t begin = (int64_t)split * chunk;
  const int64_t end = min((int64_t)V, begin + chunk);
  constexpr int EPV = Unpack<T>::kPerVec;
  const T* base = logits + (int64_t)row * row_stride;
  const int nvec = begin < end ? (int)((end - begin) / EPV) : 0;
  const int ntail = begin < end ? (int)(end - begin) - nvec * EPV : 0;
  const uint4* p = reinterpret_cast<const uint4*>(base + begin);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // the thread's elements: vectors t, t + 128, ..., then (thread 0) the ragged tail
  constexpr int NE = kVecs * EPV + EPV;
  float x[NE];
#pragma unroll
  for (int u = 0; u < kVecs; ++u) {
    float f[EPV];
    if (tid + u * kThreads < nvec) {
      Unpack<T>::get(ld_stream(p + tid + u * kThreads), f);
    } else {
#pragma unroll
      for (int e = 0; e < EPV; ++e) f[e] = -INFINITY;
    }
#pragma unroll
    for (int e = 0; e < EPV; ++e) x[u * EPV + e] = f[e];
  }
#pragma unroll
  for (int e = 0; e < EPV; ++e)
    x[kVecs * EPV + e] =
        (tid == 0 && e < ntail) ? Unpack<T>::load1(base + begin + (int64_t)nvec * EPV + e) : -INFINITY;
  auto index_of = [&](int k) -> int {  // token id of the thread's k-th element
    return k < kVecs * EPV ? (int)begin + (tid + (k / EPV) * kThreads) * EPV + k % EPV
                           : (int)begin + nvec * EPV + (k - kVecs * EPV);
  };

  __shared__ float w_val[kThreads / 32];
  __shared__ int w_idx[kThreads / 32];
  __shared__ float w_sum[kThreads / 32];
  // the thread's best remaining element; it is searched again only by the thread whose
  // element has just been taken (every other thread's best is still its best)
  float tv;
  int ti;
#define SPIFFY_DRAFT_RESCAN()                                                          \
  do {                                                                                 \
    tv = -INFINITY;                                                                    \
    ti = 0x7fffffff;                                                                   \
    _Pragma("unroll") for (int k = NE - 1; k >= 0; --k) /* descending: ties end on the lowest token */ \
      if (x[k] >= tv && x[k] != -INFINITY) {                                           \
        tv = x[k];                                                                     \
        ti = index_of(k);                                                              \
      }                                                                                \
  } while (0)
  SPIFFY_DRAFT_RESCAN();
  TopPartial out;
  out.s = 0.f;
#pragma unroll
  for (int r = 0; r < kMaxK; ++r) {
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    if (r < K) {
      // the best remaining element of the CTA: the best over the threads
      bv = tv;
      bi = ti;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        const float v2 = __shfl_xor_sync(0xffffffffu, bv, off);
        const int i2 = __shfl_xor_sync(0xffffffffu, bi, off);
        if (ahead(v2, i2, bv, bi)) { bv = v2; bi = i2; }
      }
      __syncthreads();  // the previous round's reads of w_val / w_idx are done
      if (lane == 0) { w_val[warp] = bv; w_idx[warp] = bi; }
      __syncthreads();
      bv = w_val[0];
      bi = w_idx[0];
#pragma unroll
      for (int w = 1; w < kThreads / 32; ++w)
        if (ahead(w_val[w], w_idx[w], bv, bi)) { bv = w_val[w]; bi = w_idx[w]; }
      if (r == 0) {
        // sum of exp(x - m) against the slice maximum, before anything is knocked out
        const float ml = (bv == -INFINITY) ? 0.f : bv * kLog2e;
        float s = 0.f;
#pragma unroll
        for (int k = 0; k < NE; ++k) s += ex2(fmaf(x[k], kLog2e, -ml));
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
        if (lane == 0) w_sum[warp] = s;
        __syncthreads();
        s = w_sum[0];
        for (int w = 1; w < kThreads / 32; ++w) s += w_sum[w];
        out.m = bv;
        out.s = s;
      }
      if (bv != -INFINITY && ti == bi && r + 1 < K) {  // this thread's element was taken: knock it out, search again
#pragma unroll
        for (int k = 0; k < NE; ++k)
          if (index_of(k) == bi) x[k] = -INFINITY;
        SPIFFY_DRAFT_RESCAN();
      }
    }
    out.val[r] = bv;
    out.idx[r] = bv == -INFINITY ? 0x7fffffff : bi;
  }
#undef SPIFFY_DRAFT_RESCAN
  out.pad[0] = out.pad[1] = 0;
  if (tid == 0) partials[(int64_t)row * splits + split] = out;
}

struct BuildArgs {
  const TopPartial* partials;
  int splits, L, K, D, budget, parent_cap, mask_id;
  const int32_t* state;        // [B][L]
  const int32_t* formula_off;  // [D+1]
  const int32_t* formula_i;
  const int32_t* formula_j;
  const int32_t* child_off;    // [D+1]
  const int32_t* child_idx;
  int32_t* tokens;      // [B][budget+1][L]
  int32_t* kept;        // [B][budget]
  float* score;         // [B][D]
  int32_t* parent_off;  // [B][budget+2]
  int32_t* parent_idx;  // [B][parent_cap]
  int32_t* dev_status;  // [B]
};

// Is the candidate set of formula a a strict subset of formula c's?  a < 0 is
// the current block (the empty set).
__device__ bool strict_subset(const BuildArgs& g, int a, int c) {
  const int c0 = g.formula_off[c], c1 = g.formula_off[c + 1];
  if (a < 0) return c1 > c0;
  const int a0 = g.formula_off[a], a1 = g.formula_off[a + 1];
  if (a1 - a0 >= c1 - c0) return false;
  for (int e = a0; e < a1; ++e) {
    bool found = false;
    for (int f = c0; f < c1; ++f)
      found |= g.formula_i[e] == g.formula_i[f] && g.formula_j[e] == g.formula_j[f];
    if (!found) return false;
  }
  return true;
}

// grid = B sequences, 1024 threads; dynamic shared memory, see the carve-up below.
__global__ void __launch_bounds__(kBuildThreads)
draft_build_kernel(BuildArgs g) {
  const int b = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int L = g.L, K = g.K, D = g.D;
  extern __shared__ __align__(8) unsigned char draft_smem[];
  float* cand_p = reinterpret_cast<float*>(draft_smem);      // [L][kMaxK]
  int* cand_tok = reinterpret_cast<int*>(cand_p + L * kMaxK);  // [L][kMaxK]
  int* pos_of_rank = cand_tok + L * kMaxK;                   // [L]
  float* local = reinterpret_cast<float*>(pos_of_rank + L);  // [D]
  float* total = local + D;                                  // [D]
  int* keep = reinterpret_cast<int*>(total + D);             // [D] slot + 1 of a kept formula, else 0
  int* node_formula = keep + D;                              // [budget + 1] formula of each node, -1 for node 0 / padding
  int* n_parents = node_formula + g.budget + 1;              // [budget + 1]
  __shared__ int n_masked;
  const int32_t* state = g.state + (int64_t)b * L;
  if (tid == 0) n_masked = 0;
  // The formulas are walked several times with dependent reads: when the graph
  // fits, copy it to shared memory and walk it there.  The draft graph is a
  // constant of the model (calibrated offline), not the product of earlier work on
  // the stream, so it is fetched before the wait on that work.
  __shared__ int32_t graph_smem[kGraphInts];
  {
    const int npairs = g.formula_off[D], nkids = g.child_off[D];
    if (2 * (D + 1) + 2 * npairs + nkids <= kGraphInts) {
      int32_t* f_off = graph_smem;
      int32_t* c_off = f_off + D + 1;
      int32_t* f_i = c_off + D + 1;
      int32_t* f_j = f_i + npairs;
      int32_t* c_idx = f_j + npairs;
      for (int i = tid; i <= D; i += kBuildThreads) { f_off[i] = g.formula_off[i]; c_off[i] = g.child_off[i]; }
      for (int i = tid; i < npairs; i += kBuildThreads) { f_i[i] = g.formula_i[i]; f_j[i] = g.formula_j[i]; }
      for (int i = tid; i < nkids; i += kBuildThreads) c_idx[i] = g.child_idx[i];
      g.formula_off = f_off; g.child_off = c_off; g.formula_i = f_i; g.formula_j = f_j; g.child_idx = c_idx;
    }
  }
#if __CUDA_ARCH__ >= 900
  cudaGridDependencySynchronize();  // the top-k kernel's partial results, and the caller's logits and state, are visible
#endif
  __syncthreads();

  // 1. candidates c_ij and their probabilities: one warp per position
  for (int l = warp; l < L; l += kBuildThreads / 32) {
    const bool masked = state[l] == g.mask_id;
    if (!masked) {
      if (lane < kMaxK) { cand_p[l * kMaxK + lane] = -1.f; cand_tok[l * kMaxK + lane] = state[l]; }
      continue;
    }
    const TopPartial* p = g.partials + ((int64_t)b * L + l) * g.splits;
    float m = -INFINITY, s = 0.f;
    float hv[kMaxK];
    int hi[kMaxK];
#pragma unroll
    for (int t = 0; t < kMaxK; ++t) { hv[t] = -INFINITY; hi[t] = 0x7fffffff; }
    if (g.splits <= 32) {
      // one slice per lane, fetched whole in one trip: its maximum and sum, and its K
      // candidates, which the top-k kernel left sorted
      if (lane < g.splits) {
        const uint4* q = reinterpret_cast<const uint4*>(p + lane);
        const uint4 q0 = q[0], q1 = q[1], q2 = q[2];
        m = __uint_as_float(q0.x);
        s = __uint_as_float(q0.y);
        hv[0] = __uint_as_float(q0.z); hv[1] = __uint_as_float(q0.w);
        hv[2] = __uint_as_float(q1.x); hv[3] = __uint_as_float(q1.y);
        hi[0] = (int)q1.z; hi[1] = (int)q1.w; hi[2] = (int)q2.x; hi[3] = (int)q2.y;
#pragma unroll
        for (int t = 0; t < kMaxK; ++t)
          if (t >= K || hv[t] == -INFINITY) { hv[t] = -INFINITY; hi[t] = 0x7fffffff; }
      }
    } else {
      // maximum and sum over the slices, fixed order
      for (int k = lane; k < g.splits; k += 32) {
        const float m2 = p[k].m, s2 = p[k].s, M = fmaxf(m, m2);
        s = s * ((m == M) ? 1.f : ex2((m - M) * kLog2e)) + s2 * ((m2 == M) ? 1.f : ex2((m2 - M) * kLog2e));
        m = M;
      }
      // every lane sorts the candidates it reads (each is read once)
      for (int c = lane; c < g.splits * K; c += 32) {
        float v = p[c / K].val[c % K];
        int i = p[c / K].idx[c % K];
        if (v == -INFINITY) continue;
#pragma unroll
        for (int t = 0; t < kMaxK; ++t)  // insertion into the sorted list
          if (ahead(v, i, hv[t], hi[t])) {
            const float tv = hv[t]; const int ti = hi[t];
            hv[t] = v; hi[t] = i; v = tv; i = ti;
          }
      }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const float m2 = __shfl_xor_sync(0xffffffffu, m, off), s2 = __shfl_xor_sync(0xffffffffu, s, off);
      const float M = fmaxf(m, m2);
      s = s * ((m == M) ? 1.f : ex2((m - M) * kLog2e)) + s2 * ((m2 == M) ? 1.f : ex2((m2 - M) * kLog2e));
      m = M;
    }
    if (lane == 0 && (!(fabsf(m) < INFINITY) || !(s > 0.f) || !(s < INFINITY)) && g.dev_status)
      atomicOr(g.dev_status + b, SPIFFY_DEV_NONFINITE);
    // the K best of the slices' candidates (value desc, id asc): K rounds pick the best
    // head over the lanes and pop it
    for (int r = 0; r < K; ++r) {
      float bv = hv[0];
      int bi = hi[0];
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        const float v2 = __shfl_xor_sync(0xffffffffu, bv, off);
        const int i2 = __shfl_xor_sync(0xffffffffu, bi, off);
        if (ahead(v2, i2, bv, bi)) { bv = v2; bi = i2; }
      }
      if (hi[0] == bi && bv != -INFINITY) {  // this lane's head won: pop it
#pragma unroll
        for (int t = 0; t + 1 < kMaxK; ++t) { hv[t] = hv[t + 1]; hi[t] = hi[t + 1]; }
        hv[kMaxK - 1] = -INFINITY;
        hi[kMaxK - 1] = 0x7fffffff;
      }
      if (lane == 0) {
        cand_tok[l * kMaxK + r] = bi;
        cand_p[l * kMaxK + r] = bv == -INFINITY ? 0.f : ex2((bv - m) * kLog2e) / s;
      }
    }
    if (lane == 0) atomicAdd(&n_masked, 1);
  }
  __syncthreads();
  // 2. token position ranks (Eq. token-position-sort): by maximum probability, ties to the lower position
  for (int l = tid; l < L; l += kBuildThreads) {
    const float pl = cand_p[l * kMaxK];
    if (pl < 0.f) continue;  // unmasked
    int rank = 0;
    for (int j = 0; j < L; ++j) {
      const float pj = cand_p[j * kMaxK];
      rank += (pj >= 0.f && (pj > pl || (pj == pl && j < l))) ? 1 : 0;
    }
    pos_of_rank[rank] = l;
  }
  __syncthreads();
  // 3. local score of every formula: geometric mean of its candidates' probabilities
  for (int q = tid; q < D; q += kBuildThreads) {
    const int e0 = g.formula_off[q], e1 = g.formula_off[q + 1];
    bool ok = e1 > e0;
    float logsum = 0.f;
    bool zero = false;
    for (int e = e0; e < e1 && ok; ++e) {
      const int i = g.formula_i[e], j = g.formula_j[e];
      if (i < 0 || i >= n_masked || j < 0 || j >= K) { ok = false; break; }
      const float pr = cand_p[pos_of_rank[i] * kMaxK + j];
      zero |= !(pr > 0.f);
      logsum += logf(fmaxf(pr, 1e-45f));
    }
    local[q] = !ok ? -INFINITY : (zero ? 0.f : expf(logsum / (float)(e1 - e0)));
  }
  __syncthreads();
  // 4. score = GM(local, GM(children's local scores)); a draft without buildable children keeps its local score
  for (int q = tid; q < D; q += kBuildThreads) {
    float sc = local[q];
    if (sc != -INFINITY) {
      float logsum = 0.f;
      int n = 0;
      bool zero = false;
      for (int e = g.child_off[q]; e < g.child_off[q + 1]; ++e) {
        const int x = g.child_idx[e];
        if (x < 0 || x >= D || local[x] == -INFINITY) continue;
        zero |= !(local[x] > 0.f);
        logsum += logf(fmaxf(local[x], 1e-45f));
        ++n;
      }
      if (n > 0) {
        const float child = zero ? 0.f : expf(logsum / (float)n);
        sc = sqrtf(sc * child);
      }
    }
    total[q] = sc;
    g.score[(int64_t)b * D + q] = sc;
  }
  __syncthreads();
  // 5. the D* best (score desc, formula index asc) keep their formula order
  for (int q = tid; q < D; q += kBuildThreads) {
    int rank = 0;
    const float sq = total[q];
    for (int x = 0; x < D; ++x)
      rank += (total[x] != -INFINITY && (total[x] > sq || (total[x] == sq && x < q))) ? 1 : 0;
    keep[q] = (sq != -INFINITY && rank < g.budget) ? 1 : 0;
  }
  for (int n = tid; n <= g.budget; n += kBuildThreads) node_formula[n] = -1;
  __syncthreads();
  for (int q = tid; q < D; q += kBuildThreads) {
    if (!keep[q]) continue;
    int slot = 0;
    for (int x = 0; x < q; ++x) slot += keep[x];
    node_formula[slot + 1] = q;
  }
  __syncthreads();
  // 6. blocks: the current block, then each kept draft = current block + its candidates
  int32_t* tokens = g.tokens + (int64_t)b * (g.budget + 1) * L;
  for (int i = tid; i < (g.budget + 1) * L; i += kBuildThreads) tokens[i] = state[i % L];
  for (int n = tid; n < g.budget; n += kBuildThreads) g.kept[(int64_t)b * g.budget + n] = node_formula[n + 1];
  __syncthreads();
  for (int n = 1 + warp; n <= g.budget; n += kBuildThreads / 32) {
    const int q = node_formula[n];
    if (q < 0) continue;
    for (int e = g.formula_off[q] + lane; e < g.formula_off[q + 1]; e += 32) {
      const int l = pos_of_rank[g.formula_i[e]];
      tokens[n * L + l] = cand_tok[l * kMaxK + g.formula_j[e]];
    }
  }
  // 7. parent lists: every earlier kept node whose candidate set is a strict subset.
  // One warp per child, its lanes over the candidate parents.
  auto is_parent = [&](int a, int c) {
    return a < c && (a == 0 || node_formula[a] >= 0) &&
           strict_subset(g, a == 0 ? -1 : node_formula[a], node_formula[c]);
  };
  for (int c = warp; c <= g.budget; c += kBuildThreads / 32) {
    int n = 0;
    if (c > 0 && node_formula[c] >= 0)
      for (int a0 = 0; a0 < c; a0 += 32) n += __popc(__ballot_sync(0xffffffffu, is_parent(a0 + lane, c)));
    if (lane == 0) n_parents[c] = n;
  }
  __syncthreads();
  for (int c = warp; c <= g.budget; c += kBuildThreads / 32) {
    int start = 0;
    for (int x = lane; x < c; x += 32) start += n_parents[x];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) start += __shfl_xor_sync(0xffffffffu, start, off);
    int32_t* off = g.parent_off + (int64_t)b * (g.budget + 2);
    int32_t* idx = g.parent_idx + (int64_t)b * g.parent_cap;
    if (lane == 0) {
      off[c] = min(start, g.parent_cap);
      if (c == g.budget) off[c + 1] = min(start + n_parents[c], g.parent_cap);
      if (start + n_parents[c] > g.parent_cap && g.dev_status) atomicOr(g.dev_status + b, SPIFFY_DEV_BADGRAPH);
    }
    if (c > 0 && node_formula[c] >= 0) {
      int w = start;
      for (int a0 = 0; a0 < c; a0 += 32) {
        const bool par = is_parent(a0 + lane, c);
        const unsigned mask = __ballot_sync(0xffffffffu, par);
        const int at = w + __popc(mask & ((1u << lane) - 1u));
        if (par && at < g.parent_cap) idx[at] = a0 + lane;
        w += __popc(mask);
      }
    }
  }
}

int64_t draft_chunk(const spiffy_draft_desc& d, int* splits) {
  const int64_t epv = d.logits_dtype == SPIFFY_BF16 ? 8 : 4;
  const int64_t most = (int64_t)kThreads * kVecs * epv;
  const int64_t n = (d.vocab + most - 1) / most;
  int64_t chunk = (d.vocab + n - 1) / n;
  chunk = (chunk + epv - 1) / epv * epv;
  *splits = (int)n;
  return chunk;
}

}  // namespace

size_t draft_workspace_bytes(const spiffy_draft_desc& d) {
  int splits = 1;
  draft_chunk(d, &splits);
  return (size_t)d.batch * d.block_len * splits * sizeof(TopPartial);
}

spiffy_status launch_draft(const spiffy_draft_desc& d, const void* logits, const int32_t* state,
                           const int32_t* formula_off, const int32_t* formula_i,
                           const int32_t* formula_j, const int32_t* child_off,
                           const int32_t* child_idx, int32_t* tokens, int32_t* kept, float* score,
                           int32_t* parent_off, int32_t* parent_idx, int32_t* dev_status, void* ws,
                           cudaStream_t stream) {
  int splits = 1;
  const int64_t chunk = draft_chunk(d, &splits);
  TopPartial* partials = static_cast<TopPartial*>(ws);
  const dim3 grid(splits, d.batch * d.block_len);
  cudaError_t e;
  if (d.logits_dtype == SPIFFY_BF16)
    e = launch_pdl(draft_topk_kernel<__nv_bfloat16>, grid, dim3(kThreads), (size_t)0, stream,
                   static_cast<const __nv_bfloat16*>(logits), (int64_t)d.row_stride, (int)d.vocab, chunk,
                   splits, (int)d.top_k, state, (int)d.mask_token_id, partials);
  else
    e = launch_pdl(draft_topk_kernel<float>, grid, dim3(kThreads), (size_t)0, stream,
                   static_cast<const float*>(logits), (int64_t)d.row_stride, (int)d.vocab, chunk, splits,
                   (int)d.top_k, state, (int)d.mask_token_id, partials);
  count_launch();
  if (e != cudaSuccess) return SPIFFY_ECUDA;
  BuildArgs g;
  g.partials = partials; g.splits = splits; g.L = d.block_len; g.K = d.top_k; g.D = d.n_formulas;
  g.budget = d.budget; g.parent_cap = d.parent_cap; g.mask_id = d.mask_token_id;
  g.state = state; g.formula_off = formula_off; g.formula_i = formula_i; g.formula_j = formula_j;
  g.child_off = child_off; g.child_idx = child_idx; g.tokens = tokens; g.kept = kept; g.score = score;
  g.parent_off = parent_off; g.parent_idx = parent_idx; g.dev_status = dev_status;
  const size_t smem = (size_t)d.block_len * kMaxK * 8 + (size_t)d.block_len * 4 +
                      (size_t)d.n_formulas * 12 + (size_t)(d.budget + 1) * 8 + 16;
  e = launch_pdl(draft_build_kernel, dim3(d.batch), dim3(kBuildThreads), smem, stream, g);
  count_launch();
  return e == cudaSuccess ? SPIFFY_OK : SPIFFY_ECUDA;
}

}  // namespace spiffy
