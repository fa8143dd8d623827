// Packed draft-graph attention (Sec. 4.3; mask of Fig. 3) on the fp32 CUDA
// cores.  This is the kernel for fp32 inputs (tensor cores would need TF32,
// whose 10-bit mantissa cannot hold a 1e-4 tolerance) and for shapes the
// tcgen05 kernel does not take.  The mask is never materialised: a CTA works
// on one (sequence, node, query head) and simply iterates over the context
// keys followed by that node's own block keys.
#include <math.h>

#include "common.cuh"

namespace spiffy {
namespace {

constexpr int kWarps = 4;
constexpr int kTileKeys = 32;
constexpr int kMaxRowsPerWarp = 64 / kWarps;

template <typename T>
__device__ __forceinline__ float to_f32(T v);
template <>
__device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) {
  return __bfloat162float(v);
}
template <typename T>
__device__ __forceinline__ T from_f32(float v);
template <>
__device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) {
  return __float2bfloat16_rn(v);
}

// grid = (Hq, N, B), block = 128 threads.  Warp w owns query rows w, w+4, ...
template <typename T, int D>
__global__ void __launch_bounds__(kWarps * 32)
graph_attention_simt_kernel(int N, int L, int P, int Hq, int Hkv, float scale,
                            const T* __restrict__ q, const T* __restrict__ kp,
                            const T* __restrict__ vp, const T* __restrict__ kb,
                            const T* __restrict__ vb, T* __restrict__ out) {
  constexpr int CPL = D / 32;  // output columns per lane
  const int h = blockIdx.x, n = blockIdx.y, b = blockIdx.z;
  const int g = h / (Hq / Hkv);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  extern __shared__ float smem[];
  float* sq = smem;                          // [L][D]
  float* sk = sq + (size_t)L * D;            // [32][D+1]
  float* sv = sk + kTileKeys * (D + 1);      // [32][D]

  const int64_t node = (int64_t)b * N + n;
  for (int i = threadIdx.x; i < L * D; i += blockDim.x) {
    const int l = i / D, c = i % D;
    sq[i] = to_f32(q[((node * L + l) * Hq + h) * D + c]) * scale;
  }

  float m[kMaxRowsPerWarp], z[kMaxRowsPerWarp], o[kMaxRowsPerWarp][CPL];
#pragma unroll
  for (int r = 0; r < kMaxRowsPerWarp; ++r) {
    m[r] = -INFINITY;
    z[r] = 0.f;
#pragma unroll
    for (int c = 0; c < CPL; ++c) o[r][c] = 0.f;
  }

  const int total = P + L;  // allowed keys: context, then the node's own block
  for (int t0 = 0; t0 < total; t0 += kTileKeys) {
    __syncthreads();
    for (int i = threadIdx.x; i < kTileKeys * D; i += blockDim.x) {
      const int j = i / D, c = i % D;
      const int key = t0 + j;
      float kvv = 0.f, vvv = 0.f;
      if (key < P) {
        const int64_t a = (((int64_t)b * P + key) * Hkv + g) * D + c;
        kvv = to_f32(kp[a]);
        vvv = to_f32(vp[a]);
      } else if (key < total) {
        const int64_t a = ((node * L + (key - P)) * Hkv + g) * D + c;
        kvv = to_f32(kb[a]);
        vvv = to_f32(vb[a]);
      }
      sk[j * (D + 1) + c] = kvv;
      sv[j * D + c] = vvv;
    }
    __syncthreads();
    const bool valid = t0 + lane < total;
#pragma unroll
    for (int r = 0; r < kMaxRowsPerWarp; ++r) {
      const int l = warp + r * kWarps;
      if (l >= L) break;
      float s = 0.f;
      const float* qr = sq + l * D;
      const float* kr = sk + lane * (D + 1);
#pragma unroll 8
      for (int c = 0; c < D; ++c) s = fmaf(qr[c], kr[c], s);
      s = valid ? s : -INFINITY;
      float tm = s;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1)
        tm = fmaxf(tm, __shfl_xor_sync(0xffffffffu, tm, off));
      const float mn = fmaxf(m[r], tm);  // finite: the tile holds >= 1 key
      const float corr = expf(m[r] - mn);
      const float p = valid ? expf(s - mn) : 0.f;
      float ps = p;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1)
        ps += __shfl_xor_sync(0xffffffffu, ps, off);
      z[r] = z[r] * corr + ps;
      m[r] = mn;
#pragma unroll
      for (int c = 0; c < CPL; ++c) o[r][c] *= corr;
      for (int j = 0; j < kTileKeys; ++j) {
        const float pj = __shfl_sync(0xffffffffu, p, j);
#pragma unroll
        for (int c = 0; c < CPL; ++c)
          o[r][c] = fmaf(pj, sv[j * D + lane + 32 * c], o[r][c]);
      }
    }
  }
#pragma unroll
  for (int r = 0; r < kMaxRowsPerWarp; ++r) {
    const int l = warp + r * kWarps;
    if (l >= L) break;
    const float inv = 1.0f / z[r];
#pragma unroll
    for (int c = 0; c < CPL; ++c)
      out[((node * L + l) * Hq + h) * D + lane + 32 * c] =
          from_f32<T>(o[r][c] * inv);
  }
}

template <typename T, int D>
spiffy_status launch(const spiffy_attn_desc& d, float scale, const void* q,
                     const void* kp, const void* vp, const void* kb,
                     const void* vb, void* out, cudaStream_t stream) {
  const size_t smem =
      ((size_t)d.block_len * D + kTileKeys * (D + 1) + kTileKeys * D) * sizeof(float);
  auto kern = graph_attention_simt_kernel<T, D>;
  if (smem > 48 * 1024) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)smem) != cudaSuccess)
      return SPIFFY_ECUDA;
  }
  const dim3 grid(d.n_q_heads, d.n_nodes, d.batch);
  kern<<<grid, kWarps * 32, smem, stream>>>(
      d.n_nodes, d.block_len, d.prefix_len, d.n_q_heads, d.n_kv_heads, scale,
      static_cast<const T*>(q), static_cast<const T*>(kp),
      static_cast<const T*>(vp), static_cast<const T*>(kb),
      static_cast<const T*>(vb), static_cast<T*>(out));
  count_launch();
  return check_launch();
}

}  // namespace

spiffy_status launch_attention_simt(const spiffy_attn_desc& d, const void* q,
                                    const void* kp, const void* vp,
                                    const void* kb, const void* vb, void* out,
                                    cudaStream_t stream) {
  const float scale = d.scale != 0.f ? d.scale : 1.0f / sqrtf((float)d.head_dim);
  if (d.dtype == SPIFFY_F32) {
    if (d.head_dim == 64) return launch<float, 64>(d, scale, q, kp, vp, kb, vb, out, stream);
    return launch<float, 128>(d, scale, q, kp, vp, kb, vb, out, stream);
  }
  if (d.head_dim == 64)
    return launch<__nv_bfloat16, 64>(d, scale, q, kp, vp, kb, vb, out, stream);
  return launch<__nv_bfloat16, 128>(d, scale, q, kp, vp, kb, vb, out, stream);
}

}  // namespace spiffy
