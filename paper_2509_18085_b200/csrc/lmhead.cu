// The decision step fused into the output projection: logits = H W^T are formed
// tile by tile in tensor memory and reduced there to (maximum, sum of
// exponentials, arg-max) per row, so that the [rows x vocabulary] logits are
// never written to memory (Algorithm 1, steps 1-2, on the distribution of
// Sec. 3.1 before it is materialised).
//
// H: [rows][hidden] bf16 hidden states of the B*N*L positions,
// W: [vocabulary][hidden] bf16 output embedding.  A CTA owns vocabulary tiles of
// up to 256 entries (tile n, n + grid, ...), two M-tiles of 128 rows at once, and
// runs the K loop over `hidden` in chunks of 64 (more than 256 rows are taken 256
// at a time, each pass reading the weight matrix again):
//   warp 0      TMA producer: per chunk the two H tiles and the W tile (64 KB)
//               into a three-stage ring
//   warp 1      allocates tensor memory; one lane issues tcgen05.mma, M = 128,
//               N = 256 (the shape that runs near the tensor pipe's peak: 75-88 ns
//               per K = 16 step against 64 ns for N = 128), four steps per chunk
//               and M-tile; the two fp32 accumulators fill the 512 TMEM columns
//   warps 2-9   one thread per row: reads a finished accumulator (the logits of
//               256 vocabulary entries), updates its running maximum, sum of
//               exponentials and arg-max (ties to the lower token), hands the
//               buffer back
// Each CTA leaves one partial result per row; the decision's finalize kernel
// merges them (in a fixed order) and applies the unmasking rule.
//
// Every wait is bounded; a wait that gives up raises SPIFFY_DEV_TIMEOUT.
#include <math.h>

#include "common.cuh"
#include "decide_core.cuh"
#include "sm100_ptx.cuh"
#include "tma_map.cuh"

namespace spiffy {
namespace {

using namespace sm100;

constexpr int kLmThreads = 320;
constexpr int kLmStages = 3;
constexpr int kTile = 128 * 128;        // one operand tile of a stage: 128 rows x 64 bf16 = 16 KB
constexpr int kLmN = 256;               // most vocabulary entries per tile
constexpr int kStageBytes = 4 * kTile;  // H tile 0 | H tile 1 | W tile (256 rows)
constexpr int kLmBars = 2 * kLmStages + 4;
constexpr int kLmSmem = kLmStages * kStageBytes + 8 * kLmBars + 16 + 1024;
constexpr uint32_t kLmTmemCols = 512;   // M-tile t -> columns 256 t .. 256 t + 255

struct LmParams {
  int rows, hidden, vocab;
  int n_tile;                   // vocabulary entries per tile: a multiple of 32, at most kLmN
  Partial* partials;            // [rows][gridDim.x]
  int32_t* status;              // [B], may be null
  int n_status;
  uint32_t spin_limit;          // polls of one mbarrier wait
};

__global__ void __launch_bounds__(kLmThreads, 1)
lmhead_reduce_kernel(const __grid_constant__ CUtensorMap tm_h, const __grid_constant__ CUtensorMap tm_w,
                     const LmParams p) {
  extern __shared__ uint8_t lm_smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(
      (reinterpret_cast<uintptr_t>(lm_smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kLmStages * kStageBytes);
  uint64_t* full = bars;
  uint64_t* empty = full + kLmStages;
  uint64_t* acc_full = empty + kLmStages;  // the accumulators hold a finished tile
  uint64_t* acc_empty = acc_full + 2;      // the epilogue has read them
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kLmBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_tiles = (p.vocab + p.n_tile - 1) / p.n_tile;
  const int my_tiles = (int)blockIdx.x < n_tiles ? (n_tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
  const int kc_count = p.hidden / 64;
  const int passes = (p.rows + 255) / 256;

  if (threadIdx.x == 0) {
    for (int i = 0; i < kLmStages; ++i) { mbar_init(full + i, 1); mbar_init(empty + i, 1); }
    mbar_init(acc_full, 1);
    mbar_init(acc_empty, 256u);  // every epilogue thread, also those of an M-tile beyond the rows
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc(tmem_slot, kLmTmemCols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;
  if (threadIdx.x == 0) {
    prefetch_tensormap(&tm_h);
    prefetch_tensormap(&tm_w);
  }
  cudaGridDependencySynchronize();  // H (and the tokens the finalize kernel reads) are visible

  if (warp == 0) {
    // ------------------------------------------------------------ producer --
    if (lane == 0) {
      bool ok = true;
      int it = 0, issued = 0;
      for (int g = 0; g < passes * my_tiles && ok; ++g) {
        const int pass = g / my_tiles, i = g - pass * my_tiles;
        const int n = (int)blockIdx.x + i * (int)gridDim.x;
        const int row0 = pass * 256, mt = p.rows - row0 > 128 ? 2 : 1;
        for (int kc = 0; kc < kc_count; ++kc, ++it) {
          const int stage = it % kLmStages;
          if (!mbar_wait(empty + stage, (((uint32_t)(it / kLmStages)) & 1u) ^ 1u, abort_flag, p.spin_limit)) { ok = false; break; }
          uint8_t* dst = smem + stage * kStageBytes;
          mbar_arrive_expect_tx(full + stage, (uint32_t)mt * kTile + (uint32_t)p.n_tile * 128u);
          const int c0 = (kc & 1) * 64, head = kc >> 1;
          tma_load_4d(dst, &tm_h, full + stage, c0, head, row0, 0);
          if (mt > 1) tma_load_4d(dst + kTile, &tm_h, full + stage, c0, head, row0 + 128, 0);
          tma_load_4d(dst + 2 * kTile, &tm_w, full + stage, c0, head, n * p.n_tile, 0);
          issued = it + 1;
        }
      }
      if (!ok) {  // winding down: let the copies already in flight land before exit
        for (int j = max(0, issued - kLmStages); j < issued; ++j)
          for (uint32_t s = 0; s < kSpinLimit; ++s)
            if (mbar_try_wait(full + j % kLmStages, (uint32_t)(j / kLmStages) & 1u)) break;
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------- MMA issuer --
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_f32(128, p.n_tile, false, false);
      bool ok = true;
      int it = 0;
      for (int g = 0; g < passes * my_tiles && ok; ++g) {
        const int mt = p.rows - (g / my_tiles) * 256 > 128 ? 2 : 1;
        if (!mbar_wait(acc_empty, ((uint32_t)g & 1u) ^ 1u, abort_flag, p.spin_limit)) { ok = false; break; }
        tc_fence_after_sync();
        for (int kc = 0; kc < kc_count; ++kc, ++it) {
          const int stage = it % kLmStages;
          if (!mbar_wait(full + stage, (uint32_t)(it / kLmStages) & 1u, abort_flag, p.spin_limit)) { ok = false; break; }
          tc_fence_after_sync();
          const uint32_t h0 = smem_u32(smem + stage * kStageBytes);
          const uint32_t w0 = h0 + 2 * kTile;
#pragma unroll
          for (int t = 0; t < 2; ++t) {
            if (t < mt) {
              const uint32_t d = tmem + (uint32_t)t * (uint32_t)kLmN;
#pragma unroll
              for (int kk = 0; kk < 4; ++kk)
                umma_ss(d, smem_desc_sw128(h0 + (uint32_t)t * kTile + (uint32_t)kk * 32u, 16, 1024),
                        smem_desc_sw128(w0 + (uint32_t)kk * 32u, 16, 1024), idesc, (kc > 0 || kk > 0) ? 1u : 0u);
            }
          }
          umma_commit(empty + stage);  // the stage is free once these products have read it
        }
        if (ok) umma_commit(acc_full);
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue --
    const int quad = warp & 3;
    const int t = (warp - 2) >> 2;  // M-tile of this warpgroup
    const int r = quad * 32 + lane;
    const uint32_t lane_base = (uint32_t)(quad * 32);
    bool ok = true;
    for (int pass = 0; pass < passes && ok; ++pass) {
      const int row = pass * 256 + t * 128 + r;
      const bool live = pass * 256 + t * 128 < p.rows;  // this warpgroup's M-tile holds rows in this pass
      float m_run = -INFINITY, s_run = 0.f, best = -INFINITY;
      int best_idx = 0x7fffffff;
      for (int i = 0; i < my_tiles && ok; ++i) {
        const int n = (int)blockIdx.x + i * (int)gridDim.x;
        const int g = pass * my_tiles + i;
        ok = __all_sync(0xffffffffu, mbar_wait(acc_full, (uint32_t)g & 1u, abort_flag, p.spin_limit));
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t col0 = (uint32_t)t * (uint32_t)kLmN;
#pragma unroll 1
        for (int c0 = 0; live && c0 < p.n_tile; c0 += 32) {
          uint32_t v[32];
          tmem_ld_x32(tmem_addr(tmem, lane_base, col0 + (uint32_t)c0), v);
          const int v0 = n * p.n_tile + c0;
          float cm = -INFINITY;
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            const float x = (v0 + c < p.vocab) ? __uint_as_float(v[c]) : -INFINITY;
            v[c] = __float_as_uint(x);
            cm = fmaxf(cm, x);
          }
          if (cm > m_run) {  // new reference maximum: rescale the sum
            s_run *= (m_run == -INFINITY) ? 0.f : ex2((m_run - cm) * kLog2e);
            m_run = cm;
          }
          const float ml = (m_run == -INFINITY) ? 0.f : m_run * kLog2e;
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            const float x = __uint_as_float(v[c]);
            s_run += ex2(fmaf(x, kLog2e, -ml));
            if (x > best) {  // strictly: tiles and columns come in ascending token order
              best = x;
              best_idx = v0 + c;
            }
          }
        }
        tc_fence_before_sync();
        mbar_arrive(acc_empty);
      }
      if (ok && row < p.rows) {
        // NaN logits never win a comparison: report them through the maximum
        if (!(s_run == s_run)) m_run = s_run;
        p.partials[(int64_t)row * gridDim.x + blockIdx.x] =
            Partial{m_run, s_run, best == -INFINITY ? 0x7fffffff : best_idx, 0};
      }
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, kLmTmemCols);
  }
  if (threadIdx.x == 0 && *abort_flag && p.status)
    for (int b = 0; b < p.n_status; ++b) atomicOr(p.status + b, SPIFFY_DEV_TIMEOUT);
}

}  // namespace

// Vocabulary entries per tile: the multiple of 32 (at most 256, at least 128) for which
// rounds of tiles x tile width is smallest -- a narrower tile can fill the last round.
int lmhead_tile(int vocab, int sms) {
  int best = kLmN;
  int64_t best_cost = -1;
  for (int n = kLmN; n >= 128; n -= 32) {
    const int64_t tiles = (vocab + n - 1) / n;
    const int64_t rounds = (tiles + sms - 1) / sms;
    const int64_t cost = rounds * (n + 64);  // a tile costs about its width plus a fixed part
    if (best_cost < 0 || cost < best_cost) {
      best = n;
      best_cost = cost;
    }
  }
  return best;
}

int lmhead_grid(const spiffy_decide_desc& d) {
  static int sms[64];
  int device = 0;
  if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= 64) return 0;
  if (sms[device] == 0 &&
      cudaDeviceGetAttribute(&sms[device], cudaDevAttrMultiProcessorCount, device) != cudaSuccess)
    return 0;
  const int n = lmhead_tile(d.vocab, sms[device]);
  const int n_tiles = (d.vocab + n - 1) / n;
  return n_tiles < sms[device] ? n_tiles : sms[device];
}

size_t lmhead_workspace_bytes(const spiffy_decide_desc& d, int grid) {
  return (size_t)d.batch * d.n_nodes * d.block_len * (size_t)grid * sizeof(Partial);
}

spiffy_status launch_lmhead_decide(const spiffy_decide_desc& d, int hidden, const void* hstates,
                                   const void* weight, const int32_t* block_tokens, float* conf,
                                   int32_t* top_tok, uint64_t* unmask_bits, int32_t* n_unmask,
                                   int32_t* dev_status, void* ws, cudaStream_t stream) {
  const int rows = d.batch * d.n_nodes * d.block_len;
  const int grid = lmhead_grid(d);
  if (grid <= 0) return SPIFFY_ECUDA;
  int sm_count = 0, dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return SPIFFY_ECUDA;
  const int n_tile = lmhead_tile(d.vocab, sm_count);
  CUtensorMap tm_h, tm_w;
  if (!make_map(&tm_h, hstates, hidden / 128, rows, 1, 1, 128) ||
      !make_map(&tm_w, weight, hidden / 128, d.vocab, 1, 1, n_tile))
    return SPIFFY_ECUDA;
  static bool attr_set[64];
  int device = 0;
  cudaGetDevice(&device);
  if (device >= 0 && device < 64 && !attr_set[device]) {
    if (cudaFuncSetAttribute(lmhead_reduce_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kLmSmem) !=
        cudaSuccess)
      return SPIFFY_ECUDA;
    attr_set[device] = true;
  }
  LmParams p;
  p.rows = rows;
  p.hidden = hidden;
  p.vocab = d.vocab;
  p.n_tile = n_tile;
  p.partials = static_cast<Partial*>(ws);
  p.status = dev_status;
  p.n_status = d.batch;
  p.spin_limit = mbar_poll_limit();
  cudaError_t e = launch_pdl(lmhead_reduce_kernel, dim3(grid), dim3(kLmThreads), (size_t)kLmSmem, stream,
                             tm_h, tm_w, p);
  count_launch();
  if (e != cudaSuccess) return SPIFFY_ECUDA;
  return launch_decide_finalize(d, ws, grid, block_tokens, conf, top_tok, unmask_bits, n_unmask, dev_status,
                                stream);
}

}  // namespace spiffy
