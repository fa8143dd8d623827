// Packed draft-graph attention (Sec. 4.3; mask of Fig. 3) on the sm_100a tensor
// cores: bf16 operands, head dimension 128.
//
// Work decomposition.  For one sequence b and one key/value head g, the query
// rows are all (node n, position l, query head of the group) triples; they all
// read the same P context keys, and a row of node n additionally reads the L
// keys of node n's own block.  An M-tile is TNL consecutive (n, l) positions
// times the `group` query heads of g (TNL = 128 / group, so at most 128 rows);
// a CTA owns one M-tile, or two neighbouring ones (see the kernel), and walks
// over key tiles of 128 keys: first the context tiles,
// then the tiles covering the block keys of the nodes its rows belong to.  The
// mask is never materialised: a context tile is visible to every row, and in a
// block-key tile row r sees exactly the columns of its own node, a contiguous
// column range computed from indices.
//
// Pipeline inside a CTA (320 threads):
//   warp 0      TMA producer: Q once, then K and V tiles into two rings (seven
//               32 KB tiles of shared memory in all); its first loads go out
//               before the rest of the CTA has finished setting up
//   warp 1      allocates tensor memory; one lane issues tcgen05.mma:
//               S = Q K^T (fp32 in TMEM, double buffered), O += P V
//   warps 2-9   two softmax warpgroups, one thread per row each.  With one
//               M-tile per CTA they split every key tile by columns (keys
//               0-63 and 64-127 of the tile), each with its own running
//               (maximum, sum) and accumulator O, merged once at the end; with
//               two M-tiles each warpgroup owns one.  A thread reads its scores
//               from TMEM, writes P (bf16) back over them as the A operand of
//               the second product, and rescales its O only when the maximum
//               grew by more than 2^8 (exact: O and the sum always share one
//               reference maximum).  32-column chunks of a block-key tile that
//               no row of a warp may see are skipped.
// With several splits (grid.z) each CTA handles a slice of the key tiles: two
// slices are the two CTAs of a cluster, which exchange their partials through
// each other's shared memory and finish half of the output columns each; more
// slices store unnormalised partials (O, reference maximum, sum) that a second
// kernel merges.
//
// Every wait is bounded; a wait that gives up raises SPIFFY_DEV_TIMEOUT in the
// caller's status word and the CTA winds down without touching its output.
#include <math.h>

#include "common.cuh"
#include "sm100_ptx.cuh"
#include "tma_map.cuh"

namespace spiffy {
namespace {

using namespace sm100;

constexpr int BM = 128;       // rows of an M-tile (TMEM lanes)
constexpr int BN = 128;       // keys per key tile
constexpr int HD = 128;       // head dimension
constexpr int kMaxStages = 3;  // most stages a K or V ring has
constexpr int kThreads = 320;  // producer warp, MMA warp, two softmax warpgroups
constexpr int kHalfBytes = BN * 128;           // one 64-column half of a tile: 128 rows x 128 B
constexpr int kTileBytes = 2 * kHalfBytes;     // 32 KB
constexpr uint32_t kTmemCols = 512;
// S: 2 x 128 columns (P, as bf16 pairs, overwrites the first 64 columns of its S);
// O: 2 x 128 columns, one accumulator per softmax warpgroup
constexpr uint32_t kColS = 0, kColO = 256;
constexpr float kRescaleLog2 = 8.0f;
// bytes a CTA of a pair receives from its peer: 128 rows x 64 columns of partial O, and (max, sum) per row
constexpr uint32_t kXchgBytes = BM * 64 * 4 + BM * 8;

// NQ M-tiles per CTA: NQ Q tiles, a K ring of 3 stages and a V ring of 4 - NQ
// stages: 7 tiles of 32 KB either way.
template <int NQ>
struct Smem {
  static constexpr int ks = 3, vs = 4 - NQ;
  static constexpr int q = 0;
  static constexpr int k = q + NQ * kTileBytes;
  static constexpr int v = k + ks * kTileBytes;
  static constexpr int bars = v + vs * kTileBytes;
  static constexpr int n_bars = 1 + 4 * kMaxStages + 2 + 2 + 2 + 2;
  static constexpr int tmem = bars + 8 * n_bars;
  static constexpr int abort_flag = tmem + 8;
  static constexpr int total = abort_flag + 8;
};
constexpr int kSmemBytes = Smem<1>::total + 1024;  // slack for 1024-byte alignment
static_assert(Smem<1>::total == Smem<2>::total, "both layouts use the same amount");

struct Params {
  int B, N, L, Hq, Hkv, group;
  int P, P2;    // context keys: first and second segment
  int TNL;      // (node, position) pairs per M-tile
  int NL;       // N * L
  int MT;       // M-tiles per (sequence, kv head)
  int TP1, TP;  // context key tiles: of the first segment, of both
  int splits;
  int pair;  // the two splits are the two CTAs of a cluster and merge through shared memory
  float scale_log2;
  __nv_bfloat16* out;
  float* part_o;   // [splits][B*Hkv][MT][128][128]
  float* part_ml;  // [splits][B*Hkv][MT][128][2]
  int32_t* status;
  uint32_t spin_limit;  // polls of one mbarrier wait
  int early_trigger;    // let the next kernel of the stream begin its set-up while this one runs
};

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// One thread's NC scores of a row (raw bits in s, -inf where masked): the
// maximum over the 32-column chunks flagged in `need`.
template <int NC>
__device__ __forceinline__ float row_max(const uint32_t (&s)[NC], uint32_t need) {
  float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
  for (int h = 0; h < NC / 32; ++h) {
    if ((need >> h) & 1u) {
#pragma unroll
      for (int c = 32 * h; c < 32 * h + 32; c += 8) {
        mx0 = max3(mx0, __uint_as_float(s[c]), __uint_as_float(s[c + 1]));
        mx1 = max3(mx1, __uint_as_float(s[c + 2]), __uint_as_float(s[c + 3]));
        mx2 = max3(mx2, __uint_as_float(s[c + 4]), __uint_as_float(s[c + 5]));
        mx3 = max3(mx3, __uint_as_float(s[c + 6]), __uint_as_float(s[c + 7]));
      }
    }
  }
  return fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
}

// p = 2^(s * k2 - m_use) for the flagged chunks (zero elsewhere), packed as bf16
// pairs into pk; returns the sum of the p's (fp32, before rounding to bf16).
template <int NC>
__device__ __forceinline__ float row_exps(const uint32_t (&s)[NC], uint32_t need, float k2, float m_use,
                                          uint32_t (&pk)[NC / 2]) {
  const uint64_t k22 = pack2(k2, k2), nm2 = pack2(-m_use, -m_use);
  uint64_t sum_a = pack2(0.f, 0.f), sum_b = pack2(0.f, 0.f);
#pragma unroll
  for (int h = 0; h < NC / 32; ++h) {
    if ((need >> h) & 1u) {
#pragma unroll
      for (int c = 32 * h; c < 32 * h + 32; c += 2) {
        const uint64_t x2 = fma2(pack2(__uint_as_float(s[c]), __uint_as_float(s[c + 1])), k22, nm2);
        float x0, x1;
        unpack2(x2, x0, x1);
        const float p0 = ex2(x0), p1 = ex2(x1);
        if ((c >> 1) & 1) sum_b = add2(sum_b, pack2(p0, p1)); else sum_a = add2(sum_a, pack2(p0, p1));
        pk[c >> 1] = pack_bf16(p0, p1);
      }
    } else {
#pragma unroll
      for (int c = 16 * h; c < 16 * h + 16; ++c) pk[c] = 0u;
    }
  }
  float a0, a1;
  unpack2(add2(sum_a, sum_b), a0, a1);
  return a0 + a1;
}

// Bounded wait that ignores the abort flag (used while winding down).
__device__ __forceinline__ void mbar_wait_quiet(uint64_t* bar, uint32_t parity) {
  for (uint32_t i = 0; i < kSpinLimit; ++i)
    if (mbar_try_wait(bar, parity)) return;
}

// Row r of an M-tile sees the columns [lo, hi) of key tile t (tile-relative).
struct Window {
  int lo, hi;
};
__device__ __forceinline__ Window visible_window(const Params& p, int t, int kb_start, int node) {
  Window w;
  if (t < p.TP) {  // context: every row sees every key that exists
    w.lo = 0;
    w.hi = t < p.TP1 ? min(BN, p.P - t * BN) : min(BN, p.P2 - (t - p.TP1) * BN);
  } else {  // block keys: the row's own node only
    w.lo = node * p.L - (kb_start + (t - p.TP) * BN);
    w.hi = w.lo + p.L;
  }
  return w;
}

// NQ = 1: the CTA owns one M-tile.  Its two softmax warpgroups split every key
// tile by columns: warpgroup w owns the scores of keys 64 w .. 64 w + 63 of the
// tile, keeps its own running (maximum, sum) and its own accumulator O_w, so
// that the two never exchange anything per tile and both work on every tile;
// O_0 and O_1 are merged once, at the end.
// NQ = 2: the CTA owns two neighbouring M-tiles, one per warpgroup, and every
// K/V tile brought into shared memory serves both, which halves the L2-to-SM
// traffic per flop.
template <int NQ>
__global__ void __launch_bounds__(kThreads, 1)
graph_attention_tc_kernel(const __grid_constant__ CUtensorMap tm_q,
                          const __grid_constant__ CUtensorMap tm_kp,
                          const __grid_constant__ CUtensorMap tm_vp,
                          const __grid_constant__ CUtensorMap tm_kp2,
                          const __grid_constant__ CUtensorMap tm_vp2,
                          const __grid_constant__ CUtensorMap tm_kb,
                          const __grid_constant__ CUtensorMap tm_vb, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  using SM = Smem<NQ>;
  constexpr int KS = SM::ks, VS = SM::vs;
  uint8_t* sq = smem + SM::q;
  uint8_t* sk = smem + SM::k;
  uint8_t* sv = smem + SM::v;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SM::bars);
  uint64_t* q_full = bars;
  uint64_t* k_full = bars + 1;
  uint64_t* k_empty = k_full + KS;
  uint64_t* v_full = k_empty + KS;
  uint64_t* v_empty = v_full + VS;
  uint64_t* s_full = v_empty + VS;   // [2]
  uint64_t* p_ready = s_full + 2;    // [2]
  // P V products done.  NQ = 2: one barrier per warpgroup (a thread is never more than one tile
  // ahead of its products).  NQ = 1: one per parity of the key tile: S is double buffered there, a
  // softmax thread may be two tiles ahead of the products, and the phase parity of ONE barrier
  // cannot tell "tile j - 2 still running" from "tile j - 1 done".
  uint64_t* pv_done = p_ready + 2;   // [2]
  uint64_t* xchg_ready = pv_done + 2;  // pair: the peer's Q tile and first K stage may be overwritten
  uint64_t* xchg_full = xchg_ready + 1;  // pair: the peer's partial has arrived here
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + SM::tmem);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + SM::abort_flag);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int mt = blockIdx.x * NQ;  // first M-tile of this CTA
  const int bg = blockIdx.y;
  const int b = bg / p.Hkv, g = bg % p.Hkv;
  const int split = blockIdx.z;
  const bool pair = NQ == 1 && p.pair != 0;

  // this CTA's rows and key tiles
  const int nl0 = mt * p.TNL;
  const int nl_count = min(NQ * p.TNL, p.NL - nl0);  // over all M-tiles of the CTA
  const int rows_box = p.TNL * p.group;        // rows one Q box writes
  const int n_lo = nl0 / p.L, n_hi = (nl0 + nl_count - 1) / p.L;
  const int kb_start = n_lo * p.L;
  const int TB = ((n_hi - n_lo + 1) * p.L + BN - 1) / BN;
  const int T_all = p.TP + TB;
  const int t_begin = split * T_all / p.splits;  // small numbers: splits <= T_all <= a few thousand
  const int t_end = (split + 1) * T_all / p.splits;
  const int T = t_end - t_begin;

  // ---- producers.  K tiles (and Q) are loaded by lane 0 of warp 0, V tiles by
  // lane 0 of warp 1 until that thread turns to issuing the products; each
  // initialises the barriers of its ring itself, so that its first loads go out
  // at once, ahead of the rest of the set-up (tensor-memory allocation, the
  // CTA-wide barrier).  `produce` issues tile j of one ring; may_wait = false:
  // only if its stage is still in its first round (nothing to wait for).
  int issued_k = 0, issued_v = 0;
  bool prod_ok = true;
  auto produce = [&](bool is_k, int j, bool may_wait) -> bool {
    const int depth = is_k ? KS : VS;
    const int stage = j % depth;
    const uint32_t round = (uint32_t)(j / depth);
    if (round > 0) {
      if (!may_wait) return false;
      if (!mbar_wait((is_k ? k_empty : v_empty) + stage, (round & 1u) ^ 1u, abort_flag, p.spin_limit)) {
        prod_ok = false;
        return false;
      }
    }
    uint64_t* full = (is_k ? k_full : v_full) + stage;
    const int t = t_begin + j;
    // key tiles in order: first context segment, second context segment, block keys
    const int seg = t < p.TP1 ? 0 : (t < p.TP ? 1 : 2);
    const CUtensorMap* m = is_k ? (seg == 0 ? &tm_kp : seg == 1 ? &tm_kp2 : &tm_kb)
                                : (seg == 0 ? &tm_vp : seg == 1 ? &tm_vp2 : &tm_vb);
    const int key0 = seg == 0 ? t * BN : seg == 1 ? (t - p.TP1) * BN : kb_start + (t - p.TP) * BN;
    uint8_t* dst = (is_k ? sk : sv) + stage * kTileBytes;
    mbar_arrive_expect_tx(full, kTileBytes);
    tma_load_4d(dst, m, full, 0, g, key0, b);
    tma_load_4d(dst + kHalfBytes, m, full, 64, g, key0, b);
    if (is_k) issued_k = j + 1; else issued_v = j + 1;
    return true;
  };

  if (threadIdx.x == 0) {
    prefetch_tensormap(&tm_q);  // the descriptors are kernel parameters
    prefetch_tensormap(p.TP1 > 0 ? &tm_kp : (p.TP > 0 ? &tm_kp2 : &tm_kb));
    mbar_init(q_full, 1);
    for (int i = 0; i < KS; ++i) { mbar_init(k_full + i, 1); mbar_init(k_empty + i, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(s_full + i, 1); mbar_init(p_ready + i, NQ == 1 ? 8 : 4); }  // one arrival per softmax warp
    mbar_init(pv_done, 1);
    mbar_init(pv_done + 1, 1);
    mbar_init(xchg_ready, 1);
    mbar_init(xchg_full, 1);
    *abort_flag = 0;
    mbar_fence_init();
    if (pair) mbar_arrive_expect_tx(xchg_full, kXchgBytes);  // what the peer will send in the epilogue
    cudaGridDependencySynchronize();
    if (T > 0) {
      mbar_arrive_expect_tx(q_full, (uint32_t)NQ * 2u * rows_box * 128u);
#pragma unroll
      for (int q = 0; q < NQ; ++q) {  // an M-tile beyond the last one reads as zeros
        tma_load_4d(sq + q * kTileBytes, &tm_q, q_full, 0, g * p.group, nl0 + q * p.TNL, b);
        tma_load_4d(sq + q * kTileBytes + kHalfBytes, &tm_q, q_full, 64, g * p.group,
                    nl0 + q * p.TNL, b);
      }
      while (issued_k < T && produce(true, issued_k, false)) {}
    }
  } else if (threadIdx.x == 32) {
    prefetch_tensormap(p.TP1 > 0 ? &tm_vp : (p.TP > 0 ? &tm_vp2 : &tm_vb));
    for (int i = 0; i < VS; ++i) { mbar_init(v_full + i, 1); mbar_init(v_empty + i, 1); }
    mbar_fence_init();
    cudaGridDependencySynchronize();
    while (issued_v < T && produce(false, issued_v, false)) {}
  }
  // rows of the Q tile that the TMA box does not write must be finite
  for (int i = rows_box * 8 + threadIdx.x; i < BM * 8; i += kThreads) {
    const uint4 z = make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int h = 0; h < 2 * NQ; ++h) reinterpret_cast<uint4*>(sq + h * kHalfBytes)[i] = z;
  }
  fence_proxy_async_smem();
  if (warp == 1) tmem_alloc(tmem_slot, kTmemCols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;
  // pair: both CTAs' barriers exist before either touches the other's (waited for in the epilogue)
  if (pair) cluster_arrive();
  if (p.early_trigger) pdl_launch_dependents();
  // everything above is on-chip set-up (thread 0 aside); global memory is touched from here on
  cudaGridDependencySynchronize();

  if (warp == 0) {
    // ------------------------------------------------------------ producer --
    if (lane == 0 && T > 0) {
      // the rest of both rings, in the order the products need them: K(j+1) before V(j)
      issued_v = min(T, VS);             // what warp 1's lane issued before the barrier
      int jk = issued_k, jv = issued_v;
      while (prod_ok && (jk < T || jv < T)) {
        if (jk < T && jk <= jv + 1) {
          if (produce(true, jk, true)) ++jk;
        } else if (jv < T) {
          if (produce(false, jv, true)) ++jv;
        }
      }
      if (!prod_ok) {
        // winding down: let the copies already in flight land before exit
        mbar_wait_quiet(q_full, 0);
        for (int j = max(0, issued_k - KS); j < issued_k; ++j)
          mbar_wait_quiet(k_full + j % KS, (uint32_t)(j / KS) & 1u);
        for (int j = max(0, issued_v - VS); j < issued_v; ++j)
          mbar_wait_quiet(v_full + j % VS, (uint32_t)(j / VS) & 1u);
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------- MMA issuer --
    if (lane == 0 && T > 0) {
      constexpr uint32_t idesc_s = idesc_bf16_f32(BM, BN, false, false);
      constexpr uint32_t idesc_o = idesc_bf16_f32(BM, HD, false, true);
      constexpr uint32_t hi = desc_hi_sw128(1024);
      const uint32_t q_lo = desc_lo_sw128(smem_u32(sq), 16);
      const uint32_t k_lo = desc_lo_sw128(smem_u32(sk), 16);
      const uint32_t v_lo = desc_lo_sw128(smem_u32(sv), kHalfBytes);
      bool ok = mbar_wait(q_full, 0, abort_flag, p.spin_limit);
      // S = Q K^T of key tile j into S buffer `buf`, from Q tile `qt`
      auto issue_s = [&](int j, int buf, int qt) {
        umma_ss_k128(tmem + kColS + (uint32_t)buf * BN, q_lo + (uint32_t)qt * (kTileBytes >> 4),
                     k_lo + (uint32_t)(j % KS) * (kTileBytes >> 4), hi, idesc_s, 0u);
        umma_commit(s_full + buf);
      };
      auto wait_k = [&](int j) {
        if (ok && !mbar_wait(k_full + j % KS, (uint32_t)(j / KS) & 1u, abort_flag, p.spin_limit)) ok = false;
        tc_fence_after_sync();
      };
      if constexpr (NQ == 1) {
        // the two S buffers hold consecutive key tiles
        auto s_tile = [&](int j) {
          wait_k(j);
          if (!ok) return;
          issue_s(j, j & 1, 0);
          umma_commit(k_empty + j % KS);
        };
        s_tile(0);
        if (T > 1) s_tile(1);
        for (int j = 0; j < T && ok; ++j) {
          // the operands of both products that follow P(j) are waited for first (they arrive
          // long before it), so that nothing stands between P(j) and S(j+2)
          if (!mbar_wait(v_full + j % VS, (uint32_t)(j / VS) & 1u, abort_flag, p.spin_limit)) { ok = false; break; }
          if (j + 2 < T) wait_k(j + 2);
          if (!ok) break;
          if (!mbar_wait(p_ready + (j & 1), (uint32_t)(j >> 1) & 1u, abort_flag, p.spin_limit)) { ok = false; break; }
          tc_fence_after_sync();
          // O_w (+)= P[:, 64 w .. 64 w + 63] V[64 w .. 64 w + 63, :] for both warpgroups' halves
          const uint32_t a = tmem + kColS + (uint32_t)(j & 1) * BN;
          const uint32_t vj = v_lo + (uint32_t)(j % VS) * (kTileBytes >> 4);
          umma_ts_k64(tmem + kColO, a, vj, hi, idesc_o, j > 0 ? 1u : 0u);
          umma_ts_k64(tmem + kColO + HD, a + 64u, vj + 4u * 128u, hi, idesc_o, j > 0 ? 1u : 0u);
          umma_commit(v_empty + j % VS);
          umma_commit(pv_done + (j & 1));
          if (j + 2 < T) {
            issue_s(j + 2, j & 1, 0);
            umma_commit(k_empty + (j + 2) % KS);
          }
        }
      } else {
        // S buffer q belongs to M-tile q; a key tile serves both before it is released
        wait_k(0);
        if (ok) {
          issue_s(0, 0, 0);
          issue_s(0, 1, 1);
          umma_commit(k_empty + 0);
        }
        for (int j = 0; j < T && ok; ++j) {
          if (!mbar_wait(v_full + j % VS, (uint32_t)(j / VS) & 1u, abort_flag, p.spin_limit)) { ok = false; break; }
          if (j + 1 < T) wait_k(j + 1);
          for (int q = 0; q < 2 && ok; ++q) {
            if (!mbar_wait(p_ready + q, (uint32_t)j & 1u, abort_flag, p.spin_limit)) { ok = false; break; }
            tc_fence_after_sync();
            umma_ts_k128(tmem + kColO + (uint32_t)q * HD, tmem + kColS + (uint32_t)q * BN,
                         v_lo + (uint32_t)(j % VS) * (kTileBytes >> 4), hi, idesc_o, j > 0 ? 1u : 0u);
            umma_commit(pv_done + q);
            if (j + 1 < T) issue_s(j + 1, q, q);  // after PV: P of this tile has been consumed
          }
          if (!ok) break;
          umma_commit(v_empty + j % VS);
          if (j + 1 < T) umma_commit(k_empty + (j + 1) % KS);
        }
      }
    }
  } else if (T > 0) {
    // ------------------------------------------------------------- softmax --
    const int quad = warp & 3;               // TMEM lane quadrant this warp may touch
    const int wg = (warp - 2) >> 2;
    const int r = quad * 32 + lane;          // row of the M-tile
    const int nl_tile = nl0 + (NQ == 2 ? wg * p.TNL : 0);  // first (node, position) of the rows
    const int rows_valid = max(0, min(p.TNL, p.NL - nl_tile)) * p.group;
    const bool row_ok = r < rows_valid;
    const int nl = nl_tile + r / p.group;
    const int hh = r % p.group;
    const int node = min(nl, p.NL - 1) / p.L;
    const uint32_t lane_base = (uint32_t)(quad * 32);
    const float k2 = p.scale_log2;
    float m_run = -INFINITY, l_run = 0.f;  // reference maximum (log2 units) and sum of this thread's accumulator
    bool ok = true;
    // this thread's accumulator: NQ = 1 columns half wg of every tile, NQ = 2 all of M-tile wg
    const uint32_t col_o = kColO + (uint32_t)wg * HD;
    // every product into this thread's accumulator up to key tile j has completed
    auto wait_pv = [&](int j) -> bool {
      uint64_t* bar = NQ == 1 ? pv_done + (j & 1) : pv_done + wg;
      const uint32_t parity = NQ == 1 ? (uint32_t)(j >> 1) & 1u : (uint32_t)j & 1u;
      return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag, p.spin_limit));
    };

    // O *= corr once the products that still write to it have completed
    auto rescale_o = [&](int j, float corr) -> bool {
      if (!wait_pv(j - 1)) return false;
      tc_fence_after_sync();
#pragma unroll
      for (int c0 = 0; c0 < HD; c0 += 32) {
        uint32_t o[32];
        tmem_ld_x32(tmem_addr(tmem, lane_base, col_o + c0), o);
#pragma unroll
        for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * corr);
        tmem_st_x32(tmem_addr(tmem, lane_base, col_o + c0), o);
      }
      tmem_wait_st();
      return true;
    };

    if constexpr (NQ == 1) {
      const int half0 = 64 * wg;  // first tile column of this warpgroup's half
      if (pair) cluster_wait();  // phase 1: the peer's barriers exist
      for (int j = 0; j < T; ++j) {
        const int bi = j & 1;
        const uint32_t col_s = kColS + (uint32_t)bi * BN + (uint32_t)half0;
        // wait outcomes are made warp-uniform: the TMEM accesses below are warp-collective
        if (!__all_sync(0xffffffffu, mbar_wait(s_full + bi, (uint32_t)(j >> 1) & 1u, abort_flag, p.spin_limit))) {
          ok = false;
          break;
        }
        tc_fence_after_sync();
        // the last S has been formed: the Q tile and the first K stage are free for the peer's partial
        if (pair && j == T - 1 && warp == 2 && lane == 0)
          mbar_arrive_remote(map_to_cta(smem_u32(xchg_ready), (uint32_t)split ^ 1u));
        uint32_t s[64];
        tmem_ld_x64(tmem_addr(tmem, lane_base, col_s), s);
        Window w = visible_window(p, t_begin + j, kb_start, node);
        const int lo = w.lo - half0, hi = w.hi - half0;  // relative to the half: columns [0, 64)
        // 32-column chunks that no row of the warp sees cost nothing but zeros in P
        const bool need0 = __any_sync(0xffffffffu, lo < 32 && hi > 0);
        const bool need1 = __any_sync(0xffffffffu, lo < 64 && hi > 32);
        if (!(lo <= 0 && hi >= 64)) {
#pragma unroll
          for (int c = 0; c < 64; ++c)
            s[c] = (c >= lo && c < hi) ? s[c] : 0xff800000u;  // -inf
        }
        const uint32_t chunks = (need0 ? 1u : 0u) | (need1 ? 2u : 0u);
        const float mx = row_max<64>(s, chunks);
        const float m_new = fmaxf(m_run, mx * k2);
        const bool need = (m_new - m_run) > kRescaleLog2;  // false when both are -inf
        if (__any_sync(0xffffffffu, need)) {
          float corr = 1.f;
          if (need) {
            corr = ex2(m_run - m_new);  // 0 for a row that had seen nothing yet
            l_run *= corr;
            m_run = m_new;
          }
          if (j > 0 && !rescale_o(j, corr)) {  // the accumulator holds the earlier tiles
            ok = false;
            break;
          }
        }
        const float m_use = (m_run == -INFINITY) ? 0.f : m_run;
        uint32_t pk[32];
        l_run += row_exps<64>(s, chunks, k2, m_use, pk);
        // P goes over the first half of the score columns just read (every thread owns its lane)
        tmem_st_x32(tmem_addr(tmem, lane_base, col_s), pk);
        tmem_wait_st();
        tc_fence_before_sync();
        __syncwarp();  // every lane's P is in tensor memory: one arrival speaks for the warp
        if (lane == 0) mbar_arrive(p_ready + bi);
      }
    } else {
      for (int j = 0; j < T; ++j) {
        const uint32_t col_s = kColS + (uint32_t)wg * BN;
        if (!__all_sync(0xffffffffu, mbar_wait(s_full + wg, (uint32_t)j & 1u, abort_flag, p.spin_limit))) {
          ok = false;
          break;
        }
        tc_fence_after_sync();
        uint32_t s[BN];
        tmem_ld_x128(tmem_addr(tmem, lane_base, col_s), s);
        const Window w = visible_window(p, t_begin + j, kb_start, node);
        if (!(w.lo <= 0 && w.hi >= BN)) {
#pragma unroll
          for (int c = 0; c < BN; ++c)
            s[c] = (c >= w.lo && c < w.hi) ? s[c] : 0xff800000u;  // -inf
        }
        const float mx = row_max<BN>(s, 0xfu);
        const float m_new = fmaxf(m_run, mx * k2);
        const bool need = (m_new - m_run) > kRescaleLog2;  // false when both are -inf
        if (__any_sync(0xffffffffu, need)) {
          float corr = 1.f;
          if (need) {
            corr = ex2(m_run - m_new);  // 0 for a row that had seen nothing yet
            l_run *= corr;
            m_run = m_new;
          }
          if (j > 0 && !rescale_o(j, corr)) {
            ok = false;
            break;
          }
        }
        const float m_use = (m_run == -INFINITY) ? 0.f : m_run;
        uint32_t pk[BN / 2];
        l_run += row_exps<BN>(s, 0xfu, k2, m_use, pk);
        tmem_st_x64(tmem_addr(tmem, lane_base, col_s), pk);
        tmem_wait_st();
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(p_ready + wg);
      }
    }
    // ------------------------------------------------------------ epilogue --
    // every product into this thread's accumulator has completed
    if (ok) ok = wait_pv(T - 1);
    __nv_bfloat16* dst =
        p.out + (((int64_t)b * p.NL + nl) * p.Hq + (int64_t)g * p.group + hh) * HD;
    if constexpr (NQ == 2) {
      // each warpgroup owns its rows outright: normalise (or hand on the partial) and store
      if (ok) {
        tc_fence_after_sync();
        const float inv = p.splits == 1 ? 1.0f / l_run : 1.0f;
        const int64_t tile = ((int64_t)split * gridDim.y + bg) * p.MT + mt + wg;
        float* po = p.part_o + (tile * BM + r) * HD;
#pragma unroll
        for (int c0 = 0; c0 < HD; c0 += 32) {
          uint32_t o[32];
          tmem_ld_x32(tmem_addr(tmem, lane_base, col_o + c0), o);
          if (row_ok) {
            if (p.splits == 1) {
#pragma unroll
              for (int c = 0; c < 32; c += 8) {
                uint4 w;
                w.x = pack_bf16(__uint_as_float(o[c]) * inv, __uint_as_float(o[c + 1]) * inv);
                w.y = pack_bf16(__uint_as_float(o[c + 2]) * inv, __uint_as_float(o[c + 3]) * inv);
                w.z = pack_bf16(__uint_as_float(o[c + 4]) * inv, __uint_as_float(o[c + 5]) * inv);
                w.w = pack_bf16(__uint_as_float(o[c + 6]) * inv, __uint_as_float(o[c + 7]) * inv);
                *reinterpret_cast<uint4*>(dst + c0 + c) = w;
              }
            } else {
#pragma unroll
              for (int c = 0; c < 32; c += 4)
                *reinterpret_cast<uint4*>(po + c0 + c) = make_uint4(o[c], o[c + 1], o[c + 2], o[c + 3]);
            }
          }
        }
        if (p.splits > 1 && row_ok) {
          float* pml = p.part_ml + (tile * BM + r) * 2;
          pml[0] = m_run;
          pml[1] = l_run;
        }
      }
    } else {
      // The two warpgroups exchange their (reference maximum, sum) per row through
      // spare columns of the first S buffer (every product has completed), and
      // each then merges and stores one half of the output columns of every row.
      constexpr uint32_t kColMl = kColS + 32;  // S columns 32..63 hold no P
      tmem_st_x2(tmem_addr(tmem, lane_base, kColMl + 2u * (uint32_t)wg), __float_as_uint(m_run),
                 __float_as_uint(l_run));
      tmem_wait_st();
      tc_fence_before_sync();
      asm volatile("bar.sync 1, 256;" ::: "memory");  // all eight softmax warps, whatever `ok` says
      tc_fence_after_sync();
      uint32_t um, ul;
      tmem_ld_x2(tmem_addr(tmem, lane_base, kColMl + 2u * (uint32_t)(wg ^ 1)), um, ul);
      const float m_o = __uint_as_float(um), l_o = __uint_as_float(ul);
      const float m_a = wg == 0 ? m_run : m_o, l_a = wg == 0 ? l_run : l_o;
      const float m_b = wg == 0 ? m_o : m_run, l_b = wg == 0 ? l_o : l_run;
      const float m_all = fmaxf(m_a, m_b);
      // an accumulator whose half held no visible key of this row is left out
      const bool has_a = m_a != -INFINITY, has_b = m_b != -INFINITY;
      const float w_a = has_a ? ex2(m_a - m_all) : 0.f;
      const float w_b = has_b ? ex2(m_b - m_all) : 0.f;
      const float l_all = w_a * l_a + w_b * l_b;
      // 32 columns of this CTA's two accumulators, merged against m_all and scaled by f
      auto merged = [&](int c0, float f, float (&o)[32]) {
        uint32_t oa[32], ob[32];
        tmem_ld_x32(tmem_addr(tmem, lane_base, kColO + c0), oa);
        tmem_ld_x32(tmem_addr(tmem, lane_base, kColO + HD + c0), ob);
        const float f_a = w_a * f, f_b = w_b * f;
#pragma unroll
        for (int c = 0; c < 32; ++c)
          o[c] = (has_a ? __uint_as_float(oa[c]) * f_a : 0.f) +
                 (has_b ? __uint_as_float(ob[c]) * f_b : 0.f);
      };
      auto store_bf16 = [&](__nv_bfloat16* at, const float (&o)[32]) {
#pragma unroll
        for (int c = 0; c < 32; c += 8) {
          uint4 w;
          w.x = pack_bf16(o[c], o[c + 1]);
          w.y = pack_bf16(o[c + 2], o[c + 3]);
          w.z = pack_bf16(o[c + 4], o[c + 5]);
          w.w = pack_bf16(o[c + 6], o[c + 7]);
          *reinterpret_cast<uint4*>(at + c) = w;
        }
      };
      if (pair) {
        // The other half of the key tiles went to the peer CTA of the cluster.  Each of the
        // two finishes 64 of the 128 output columns: it sends its partial of the peer's
        // columns into the peer's shared memory (the Q tile and the first K stage, idle
        // since the last S) and merges what it gets.  Hand-over by mbarriers: xchg_ready =
        // "my buffers are free" (sent from the tile loop), xchg_full = "your partial has
        // landed", completed by the byte count of the asynchronous stores themselves.
        const uint32_t rank = (uint32_t)split, peer = rank ^ 1u;
        if (ok) ok = __all_sync(0xffffffffu, mbar_wait_cluster(xchg_ready, 0, abort_flag, p.spin_limit));
        if (ok) {
          tc_fence_after_sync();
          const uint32_t q_peer = map_to_cta(smem_u32(sq), peer);
          const uint32_t bar_peer = map_to_cta(smem_u32(xchg_full), peer);
          float o[32];
          merged(64 * (int)peer + 32 * wg, 1.0f, o);
#pragma unroll
          for (int k = 0; k < 8; ++k)  // 16-byte chunk (8 wg + k) of row r: chunk-major, rows contiguous
            st_async_f4(q_peer + (uint32_t)(8 * wg + k) * 2048u + (uint32_t)r * 16u, bar_peer, o[4 * k],
                        o[4 * k + 1], o[4 * k + 2], o[4 * k + 3]);
          if (wg == 0) st_async_f2(map_to_cta(smem_u32(sk), peer) + (uint32_t)r * 8u, bar_peer, m_all, l_all);
        }
        cluster_arrive();  // phase 2: this thread issues nothing more towards the peer
        // this CTA's own share of its output columns, read while the peer's partial travels
        float o[32];
        merged(64 * (int)rank + 32 * wg, 1.0f, o);
        if (ok) ok = __all_sync(0xffffffffu, mbar_wait_cluster(xchg_full, 0, abort_flag, p.spin_limit));
        if (ok) {
          const float2 mlp = *reinterpret_cast<const float2*>(sk + r * 8);
          const float m_p = mlp.x, l_p = mlp.y;
          const float m_fin = fmaxf(m_all, m_p);
          const float w_l = m_all != -INFINITY ? ex2(m_all - m_fin) : 0.f;
          const float w_p = m_p != -INFINITY ? ex2(m_p - m_fin) : 0.f;
          const float inv = 1.0f / (w_l * l_all + w_p * l_p);
          const float f_l = w_l * inv, f_p = w_p * inv;
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const float4 q4 = *reinterpret_cast<const float4*>(sq + (8 * wg + k) * 2048 + r * 16);
            o[4 * k] = o[4 * k] * f_l + (w_p != 0.f ? q4.x * f_p : 0.f);
            o[4 * k + 1] = o[4 * k + 1] * f_l + (w_p != 0.f ? q4.y * f_p : 0.f);
            o[4 * k + 2] = o[4 * k + 2] * f_l + (w_p != 0.f ? q4.z * f_p : 0.f);
            o[4 * k + 3] = o[4 * k + 3] * f_l + (w_p != 0.f ? q4.w * f_p : 0.f);
          }
          if (row_ok) store_bf16(dst + 64 * (int)rank + 32 * wg, o);
        }
      } else if (ok) {
        tc_fence_after_sync();
        const float inv = p.splits == 1 ? 1.0f / l_all : 1.0f;
        const int64_t tile = ((int64_t)split * gridDim.y + bg) * p.MT + mt;
        float* po = p.part_o + (tile * BM + r) * HD;
        for (int c0 = wg * 64; c0 < wg * 64 + 64; c0 += 32) {  // each warpgroup stores one half
          float o[32];
          merged(c0, inv, o);
          if (row_ok) {
            if (p.splits == 1) {
              store_bf16(dst + c0, o);
            } else {
#pragma unroll
              for (int c = 0; c < 32; c += 4)
                *reinterpret_cast<float4*>(po + c0 + c) = make_float4(o[c], o[c + 1], o[c + 2], o[c + 3]);
            }
          }
        }
        if (p.splits > 1 && row_ok && wg == 0) {
          float* pml = p.part_ml + (tile * BM + r) * 2;
          pml[0] = m_all;
          pml[1] = l_all;
        }
      }
    }  // NQ == 1
  }

  if (pair) {
    // No CTA of the pair leaves while the other may still write into its shared
    // memory or arrive on its barriers: a second phase of the cluster barrier
    // (the softmax warps have arrived on it in the epilogue).
    if (warp < 2 || T <= 0) {
      cluster_wait();  // phase 1
      cluster_arrive();
    }
    cluster_wait();
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, kTmemCols);
  }
  if (threadIdx.x == 0 && *abort_flag && p.status) atomicOr(p.status, SPIFFY_DEV_TIMEOUT);
}

// Merge of the per-split partials: one warp per output row, lane = 4 columns.
__global__ void __launch_bounds__(256)
graph_attention_combine_kernel(const Params p) {
  cudaGridDependencySynchronize();  // the partials are visible
  const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);  // (b, nl, h)
  const int lane = threadIdx.x & 31;
  const int64_t rows = (int64_t)p.B * p.NL * p.Hq;
  if (row >= rows) return;
  const int h = (int)(row % p.Hq);
  const int nl = (int)((row / p.Hq) % p.NL);
  const int b = (int)(row / ((int64_t)p.Hq * p.NL));
  const int g = h / p.group, hh = h % p.group;
  const int mt = nl / p.TNL;
  const int r = (nl - mt * p.TNL) * p.group + hh;
  const int64_t BG = (int64_t)p.B * p.Hkv;
  float M = -INFINITY;
  for (int s = 0; s < p.splits; ++s) {
    const int64_t tile = ((int64_t)s * BG + (int64_t)b * p.Hkv + g) * p.MT + mt;
    M = fmaxf(M, p.part_ml[(tile * BM + r) * 2]);
  }
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  float l = 0.f;
  for (int s = 0; s < p.splits; ++s) {
    const int64_t tile = ((int64_t)s * BG + (int64_t)b * p.Hkv + g) * p.MT + mt;
    const float m = p.part_ml[(tile * BM + r) * 2];
    if (m == -INFINITY) continue;  // this slice held no visible key for the row
    const float w = ex2(m - M);
    l += w * p.part_ml[(tile * BM + r) * 2 + 1];
    const float4 o = *reinterpret_cast<const float4*>(p.part_o + (tile * BM + r) * HD + lane * 4);
    acc.x += w * o.x; acc.y += w * o.y; acc.z += w * o.z; acc.w += w * o.w;
  }
  const float inv = 1.0f / l;
  uint2 w2;
  w2.x = pack_bf16(acc.x * inv, acc.y * inv);
  w2.y = pack_bf16(acc.z * inv, acc.w * inv);
  *reinterpret_cast<uint2*>(p.out + row * HD + lane * 4) = w2;
}

// ------------------------------------------------------------------ host ----
struct Plan {
  int group, TNL, NL, MT, TP1, TP, splits;
  int nq;    // M-tiles per CTA
  int pair;  // key tiles split over the two CTAs of a cluster (no workspace, no merge kernel)
  int64_t tiles;  // B * Hkv * MT
};

Plan make_plan(const spiffy_attn_desc& d, int ctx2_len) {
  Plan pl;
  pl.group = d.n_q_heads / d.n_kv_heads;
  pl.TNL = BM / pl.group;
  pl.NL = d.n_nodes * d.block_len;
  pl.MT = (pl.NL + pl.TNL - 1) / pl.TNL;
  pl.TP1 = (d.prefix_len + BN - 1) / BN;
  pl.TP = pl.TP1 + (ctx2_len + BN - 1) / BN;
  pl.tiles = (int64_t)d.batch * d.n_kv_heads * pl.MT;
  // Two M-tiles per CTA once the paired CTAs still fill the machine: every K/V
  // tile then serves twice as many rows per trip from L2.
  pl.nq = ((int64_t)d.batch * d.n_kv_heads * ((pl.MT + 1) / 2) >= 148) ? 2 : 1;
  // Fewer CTAs than SMs: cut the key tiles of each M-tile into slices so that
  // the context streams through more SMs at once.  Many slices go through the
  // workspace and a merge kernel (which costs about three key tiles); two
  // slices are the two CTAs of a cluster and merge through shared memory.
  int splits = 1;
  pl.pair = 0;
  if (pl.tiles < 120 && pl.TP + 1 >= 8 && 148 / pl.tiles >= 3) {
    splits = (int)(148 / pl.tiles);
    if (splits > pl.TP + 1) splits = pl.TP + 1;
  } else if (pl.nq == 1 && 2 * pl.tiles <= 148 && pl.TP + 1 >= 4) {
    splits = 2;
    pl.pair = 1;
  }
  pl.splits = splits;
  return pl;
}

}  // namespace

bool attention_tc_supported(const spiffy_attn_desc& d) {
  if (d.dtype != SPIFFY_BF16 || d.head_dim != HD) return false;
  const int group = d.n_q_heads / d.n_kv_heads;
  if (group > BM) return false;
  if ((int64_t)d.batch * d.n_kv_heads > 65535) return false;
  return true;
}

size_t attention_tc_workspace_bytes(const spiffy_attn_desc& d, int ctx2_len) {
  const Plan pl = make_plan(d, ctx2_len);
  if (pl.splits == 1 || pl.pair) return 0;
  return (size_t)pl.splits * pl.tiles * BM * (HD + 2) * sizeof(float);
}

spiffy_status launch_attention_tc(const spiffy_attn_desc& d, const void* q, const AttnContext& ctx,
                                  const AttnContext& ctx2, const void* kb, const void* vb, void* out,
                                  int32_t* dev_status, void* ws, cudaStream_t stream) {
  const Plan pl = make_plan(d, ctx2.len);
  CUtensorMap tm_q, tm_kp, tm_vp, tm_kp2, tm_vp2, tm_kb, tm_vb;
  bool ok = make_map(&tm_q, q, d.n_q_heads, pl.NL, d.batch, pl.group, pl.TNL);
  ok = ok && make_map(&tm_kb, kb, d.n_kv_heads, pl.NL, d.batch, 1, BN);
  ok = ok && make_map(&tm_vb, vb, d.n_kv_heads, pl.NL, d.batch, 1, BN);
  if (ctx.len > 0) {
    ok = ok && make_map(&tm_kp, ctx.k, d.n_kv_heads, ctx.len, d.batch, 1, BN, ctx.batch_stride_rows);
    ok = ok && make_map(&tm_vp, ctx.v, d.n_kv_heads, ctx.len, d.batch, 1, BN, ctx.batch_stride_rows);
  } else {  // never dereferenced: the segment has no tile
    tm_kp = tm_kb;
    tm_vp = tm_vb;
  }
  if (ctx2.len > 0) {
    ok = ok && make_map(&tm_kp2, ctx2.k, d.n_kv_heads, ctx2.len, d.batch, 1, BN, ctx2.batch_stride_rows);
    ok = ok && make_map(&tm_vp2, ctx2.v, d.n_kv_heads, ctx2.len, d.batch, 1, BN, ctx2.batch_stride_rows);
  } else {
    tm_kp2 = tm_kb;
    tm_vp2 = tm_vb;
  }
  if (!ok) return SPIFFY_ECUDA;

  Params p;
  p.B = d.batch; p.N = d.n_nodes; p.L = d.block_len; p.P = ctx.len; p.P2 = ctx2.len;
  p.Hq = d.n_q_heads; p.Hkv = d.n_kv_heads; p.group = pl.group;
  p.TNL = pl.TNL; p.NL = pl.NL; p.MT = pl.MT; p.TP1 = pl.TP1; p.TP = pl.TP; p.splits = pl.splits;
  p.pair = pl.pair;
  const float scale = d.scale != 0.f ? d.scale : 1.0f / sqrtf((float)d.head_dim);
  p.scale_log2 = scale * kLog2e;
  p.out = static_cast<__nv_bfloat16*>(out);
  p.part_o = static_cast<float*>(ws);
  p.part_ml = p.part_o ? p.part_o + (size_t)pl.splits * pl.tiles * BM * HD : nullptr;
  p.status = dev_status;
  p.spin_limit = mbar_poll_limit();
  p.early_trigger = (d.kernel & SPIFFY_ATTN_EARLY_DEPENDENTS) ? 1 : 0;

  if (cudaFuncSetAttribute(graph_attention_tc_kernel<1>,
                           cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess ||
      cudaFuncSetAttribute(graph_attention_tc_kernel<2>,
                           cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess)
    return SPIFFY_ECUDA;
  const dim3 grid((pl.MT + pl.nq - 1) / pl.nq, d.batch * d.n_kv_heads, pl.splits);
  auto kern = pl.nq == 2 ? graph_attention_tc_kernel<2> : graph_attention_tc_kernel<1>;
  {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;  // pairs along grid.z, only when asked for
    attr[1].val.clusterDim.x = 1;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 2;
    cfg.attrs = attr;
    cfg.numAttrs = pl.pair ? 2 : 1;
    if (cudaLaunchKernelEx(&cfg, kern, tm_q, tm_kp, tm_vp, tm_kp2, tm_vp2, tm_kb, tm_vb, p) != cudaSuccess)
      return SPIFFY_ECUDA;
  }
  count_launch();
  if (pl.splits > 1 && !pl.pair) {
    const int64_t rows = (int64_t)d.batch * pl.NL * d.n_q_heads;
    if (launch_pdl(graph_attention_combine_kernel, dim3((unsigned)((rows + 7) / 8)), dim3(256),
                   (size_t)0, stream, p) != cudaSuccess)
      return SPIFFY_ECUDA;
    count_launch();
  }
  return SPIFFY_OK;
}

}  // namespace spiffy
