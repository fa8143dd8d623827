// Thin inline-PTX wrappers for the sm_100a features the attention kernel uses:
// mbarriers, TMA tile loads, tensor memory (TMEM) and tcgen05 MMA.  Encodings
// follow the PTX ISA's tcgen05 chapter (shared-memory matrix descriptor,
// instruction descriptor of .kind::f16, tensor-memory addressing).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace spiffy {
namespace sm100 {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}

// ---------------------------------------------------------------- mbarrier --
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count)
               : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}

// Bounded wait: gives up after `limit` polls (kSpinLimit unless the host lowered
// it) or as soon as another thread of the CTA has given up (*abort != 0); the
// first to give up raises *abort.  A limit of 0 gives up without polling.
constexpr uint32_t kSpinLimit = 1u << 20;
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort,
                                          uint32_t limit) {
  for (uint32_t i = 0; i < limit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 15u) == 15u && *abort) return false;
  }
  *abort = 1;
  return false;
}

// --------------------------------------------------------------------- TMA --
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* m) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(m)) : "memory");
}
// 4-D tile load global -> shared, into this CTA alone; completion is
// signalled on `bar` as transferred bytes.  c0 is the innermost coordinate and
// must be a multiple of 8 for 16-bit elements.
__device__ __forceinline__ void tma_load_4d(void* smem_dst, const CUtensorMap* m, uint64_t* bar,
                                            int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4, %5, %6}], [%2];"
      :
      : "r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(c0),
        "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
// Generic-proxy writes to shared memory become visible to the async proxy
// (TMA stores, tensor-core operand reads).
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// The two halves of the cluster barrier: a thread that has arrived may go on
// with work that does not depend on the other CTAs and wait later.  Every
// thread of every CTA of the cluster takes part in each phase.
__device__ __forceinline__ void cluster_arrive() {
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait() {
  asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}
// One arrival on an mbarrier of another CTA of the cluster (`addr` from
// map_to_cta); orders this thread's earlier writes, also those into that CTA's
// shared memory, before the arrival.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(addr) : "memory");
}
// 16 bytes into another CTA's shared memory without waiting for them: the
// destination CTA's mbarrier `bar` (same CTA as `addr`) counts the bytes as a
// transaction, so whoever waits on it with the byte count expected sees them.
__device__ __forceinline__ void st_async_f4(uint32_t addr, uint32_t bar, float a, float b, float c, float d) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%0], {%2, %3, %4, %5}, [%1];"
               ::"r"(addr), "r"(bar), "f"(a), "f"(b), "f"(c), "f"(d)
               : "memory");
}
__device__ __forceinline__ void st_async_f2(uint32_t addr, uint32_t bar, float a, float b) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.f32 [%0], {%2, %3}, [%1];"
               ::"r"(addr), "r"(bar), "f"(a), "f"(b)
               : "memory");
}
// try_wait that also acquires what threads of other CTAs released with
// mbar_arrive_remote.
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity, volatile int* abort,
                                                  uint32_t limit) {
  for (uint32_t i = 0; i < limit; ++i) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    if ((i & 15u) == 15u && *abort) return false;
  }
  *abort = 1;
  return false;
}
// The address, in the shared window of the cluster, of `smem_addr` in CTA `rank`.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
// -------------------------------------------------------------------- TMEM --
// Whole-warp calls (.sync.aligned).  The allocated base address (lane 0,
// first column) is written to *smem_result.
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_result, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                   smem_u32(smem_result)),
               "r"(ncols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after_sync() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tmem_wait_st() {
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
// A tensor-memory address: lane in bits 31..16, column in bits 15..0.
__device__ __forceinline__ uint32_t tmem_addr(uint32_t base, uint32_t lane, uint32_t col) {
  return base + (lane << 16) + col;
}

// Row `lane` of the warp's TMEM quadrant, 32 consecutive 32-bit columns from
// `taddr`, into r[0..31]; returns once the data has arrived.
__device__ __forceinline__ void tmem_ld_x32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
      "tcgen05.wait::ld.sync.aligned;\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}

// Row `lane` of the warp's TMEM quadrant, 64 consecutive 32-bit columns from
// `taddr`, into r[0..63]; returns once the data has arrived.
__device__ __forceinline__ void tmem_ld_x64(uint32_t taddr, uint32_t (&r)[64]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x64.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32,%33,%34,%35,%36,%37,%38,%39,%40,%41,%42,%43,%44,%45,%46,%47,%48,%49,%50,%51,%52,%53,%54,%55,%56,%57,%58,%59,%60,%61,%62,%63}, [%64];\n"
      "tcgen05.wait::ld.sync.aligned;\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
      : "r"(taddr)
      : "memory");
}

// Row `lane` of the warp's TMEM quadrant, 128 consecutive 32-bit columns from
// `taddr`, into r[0..127]; returns once the data has arrived.
__device__ __forceinline__ void tmem_ld_x128(uint32_t taddr, uint32_t (&r)[128]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x128.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32,%33,%34,%35,%36,%37,%38,%39,%40,%41,%42,%43,%44,%45,%46,%47,%48,%49,%50,%51,%52,%53,%54,%55,%56,%57,%58,%59,%60,%61,%62,%63,%64,%65,%66,%67,%68,%69,%70,%71,%72,%73,%74,%75,%76,%77,%78,%79,%80,%81,%82,%83,%84,%85,%86,%87,%88,%89,%90,%91,%92,%93,%94,%95,%96,%97,%98,%99,%100,%101,%102,%103,%104,%105,%106,%107,%108,%109,%110,%111,%112,%113,%114,%115,%116,%117,%118,%119,%120,%121,%122,%123,%124,%125,%126,%127}, [%128];\n"
      "tcgen05.wait::ld.sync.aligned;\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63]), "=r"(r[64]), "=r"(r[65]), "=r"(r[66]), "=r"(r[67]), "=r"(r[68]), "=r"(r[69]), "=r"(r[70]), "=r"(r[71]), "=r"(r[72]), "=r"(r[73]), "=r"(r[74]), "=r"(r[75]), "=r"(r[76]), "=r"(r[77]), "=r"(r[78]), "=r"(r[79]), "=r"(r[80]), "=r"(r[81]), "=r"(r[82]), "=r"(r[83]), "=r"(r[84]), "=r"(r[85]), "=r"(r[86]), "=r"(r[87]), "=r"(r[88]), "=r"(r[89]), "=r"(r[90]), "=r"(r[91]), "=r"(r[92]), "=r"(r[93]), "=r"(r[94]), "=r"(r[95]), "=r"(r[96]), "=r"(r[97]), "=r"(r[98]), "=r"(r[99]), "=r"(r[100]), "=r"(r[101]), "=r"(r[102]), "=r"(r[103]), "=r"(r[104]), "=r"(r[105]), "=r"(r[106]), "=r"(r[107]), "=r"(r[108]), "=r"(r[109]), "=r"(r[110]), "=r"(r[111]), "=r"(r[112]), "=r"(r[113]), "=r"(r[114]), "=r"(r[115]), "=r"(r[116]), "=r"(r[117]), "=r"(r[118]), "=r"(r[119]), "=r"(r[120]), "=r"(r[121]), "=r"(r[122]), "=r"(r[123]), "=r"(r[124]), "=r"(r[125]), "=r"(r[126]), "=r"(r[127])
      : "r"(taddr)
      : "memory");
}

// r[0..31] into row `lane` of the warp's TMEM quadrant, 32 consecutive columns
// from `taddr` (issue only; follow with tmem_wait_st()).
__device__ __forceinline__ void tmem_st_x32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};\n"
      :
      : "r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}

// r[0..63] into row `lane` of the warp's TMEM quadrant, 64 consecutive columns
// from `taddr` (issue only; follow with tmem_wait_st()).
__device__ __forceinline__ void tmem_st_x64(uint32_t taddr, const uint32_t (&r)[64]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x64.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32,%33,%34,%35,%36,%37,%38,%39,%40,%41,%42,%43,%44,%45,%46,%47,%48,%49,%50,%51,%52,%53,%54,%55,%56,%57,%58,%59,%60,%61,%62,%63,%64};\n"
      :
      : "r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]), "r"(r[32]), "r"(r[33]), "r"(r[34]), "r"(r[35]), "r"(r[36]), "r"(r[37]), "r"(r[38]), "r"(r[39]), "r"(r[40]), "r"(r[41]), "r"(r[42]), "r"(r[43]), "r"(r[44]), "r"(r[45]), "r"(r[46]), "r"(r[47]), "r"(r[48]), "r"(r[49]), "r"(r[50]), "r"(r[51]), "r"(r[52]), "r"(r[53]), "r"(r[54]), "r"(r[55]), "r"(r[56]), "r"(r[57]), "r"(r[58]), "r"(r[59]), "r"(r[60]), "r"(r[61]), "r"(r[62]), "r"(r[63])
      : "memory");
}

// Two columns of row `lane` of the warp's TMEM quadrant.
__device__ __forceinline__ void tmem_ld_x2(uint32_t taddr, uint32_t& r0, uint32_t& r1) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x2.b32 {%0,%1}, [%2];\n"
      "tcgen05.wait::ld.sync.aligned;\n"
      : "=r"(r0), "=r"(r1)
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st_x2(uint32_t taddr, uint32_t r0, uint32_t r1) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x2.b32 [%0], {%1,%2};\n"
               :
               : "r"(taddr), "r"(r0), "r"(r1)
               : "memory");
}

// --------------------------------------------------------------------- MMA --
// Shared-memory matrix descriptor of a 128-byte-swizzled operand tile whose
// 8-row (1024-byte) swizzle atoms are `sbo_bytes` apart; `lbo_bytes` is the
// distance between 64-element blocks along M/N of an MN-major operand (unused
// for K-major).  The tile base must be 1024-byte aligned; `addr` may point
// 32, 64 or 96 bytes into a row to step along K inside the swizzle span.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr, uint32_t lbo_bytes,
                                                    uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);          // bits  0..13 start address
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;  // bits 16..29 leading byte offset
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;  // bits 32..45 stride byte offset
  d |= (uint64_t)1 << 46;                           // bits 46..48 fixed 0b001
  d |= (uint64_t)2 << 61;                           // bits 61..63 swizzle mode: 128 bytes
  return d;
}
// Instruction descriptor of tcgen05.mma.kind::f16 with bf16 operands and fp32
// accumulation; *_mn_major = operand stored with M/N (not K) contiguous.
__host__ __device__ constexpr uint32_t idesc_bf16_f32(int m, int n, bool a_mn_major,
                                                      bool b_mn_major) {
  return (1u << 4)                       // D format: fp32
         | (1u << 7)                     // A format: bf16
         | (1u << 10)                    // B format: bf16
         | ((a_mn_major ? 1u : 0u) << 15)
         | ((b_mn_major ? 1u : 0u) << 16)
         | ((uint32_t)(n >> 3) << 17)
         | ((uint32_t)(m >> 4) << 24);
}
// D[tmem] (+)= A[smem] * B[smem]; issued by one thread.
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                        uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n"
      :
      : "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// ------------------------------------------------- lean issue of MMA groups --
// One thread issues every MMA of a CTA; what it spends per instruction on
// building descriptors bounds the tensor pipe's rate (a 128 x 128 x 16 product
// lasts 64 cycles).  The groups below take the descriptors split into their low
// word (address and leading offset: advanced by a constant per K step) and
// their high word (stride offset, fixed bits, swizzle: the same for all).
__device__ __forceinline__ uint32_t desc_lo_sw128(uint32_t addr, uint32_t lbo_bytes) {
  return ((addr & 0x3FFFFu) >> 4) | ((lbo_bytes >> 4) << 16);
}
__host__ __device__ constexpr uint32_t desc_hi_sw128(uint32_t sbo_bytes) {
  return ((sbo_bytes >> 4) & 0x3FFFu) | (1u << 14) | (2u << 29);
}
// D[tmem] (+)= A B^T over K = 128: A and B K-major tiles of 128-byte-swizzled
// rows, stored as two 64-element halves 16 KB apart (eight K steps of 16).
__device__ __forceinline__ void umma_ss_k128(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi,
                                             uint32_t idesc, uint32_t accumulate_first) {
  asm volatile(
      "{\n"
      ".reg .pred p0, p1;\n"
      ".reg .b32 al, bl;\n"
      ".reg .b64 da, db;\n"
      "setp.ne.b32 p0, %5, 0;\n"
      "setp.eq.b32 p1, %5, %5;\n"
      "add.u32 al, %1, 0;\n"
      "add.u32 bl, %2, 0;\n"
      "mov.b64 da, {al, %3};\n"
      "mov.b64 db, {bl, %3};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p0;\n"
      "add.u32 al, %1, 2;\n"
      "add.u32 bl, %2, 2;\n"
      "mov.b64 da, {al, %3};\n"
      "mov.b64 db, {bl, %3};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p1;\n"
      "add.u32 al, %1, 4;\n"
      "add.u32 bl, %2, 4;\n"
      "mov.b64 da, {al, %3};\n"
      "mov.b64 db, {bl, %3};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p1;\n"
      "add.u32 al, %1, 6;\n"
      "add.u32 bl, %2, 6;\n"
      "mov.b64 da, {al, %3};\n"
      "mov.b64 db, {bl, %3};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p1;\n"
      "add.u32 al, %1, 1024;\n"
      "add.u32 bl, %2, 1024;\n"
      "mov.b64 da, {al, %3};\n"
      "mov.b64 db, {bl, %3};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p1;\n"
      "add.u32 al, %1, 1026;\n"
      "add.u32 bl, %2, 1026;\n"
      "mov.b64 da, {al, %3};\n"
      "mov.b64 db, {bl, %3};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p1;\n"
      "add.u32 al, %1, 1028;\n"
      "add.u32 bl, %2, 1028;\n"
      "mov.b64 da, {al, %3};\n"
      "mov.b64 db, {bl, %3};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p1;\n"
      "add.u32 al, %1, 1030;\n"
      "add.u32 bl, %2, 1030;\n"
      "mov.b64 da, {al, %3};\n"
      "mov.b64 db, {bl, %3};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p1;\n"
      "}\n"
      :
      : "r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate_first)
      : "memory");
}
// D[tmem] (+)= A[tmem] B over `steps` K steps of 16: A = bf16 pairs in tensor
// memory (8 columns per step), B an MN-major tile whose rows of 16 keys are
// 2048 bytes apart.
__device__ __forceinline__ void umma_ts_k64(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t hi,
                                            uint32_t idesc, uint32_t accumulate_first) {
  asm volatile(
      "{\n"
      ".reg .pred p0, p1;\n"
      ".reg .b32 at, bl;\n"
      ".reg .b64 db;\n"
      "setp.ne.b32 p0, %5, 0;\n"
      "setp.eq.b32 p1, %5, %5;\n"
      "add.u32 at, %1, 0;\n"
      "add.u32 bl, %2, 0;\n"
      "mov.b64 db, {bl, %3};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, p0;\n"
      "add.u32 at, %1, 8;\n"
      "add.u32 bl, %2, 128;\n"
      "mov.b64 db, {bl, %3};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, p1;\n"
      "add.u32 at, %1, 16;\n"
      "add.u32 bl, %2, 256;\n"
      "mov.b64 db, {bl, %3};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, p1;\n"
      "add.u32 at, %1, 24;\n"
      "add.u32 bl, %2, 384;\n"
      "mov.b64 db, {bl, %3};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, p1;\n"
      "}\n"
      :
      : "r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate_first)
      : "memory");
}
__device__ __forceinline__ void umma_ts_k128(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t hi,
                                             uint32_t idesc, uint32_t accumulate_first) {
  asm volatile(
      "{\n"
      ".reg .pred p0, p1;\n"
      ".reg .b32 at, bl;\n"
      ".reg .b64 db;\n"
      "setp.ne.b32 p0, %5, 0;\n"
      "setp.eq.b32 p1, %5, %5;\n"
      "add.u32 at, %1, 0;\n"
      "add.u32 bl, %2, 0;\n"
      "mov.b64 db, {bl, %3};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, p0;\n"
      "add.u32 at, %1, 8;\n"
      "add.u32 bl, %2, 128;\n"
      "mov.b64 db, {bl, %3};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, p1;\n"
      "add.u32 at, %1, 16;\n"
      "add.u32 bl, %2, 256;\n"
      "mov.b64 db, {bl, %3};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, p1;\n"
      "add.u32 at, %1, 24;\n"
      "add.u32 bl, %2, 384;\n"
      "mov.b64 db, {bl, %3};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, p1;\n"
      "add.u32 at, %1, 32;\n"
      "add.u32 bl, %2, 512;\n"
      "mov.b64 db, {bl, %3};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, p1;\n"
      "add.u32 at, %1, 40;\n"
      "add.u32 bl, %2, 640;\n"
      "mov.b64 db, {bl, %3};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, p1;\n"
      "add.u32 at, %1, 48;\n"
      "add.u32 bl, %2, 768;\n"
      "mov.b64 db, {bl, %3};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, p1;\n"
      "add.u32 at, %1, 56;\n"
      "add.u32 bl, %2, 896;\n"
      "mov.b64 db, {bl, %3};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, p1;\n"
      "}\n"
      :
      : "r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate_first)
      : "memory");
}

// The mbarrier receives one arrival when every MMA issued so far by this
// thread has completed (implies tcgen05.fence::before_thread_sync).
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                   smem_u32(bar))
               : "memory");
}

}  // namespace sm100
}  // namespace spiffy
