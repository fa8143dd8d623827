// spiffy_verify_step_host: one whole verification step (Sec. 4.3 packed
// attention for one layer, then Algorithm 1 steps 1-5) for a caller whose
// tensors sit in HOST memory.  The call stages the inputs on the device, runs the
// three kernels of the step and brings the verdict back; see include/spiffy.h.
//
// Staging.  Everything but the logits goes through the copy engine on a helper
// stream of the library; meanwhile, on the caller's stream, one kernel pulls the
// logits rows of still-masked positions (the only rows the decision reads)
// straight out of the pinned host buffer.  Both meet before the first kernel.
#include <mutex>

#include "common.cuh"

namespace spiffy {
namespace {

constexpr size_t kAlign = 256;
size_t up(size_t n) { return (n + kAlign - 1) / kAlign * kAlign; }

struct Layout {
  size_t q, kp, vp, kb, vb, logits, tokens, poff, pidx;       // inputs
  size_t qn, pn, bn;                                          // bytes of q, of a prefix tensor, of a block tensor
  size_t attn_out, conf, top_tok, bits, n_unmask;             // intermediate results
  size_t accepted, n_accepted, path, next_block;              // verdict
  size_t status;                                              // [attention | decision[B] | walk[B]]
  size_t attn_ws, decide_ws, total;
};

Layout layout_of(const spiffy_step_desc& s) {
  const spiffy_attn_desc& a = s.attn;
  const spiffy_decide_desc& d = s.decide;
  const size_t e = a.dtype == SPIFFY_BF16 ? 2 : 4, le = d.logits_dtype == SPIFFY_BF16 ? 2 : 4;
  const size_t B = a.batch, N = a.n_nodes, L = a.block_len;
  Layout l;
  l.qn = B * N * L * a.n_q_heads * a.head_dim * e;
  l.pn = B * (size_t)a.prefix_len * a.n_kv_heads * a.head_dim * e;
  l.bn = B * N * L * a.n_kv_heads * a.head_dim * e;
  size_t o = 0;
  auto take = [&](size_t bytes) { const size_t at = o; o += up(bytes); return at; };
  l.q = take(l.qn); l.kp = take(l.pn); l.vp = take(l.pn); l.kb = take(l.bn); l.vb = take(l.bn);
  l.logits = take(B * N * L * (size_t)d.row_stride * le);
  l.tokens = take(B * N * L * 4);
  l.poff = take(B * (N + 1) * 4);
  l.pidx = take(B * (size_t)s.parent_cap * 4);
  l.attn_out = take(l.qn);
  l.conf = take(B * N * L * 4); l.top_tok = take(B * N * L * 4);
  l.bits = take(B * N * 8); l.n_unmask = take(B * N * 4);
  l.accepted = take(B * 4); l.n_accepted = take(B * 4); l.path = take(B * N * 4); l.next_block = take(B * L * 4);
  l.status = take((1 + 2 * B) * 4);
  l.attn_ws = take(spiffy_graph_attention_workspace(&a));
  l.decide_ws = take(decide_workspace_bytes(d));
  l.total = o;
  return l;
}

spiffy_status check(const spiffy_step_desc* s) {
  if (!s) return SPIFFY_EINVAL;
  if (s->attn.batch != s->decide.batch || s->attn.n_nodes != s->decide.n_nodes ||
      s->attn.block_len != s->decide.block_len || s->parent_cap < 1)
    return SPIFFY_EINVAL;
  if (s->attn.block_len > 64) return SPIFFY_EUNSUPPORTED;
  // the component calls check the rest; their workspace queries return 0 for a bad descriptor
  if (spiffy_unmask_decide_workspace(&s->decide) == 0) return SPIFFY_EINVAL;
  return SPIFFY_OK;
}

// One helper stream and two events per device, created at the first call there.
struct Helper {
  cudaStream_t stream = nullptr;
  cudaEvent_t start = nullptr, done = nullptr;
};
std::mutex g_mutex;
Helper g_helper[64];

spiffy_status helper_for_current_device(Helper** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SPIFFY_ECUDA;
  std::lock_guard<std::mutex> lock(g_mutex);
  Helper& h = g_helper[dev];
  if (!h.stream) {
    if (cudaStreamCreateWithFlags(&h.stream, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&h.start, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h.done, cudaEventDisableTiming) != cudaSuccess)
      return SPIFFY_ECUDA;
  }
  *out = &h;
  return SPIFFY_OK;
}

bool device_can_read(const void* host_ptr) {
  cudaPointerAttributes at;
  if (cudaPointerGetAttributes(&at, host_ptr) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  return at.type == cudaMemoryTypeHost || at.type == cudaMemoryTypeManaged || at.type == cudaMemoryTypeDevice;
}

}  // namespace
}  // namespace spiffy

using namespace spiffy;

extern "C" {

size_t spiffy_verify_step_host_workspace(const spiffy_step_desc* desc) {
  if (check(desc) != SPIFFY_OK) return 0;
  return layout_of(*desc).total;
}

spiffy_status spiffy_verify_step_host(const spiffy_step_desc* desc, const void* q, const void* k_prefix,
                                      const void* v_prefix, const void* k_block, const void* v_block,
                                      const void* logits, const int32_t* block_tokens,
                                      const int32_t* parent_off, const int32_t* parent_idx,
                                      int32_t* accepted_node, int32_t* n_accepted, int32_t* path,
                                      int32_t* next_block, int32_t* status, void* device_workspace,
                                      size_t workspace_bytes, void* cuda_stream) {
  spiffy_status st = check(desc);
  if (st != SPIFFY_OK) return st;
  const spiffy_step_desc s = *desc;
  if (!q || !k_block || !v_block || !logits || !block_tokens || !parent_off || !parent_idx ||
      !accepted_node || !n_accepted || !path || !next_block || !status)
    return SPIFFY_EINVAL;
  if (s.attn.prefix_len > 0 && (!k_prefix || !v_prefix)) return SPIFFY_EINVAL;
  const Layout l = layout_of(s);
  if (!device_workspace || workspace_bytes < l.total ||
      (reinterpret_cast<uintptr_t>(device_workspace) & (kAlign - 1)) != 0)
    return SPIFFY_EWORKSPACE;
  Helper* h = nullptr;
  st = helper_for_current_device(&h);
  if (st != SPIFFY_OK) return st;

  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(device_workspace);
  const size_t B = s.attn.batch, N = s.attn.n_nodes, L = s.attn.block_len;
  const size_t le = s.decide.logits_dtype == SPIFFY_BF16 ? 2 : 4;
  const size_t rows = B * N * L;
  bool ok = true;
  auto h2d = [&](size_t at, const void* src, size_t bytes, cudaStream_t on) {
    if (bytes) ok = ok && cudaMemcpyAsync(ws + at, src, bytes, cudaMemcpyHostToDevice, on) == cudaSuccess;
  };
  // the staging buffers are free once earlier work on the caller's stream is done
  ok = ok && cudaEventRecord(h->start, stream) == cudaSuccess;
  ok = ok && cudaStreamWaitEvent(h->stream, h->start, 0) == cudaSuccess;
  h2d(l.tokens, block_tokens, rows * 4, stream);  // the row-staging kernel below reads them
  h2d(l.q, q, l.qn, h->stream);
  h2d(l.kp, k_prefix, l.pn, h->stream);
  h2d(l.vp, v_prefix, l.pn, h->stream);
  h2d(l.kb, k_block, l.bn, h->stream);
  h2d(l.vb, v_block, l.bn, h->stream);
  h2d(l.poff, parent_off, B * (N + 1) * 4, h->stream);
  h2d(l.pidx, parent_idx, B * (size_t)s.parent_cap * 4, h->stream);
  ok = ok && cudaEventRecord(h->done, h->stream) == cudaSuccess;
  if (!ok) return SPIFFY_ECUDA;
  // logits: only the rows of still-masked positions cross the bus
  const size_t row_bytes = (size_t)s.decide.row_stride * le;
  if (device_can_read(logits) && rows <= 65535) {
    st = launch_stage_masked_rows(logits, ws + l.logits, (int64_t)row_bytes,
                                  reinterpret_cast<const int32_t*>(ws + l.tokens), s.decide.mask_token_id,
                                  (int64_t)rows, stream);
    if (st != SPIFFY_OK) return st;
  } else {  // pageable memory: the runtime stages it; all rows go
    h2d(l.logits, logits, rows * row_bytes, stream);
  }
  ok = ok && cudaStreamWaitEvent(stream, h->done, 0) == cudaSuccess;
  if (!ok) return SPIFFY_ECUDA;

  // the status words are OR-ed into by the kernels: [attention | decision per sequence | walk per sequence]
  if (cudaMemsetAsync(ws + l.status, 0, (1 + 2 * B) * 4, stream) != cudaSuccess) return SPIFFY_ECUDA;
  int32_t* dev_status = reinterpret_cast<int32_t*>(ws + l.status);
  st = spiffy_graph_attention(&s.attn, ws + l.q, s.attn.prefix_len ? ws + l.kp : nullptr,
                              s.attn.prefix_len ? ws + l.vp : nullptr, ws + l.kb, ws + l.vb, ws + l.attn_out,
                              dev_status, ws + l.attn_ws, l.decide_ws - l.attn_ws, cuda_stream);
  if (st != SPIFFY_OK) return st;
  st = spiffy_decide_walk(&s.decide, ws + l.logits, reinterpret_cast<const int32_t*>(ws + l.tokens),
                          reinterpret_cast<const int32_t*>(ws + l.poff),
                          reinterpret_cast<const int32_t*>(ws + l.pidx), s.parent_cap,
                          reinterpret_cast<float*>(ws + l.conf), reinterpret_cast<int32_t*>(ws + l.top_tok),
                          reinterpret_cast<uint64_t*>(ws + l.bits), reinterpret_cast<int32_t*>(ws + l.n_unmask),
                          dev_status + 1, reinterpret_cast<int32_t*>(ws + l.accepted),
                          reinterpret_cast<int32_t*>(ws + l.n_accepted), reinterpret_cast<int32_t*>(ws + l.path),
                          reinterpret_cast<int32_t*>(ws + l.next_block), dev_status + 1 + B,
                          ws + l.decide_ws, l.total - l.decide_ws, cuda_stream);
  if (st != SPIFFY_OK) return st;
  // the verdict: four small arrays and the status words
  auto d2h = [&](void* dst, size_t at, size_t bytes) {
    ok = ok && cudaMemcpyAsync(dst, ws + at, bytes, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
  };
  d2h(accepted_node, l.accepted, B * 4);
  d2h(n_accepted, l.n_accepted, B * 4);
  d2h(path, l.path, B * N * 4);
  d2h(next_block, l.next_block, B * L * 4);
  d2h(status, l.status, (1 + 2 * B) * 4);
  ok = ok && cudaStreamSynchronize(stream) == cudaSuccess;
  return ok ? SPIFFY_OK : SPIFFY_ECUDA;
}

}  // extern "C"
