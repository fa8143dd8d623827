// C ABI of libspiffy: argument validation and dispatch.  See include/spiffy.h
// for the contract of every entry point.
#include <atomic>

#include "common.cuh"

namespace spiffy {

static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

// defaults: 2^20 mbarrier polls; 2^21 polls of about 100 ns each on a global word
static std::atomic<uint32_t> g_mbar_polls{1u << 20};
static std::atomic<uint32_t> g_flag_polls{1u << 21};
static std::atomic<int32_t> g_lazy_extra{0};
uint32_t mbar_poll_limit() { return g_mbar_polls.load(std::memory_order_relaxed); }
uint32_t flag_poll_limit() { return g_flag_polls.load(std::memory_order_relaxed); }
int32_t lazy_extra_arrivals() { return g_lazy_extra.load(std::memory_order_relaxed); }

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

spiffy_status check_attn_desc(const spiffy_attn_desc* d) {
  if (!d) return SPIFFY_EINVAL;
  if (d->batch < 1 || d->n_nodes < 1 || d->block_len < 1 || d->prefix_len < 0 ||
      d->n_q_heads < 1 || d->n_kv_heads < 1)
    return SPIFFY_EINVAL;
  if (d->n_q_heads % d->n_kv_heads != 0) return SPIFFY_EINVAL;
  if (d->dtype != SPIFFY_F32 && d->dtype != SPIFFY_BF16) return SPIFFY_EINVAL;
  if (!(d->scale >= 0.f) || !(d->scale < INFINITY)) return SPIFFY_EINVAL;
  if (d->kernel & ~(0xff | SPIFFY_ATTN_EARLY_DEPENDENTS)) return SPIFFY_EINVAL;
  if ((d->kernel & 0xff) > SPIFFY_ATTN_TCGEN05) return SPIFFY_EINVAL;
  if (d->block_len > 1024) return SPIFFY_EUNSUPPORTED;
  if (d->head_dim != 64 && d->head_dim != 128) return SPIFFY_EUNSUPPORTED;
  if (d->n_nodes > 65535 || d->batch > 65535) return SPIFFY_EUNSUPPORTED;
  return SPIFFY_OK;
}

bool use_tc(const spiffy_attn_desc& d) {
  if ((d.kernel & 0xff) == SPIFFY_ATTN_SIMT) return false;
  return attention_tc_supported(d);
}

spiffy_status check_decide_desc(const spiffy_decide_desc* d, bool need_vocab) {
  if (!d) return SPIFFY_EINVAL;
  if (d->batch < 1 || d->n_nodes < 1 || d->block_len < 1) return SPIFFY_EINVAL;
  if (d->block_len > 64) return SPIFFY_EUNSUPPORTED;
  if ((int64_t)d->batch * d->n_nodes > 65535) return SPIFFY_EUNSUPPORTED;
  if ((int64_t)d->batch * d->n_nodes * d->block_len > 65535) return SPIFFY_EUNSUPPORTED;
  if (!need_vocab) return SPIFFY_OK;
  if (d->vocab < 1) return SPIFFY_EINVAL;
  if (d->logits_dtype != SPIFFY_F32 && d->logits_dtype != SPIFFY_BF16) return SPIFFY_EINVAL;
  if (d->row_stride < d->vocab) return SPIFFY_EINVAL;
  const int64_t esize = d->logits_dtype == SPIFFY_BF16 ? 2 : 4;
  if ((d->row_stride * esize) % 16 != 0) return SPIFFY_EINVAL;
  if (d->rule != SPIFFY_RULE_TOPS && d->rule != SPIFFY_RULE_THRESHOLD) return SPIFFY_EINVAL;
  if (d->rule == SPIFFY_RULE_TOPS && d->top_s < 1) return SPIFFY_EINVAL;
  if (d->rule == SPIFFY_RULE_THRESHOLD && !(d->threshold == d->threshold)) return SPIFFY_EINVAL;
  return SPIFFY_OK;
}

spiffy_status check_draft_desc(const spiffy_draft_desc* d) {
  if (!d) return SPIFFY_EINVAL;
  if (d->batch < 1 || d->block_len < 1 || d->vocab < 1 || d->n_formulas < 1) return SPIFFY_EINVAL;
  if (d->logits_dtype != SPIFFY_F32 && d->logits_dtype != SPIFFY_BF16) return SPIFFY_EINVAL;
  if (d->row_stride < d->vocab) return SPIFFY_EINVAL;
  if ((d->row_stride * (d->logits_dtype == SPIFFY_BF16 ? 2 : 4)) % 16 != 0) return SPIFFY_EINVAL;
  if (d->top_k < 1 || d->budget < 1 || d->budget > d->n_formulas || d->parent_cap < 1) return SPIFFY_EINVAL;
  if (d->block_len > 64 || d->top_k > 4 || d->n_formulas > 1024) return SPIFFY_EUNSUPPORTED;
  if ((int64_t)d->batch * d->block_len > 65535) return SPIFFY_EUNSUPPORTED;
  return SPIFFY_OK;
}

}  // namespace
}  // namespace spiffy

using namespace spiffy;

extern "C" {

size_t spiffy_graph_attention_workspace(const spiffy_attn_desc* desc) {
  if (check_attn_desc(desc) != SPIFFY_OK) return 0;
  return use_tc(*desc) ? attention_tc_workspace_bytes(*desc, 0) : 0;
}

spiffy_status spiffy_graph_attention(const spiffy_attn_desc* desc, const void* q,
                                     const void* k_prefix, const void* v_prefix,
                                     const void* k_block, const void* v_block,
                                     void* out, int32_t* dev_status,
                                     void* workspace, size_t workspace_bytes,
                                     void* cuda_stream) {
  const spiffy_status st = check_attn_desc(desc);
  if (st != SPIFFY_OK) return st;
  const spiffy_attn_desc d = *desc;
  if (!q || !k_block || !v_block || !out) return SPIFFY_EINVAL;
  if (d.prefix_len > 0 && (!k_prefix || !v_prefix)) return SPIFFY_EINVAL;
  if (!aligned16(q) || !aligned16(k_block) || !aligned16(v_block) || !aligned16(out) ||
      !aligned16(k_prefix) || !aligned16(v_prefix))
    return SPIFFY_EINVAL;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (use_tc(d)) {
    const size_t need = attention_tc_workspace_bytes(d, 0);
    if (need > 0 && (!workspace || workspace_bytes < need || !aligned16(workspace)))
      return SPIFFY_EWORKSPACE;
    const AttnContext ctx = {k_prefix, v_prefix, d.prefix_len, 0};
    const AttnContext none = {nullptr, nullptr, 0, 0};
    return launch_attention_tc(d, q, ctx, none, k_block, v_block, out, dev_status, workspace, stream);
  }
  if ((d.kernel & 0xff) == SPIFFY_ATTN_TCGEN05) return SPIFFY_EUNSUPPORTED;
  if (d.block_len > 64) return SPIFFY_EUNSUPPORTED;  // the CUDA-core kernel keeps a block's rows in registers
  return launch_attention_simt(d, q, k_prefix, v_prefix, k_block, v_block, out, stream);
}

namespace {
// The second launch of the full-sequence call: the suffix rows as one node whose block is the suffix.
spiffy_attn_desc suffix_desc(const spiffy_attn_desc& d, int32_t suffix_len) {
  spiffy_attn_desc s = d;
  s.n_nodes = 1;
  s.block_len = suffix_len;
  return s;
}
spiffy_status check_full_sequence(const spiffy_attn_desc* desc, int32_t suffix_len) {
  const spiffy_status st = check_attn_desc(desc);
  if (st != SPIFFY_OK) return st;
  if (suffix_len < 0) return SPIFFY_EINVAL;
  if (suffix_len > 1024) return SPIFFY_EUNSUPPORTED;
  if (!use_tc(*desc)) return SPIFFY_EUNSUPPORTED;  // bf16, head dimension 128 only
  return SPIFFY_OK;
}
}  // namespace

size_t spiffy_full_sequence_attention_workspace(const spiffy_attn_desc* desc, int32_t suffix_len) {
  if (check_full_sequence(desc, suffix_len) != SPIFFY_OK) return 0;
  const size_t nodes = attention_tc_workspace_bytes(*desc, suffix_len);
  const size_t suffix = suffix_len > 0 ? attention_tc_workspace_bytes(suffix_desc(*desc, suffix_len), desc->block_len) : 0;
  return nodes > suffix ? nodes : suffix;
}

spiffy_status spiffy_full_sequence_attention(const spiffy_attn_desc* desc, int32_t suffix_len,
                                             const void* q_nodes, const void* q_suffix,
                                             const void* k_prefix, const void* v_prefix,
                                             const void* k_suffix, const void* v_suffix,
                                             const void* k_block, const void* v_block, void* out_nodes,
                                             void* out_suffix, int32_t* dev_status, void* workspace,
                                             size_t workspace_bytes, void* cuda_stream) {
  const spiffy_status st = check_full_sequence(desc, suffix_len);
  if (st != SPIFFY_OK) return st;
  const spiffy_attn_desc d = *desc;
  if (!q_nodes || !k_block || !v_block || !out_nodes) return SPIFFY_EINVAL;
  if (d.prefix_len > 0 && (!k_prefix || !v_prefix)) return SPIFFY_EINVAL;
  if (suffix_len > 0 && (!q_suffix || !k_suffix || !v_suffix || !out_suffix)) return SPIFFY_EINVAL;
  const void* all[] = {q_nodes, q_suffix, k_prefix, v_prefix, k_suffix, v_suffix, k_block, v_block, out_nodes, out_suffix};
  for (const void* ptr : all)
    if (!aligned16(ptr)) return SPIFFY_EINVAL;
  const size_t need = spiffy_full_sequence_attention_workspace(desc, suffix_len);
  if (need > 0 && (!workspace || workspace_bytes < need || !aligned16(workspace))) return SPIFFY_EWORKSPACE;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const AttnContext prefix = {k_prefix, v_prefix, d.prefix_len, 0};
  // nodes: context = [prefix ; suffix]; every node's own block as always
  const AttnContext suffix = {k_suffix, v_suffix, suffix_len, 0};
  spiffy_status rc = launch_attention_tc(d, q_nodes, prefix, suffix, k_block, v_block, out_nodes, dev_status,
                                         workspace, stream);
  if (rc != SPIFFY_OK || suffix_len == 0) return rc;
  // suffix rows: one node whose block is the suffix; context = [prefix ; the true block], the
  // latter being node 0 of every sequence's blocks (sequences N * L rows apart)
  const AttnContext true_block = {k_block, v_block, d.block_len, (int64_t)d.n_nodes * d.block_len};
  return launch_attention_tc(suffix_desc(d, suffix_len), q_suffix, prefix, true_block, k_suffix, v_suffix,
                             out_suffix, dev_status, workspace, stream);
}

size_t spiffy_unmask_decide_workspace(const spiffy_decide_desc* desc) {
  if (check_decide_desc(desc, true) != SPIFFY_OK) return 0;
  return decide_workspace_bytes(*desc);
}

spiffy_status spiffy_unmask_decide(const spiffy_decide_desc* desc,
                                   const void* logits,
                                   const int32_t* block_tokens, float* conf,
                                   int32_t* top_tok, uint64_t* unmask_bits,
                                   int32_t* n_unmask, int32_t* dev_status,
                                   void* workspace, size_t workspace_bytes,
                                   void* cuda_stream) {
  const spiffy_status st = check_decide_desc(desc, true);
  if (st != SPIFFY_OK) return st;
  if (!logits || !block_tokens || !conf || !top_tok || !unmask_bits || !n_unmask)
    return SPIFFY_EINVAL;
  if (!aligned16(logits)) return SPIFFY_EINVAL;
  const size_t need = decide_workspace_bytes(*desc);
  if (!workspace || workspace_bytes < need || !aligned16(workspace)) return SPIFFY_EWORKSPACE;
  return launch_decide(*desc, logits, block_tokens, conf, top_tok, unmask_bits,
                       n_unmask, dev_status, workspace,
                       static_cast<cudaStream_t>(cuda_stream));
}

spiffy_status spiffy_accept_walk(const spiffy_decide_desc* desc,
                                 const int32_t* block_tokens,
                                 const int32_t* parent_off,
                                 const int32_t* parent_idx, int32_t parent_cap,
                                 const int32_t* top_tok,
                                 const uint64_t* unmask_bits,
                                 int32_t* accepted_node, int32_t* n_accepted,
                                 int32_t* path, int32_t* next_block,
                                 int32_t* dev_status, void* cuda_stream) {
  const spiffy_status st = check_decide_desc(desc, false);
  if (st != SPIFFY_OK) return st;
  if (!block_tokens || !parent_off || !parent_idx || !top_tok || !unmask_bits ||
      !accepted_node || !n_accepted || !path || !next_block)
    return SPIFFY_EINVAL;
  if (parent_cap < 0) return SPIFFY_EINVAL;
  return launch_walk(*desc, block_tokens, parent_off, parent_idx, parent_cap,
                     top_tok, unmask_bits, accepted_node, n_accepted, path,
                     next_block, dev_status, static_cast<cudaStream_t>(cuda_stream));
}

spiffy_status spiffy_decide_walk(const spiffy_decide_desc* desc, const void* logits,
                                 const int32_t* block_tokens, const int32_t* parent_off,
                                 const int32_t* parent_idx, int32_t parent_cap, float* conf,
                                 int32_t* top_tok, uint64_t* unmask_bits, int32_t* n_unmask,
                                 int32_t* decide_status, int32_t* accepted_node,
                                 int32_t* n_accepted, int32_t* path, int32_t* next_block,
                                 int32_t* walk_status, void* workspace, size_t workspace_bytes,
                                 void* cuda_stream) {
  const spiffy_status st = check_decide_desc(desc, true);
  if (st != SPIFFY_OK) return st;
  if (!logits || !block_tokens || !conf || !top_tok || !unmask_bits || !n_unmask || !parent_off ||
      !parent_idx || !accepted_node || !n_accepted || !path || !next_block)
    return SPIFFY_EINVAL;
  if (!aligned16(logits) || parent_cap < 0) return SPIFFY_EINVAL;
  const size_t need = decide_workspace_bytes(*desc);
  if (!workspace || workspace_bytes < need || !aligned16(workspace)) return SPIFFY_EWORKSPACE;
  return launch_decide_walk(*desc, logits, block_tokens, conf, top_tok, unmask_bits, n_unmask,
                            decide_status, parent_off, parent_idx, parent_cap, accepted_node,
                            n_accepted, path, next_block, walk_status, workspace,
                            static_cast<cudaStream_t>(cuda_stream));
}

size_t spiffy_decide_walk_lazy_workspace(const spiffy_decide_desc* desc) {
  if (check_decide_desc(desc, true) != SPIFFY_OK) return 0;
  return decide_lazy_workspace_bytes(*desc);
}

spiffy_status spiffy_decide_walk_lazy(const spiffy_decide_desc* desc, const void* logits,
                                      const int32_t* block_tokens, const int32_t* parent_off,
                                      const int32_t* parent_idx, int32_t parent_cap, float* conf,
                                      int32_t* top_tok, uint64_t* unmask_bits, int32_t* n_unmask,
                                      int32_t* decide_status, int32_t* accepted_node,
                                      int32_t* n_accepted, int32_t* path, int32_t* next_block,
                                      int32_t* walk_status, void* workspace,
                                      size_t workspace_bytes, void* cuda_stream) {
  const spiffy_status st = check_decide_desc(desc, true);
  if (st != SPIFFY_OK) return st;
  if (!logits || !block_tokens || !conf || !top_tok || !unmask_bits || !n_unmask || !parent_off ||
      !parent_idx || !accepted_node || !n_accepted || !path || !next_block)
    return SPIFFY_EINVAL;
  if (!aligned16(logits) || parent_cap < 0) return SPIFFY_EINVAL;
  const size_t need = decide_lazy_workspace_bytes(*desc);
  if (!workspace || workspace_bytes < need || !aligned16(workspace)) return SPIFFY_EWORKSPACE;
  return launch_decide_walk_lazy(*desc, logits, block_tokens, conf, top_tok, unmask_bits, n_unmask,
                                 decide_status, parent_off, parent_idx, parent_cap, accepted_node,
                                 n_accepted, path, next_block, walk_status, workspace,
                                 static_cast<cudaStream_t>(cuda_stream));
}

spiffy_status spiffy_stage_masked_rows(const void* src_rows, void* dst_rows, int64_t row_bytes,
                                       const int32_t* tokens, int32_t mask_token_id,
                                       int64_t n_rows, void* cuda_stream) {
  if (!src_rows || !dst_rows || !tokens) return SPIFFY_EINVAL;
  if (row_bytes < 16 || row_bytes % 16 != 0 || n_rows < 1) return SPIFFY_EINVAL;
  if (!aligned16(src_rows) || !aligned16(dst_rows)) return SPIFFY_EINVAL;
  if (n_rows > 65535) return SPIFFY_EUNSUPPORTED;
  return launch_stage_masked_rows(src_rows, dst_rows, row_bytes, tokens, mask_token_id, n_rows,
                                  static_cast<cudaStream_t>(cuda_stream));
}

size_t spiffy_unmask_decide_sampled_workspace(const spiffy_decide_desc* desc) {
  if (check_decide_desc(desc, true) != SPIFFY_OK) return 0;
  return decide_sampled_workspace_bytes(*desc);
}

int64_t spiffy_sampled_slice_width(const spiffy_decide_desc* desc) {
  if (check_decide_desc(desc, true) != SPIFFY_OK) return 0;
  int64_t chunk = 0;
  decide_splits(*desc, &chunk);
  return chunk;
}

spiffy_status spiffy_unmask_decide_sampled(const spiffy_decide_desc* desc,
                                           const spiffy_sample_desc* sample, const void* logits,
                                           const int32_t* block_tokens, float* conf,
                                           int32_t* top_tok, uint64_t* unmask_bits,
                                           int32_t* n_unmask, int32_t* dev_status,
                                           void* workspace, size_t workspace_bytes,
                                           void* cuda_stream) {
  const spiffy_status st = check_decide_desc(desc, true);
  if (st != SPIFFY_OK) return st;
  if (!sample || !(sample->temperature > 0.f) || !(sample->temperature < INFINITY)) return SPIFFY_EINVAL;
  if (!logits || !block_tokens || !conf || !top_tok || !unmask_bits || !n_unmask)
    return SPIFFY_EINVAL;
  if (!aligned16(logits)) return SPIFFY_EINVAL;
  const size_t need = decide_sampled_workspace_bytes(*desc);
  if (!workspace || workspace_bytes < need || !aligned16(workspace)) return SPIFFY_EWORKSPACE;
  return launch_decide_sampled(*desc, sample->temperature, sample->seed, logits, block_tokens, conf,
                               top_tok, unmask_bits, n_unmask, dev_status, workspace,
                               static_cast<cudaStream_t>(cuda_stream));
}

namespace {
// The descriptor of the fused call names no logits: fill those fields in so that the
// common checks apply.
spiffy_status lmhead_desc(const spiffy_decide_desc* desc, int32_t hidden, spiffy_decide_desc* out) {
  if (!desc) return SPIFFY_EINVAL;
  *out = *desc;
  out->logits_dtype = SPIFFY_BF16;
  out->row_stride = ((int64_t)desc->vocab + 7) / 8 * 8;
  const spiffy_status st = check_decide_desc(out, true);
  if (st != SPIFFY_OK) return st;
  if (hidden < 128 || hidden % 128 != 0) return SPIFFY_EUNSUPPORTED;
  return SPIFFY_OK;
}
}  // namespace

size_t spiffy_lmhead_decide_workspace(const spiffy_decide_desc* desc, int32_t hidden) {
  spiffy_decide_desc d;
  if (lmhead_desc(desc, hidden, &d) != SPIFFY_OK) return 0;
  const int grid = lmhead_grid(d);
  return grid > 0 ? lmhead_workspace_bytes(d, grid) : 0;
}

spiffy_status spiffy_lmhead_decide(const spiffy_decide_desc* desc, int32_t hidden,
                                   const void* hidden_states, const void* weight,
                                   const int32_t* block_tokens, float* conf, int32_t* top_tok,
                                   uint64_t* unmask_bits, int32_t* n_unmask, int32_t* dev_status,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream) {
  spiffy_decide_desc d;
  const spiffy_status st = lmhead_desc(desc, hidden, &d);
  if (st != SPIFFY_OK) return st;
  if (!hidden_states || !weight || !block_tokens || !conf || !top_tok || !unmask_bits || !n_unmask)
    return SPIFFY_EINVAL;
  if (!aligned16(hidden_states) || !aligned16(weight)) return SPIFFY_EINVAL;
  const int grid = lmhead_grid(d);
  if (grid <= 0) return SPIFFY_ECUDA;
  const size_t need = lmhead_workspace_bytes(d, grid);
  if (!workspace || workspace_bytes < need || !aligned16(workspace)) return SPIFFY_EWORKSPACE;
  return launch_lmhead_decide(d, hidden, hidden_states, weight, block_tokens, conf, top_tok,
                              unmask_bits, n_unmask, dev_status, workspace,
                              static_cast<cudaStream_t>(cuda_stream));
}

size_t spiffy_draft_blocks_workspace(const spiffy_draft_desc* desc) {
  if (check_draft_desc(desc) != SPIFFY_OK) return 0;
  return draft_workspace_bytes(*desc);
}

spiffy_status spiffy_draft_blocks(const spiffy_draft_desc* desc, const void* logits,
                                  const int32_t* state, const int32_t* formula_off,
                                  const int32_t* formula_i, const int32_t* formula_j,
                                  const int32_t* child_off, const int32_t* child_idx,
                                  int32_t* draft_tokens, int32_t* kept, float* score,
                                  int32_t* parent_off, int32_t* parent_idx,
                                  int32_t* dev_status, void* workspace,
                                  size_t workspace_bytes, void* cuda_stream) {
  const spiffy_status st = check_draft_desc(desc);
  if (st != SPIFFY_OK) return st;
  if (!logits || !state || !formula_off || !formula_i || !formula_j || !child_off || !child_idx ||
      !draft_tokens || !kept || !score || !parent_off || !parent_idx)
    return SPIFFY_EINVAL;
  if (!aligned16(logits)) return SPIFFY_EINVAL;
  const size_t need = draft_workspace_bytes(*desc);
  if (!workspace || workspace_bytes < need || !aligned16(workspace)) return SPIFFY_EWORKSPACE;
  return launch_draft(*desc, logits, state, formula_off, formula_i, formula_j, child_off, child_idx,
                      draft_tokens, kept, score, parent_off, parent_idx, dev_status, workspace,
                      static_cast<cudaStream_t>(cuda_stream));
}

const char* spiffy_status_string(spiffy_status status) {
  switch (status) {
    case SPIFFY_OK: return "ok";
    case SPIFFY_EINVAL: return "invalid argument (null, size, alignment)";
    case SPIFFY_EUNSUPPORTED: return "shape or dtype outside the supported limits";
    case SPIFFY_EWORKSPACE: return "workspace missing, misaligned or too small";
    case SPIFFY_EGRAPH: return "malformed draft graph";
    case SPIFFY_ECUDA: return "CUDA runtime error at launch";
  }
  return "unknown status";
}

void spiffy_set_wait_limits(int64_t mbarrier_polls, int64_t flag_polls, int32_t lazy_extra_arrivals) {
  g_mbar_polls.store(mbarrier_polls < 0 ? (1u << 20) : (uint32_t)(mbarrier_polls > (1 << 20) ? (1 << 20) : mbarrier_polls),
                     std::memory_order_relaxed);
  g_flag_polls.store(flag_polls < 0 ? (1u << 21) : (uint32_t)(flag_polls > (1 << 21) ? (1 << 21) : flag_polls),
                     std::memory_order_relaxed);
  g_lazy_extra.store(lazy_extra_arrivals < 0 ? 0 : lazy_extra_arrivals, std::memory_order_relaxed);
}

uint64_t spiffy_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
