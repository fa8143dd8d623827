/*
 * spiffy.h -- C ABI of libspiffy: the verification hot path of Spiffy
 * (speculative decoding for masked-diffusion LLMs with directed draft graphs),
 * written for NVIDIA B200 (sm_100a).
 *
 * One verification step scores N draft states of one L-token block in a single
 * packed forward pass of the target model and then decides how far the block
 * may advance.  This library holds the two model-independent, data-parallel
 * pieces of that step:
 *
 *   spiffy_graph_attention   the packed attention of Sec. 4.3 (mask of Fig. 3):
 *                            every draft state attends to the cached context
 *                            and, bidirectionally, to its own block only;
 *   spiffy_full_sequence_attention
 *                            the same with trailing masked blocks as extra
 *                            queries (full-sequence models, App. A.2);
 *   spiffy_unmask_decide     steps 1-4 of Algorithm 1 (the function Next() of
 *                            App. A) evaluated for every node of the graph;
 *   spiffy_accept_walk       step 5 of Algorithm 1: the walk through the draft
 *                            graph (Sec. 4.4.1, Eqs. draft-graph-1..3) to the
 *                            deepest accepted node;
 *   spiffy_decide_walk       the two above in one call (steps 1-5), fused on
 *                            the device where the graph is small;
 *   spiffy_decide_walk_lazy  steps 1-5 with the decision evaluated only for the
 *                            nodes the walk reaches (fewer bytes read);
 *   spiffy_unmask_decide_sampled
 *                            steps 1-4 at sampling temperature T > 0;
 *   spiffy_lmhead_decide     steps 1-4 fused into the output projection: the
 *                            logits are reduced on the tensor cores, never stored;
 *   spiffy_draft_blocks      drafting and pruning (Sec. 4.4.2, Sec. 4.4.4): the
 *                            draft blocks and parent lists of the next step;
 *   spiffy_verify_step_host  one whole step (attention of one layer, steps 1-5)
 *                            from tensors in host memory, copies included;
 *   spiffy_stage_masked_rows, spiffy_unmask_decide_static
 *                            helpers without a counterpart in the paper: staging
 *                            of logits from pinned host memory, and the decision
 *                            step with its scratch inside the library.
 *
 * Vocabulary (paper notation in brackets where it differs):
 *   B  batch of independent sequences            N  nodes of the draft graph,
 *   L  block length [L]                             node 0 = the true block
 *   P  cached context length (keys/values of X')    X_k(t), nodes 1..N-1 = the
 *   Hq, Hkv  query / key-value heads                draft blocks [D = N-1]
 *   d  head dimension                            V  vocabulary size [V]
 *   tau  confidence threshold of dynamic unmasking; S  static unmasking rate
 *
 * Conventions common to every entry point
 *   - Every data pointer is a DEVICE pointer owned by the caller (the source of
 *     spiffy_stage_masked_rows may also be mapped pinned host memory); the
 *     library neither allocates nor frees device memory.  Descriptors are plain host
 *     structs, read before the call returns.
 *   - Calls are asynchronous on `cuda_stream` (a cudaStream_t passed as void*,
 *     NULL = the default stream) and never synchronise the device.
 *   - Scratch memory is caller-provided: size it with the *_workspace() query.
 *     Its contents on entry are arbitrary; calls sharing one workspace must be
 *     ordered on one stream.  (spiffy_unmask_decide_static is the exception: it
 *     keeps its scratch inside the library.)
 *   - Tensor base addresses must be 16-byte aligned, else SPIFFY_EINVAL.
 *   - Host-detectable problems return a status code and launch nothing.
 *     Device-detectable problems set bits in a caller-provided status word and
 *     yield a defined output; no kernel traps, asserts or waits unboundedly.
 *   - Thread-safe for calls on distinct streams with distinct workspaces.
 */
#ifndef SPIFFY_H_
#define SPIFFY_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SPIFFY_OK = 0,
  SPIFFY_EINVAL = 1,       /* null pointer, bad size, misaligned tensor */
  SPIFFY_EUNSUPPORTED = 2, /* shape or dtype outside the stated limits */
  SPIFFY_EWORKSPACE = 3,   /* workspace missing or too small */
  SPIFFY_EGRAPH = 4,       /* reserved for host-side graph validation */
  SPIFFY_ECUDA = 5         /* a CUDA runtime call failed (launch error) */
} spiffy_status;

typedef enum { SPIFFY_F32 = 0, SPIFFY_BF16 = 1 } spiffy_dtype;

/* Unmasking rule of step 3 of Algorithm 1.
 * TOPS:      the S most confident still-masked positions (Sec. 3.1, S_t = S).
 * THRESHOLD: every still-masked position whose confidence is > tau (strict,
 *            Sec. 3.1 "threshold-based dynamic unmasking"); when none passes,
 *            the single most confident one, so that decoding always advances. */
typedef enum { SPIFFY_RULE_TOPS = 0, SPIFFY_RULE_THRESHOLD = 1 } spiffy_rule;

/* Bits of the device status words. */
#define SPIFFY_DEV_NONFINITE 1 /* a logits row held NaN/+inf or only -inf     */
#define SPIFFY_DEV_BADGRAPH 2  /* parent list malformed (offsets or indices)   */
#define SPIFFY_DEV_TIMEOUT 4   /* a bounded on-chip wait gave up               */

/* Attention kernel selection (spiffy_attn_desc.kernel). */
#define SPIFFY_ATTN_AUTO 0   /* tensor-core kernel when the shape allows it   */
#define SPIFFY_ATTN_SIMT 1   /* fp32 CUDA-core kernel (any supported shape)   */
#define SPIFFY_ATTN_TCGEN05 2 /* tcgen05/TMEM kernel or SPIFFY_EUNSUPPORTED   */
/* Flag, OR-ed into spiffy_attn_desc.kernel: the next kernel of the stream may be
 * scheduled while this call's kernel still runs (it is launched as soon as every
 * thread block of this kernel has started; kernels that order themselves with
 * cudaGridDependencySynchronize(), as all kernels of this library do, still see
 * this call's complete output).  For the layer loop of a model, where the next
 * kernel's set-up then overlaps this kernel's tail.  Tensor-core kernel only. */
#define SPIFFY_ATTN_EARLY_DEPENDENTS 0x100

/* ------------------------------------------------------------------------- */
/* Packed draft-graph attention (Sec. 4.3; mask semantics: caption of Fig. 3) */
/* ------------------------------------------------------------------------- */
typedef struct {
  int32_t batch;      /* B >= 1                                              */
  int32_t n_nodes;    /* N >= 1                                              */
  int32_t block_len;  /* L in [1, 1024]; [1, 64] on the CUDA-core kernel        */
  int32_t prefix_len; /* P >= 0 context keys shared by all nodes             */
  int32_t n_q_heads;  /* Hq                                                  */
  int32_t n_kv_heads; /* Hkv, divides Hq; query head h reads kv head
                         h / (Hq/Hkv)                                        */
  int32_t head_dim;   /* d in {64, 128}                                      */
  int32_t dtype;      /* spiffy_dtype of q, k, v and out                     */
  float scale;        /* softmax scale; 0 means 1/sqrt(d)                    */
  int32_t kernel;     /* SPIFFY_ATTN_AUTO/SIMT/TCGEN05, | SPIFFY_ATTN_EARLY_DEPENDENTS */
} spiffy_attn_desc;

/* Bytes of scratch spiffy_graph_attention needs for this shape (may be 0). */
size_t spiffy_graph_attention_workspace(const spiffy_attn_desc* desc);

/*
 * out[b,n,l,h,:] = sum_j softmax_j(scale * <q[b,n,l,h,:], k_j>) * v_j, where j
 * runs over the P context keys of sequence b and the L keys of node n's OWN
 * block -- no other node's block, the root's included.  Attention inside the
 * block is bidirectional.  Positional encoding is the caller's: q and k arrive
 * already rotated, every node using the true block's positions (Sec. 4.3).
 *
 * Layouts (row-major, innermost last), all of dtype desc->dtype:
 *   q, out             [B][N][L][Hq][d]
 *   k_prefix, v_prefix [B][P][Hkv][d]     (may be NULL when P == 0)
 *   k_block, v_block   [B][N][L][Hkv][d]
 * dev_status: one int32 on the device, OR-ed with SPIFFY_DEV_* bits; may be
 * NULL.  Accumulation is fp32; the result is rounded once to desc->dtype.
 */
spiffy_status spiffy_graph_attention(const spiffy_attn_desc* desc,
                                     const void* q, const void* k_prefix,
                                     const void* v_prefix, const void* k_block,
                                     const void* v_block, void* out,
                                     int32_t* dev_status, void* workspace,
                                     size_t workspace_bytes, void* cuda_stream);

/*
 * The verification attention of a full-sequence bidirectional model that caches
 * only its prefix (caption of Fig. 3; App. A.2): the block being decoded (node 0)
 * and the S trailing, still fully masked positions attend to the whole true
 * sequence -- prefix, true block, suffix --, every draft block to the prefix, the
 * suffix and itself (every block of the true sequence except the one it is a
 * draft of).  Two launches of the tensor-core kernel, no copy: the nodes with
 * the context given as two segments [prefix ; suffix], then the suffix rows as
 * one node whose block is the suffix and whose context is [prefix ; true block].
 *
 *   desc      batch, n_nodes, block_len, prefix_len, heads, head_dim, scale of the
 *             nodes' call; dtype bf16 and head_dim 128 (else SPIFFY_EUNSUPPORTED)
 *   suffix_len S in [0, 1024]; 0 makes this spiffy_graph_attention
 *   q_nodes, out_nodes   [B][N][L][Hq][d]     q_suffix, out_suffix [B][S][Hq][d]
 *   k/v_prefix [B][P][Hkv][d]   k/v_suffix [B][S][Hkv][d]   k/v_block [B][N][L][Hkv][d]
 * dev_status, stream and error behaviour as in spiffy_graph_attention; the
 * workspace (spiffy_full_sequence_attention_workspace) serves both launches.
 */
size_t spiffy_full_sequence_attention_workspace(const spiffy_attn_desc* desc, int32_t suffix_len);
spiffy_status spiffy_full_sequence_attention(const spiffy_attn_desc* desc, int32_t suffix_len,
                                             const void* q_nodes, const void* q_suffix,
                                             const void* k_prefix, const void* v_prefix,
                                             const void* k_suffix, const void* v_suffix,
                                             const void* k_block, const void* v_block,
                                             void* out_nodes, void* out_suffix,
                                             int32_t* dev_status, void* workspace,
                                             size_t workspace_bytes, void* cuda_stream);

/* ------------------------------------------------------------------------- */
/* Decision: steps 1-4 of Algorithm 1 for every node (Next() of App. A)      */
/* ------------------------------------------------------------------------- */
typedef struct {
  int32_t batch;         /* B                                                */
  int32_t n_nodes;       /* N                                                */
  int32_t block_len;     /* L in [1, 64]                                     */
  int32_t vocab;         /* V >= 1                                           */
  int32_t logits_dtype;  /* spiffy_dtype                                     */
  int64_t row_stride;    /* elements between consecutive logits rows, >= V;
                            row_stride * sizeof(element) must be a multiple
                            of 16                                            */
  int32_t mask_token_id; /* token id that marks a still-masked position      */
  int32_t rule;          /* spiffy_rule                                      */
  int32_t top_s;         /* S of RULE_TOPS (>= 1); ignored by THRESHOLD      */
  float threshold;       /* tau of RULE_THRESHOLD                            */
} spiffy_decide_desc;

size_t spiffy_unmask_decide_workspace(const spiffy_decide_desc* desc);

/*
 * For every node (b,n) and every position l with block_tokens[b,n,l] ==
 * mask_token_id, reduce the V logits of row (b,n,l) to
 *   top_tok = argmax_v x_v (lowest v on ties),
 *   conf    = max_v softmax(x)_v = 1 / sum_v exp(x_v - max x)
 * (steps 1-2), then choose the set U of positions to unmask by desc->rule
 * (step 3; ties in confidence go to the lower position).  Step 4, the next
 * state, is state with top_tok written at the positions of U; it is returned
 * implicitly as (top_tok, unmask_bits).
 *
 *   logits       [B][N][L] rows of V elements, desc->row_stride apart; rows of
 *                already-unmasked positions are never read
 *   block_tokens [B][N][L] int32, the state of every node
 *   conf         [B][N][L] fp32; -inf at unmasked positions
 *   top_tok      [B][N][L] int32; the existing token at unmasked positions
 *   unmask_bits  [B][N] uint64, bit l set when l is in U
 *   n_unmask     [B][N] int32, |U| (0 for a node with nothing left to unmask)
 *   dev_status   [B] int32, OR-ed with SPIFFY_DEV_NONFINITE when a row that was
 *                read is not finite (its conf/top_tok are then unspecified);
 *                may be NULL
 * Math is fp32 on exactly up-converted inputs; the argmax compares input
 * values, never probabilities.
 */
spiffy_status spiffy_unmask_decide(const spiffy_decide_desc* desc,
                                   const void* logits,
                                   const int32_t* block_tokens, float* conf,
                                   int32_t* top_tok, uint64_t* unmask_bits,
                                   int32_t* n_unmask, int32_t* dev_status,
                                   void* workspace, size_t workspace_bytes,
                                   void* cuda_stream);

/*
 * The same decision step for callers that cannot provide scratch memory.  (The
 * paper has no counterpart: this is a packaging variant of the call above.)
 *
 * Who needs it: code that must not, or cannot, allocate device memory when it
 * calls -- a plug-in inside a serving engine that has already claimed the
 * whole device for its own pool, so that cudaMalloc would fail; a decode loop
 * whose latency budget does not tolerate cudaMalloc's device-wide
 * synchronisation; a caller that simply has no allocator at hand.  Such a
 * caller still passes its inputs and outputs, but no workspace: the partial
 * results of the vocabulary reduction go to one fixed array of
 * SPIFFY_DECIDE_STATIC_BYTES bytes that is part of the library image (every GPU
 * on which the library is loaded holds that array until the process exits).
 * The call performs no cudaMalloc, cudaFree or other allocation.
 *
 * Arguments, layouts, results and status bits are those of
 * spiffy_unmask_decide.  Differences:
 *   - A shape whose scratch need (spiffy_unmask_decide_workspace) exceeds
 *     SPIFFY_DECIDE_STATIC_BYTES is refused with SPIFFY_EUNSUPPORTED and nothing
 *     is launched.  The limit (2 MiB) covers every benchmark shape, the
 *     largest being B*N*L = 4096 rows of a 126k vocabulary (1 MiB); batches of
 *     ten thousand rows and more go beyond it and have to use the regular
 *     entry point.
 *   - The first call on each device looks up the array's device address
 *     (cudaGetSymbolAddress, with that device current) and keeps it; make that
 *     first call outside any stream capture.
 *   - All calls in the process share the one array, and it keeps whatever the
 *     last call left.  Nothing in it needs clearing between calls, but two
 *     calls that overlap on the GPU (different streams, or one device used
 *     from two threads without ordering) race on it and give undefined
 *     results: order them on one stream or with events.
 */
#define SPIFFY_DECIDE_STATIC_BYTES (2u << 20)
spiffy_status spiffy_unmask_decide_static(const spiffy_decide_desc* desc,
                                          const void* logits,
                                          const int32_t* block_tokens,
                                          float* conf, int32_t* top_tok,
                                          uint64_t* unmask_bits,
                                          int32_t* n_unmask,
                                          int32_t* dev_status,
                                          void* cuda_stream);

/*
 * The decision step at sampling temperature T > 0 (Sec. 5.3, "Effect of Temperature", runs Spiffy at
 * T > 0; the sampler itself is not given in the paper and is fixed here).
 * Per still-masked position the token is drawn from softmax(z), z = x / T, in
 * two levels over vocabulary slices of W = spiffy_sampled_slice_width(desc)
 * consecutive entries (slice s = entries s W ... s W + W - 1):
 *   1. the slice  s* = argmax_s (ln Z_s + g_s),  Z_s = sum over the slice of
 *      exp(z_v),  g_s = -ln(-ln u_s)   (Gumbel-max on the slices' weights; ties
 *      to the lower slice, a slice without weight never wins);
 *   2. top_tok = the first entry v of slice s*, ascending, whose running sum
 *      sum_{w <= v in s*} exp(z_w) reaches u' Z_s*   (inversion inside the slice);
 * conf is its probability softmax(z)[top_tok]; the unmasking rule then runs on
 * conf exactly as in spiffy_unmask_decide, and every other argument, layout and
 * status bit is that call's.  One pass over the logits plus one slice per row:
 * the cost of the greedy decision, not of V random numbers per row.
 * The uniforms come from the counter-based generator Philox4x32-10 (Salmon,
 * Moraes, Dror, Shaw, SC 2011):
 *   counter = (slice s, position l, sequence b, number of still-masked
 *              positions of the node),  key = (seed & 0xffffffff, seed >> 32),
 *   u_s = (output word 0 + 0.5) / 2^32,  u' = (output word 1 + 0.5) / 2^32 of
 *   the chosen slice's counter.
 * W is the width of the slices the kernels reduce in one piece: the vocabulary
 * cut into the fewest equal slices of at most 8192 (bf16) or 4096 (fp32)
 * entries, rounded up to a multiple of 8 (bf16) or 4 (fp32); 0 for a bad
 * descriptor.  It is part of the sampler's definition: another W gives other
 * (equally distributed) tokens for the same seed.
 * The noise depends on the state of the block, not on the node's index: a
 * draft block and the true block that equals it draw the same tokens, which is
 * what the losslessness argument of App. A needs.  A caller that wants fresh
 * noise for another block or request changes the seed.
 * Workspace: spiffy_unmask_decide_sampled_workspace(desc).
 */
typedef struct {
  float temperature; /* T > 0 */
  uint32_t reserved; /* 0 */
  uint64_t seed;
} spiffy_sample_desc;

size_t spiffy_unmask_decide_sampled_workspace(const spiffy_decide_desc* desc);
int64_t spiffy_sampled_slice_width(const spiffy_decide_desc* desc);
spiffy_status spiffy_unmask_decide_sampled(const spiffy_decide_desc* desc,
                                           const spiffy_sample_desc* sample, const void* logits,
                                           const int32_t* block_tokens, float* conf,
                                           int32_t* top_tok, uint64_t* unmask_bits,
                                           int32_t* n_unmask, int32_t* dev_status,
                                           void* workspace, size_t workspace_bytes,
                                           void* cuda_stream);

/*
 * Steps 1-4 of Algorithm 1 straight from the hidden states: the logits
 *   x[r][v] = sum_k hidden_states[r][k] * weight[v][k]       (fp32 accumulation)
 * are formed tile by tile on the tensor cores and reduced there, so that the
 * [rows x V] logits are never written to memory; the result is what
 * spiffy_unmask_decide gives on those (unrounded, fp32) logits.
 *   hidden_states [B*N*L][hidden] bf16, row r = (b * N + n) * L + l; rows of
 *                 unmasked positions are computed and ignored
 *   weight        [V][hidden] bf16 (the output embedding, one row per token)
 *   desc          batch, n_nodes, block_len, vocab, mask_token_id, rule, top_s,
 *                 threshold are used; logits_dtype and row_stride are ignored
 * Limit: hidden a multiple of 128, else SPIFFY_EUNSUPPORTED.  Rows are taken 256 at a
 * time and every such pass reads the weight matrix again: the call is made for
 * the few hundred rows of one verification step.
 * Outputs, status bits and the finalize step are those of spiffy_unmask_decide.
 * The paper evaluates the decision on materialised logits; fusing it into the
 * output projection is this library's addition.
 * Workspace: spiffy_lmhead_decide_workspace(desc, hidden) (depends on the
 * device's SM count; 0 when the shape is not supported).
 */
size_t spiffy_lmhead_decide_workspace(const spiffy_decide_desc* desc, int32_t hidden);
spiffy_status spiffy_lmhead_decide(const spiffy_decide_desc* desc, int32_t hidden,
                                   const void* hidden_states, const void* weight,
                                   const int32_t* block_tokens, float* conf, int32_t* top_tok,
                                   uint64_t* unmask_bits, int32_t* n_unmask, int32_t* dev_status,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ------------------------------------------------------------------------- */
/* Acceptance: step 5 of Algorithm 1 over the draft graph of Sec. 4.4.1      */
/* ------------------------------------------------------------------------- */
/*
 * Per sequence b: cur = 0 (the true block).  Repeat: let next(cur) be
 * state(cur) with top_tok written at unmask_bits(cur).  Among the nodes m that
 * list cur as a parent, in ascending m, take the first whose state equals
 * next(cur) on all L tokens; if there is one it is accepted (its distribution
 * replaces the target's), cur = m; otherwise stop.  A node with an empty
 * unmask set ends the walk.
 *
 *   parent_off [B][N+1] int32, CSR offsets into parent_idx, relative to the
 *              start of sequence b's own slice: the slice of sequence b begins
 *              at parent_idx + b * parent_cap
 *   parent_idx [B][parent_cap] int32, parents of node m at
 *              [parent_off[b][m], parent_off[b][m+1]); a parent index must be
 *              smaller than its child's (topological order), node 0 has none
 *   accepted_node [B] deepest accepted node (0 = no draft accepted)
 *   n_accepted    [B] number of accepted drafts = hops taken; the block has
 *                 advanced n_accepted + 1 denoising steps on one model call
 *   path          [B][N] visited nodes, root first, padded with -1
 *   next_block    [B][L] next(accepted_node): the new true block
 *   dev_status    [B] OR-ed with SPIFFY_DEV_BADGRAPH when an offset or index is
 *                 out of range (such entries are ignored); may be NULL
 * Uses desc->batch, n_nodes, block_len only.
 * Ordering: block_tokens and the parent lists (here, in spiffy_decide_walk and in
 * the lazy call) are fetched while earlier work of the stream may still be
 * draining.  They must be complete in memory before the kernel that precedes
 * this call in the stream can let its dependents start, which holds for every
 * kernel of this library and for any kernel that does not use programmatic
 * dependent launch; do not produce them with an early-triggering kernel of your
 * own placed directly before the call.
 */
spiffy_status spiffy_accept_walk(const spiffy_decide_desc* desc,
                                 const int32_t* block_tokens,
                                 const int32_t* parent_off,
                                 const int32_t* parent_idx, int32_t parent_cap,
                                 const int32_t* top_tok,
                                 const uint64_t* unmask_bits,
                                 int32_t* accepted_node, int32_t* n_accepted,
                                 int32_t* path, int32_t* next_block,
                                 int32_t* dev_status, void* cuda_stream);

/*
 * Steps 1-5 of Algorithm 1 in one call: exactly spiffy_unmask_decide followed
 * by spiffy_accept_walk on its top_tok / unmask_bits, with the same arguments,
 * layouts, outputs (bit for bit) and status codes; decide_status and
 * walk_status are the dev_status arrays of the two calls (either may be NULL).
 * When a sequence's graph is small (N * L <= 512 and its arrays fit the
 * default shared memory of one CTA) the merge of the vocabulary slices, the
 * unmasking rule and the walk run in one kernel per sequence, one launch
 * fewer than the two separate calls; otherwise this is the two calls.
 * Workspace: spiffy_unmask_decide_workspace(desc).
 */
spiffy_status spiffy_decide_walk(const spiffy_decide_desc* desc, const void* logits,
                                 const int32_t* block_tokens, const int32_t* parent_off,
                                 const int32_t* parent_idx, int32_t parent_cap, float* conf,
                                 int32_t* top_tok, uint64_t* unmask_bits, int32_t* n_unmask,
                                 int32_t* decide_status, int32_t* accepted_node,
                                 int32_t* n_accepted, int32_t* path, int32_t* next_block,
                                 int32_t* walk_status, void* workspace, size_t workspace_bytes,
                                 void* cuda_stream);

/*
 * Lazy chain evaluation of steps 1-5 of Algorithm 1: the decision is computed
 * only for the nodes the walk reaches (the true block, then each accepted
 * draft), level by level inside one kernel, instead of for all N nodes.  Only
 * 1 + n_accepted of the N nodes' logits are read.  The paper has no
 * counterpart; it evaluates every draft's distribution (Sec. 4.3).
 *
 * Same arguments and layouts as spiffy_decide_walk.  On return
 *   - accepted_node, n_accepted, path, next_block are those of
 *     spiffy_decide_walk, bit for bit;
 *   - conf, top_tok, unmask_bits, n_unmask hold, for the nodes on the path, the
 *     bits spiffy_unmask_decide gives; for every other node n_unmask is -1 and
 *     the other three are left untouched;
 *   - walk_status reports a malformed parent list only if the walk scanned it;
 *     SPIFFY_DEV_TIMEOUT in both status words when a bounded wait between the
 *     levels ran out (results are then unspecified).
 * There is no grid-wide barrier: per sequence, the thread blocks that reduce
 * the current node's rows count themselves in on an arrival counter, the block
 * that owns the sequence waits for that count, decides, and publishes the next
 * node under an epoch number the reducers wait for; sequences never wait for one
 * another.  A level still costs two such round trips through memory, so the
 * call pays off when one node's share of the logits is large (long
 * vocabularies, batches) and loses to spiffy_decide_walk on a single short
 * graph.  SPIFFY_EUNSUPPORTED when the batch exceeds the number of thread blocks
 * the device holds at once.
 * Workspace: spiffy_decide_walk_lazy_workspace(desc); contents on entry
 * arbitrary (the call zeroes the few bytes it needs with a memset on the
 * stream).
 */
size_t spiffy_decide_walk_lazy_workspace(const spiffy_decide_desc* desc);
spiffy_status spiffy_decide_walk_lazy(const spiffy_decide_desc* desc, const void* logits,
                                      const int32_t* block_tokens, const int32_t* parent_off,
                                      const int32_t* parent_idx, int32_t parent_cap, float* conf,
                                      int32_t* top_tok, uint64_t* unmask_bits, int32_t* n_unmask,
                                      int32_t* decide_status, int32_t* accepted_node,
                                      int32_t* n_accepted, int32_t* path, int32_t* next_block,
                                      int32_t* walk_status, void* workspace,
                                      size_t workspace_bytes, void* cuda_stream);

/* ------------------------------------------------------------------------- */
/* One whole verification step from HOST memory                                */
/* ------------------------------------------------------------------------- */
/*
 * For a caller whose tensors are in host memory (the paper has no counterpart:
 * its tensors never leave the device): copies the inputs of one verification
 * step to the device, runs spiffy_graph_attention (one layer; Sec. 4.3) and
 * spiffy_decide_walk (Algorithm 1, steps 1-5) on them, copies the verdict back
 * and returns when it has arrived (the call synchronises `cuda_stream`).
 *
 * All tensor arguments are HOST pointers with the layouts of the component
 * calls.  Pinned memory (cudaHostAlloc / cudaHostRegister) makes the copies
 * asynchronous and lets one kernel read, of the logits, only the rows of
 * still-masked positions -- the only ones the decision reads -- over the bus;
 * pageable memory works too, through the runtime's staging, with all rows
 * copied.  Everything but the logits travels on a helper stream of the library
 * (created at the first call on a device) at the same time.
 *
 *   desc->attn, desc->decide   descriptors of the two component calls; batch,
 *                    n_nodes and block_len must agree, block_len <= 64
 *   desc->parent_cap entries per sequence in parent_idx
 *   q .. parent_idx  inputs (k_prefix, v_prefix may be NULL when prefix_len == 0)
 *   accepted_node [B], n_accepted [B], path [B][N], next_block [B][L]   the verdict
 *   status [1 + 2B]  device status words: [0] attention, [1 .. B] decision per
 *                    sequence, [1+B .. 2B] walk per sequence (SPIFFY_DEV_* bits)
 *   device_workspace DEVICE memory, 256-byte aligned, of
 *                    spiffy_verify_step_host_workspace(desc) bytes: staging copies
 *                    of every input, the attention output and the decision's
 *                    per-node results (which stay there), the kernels' scratch
 * Calls sharing a workspace, or made from several threads on one device, must
 * not overlap (the helper stream is shared).
 */
typedef struct {
  spiffy_attn_desc attn;
  spiffy_decide_desc decide;
  int32_t parent_cap;
} spiffy_step_desc;

size_t spiffy_verify_step_host_workspace(const spiffy_step_desc* desc);
spiffy_status spiffy_verify_step_host(const spiffy_step_desc* desc, const void* q,
                                      const void* k_prefix, const void* v_prefix,
                                      const void* k_block, const void* v_block,
                                      const void* logits, const int32_t* block_tokens,
                                      const int32_t* parent_off, const int32_t* parent_idx,
                                      int32_t* accepted_node, int32_t* n_accepted, int32_t* path,
                                      int32_t* next_block, int32_t* status,
                                      void* device_workspace, size_t workspace_bytes,
                                      void* cuda_stream);

/*
 * Staging helper for callers whose logits sit in pinned host memory (the paper
 * has no counterpart: its logits never leave the device).  Copies row r
 * (row_bytes bytes, a multiple of 16) from src_rows to dst_rows for every r in
 * [0, n_rows) with tokens[r] == mask_token_id, i.e. exactly the rows
 * spiffy_unmask_decide will read; other rows of dst_rows are left as they are.
 *   src_rows, tokens: memory the DEVICE can read -- device memory, or pinned
 *             host memory that is mapped into the device's address space (with
 *             unified addressing every cudaHostAlloc / cudaHostRegister
 *             allocation is); 16-byte aligned
 *   dst_rows: device memory, 16-byte aligned, same row layout as src_rows
 * One kernel reads the rows over the bus; n_rows <= 65535.
 */
spiffy_status spiffy_stage_masked_rows(const void* src_rows, void* dst_rows, int64_t row_bytes,
                                       const int32_t* tokens, int32_t mask_token_id,
                                       int64_t n_rows, void* cuda_stream);

/* ------------------------------------------------------------------------- */
/* Drafting and pruning (Sec. 4.4.2 "Drafting Source", Sec. 4.4.4 "Pruning")  */
/* ------------------------------------------------------------------------- */
typedef struct {
  int32_t batch;         /* B                                                */
  int32_t block_len;     /* L in [1, 64]                                     */
  int32_t vocab;         /* V                                                */
  int32_t logits_dtype;  /* spiffy_dtype                                     */
  int64_t row_stride;    /* elements between logits rows, as in the decision */
  int32_t mask_token_id;
  int32_t n_formulas;    /* D draft formulas of the calibrated graph, <= 1024 */
  int32_t top_k;         /* vocabulary ranks a formula may use, 1..4         */
  int32_t budget;        /* D* drafts kept after pruning, 1..D               */
  int32_t parent_cap;    /* entries per sequence in parent_idx               */
} spiffy_draft_desc;

size_t spiffy_draft_blocks_workspace(const spiffy_draft_desc* desc);

/*
 * Builds the draft blocks of the next verification step from the target
 * distribution of the current block.  Per sequence: the still-masked positions
 * are ranked by their maximum probability (token position rank i, 0 = most
 * confident; ties to the lower position) and per position the vocabulary by
 * probability (vocabulary rank j; ties to the lower token id); candidate c_ij
 * is the token of rank j at the position of rank i (Sec. 4.4.2).  Draft formula
 * q is a fixed list of (i, j) pairs from the offline calibration; its block is
 * the current block with its candidates written in.  Pruning (Sec. 4.4.4):
 * localScore = geometric mean of the candidates' probabilities, childScore =
 * geometric mean of the local scores of the formula's children, score = their
 * geometric mean (just localScore without children); the `budget` best formulas
 * are kept (ties to the lower index).  A formula that asks for a position rank
 * beyond the number of masked positions cannot be built: score -inf, never kept.
 *
 *   logits      [B][L] rows of V: the distribution to draft from (that of the
 *               node accepted last); rows of unmasked positions are not read
 *   state       [B][L] int32 current block
 *   formula_off [D+1], formula_i, formula_j: CSR of the (i, j) pairs, shared
 *               by all sequences; parents before children
 *   child_off   [D+1], child_idx: children of each formula in the draft graph.
 *               These five arrays are constants of the model: they must be
 *               complete in device memory before the call is made (the kernels
 *               read them without waiting for earlier work on the stream)
 *   draft_tokens [B][D*+1][L]: node 0 = the current block, then the kept drafts
 *               in formula order; unused nodes repeat the current block
 *   kept        [B][D*] formula index of every kept draft, -1 for unused nodes
 *   score       [B][D] fp32 score of every formula
 *   parent_off  [B][D*+2], parent_idx [B][parent_cap]: parent lists over the
 *               D*+1 nodes in the layout spiffy_accept_walk reads: node a is a
 *               parent of node c when a's candidate set is a strict subset of
 *               c's (Eqs. draft-graph-2/3; node 0 is the empty set)
 *   dev_status  [B]: SPIFFY_DEV_NONFINITE for an unusable logits row,
 *               SPIFFY_DEV_BADGRAPH when parent_cap was too small (lists cut)
 */
spiffy_status spiffy_draft_blocks(const spiffy_draft_desc* desc, const void* logits,
                                  const int32_t* state, const int32_t* formula_off,
                                  const int32_t* formula_i, const int32_t* formula_j,
                                  const int32_t* child_off, const int32_t* child_idx,
                                  int32_t* draft_tokens, int32_t* kept, float* score,
                                  int32_t* parent_off, int32_t* parent_idx,
                                  int32_t* dev_status, void* workspace,
                                  size_t workspace_bytes, void* cuda_stream);

/*
 * Failure-detection hook (the paper has no counterpart).  Every device-side wait
 * of this library is bounded: an mbarrier wait of the tensor-core kernels gives
 * up after a number of polls, a wait on a global-memory word of
 * spiffy_decide_walk_lazy likewise; the kernel then sets SPIFFY_DEV_TIMEOUT in
 * the caller's status word(s), lets copies in flight land, frees its tensor
 * memory and returns, so the context stays usable.  This call changes those
 * limits for all later launches of the process, so that a test can make a wait
 * run out without hanging or faulting anything:
 *   mbarrier_polls       polls per mbarrier wait; 0 = give up without waiting
 *                        (the kernel then issues no copy it does not wait for
 *                        and no tensor-core product); < 0 restores the default
 *   flag_polls           polls (about 100 ns apart) per wait of the lazy call;
 *                        < 0 restores the default
 *   lazy_extra_arrivals  sequence 0 of the lazy call waits for this many
 *                        arrivals more than can come (0 = normal operation)
 * Values above the defaults are clamped to them.  Not for production use.
 */
void spiffy_set_wait_limits(int64_t mbarrier_polls, int64_t flag_polls,
                            int32_t lazy_extra_arrivals);

/* Static description of a status code; never NULL. */
const char* spiffy_status_string(spiffy_status status);

/* Launch counter: number of kernels this library has launched in this process
 * since load (all entry points, all threads).  For benchmarks' bookkeeping. */
uint64_t spiffy_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SPIFFY_H_ */
