// spiffy_oracle.cpp -- TEST INFRASTRUCTURE, not a product path.
//
// A plain, slow, double-precision CPU statement of what one Spiffy draft-graph
// verification step computes.  It exists so that the CUDA library can be
// checked against something written straight from the paper; it shares no code
// with the CUDA path and nothing in the product may call it.  Only the tests,
// the smoke check and the benchmark's CPU-baseline leg use it.
//
// The method is exact (not an approximation), so each function below is the
// definition written out, with no blocking, fusion or reordering:
//   oracle_graph_attention  Sec. 4.3 + the mask described in Fig. 3's caption
//   oracle_unmask_decide    Algorithm 1 steps 1-4 (Next() of App. A), with the
//                           unmasking rules of Sec. 3.1
//   oracle_accept_walk      Algorithm 1 step 5 over the graph of Sec. 4.4.1
//
// Pins (tests/test_oracle_*.py): softmax rows sum to one; packing invariance
// against an explicit-mask formulation; closed forms (equal values, equal
// keys, one dominant key); a library SDPA in float64 on the P = 0, N = 1 case;
// naive long-double softmax; hand-built rule cases; brute-force DAG search;
// the losslessness invariant of App. A on a toy model.  No numeric example is
// printed in the paper, so absolute values are pinned by those alone.
//
// Build: g++ -O2 -fopenmp -shared -fPIC (OpenMP only spreads independent
// (sequence, node) pairs over cores; per-element arithmetic order is fixed).

#include <cmath>
#include <cstdint>
#include <limits>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

extern "C" {

// ---------------------------------------------------------------------------
// Sec. 4.3 / Fig. 3: node n's queries see the P context keys and the L keys of
// node n's own block, nothing else.  Inputs are fp32 (bf16 values up-converted
// exactly by the caller); all arithmetic is double.
//   q, out            [B][N][L][Hq][d]
//   kp, vp            [B][P][Hkv][d]
//   kb, vb            [B][N][L][Hkv][d]
//   probs (optional)  [B][N][L][Hq][P+L] softmax rows, for the sum-to-one pin
// ---------------------------------------------------------------------------
void oracle_graph_attention(int B, int N, int L, int P, int Hq, int Hkv, int d,
                            double scale, const float* q, const float* kp,
                            const float* vp, const float* kb, const float* vb,
                            double* out, double* probs) {
  const int group = Hq / Hkv;
  const long long n_tasks = (long long)B * N;
#pragma omp parallel for schedule(dynamic)
  for (long long task = 0; task < n_tasks; ++task) {
    const int b = (int)(task / N), n = (int)(task % N);
    std::vector<double> s(P + L);
    for (int l = 0; l < L; ++l) {
      for (int h = 0; h < Hq; ++h) {
        const int g = h / group;
        const float* qv = q + ((((size_t)b * N + n) * L + l) * Hq + h) * d;
        // scores over the context keys, then over the node's own block keys
        for (int j = 0; j < P; ++j) {
          const float* kv = kp + (((size_t)b * P + j) * Hkv + g) * d;
          double acc = 0.0;
          for (int c = 0; c < d; ++c) acc += (double)qv[c] * (double)kv[c];
          s[j] = scale * acc;
        }
        for (int r = 0; r < L; ++r) {
          const float* kv = kb + ((((size_t)b * N + n) * L + r) * Hkv + g) * d;
          double acc = 0.0;
          for (int c = 0; c < d; ++c) acc += (double)qv[c] * (double)kv[c];
          s[P + r] = scale * acc;
        }
        // softmax over the P + L allowed keys
        double m = -std::numeric_limits<double>::infinity();
        for (int j = 0; j < P + L; ++j) m = s[j] > m ? s[j] : m;
        double z = 0.0;
        for (int j = 0; j < P + L; ++j) {
          s[j] = std::exp(s[j] - m);
          z += s[j];
        }
        for (int j = 0; j < P + L; ++j) s[j] /= z;
        if (probs) {
          double* pr =
              probs + ((((size_t)b * N + n) * L + l) * Hq + h) * (size_t)(P + L);
          for (int j = 0; j < P + L; ++j) pr[j] = s[j];
        }
        // weighted sum of the values
        double* o = out + ((((size_t)b * N + n) * L + l) * Hq + h) * d;
        for (int c = 0; c < d; ++c) o[c] = 0.0;
        for (int j = 0; j < P; ++j) {
          const float* vv = vp + (((size_t)b * P + j) * Hkv + g) * d;
          for (int c = 0; c < d; ++c) o[c] += s[j] * (double)vv[c];
        }
        for (int r = 0; r < L; ++r) {
          const float* vv = vb + ((((size_t)b * N + n) * L + r) * Hkv + g) * d;
          for (int c = 0; c < d; ++c) o[c] += s[P + r] * (double)vv[c];
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------
// Algorithm 1 steps 1-4 for every node.  rule: 0 = top-S, 1 = threshold.
//   logits        rows (b,n,l) of V floats, row_stride apart
//   block_tokens  [B][N][L]
//   conf          [B][N][L] double, -inf at unmasked positions
//   top_tok       [B][N][L], the existing token at unmasked positions
//   unmask_bits   [B][N], n_unmask [B][N]
//   next_tokens   [B][N][L] the state after step 4
//   margin        [B][N] distance of the decision from flipping: for the
//                 threshold rule min_l |conf_l - tau| (and, when the fallback
//                 fires, the gap between the two best confidences); for top-S
//                 the gap between the S-th and (S+1)-th confidence; +inf when
//                 nothing could flip
//   bad_row       [B][N] 1 when a row that was read is not finite
// ---------------------------------------------------------------------------
void oracle_unmask_decide(int B, int N, int L, int V, long long row_stride,
                          int mask_id, int rule, int top_s, double tau,
                          const float* logits, const int32_t* block_tokens,
                          double* conf, int32_t* top_tok, uint64_t* unmask_bits,
                          int32_t* n_unmask, int32_t* next_tokens,
                          double* margin, int32_t* bad_row) {
  const double inf = std::numeric_limits<double>::infinity();
  const long long n_tasks = (long long)B * N;
#pragma omp parallel for schedule(dynamic)
  for (long long node = 0; node < n_tasks; ++node) {
    const int32_t* state = block_tokens + node * L;
    int bad = 0;
    std::vector<int> masked;
    for (int l = 0; l < L; ++l) {
      const size_t pos = (size_t)node * L + l;
      if (state[l] != mask_id) {
        conf[pos] = -inf;
        top_tok[pos] = state[l];
        continue;
      }
      masked.push_back(l);
      const float* x = logits + pos * (size_t)row_stride;
      // step 2: max and argmax of the marginal; softmax is monotone, so both
      // are taken on the logits; ties go to the lowest vocabulary index
      double m = -inf;
      for (int v = 0; v < V; ++v) m = (double)x[v] > m ? (double)x[v] : m;
      int tok = 0;
      for (int v = 0; v < V; ++v)
        if ((double)x[v] == m) { tok = v; break; }
      double z = 0.0;
      for (int v = 0; v < V; ++v) z += std::exp((double)x[v] - m);
      const double c = 1.0 / z;  // = exp(m - m) / z, the top-1 probability
      if (!(c == c) || !std::isfinite(m)) bad = 1;
      conf[pos] = c;
      top_tok[pos] = tok;
    }
    // step 3: positions ordered by (confidence desc, position asc)
    std::vector<int> order(masked);
    for (size_t i = 1; i < order.size(); ++i) {  // insertion sort, stable
      int key = order[i];
      size_t j = i;
      while (j > 0 && conf[(size_t)node * L + order[j - 1]] <
                          conf[(size_t)node * L + key]) {
        order[j] = order[j - 1];
        --j;
      }
      order[j] = key;
    }
    uint64_t bits = 0;
    double mar = inf;
    const size_t n_masked = order.size();
    if (n_masked > 0) {
      if (rule == 0) {
        const size_t take = (size_t)top_s < n_masked ? (size_t)top_s : n_masked;
        for (size_t i = 0; i < take; ++i) bits |= 1ull << order[i];
        if (take < n_masked)
          mar = conf[(size_t)node * L + order[take - 1]] -
                conf[(size_t)node * L + order[take]];
      } else {
        for (size_t i = 0; i < n_masked; ++i) {
          const double c = conf[(size_t)node * L + order[i]];
          if (c > tau) bits |= 1ull << order[i];
          const double gap = std::fabs(c - tau);
          mar = gap < mar ? gap : mar;
        }
        if (bits == 0) {  // nothing passes: unmask the single best position
          bits = 1ull << order[0];
          if (n_masked > 1) {
            const double gap = conf[(size_t)node * L + order[0]] -
                               conf[(size_t)node * L + order[1]];
            mar = gap < mar ? gap : mar;
          }
        }
      }
    }
    // step 4: the next state
    int cnt = 0;
    for (int l = 0; l < L; ++l) {
      const bool u = (bits >> l) & 1ull;
      next_tokens[(size_t)node * L + l] =
          u ? top_tok[(size_t)node * L + l] : state[l];
      cnt += u ? 1 : 0;
    }
    unmask_bits[node] = bits;
    n_unmask[node] = cnt;
    margin[node] = mar;
    bad_row[node] = bad;
  }
}

// ---------------------------------------------------------------------------
// Algorithm 1 step 5.  The graph is given as parent lists (CSR per sequence,
// offsets relative to the sequence's slice of parent_idx, parent_cap entries
// per sequence).  next_tokens is step 4's output for every node.
// ---------------------------------------------------------------------------
void oracle_accept_walk(int B, int N, int L, const int32_t* block_tokens,
                        const int32_t* parent_off, const int32_t* parent_idx,
                        int parent_cap, const int32_t* next_tokens,
                        const uint64_t* unmask_bits, int32_t* accepted_node,
                        int32_t* n_accepted, int32_t* path,
                        int32_t* next_block) {
  for (int b = 0; b < B; ++b) {
    const int32_t* off = parent_off + (size_t)b * (N + 1);
    const int32_t* idx = parent_idx + (size_t)b * parent_cap;
    const int32_t* state = block_tokens + (size_t)b * N * L;
    const int32_t* next = next_tokens + (size_t)b * N * L;
    int32_t* pth = path + (size_t)b * N;
    for (int i = 0; i < N; ++i) pth[i] = -1;
    int cur = 0, hops = 0;
    pth[0] = 0;
    while (hops < N - 1) {  // a path visits each node at most once
      if (unmask_bits[(size_t)b * N + cur] == 0) break;  // nothing left to do
      int found = -1;
      for (int m = 0; m < N && found < 0; ++m) {
        bool is_child = false;
        for (int e = off[m]; e < off[m + 1]; ++e)
          if (idx[e] == cur) is_child = true;
        if (!is_child) continue;
        bool equal = true;
        for (int l = 0; l < L; ++l)
          if (state[(size_t)m * L + l] != next[(size_t)cur * L + l]) equal = false;
        if (equal) found = m;
      }
      if (found < 0) break;
      cur = found;  // accept: its distribution becomes the target's
      pth[++hops] = cur;
    }
    accepted_node[b] = cur;
    n_accepted[b] = hops;
    for (int l = 0; l < L; ++l) next_block[(size_t)b * L + l] = next[(size_t)cur * L + l];
  }
}

int oracle_max_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void oracle_set_threads(int n) {
#ifdef _OPENMP
  omp_set_num_threads(n);
#else
  (void)n;
#endif
}

}  // extern "C"
