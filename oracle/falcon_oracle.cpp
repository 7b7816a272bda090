// CPU oracle for the tree-verification step of Falcon speculative decoding.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
// verification step computes; tests compare the CUDA library against it and the
// benchmark times it as a CPU baseline.  Nothing in the product path may call
// it, and it shares no code with the CUDA sources.
//
// What is computed, and where the paper says so:
//   * tree-masked attention: the target model scores all drafted tree tokens in
//     one forward pass, each token attending to the sequence's prefix and to its
//     own root-to-node chain (Section 3.4 verifies the whole tree in one parallel
//     pass the way SpecInfer does; Section 4.5 uses tree attention when drafting
//     and when verifying).  The paper writes no attention formula; standard
//     scaled-dot-product softmax is taken.
//   * greedy acceptance: temperature 0 (Section 4.1); a drafted child is accepted
//     when its token equals the target's argmax at its parent; the accepted
//     length is the tau of Section 4.2.
//   * compaction: after verification the accepted tokens and their features are
//     kept for the next drafting phase (Section 3.4); this is the KV-cache form.
//   * top-m selection (the step before verification): every tree node is expanded
//     with the m most probable tokens of the drafter's distribution (Appendix A).
//   * the LM head with the greedy token taken directly (Section 3.1, Eq. 6).
//   * non-greedy decoding: the target's own draw at every node (Section 3.1).  The
//     paper states no acceptance rule for this case; oracle_sample_tokens follows
//     a reading stated at the function, so it is "parity unpinned" with respect to
//     the paper (its arithmetic is pinned like the rest).
//
// Every routine is the plain definition: visible sets by walking parent
// pointers, two-pass softmax with double accumulators, sequential argmax scan,
// alive-node search over all nodes, out-of-place gather.  No blocking, fusion
// or bit tricks.  All outputs have pins in tests/ (closed forms, hand-worked
// trees, chain == causal attention, brute-force path enumeration, invariants).
//
// Build: g++ -O2 -fopenmp -shared -fPIC (see oracle/build_oracle.py).

#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// bf16 is the upper half of an IEEE fp32: widening is exact.
inline float bf16_to_float(uint16_t h) {
  uint32_t u = static_cast<uint32_t>(h) << 16;
  float f;
  std::memcpy(&f, &u, sizeof f);
  return f;
}

// A(i): node i, its parent, its grandparent, ... up to the root (Section 3.4:
// a token sees the tokens that precede it in the tree; verification uses the strict
// ancestor-or-self set).  Returns false on a malformed tree.
bool ancestor_chain(const int32_t* parent, int32_t T, int32_t i, std::vector<int32_t>& chain) {
  chain.clear();
  int32_t u = i;
  for (int32_t steps = 0; steps <= T; ++steps) {
    if (u < 0 || u >= T) return false;
    chain.push_back(u);
    if (u == 0) return true;
    u = parent[u];
  }
  return false;  // cycle
}

bool tree_ok(const int32_t* parent, int32_t T) {
  if (T < 1 || parent[0] != -1) return false;
  for (int32_t i = 1; i < T; ++i)
    if (parent[i] < 0 || parent[i] >= i) return false;
  return true;
}

int pick_threads(int n_threads) {
#ifdef _OPENMP
  return n_threads > 0 ? n_threads : omp_get_max_threads();
#else
  (void)n_threads;
  return 1;
#endif
}

}  // namespace

extern "C" {

int oracle_max_threads() { return pick_threads(0); }

// 0 when parent[0] == -1 and 0 <= parent[i] < i for i >= 1, else 1.
int oracle_tree_validate(const int32_t* parent, int32_t T) { return tree_ok(parent, T) ? 0 : 1; }

// Writes A(i) in walk order (i first, root last) to out[]; returns its size, or -1.
int oracle_ancestors(const int32_t* parent, int32_t T, int32_t i, int32_t* out) {
  std::vector<int32_t> chain;
  if (!ancestor_chain(parent, T, i, chain)) return -1;
  for (size_t j = 0; j < chain.size(); ++j) out[j] = chain[j];
  return static_cast<int>(chain.size());
}

// Masked softmax attention with an explicit visibility rule.
//
// For sequence b with prefix length L and tree size T, node i of the tree and
// query head h (KV head h / G, consecutive query heads sharing a KV head) see
// the keys  {0..L-1}  and  {L + t : t in S(i)}  where S(i) = A(i) when
// tree_mask == nullptr, else the set bits of tree_mask row i (a caller-given
// T-bit row, two 64-bit words per node; used for the drafter's relaxed mask).
//   s_j = sm_scale * <q[i,h,:], K[j,:]>,  m = max_j s_j,  p_j = exp(s_j - m),
//   out[i,h,:] = sum_j p_j V[j,:] / sum_j p_j
// Tree keys are cache rows L + t unless k_tree/v_tree are given, in which case
// tree key t of sequence b is row node_off[b] + t of those [N, Hkv, D] arrays.
int oracle_tree_attn(int32_t B, const int32_t* node_off, const int32_t* parent, const int32_t* prefix_len,
                     int32_t Hq, int32_t Hkv, int32_t D, float sm_scale, const uint16_t* q,
                     const uint16_t* k_cache, const uint16_t* v_cache, int64_t stride_b, int64_t stride_h,
                     int64_t stride_s, const uint16_t* k_tree, const uint16_t* v_tree,
                     const uint64_t* tree_mask, float* out, int n_threads) {
  if (B < 1 || Hq < 1 || Hkv < 1 || Hq % Hkv != 0 || D < 1) return 1;
  const int32_t G = Hq / Hkv;
  for (int32_t b = 0; b < B; ++b)
    if (!tree_ok(parent + node_off[b], node_off[b + 1] - node_off[b])) return 4;

  // One work item per (sequence, node, query head).
  struct Item { int32_t b, i, h; };
  std::vector<Item> items;
  for (int32_t b = 0; b < B; ++b)
    for (int32_t i = 0; i < node_off[b + 1] - node_off[b]; ++i)
      for (int32_t h = 0; h < Hq; ++h) items.push_back({b, i, h});

  const int nt = pick_threads(n_threads);
  (void)nt;
#pragma omp parallel for schedule(dynamic, 8) num_threads(nt)
  for (int64_t w = 0; w < static_cast<int64_t>(items.size()); ++w) {
    const int32_t b = items[w].b, i = items[w].i, h = items[w].h;
    const int32_t base = node_off[b];
    const int32_t T = node_off[b + 1] - base;
    const int32_t L = prefix_len[b];
    const int32_t kvh = h / G;
    const int32_t* par = parent + base;

    // visible tree nodes
    std::vector<int32_t> tree_vis;
    if (tree_mask) {
      const uint64_t* row = tree_mask + 2 * static_cast<int64_t>(base + i);
      for (int32_t t = 0; t < T; ++t)
        if ((row[t >> 6] >> (t & 63)) & 1ull) tree_vis.push_back(t);
    } else {
      ancestor_chain(par, T, i, tree_vis);
    }

    // key/value row pointers of the visible set, prefix first
    std::vector<const uint16_t*> kp, vp;
    const uint16_t* kb = k_cache + b * stride_b + kvh * stride_h;
    const uint16_t* vb = v_cache + b * stride_b + kvh * stride_h;
    for (int32_t j = 0; j < L; ++j) {
      kp.push_back(kb + j * stride_s);
      vp.push_back(vb + j * stride_s);
    }
    for (int32_t t : tree_vis) {
      if (k_tree) {
        const int64_t r = (static_cast<int64_t>(base + t) * Hkv + kvh) * D;
        kp.push_back(k_tree + r);
        vp.push_back(v_tree + r);
      } else {
        kp.push_back(kb + (L + t) * stride_s);
        vp.push_back(vb + (L + t) * stride_s);
      }
    }

    const uint16_t* qrow = q + (static_cast<int64_t>(base + i) * Hq + h) * D;
    float* orow = out + (static_cast<int64_t>(base + i) * Hq + h) * D;
    const size_t n = kp.size();
    if (n == 0) {  // only reachable with an all-zero caller mask and L == 0
      for (int32_t d = 0; d < D; ++d) orow[d] = 0.0f;
      continue;
    }
    std::vector<double> s(n);
    double m = -std::numeric_limits<double>::infinity();
    for (size_t j = 0; j < n; ++j) {
      double acc = 0.0;
      for (int32_t d = 0; d < D; ++d)
        acc += static_cast<double>(bf16_to_float(qrow[d])) * static_cast<double>(bf16_to_float(kp[j][d]));
      s[j] = static_cast<double>(sm_scale) * acc;
      if (s[j] > m) m = s[j];
    }
    double denom = 0.0;
    std::vector<double> o(D, 0.0);
    for (size_t j = 0; j < n; ++j) {
      const double p = std::exp(s[j] - m);
      denom += p;
      for (int32_t d = 0; d < D; ++d) o[d] += p * static_cast<double>(bf16_to_float(vp[j][d]));
    }
    for (int32_t d = 0; d < D; ++d) orow[d] = static_cast<float>(o[d] / denom);
  }
  return 0;
}

// Ordinary causal attention of T new tokens appended to a prefix of L tokens:
// new token i sees keys 0 .. L+i.  Written separately from oracle_tree_attn
// (score matrix first, then a row softmax in long double) as the second
// opinion for chain-shaped trees (Section 4.5: a chain of the tree's height).
// q [T, Hq, D]; k, v [Hkv, L+T, D] contiguous; out fp32 [T, Hq, D].
int oracle_causal_attn(int32_t L, int32_t T, int32_t Hq, int32_t Hkv, int32_t D, float sm_scale,
                       const uint16_t* q, const uint16_t* k, const uint16_t* v, float* out) {
  if (Hq % Hkv != 0) return 1;
  const int32_t G = Hq / Hkv, S = L + T;
  std::vector<long double> score(static_cast<size_t>(T) * S);
  for (int32_t h = 0; h < Hq; ++h) {
    const uint16_t* kh = k + static_cast<int64_t>(h / G) * S * D;
    const uint16_t* vh = v + static_cast<int64_t>(h / G) * S * D;
    for (int32_t i = 0; i < T; ++i)
      for (int32_t j = 0; j < S; ++j) {
        long double acc = 0.0L;
        for (int32_t d = 0; d < D; ++d)
          acc += static_cast<long double>(bf16_to_float(q[(static_cast<int64_t>(i) * Hq + h) * D + d])) *
                 static_cast<long double>(bf16_to_float(kh[static_cast<int64_t>(j) * D + d]));
        score[static_cast<size_t>(i) * S + j] = acc * static_cast<long double>(sm_scale);
      }
    for (int32_t i = 0; i < T; ++i) {
      const int32_t last = L + i;  // inclusive
      long double mx = score[static_cast<size_t>(i) * S];
      for (int32_t j = 1; j <= last; ++j) mx = std::fmax(mx, score[static_cast<size_t>(i) * S + j]);
      long double z = 0.0L;
      for (int32_t j = 0; j <= last; ++j) z += std::exp(score[static_cast<size_t>(i) * S + j] - mx);
      for (int32_t d = 0; d < D; ++d) {
        long double acc = 0.0L;
        for (int32_t j = 0; j <= last; ++j)
          acc += std::exp(score[static_cast<size_t>(i) * S + j] - mx) / z *
                 static_cast<long double>(bf16_to_float(vh[static_cast<int64_t>(j) * D + d]));
        out[(static_cast<int64_t>(i) * Hq + h) * D + d] = static_cast<float>(acc);
      }
    }
  }
  return 0;
}

// g[i] = lowest index attaining the row maximum of logits[i, 0..V-1]
// (greedy decoding, Section 4.1).  Sequential scan with a strict '>' test: a
// NaN never wins, +0 and -0 tie (lower index wins), an all-NaN or all -inf
// row gives 0.
int oracle_argmax(const float* logits, int32_t N, int32_t V, int64_t stride, int32_t* g, int n_threads) {
  if (N < 0 || V < 1 || stride < V) return 1;
  const int nt = pick_threads(n_threads);
  (void)nt;
#pragma omp parallel for num_threads(nt)
  for (int32_t i = 0; i < N; ++i) {
    const float* row = logits + static_cast<int64_t>(i) * stride;
    float best = -std::numeric_limits<float>::infinity();
    int32_t idx = 0;
    for (int32_t v = 0; v < V; ++v)
      if (row[v] > best) {
        best = row[v];
        idx = v;
      }
    g[i] = idx;
  }
  return 0;
}

// The target model's own token at every node when decoding is not greedy.  Section 3.1: the next
// token is drawn from the distribution that the LM head computes; Appendix A only says that in a
// non-greedy setting the drafted children are sampled, and Section 3.4 that verification follows
// SpecInfer - the paper states no acceptance rule of its own.
// The reading taken here is the simplest lossless one: at every node the target draws its token
// from softmax(logits / temperature), and a drafted child is accepted when it carries that token
// (with temperature -> 0 this is the greedy rule).  The draw is the inverse-CDF one, with the
// uniform number u[i] in [0, 1) supplied by the caller:
//   w_v = exp((logits[i, v] - max_v logits[i, v]) / temperature)   (a NaN logit has weight 0),
//   g[i] = the lowest v with  sum_{k <= v} w_k  >  u[i] * sum_k w_k,
// sums in vocabulary order, in double; if rounding leaves no such v, the last v with w_v > 0; a row
// with no finite maximum (all NaN or -inf) gives 0.  cdf (optional, [N, V] doubles) receives the
// normalised partial sums.  The accepted path then follows from g exactly as in the greedy case.
int oracle_sample_tokens(const float* logits, int32_t N, int32_t V, int64_t stride, double temperature, const float* u,
                         int32_t* g, double* cdf, int n_threads) {
  if (N < 0 || V < 1 || stride < V || !(temperature > 0.0)) return 1;
  const int nt = pick_threads(n_threads);
  (void)nt;
#pragma omp parallel for num_threads(nt)
  for (int32_t i = 0; i < N; ++i) {
    const float* row = logits + static_cast<int64_t>(i) * stride;
    double top = -std::numeric_limits<double>::infinity();
    for (int32_t v = 0; v < V; ++v)
      if (static_cast<double>(row[v]) > top) top = row[v];
    if (!std::isfinite(top)) {  // nothing to draw from (or a +inf logit, which takes everything: its first position)
      int32_t idx = 0;
      if (top > 0)
        for (int32_t v = 0; v < V; ++v)
          if (static_cast<double>(row[v]) == top) {
            idx = v;
            break;
          }
      g[i] = idx;
      if (cdf)
        for (int32_t v = 0; v < V; ++v) cdf[static_cast<int64_t>(i) * V + v] = v >= idx ? 1.0 : 0.0;
      continue;
    }
    double total = 0.0;
    for (int32_t v = 0; v < V; ++v) {
      const double x = row[v];
      if (x == x) total += std::exp((x - top) / temperature);
    }
    const double target = static_cast<double>(u[i]) * total;
    double run = 0.0;
    int32_t idx = -1, last = 0;
    for (int32_t v = 0; v < V; ++v) {
      const double x = row[v];
      const double w = (x == x) ? std::exp((x - top) / temperature) : 0.0;
      run += w;
      if (w > 0.0) last = v;
      if (idx < 0 && run > target) idx = v;
      if (cdf) cdf[static_cast<int64_t>(i) * V + v] = run / total;
    }
    g[i] = idx >= 0 ? idx : last;
  }
  return 0;
}

// LM-head logits of the tree's nodes and their greedy argmax without a logits matrix in
// between.  The verification pass ends in the target model's LM head, which turns the
// aggregated features into the distribution over the vocabulary (Section 3.1); Eq. 6 writes
// p = Softmax(LM(f)); with temperature 0 (Section 4.1) only the position of the largest logit
// is needed, and the softmax does not move it.  The LM head is taken as a bias-free linear map
// (the LLaMA / Vicuna heads the paper evaluates have no bias):
//   logit[i, v] = sum_k feat[i, k] * head[v, k],      g[i] = lowest v attaining max_v logit[i, v].
// feat: bf16 bit patterns [N, feat_stride], head: bf16 [V, head_stride] (both row-major, the
// first `hidden` columns used).  Products of bf16 values are exact in double and the sum runs
// over k in order in double.  Same tie and NaN rules as oracle_argmax (strict '>' scan).
// best[i] (optional) receives the winning logit; logits_out (optional, [N, V] doubles) all of them.
int oracle_lm_head_argmax(const uint16_t* feat, int64_t feat_stride, const uint16_t* head, int64_t head_stride, int32_t N,
                          int32_t hidden, int32_t V, int32_t* g, double* best, double* logits_out, int n_threads) {
  if (N < 0 || hidden < 1 || V < 1 || feat_stride < hidden || head_stride < hidden) return 1;
  const int nt = pick_threads(n_threads);
  (void)nt;
#pragma omp parallel for num_threads(nt)
  for (int32_t i = 0; i < N; ++i) {
    const uint16_t* f = feat + static_cast<int64_t>(i) * feat_stride;
    double top = -std::numeric_limits<double>::infinity();
    int32_t idx = 0;
    for (int32_t v = 0; v < V; ++v) {
      const uint16_t* w = head + static_cast<int64_t>(v) * head_stride;
      double acc = 0.0;
      for (int32_t k = 0; k < hidden; ++k)
        acc += static_cast<double>(bf16_to_float(f[k])) * static_cast<double>(bf16_to_float(w[k]));
      if (logits_out) logits_out[static_cast<int64_t>(i) * V + v] = acc;
      if (acc > top) {
        top = acc;
        idx = v;
      }
    }
    g[i] = idx;
    if (best) best[i] = top;
  }
  return 0;
}

// Top-m entries of every row, best first: the children a tree node is given when the tree is
// grown (in the greedy setting the m most probable tokens, Appendix A; m = 20 at the root there).
// Plain definition: m passes over the row, each taking the best entry not taken yet.  Order:
// larger value first, the lower index among equal values (+0 and -0 are equal); a NaN counts as
// -inf and is reported as -inf.  Needs 1 <= m <= V.
int oracle_topm(const float* logits, int32_t N, int32_t V, int64_t stride, int32_t m, float* top_val,
                int32_t* top_idx, int n_threads) {
  if (N < 0 || V < 1 || stride < V || m < 1 || m > V) return 1;
  const int nt = pick_threads(n_threads);
  (void)nt;
#pragma omp parallel for num_threads(nt)
  for (int32_t i = 0; i < N; ++i) {
    const float* row = logits + static_cast<int64_t>(i) * stride;
    std::vector<char> taken(static_cast<size_t>(V), 0);
    for (int32_t r = 0; r < m; ++r) {
      const float ninf = -std::numeric_limits<float>::infinity();
      float best = ninf;
      int32_t idx = -1;
      for (int32_t v = 0; v < V; ++v) {
        if (taken[v]) continue;
        const float x = (row[v] != row[v]) ? ninf : row[v];
        if (idx < 0 || x > best) {  // strict: the first (lowest) index among equals stays
          best = x;
          idx = v;
        }
      }
      taken[idx] = 1;
      top_val[static_cast<int64_t>(i) * m + r] = best;
      top_idx[static_cast<int64_t>(i) * m + r] = idx;
    }
  }
  return 0;
}

// Greedy tree acceptance (Section 3.4 with Section 4.1's temperature 0).
// The root (local node 0) is always on the path.  A non-root node c is alive
// when every node a on its chain other than the root satisfies
// token[a] == g[parent[a]].  The result is the alive node of greatest depth,
// lowest index among equals; path = its root-to-node chain; n_path = depth+1;
// next_token = g[last node of the path] (the target's own next token).
int oracle_tree_accept(int32_t B, const int32_t* node_off, const int32_t* parent, const int32_t* token,
                       const int32_t* g, int32_t* path, int32_t path_stride, int32_t* n_path,
                       int32_t* next_token) {
  std::vector<int32_t> chain;
  for (int32_t b = 0; b < B; ++b) {
    const int32_t base = node_off[b], T = node_off[b + 1] - base;
    const int32_t* par = parent + base;
    const int32_t* tok = token + base;
    const int32_t* gb = g + base;
    if (!tree_ok(par, T)) return 4;
    int32_t best = 0, best_depth = 0;
    for (int32_t c = 0; c < T; ++c) {
      if (!ancestor_chain(par, T, c, chain)) return 4;
      bool alive = true;
      for (int32_t a : chain)
        if (a != 0 && tok[a] != gb[par[a]]) alive = false;
      const int32_t depth = static_cast<int32_t>(chain.size()) - 1;
      if (alive && depth > best_depth) {  // strict: lowest index wins ties
        best = c;
        best_depth = depth;
      }
    }
    ancestor_chain(par, T, best, chain);
    if (static_cast<int32_t>(chain.size()) > path_stride) return 5;
    for (int32_t j = 0; j < path_stride; ++j) path[static_cast<int64_t>(b) * path_stride + j] = -1;
    for (size_t j = 0; j < chain.size(); ++j)  // chain is node-first; the path is root-first
      path[static_cast<int64_t>(b) * path_stride + j] = chain[chain.size() - 1 - j];
    n_path[b] = static_cast<int32_t>(chain.size());
    next_token[b] = gb[best];
  }
  return 0;
}

// Second opinion for acceptance: enumerate every root-to-leaf path, scan each
// from the root and stop at the first node whose token differs from the
// argmax at its parent; keep the longest accepted prefix (ties: lowest index
// of the prefix's last node).
int oracle_bruteforce_accept(int32_t B, const int32_t* node_off, const int32_t* parent, const int32_t* token,
                             const int32_t* g, int32_t* path, int32_t path_stride, int32_t* n_path,
                             int32_t* next_token) {
  for (int32_t b = 0; b < B; ++b) {
    const int32_t base = node_off[b], T = node_off[b + 1] - base;
    const int32_t* par = parent + base;
    const int32_t* tok = token + base;
    const int32_t* gb = g + base;
    if (!tree_ok(par, T)) return 4;
    std::vector<char> has_child(T, 0);
    for (int32_t i = 1; i < T; ++i) has_child[par[i]] = 1;
    std::vector<int32_t> best_path{0};
    for (int32_t leaf = 0; leaf < T; ++leaf) {
      if (has_child[leaf]) continue;
      std::vector<int32_t> rev;
      for (int32_t u = leaf; u != -1; u = par[u]) rev.push_back(u);
      std::vector<int32_t> p(rev.rbegin(), rev.rend());  // root first
      size_t keep = 1;
      while (keep < p.size() && tok[p[keep]] == gb[p[keep - 1]]) ++keep;
      p.resize(keep);
      if (p.size() > best_path.size() || (p.size() == best_path.size() && p.back() < best_path.back()))
        best_path = p;
    }
    if (static_cast<int32_t>(best_path.size()) > path_stride) return 5;
    for (int32_t j = 0; j < path_stride; ++j) path[static_cast<int64_t>(b) * path_stride + j] = -1;
    for (size_t j = 0; j < best_path.size(); ++j) path[static_cast<int64_t>(b) * path_stride + j] = best_path[j];
    n_path[b] = static_cast<int32_t>(best_path.size());
    next_token[b] = gb[best_path.back()];
  }
  return 0;
}

// Compaction of one cache (K or V of one layer): the accepted path's rows
// become cache rows L_b .. L_b + n_path - 1 in path order (Section 3.4: the
// accepted tokens and their features are kept for the next drafting phase).
// Out of place: rows are read from a pristine copy, so the overlap between
// source and destination rows cannot matter.  tree_rows == nullptr means tree
// row t is cache row L_b + t; else it is row node_off[b] + t of [N, Hkv, D].
// cache is modified in place on the host; new_len (optional) = L_b + n_path.
int oracle_kv_compact(int32_t B, const int32_t* node_off, const int32_t* prefix_len, int32_t Hkv, int32_t D,
                      uint16_t* cache, int64_t stride_b, int64_t stride_h, int64_t stride_s, int32_t s_cap,
                      const uint16_t* tree_rows, const int32_t* path, int32_t path_stride,
                      const int32_t* n_path, int32_t* new_len) {
  for (int32_t b = 0; b < B; ++b) {
    const int32_t L = prefix_len[b], T = node_off[b + 1] - node_off[b];
    if (n_path[b] < 1 || n_path[b] > T || L + T > s_cap) return 5;
    for (int32_t h = 0; h < Hkv; ++h) {
      uint16_t* base = cache + b * stride_b + h * stride_h;
      std::vector<uint16_t> pristine(static_cast<size_t>(T) * D);
      for (int32_t t = 0; t < T; ++t) {
        const uint16_t* src = tree_rows
                                  ? tree_rows + (static_cast<int64_t>(node_off[b] + t) * Hkv + h) * D
                                  : base + static_cast<int64_t>(L + t) * stride_s;
        std::memcpy(&pristine[static_cast<size_t>(t) * D], src, sizeof(uint16_t) * D);
      }
      for (int32_t j = 0; j < n_path[b]; ++j) {
        const int32_t t = path[static_cast<int64_t>(b) * path_stride + j];
        if (t < 0 || t >= T) return 4;
        std::memcpy(base + static_cast<int64_t>(L + j) * stride_s, &pristine[static_cast<size_t>(t) * D],
                    sizeof(uint16_t) * D);
      }
    }
    if (new_len) new_len[b] = L + n_path[b];
  }
  return 0;
}

// Accepted tokens and their features (Section 3.4: they are kept after verification, as the
// input of the next drafting phase): for every node on the accepted
// path, in path order, its drafted token and its row of the [N, hidden] feature matrix (16-bit
// elements, copied bit for bit).  feat_out is [B, out_rows, hidden], tok_out [B, out_rows]; only
// the first n_path[b] rows of a sequence are written.
int oracle_feature_gather(int32_t B, const int32_t* node_off, const int32_t* path, int32_t path_stride,
                          const int32_t* n_path, const int32_t* token, const uint16_t* feat, int32_t hidden,
                          int64_t feat_stride, int32_t out_rows, uint16_t* feat_out, int32_t* tok_out) {
  for (int32_t b = 0; b < B; ++b) {
    const int32_t T = node_off[b + 1] - node_off[b];
    if (n_path[b] < 1 || n_path[b] > T || n_path[b] > out_rows) return 5;
    for (int32_t j = 0; j < n_path[b]; ++j) {
      const int32_t t = path[static_cast<int64_t>(b) * path_stride + j];
      if (t < 0 || t >= T) return 4;
      const int64_t node = node_off[b] + t;
      tok_out[static_cast<int64_t>(b) * out_rows + j] = token[node];
      for (int32_t c = 0; c < hidden; ++c)
        feat_out[(static_cast<int64_t>(b) * out_rows + j) * hidden + c] = feat[node * feat_stride + c];
    }
  }
  return 0;
}

}  // extern "C"
