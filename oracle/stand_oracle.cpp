// STAND oracle: a plain, slow, double-precision CPU statement of what one
// speculative-sampling step computes.
//
// THIS IS TEST INFRASTRUCTURE.  Only the tests, the smoke check and the
// benchmark's CPU-baseline leg may build, load or call it.  It shares no code
// with the CUDA library: no headers, no tables, no helpers.
//
// What it follows (section numbers are the paper's):
//   * Sec. 3.2  speculative sampling: draft x ~ q, accept with min(1, p/q),
//               otherwise resample from norm(max(0, p - q)).
//   * Sec. 4.1  logit-based N-gram module, one table per order 1..n_max; the
//               "efficient logit approximation": keep top-k (id, probability),
//               merge a repeat with weights c/(c+1) and 1/(c+1), missing ids
//               count as zero, truncate to top-k again.
//   * Sec. 4.2  stochastic tree drafting: look up the longest matching order
//               first, take the first hit, draw as many children as the
//               static tree asks for without replacement; Gumbel-Top-K:
//               phi' = phi - log(-log U), keep the largest.
//   * Sec. 5    sampling temperature T (softmax of logits / T).
//   * Sec. 3.2  deterministic drafting as a variant: the drafts of a node are
//               its most probable candidates, each verified as a one-hot draft.
//
// Readings where the paper is silent (multi-draft verification by recursive
// rejection, what q is, inverse-CDF order, canonical update order, ...) are
// listed in the repository's design document; every one of them is written
// out below where it is used.
//
// Pins (tests marked "not gpu"): Philox known-answer vectors; softmax and
// top-k against library routines; losslessness of verification by black-box
// threshold search and by chi-square; Gumbel-Top-K against the Plackett-Luce
// closed form; table contents against a recount of the token stream, both
// for bulk rows and for whole steps on one-hot targets (which pins the
// pairing of accepted-path rows with their context windows); hand cases for
// the merge, the lookup order and the contexts of nodes deep in the tree.
// Parity unpinned: the canonical order of same-step updates from different
// sequences (a convention, the paper fixes none).
//
// Everything floating point is double.  Nothing is blocked, fused or
// reordered: vectors over the whole vocabulary are used wherever the
// definition speaks of a distribution.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <map>
#include <utility>
#include <vector>

namespace {

// ---------------------------------------------------------------------------
// Randomness: Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw 2011).
// counter = (sequence b, step s, tree node u, slot), key = (seed lo, seed hi).
// Only output word 0 is used.
// ---------------------------------------------------------------------------
void philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2], uint32_t out[4]) {
  uint32_t c0 = ctr_in[0], c1 = ctr_in[1], c2 = ctr_in[2], c3 = ctr_in[3];
  uint32_t k0 = key_in[0], k1 = key_in[1];
  for (int round = 0; round < 10; ++round) {
    const uint64_t prod0 = (uint64_t)0xD2511F53u * c0;
    const uint64_t prod1 = (uint64_t)0xCD9E8D57u * c2;
    const uint32_t n0 = (uint32_t)(prod1 >> 32) ^ c1 ^ k0;
    const uint32_t n1 = (uint32_t)prod1;
    const uint32_t n2 = (uint32_t)(prod0 >> 32) ^ c3 ^ k1;
    const uint32_t n3 = (uint32_t)prod0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

const uint32_t SLOT_FINAL = 0x40000000u;   // the one token sampled at the end of a walk
const uint32_t SLOT_GUMBEL = 0x80000000u;  // | token id: Gumbel noise of that candidate

uint32_t random_u24(uint64_t seed, uint32_t b, uint32_t step, uint32_t node, uint32_t slot) {
  const uint32_t ctr[4] = {b, step, node, slot};
  const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  uint32_t out[4];
  philox4x32_10(ctr, key, out);
  return out[0] >> 8;
}
// U in [0,1): accept tests and the final inverse-CDF sample.
double uniform_half_open(uint32_t u24) { return (double)u24 / 16777216.0; }
// U in (0,1): Gumbel noise, so that log(-log U) is finite.
double uniform_open(uint32_t u24) { return ((double)u24 + 0.5) / 16777216.0; }

// ---------------------------------------------------------------------------
// Input element -> double (exact).  dtype 0: IEEE float.  dtype 1: bfloat16,
// i.e. the upper 16 bits of an IEEE float.
// ---------------------------------------------------------------------------
double element(const void* base, int dtype, int64_t index) {
  if (dtype == 0) return (double)((const float*)base)[index];
  const uint32_t bits = (uint32_t)((const uint16_t*)base)[index] << 16;
  float f;
  std::memcpy(&f, &bits, 4);
  return (double)f;
}

// ---------------------------------------------------------------------------
// Sec. 5: temperature softmax of one row.  z_v = x_v / T,
// p_v = exp(z_v - max z) / sum.  Also returns the log-sum-exp of z.
// ---------------------------------------------------------------------------
void softmax_row(const void* row, int dtype, int V, double T, std::vector<double>& p, double* lse) {
  p.resize(V);
  double zmax = -INFINITY;
  for (int v = 0; v < V; ++v) {
    p[v] = element(row, dtype, v) / T;
    if (p[v] > zmax) zmax = p[v];
  }
  double sum = 0.0;
  for (int v = 0; v < V; ++v) {
    p[v] = std::exp(p[v] - zmax);
    sum += p[v];
  }
  for (int v = 0; v < V; ++v) p[v] /= sum;
  if (lse) *lse = zmax + std::log(sum);
}

// Sec. 4.1: the k entries of a row kept by the table: largest input value
// first, equal values by lower token id.
std::vector<int> topk_ids(const void* row, int dtype, int V, int k) {
  std::vector<int> order(V);
  for (int v = 0; v < V; ++v) order[v] = v;
  const int kk = std::min(k, V);
  std::partial_sort(order.begin(), order.begin() + kk, order.end(), [&](int a, int b) {
    const double xa = element(row, dtype, a), xb = element(row, dtype, b);
    if (xa != xb) return xa > xb;
    return a < b;
  });
  order.resize(kk);
  return order;
}

// ---------------------------------------------------------------------------
// Decision margins: how far a decision was from going the other way.  A GPU
// run may differ from the oracle only where the margin is tiny.
// ---------------------------------------------------------------------------
enum MarginKind { MARGIN_ACCEPT = 0, MARGIN_FINAL = 1, MARGIN_GUMBEL = 2, MARGIN_MERGE = 3 };
struct MarginRec {
  int32_t kind, b, node, aux;
  int32_t key[4];
  double margin;
};

// Inverse CDF in token-index order: the smallest y with U*W < sum_{v<=y} w_v,
// W = sum of all weights.  Falls back to the last token with positive weight.
int inverse_cdf(const std::vector<double>& w, double U, double* margin) {
  double W = 0.0;
  for (double x : w) W += x;
  const double target = U * W;
  double acc = 0.0;
  int last_positive = -1;
  for (int v = 0; v < (int)w.size(); ++v) {
    const double before = acc;
    acc += w[v];
    if (w[v] > 0.0) last_positive = v;
    if (target < acc) {
      if (margin) *margin = std::min(target - before, acc - target) / W;
      return v;
    }
  }
  if (margin) *margin = 0.0;
  return last_positive;
}

// ---------------------------------------------------------------------------
// Sec. 3.2 applied to the ordered children of ONE tree node (the drafts were
// drawn without replacement from q, in this order).  Recursive rejection:
// test child j against the current target pt with the current draft
// distribution q; on rejection the target becomes norm(max(0, pt - q)) and
// the rejected token leaves q, which is renormalised.  If every child is
// rejected one token is drawn from the final residual.
//   p        target distribution of the node (length V)
//   cand_*   the candidate list the children were drawn from (q = phi / sum)
//   child    drafted tokens in draft-rank order
//   u_acc    one uniform in [0,1) per child, u_final one for the resample
// Returns the rank of the accepted child, or -1 with *resampled set.
// ---------------------------------------------------------------------------
int verify_children(const std::vector<double>& p, const std::vector<int>& cand_id,
                    const std::vector<double>& cand_phi, const std::vector<int>& child,
                    const std::vector<double>& u_acc, double u_final, int* resampled,
                    std::vector<double>* accept_margins, double* final_margin) {
  const int V = (int)p.size();
  std::vector<double> pt(p);
  std::vector<double> q(V, 0.0);
  double phi_sum = 0.0;
  for (double f : cand_phi) phi_sum += f;
  for (size_t i = 0; i < cand_id.size(); ++i) q[cand_id[i]] += cand_phi[i] / phi_sum;

  for (size_t j = 0; j < child.size(); ++j) {
    const int x = child[j];
    // accept with probability min(1, pt(x)/q(x)), written without a division
    const bool accept = u_acc[j] * q[x] < pt[x];
    if (accept_margins)
      accept_margins->push_back(q[x] > 0.0 ? std::fabs(u_acc[j] - pt[x] / q[x]) : 1.0);
    if (accept) return (int)j;
    // rejected: residual target, and x leaves the draft distribution
    double rsum = 0.0;
    for (int v = 0; v < V; ++v) {
      pt[v] = std::max(0.0, pt[v] - q[v]);
      rsum += pt[v];
    }
    for (int v = 0; v < V; ++v) pt[v] /= rsum;
    q[x] = 0.0;
    double qsum = 0.0;
    for (int v = 0; v < V; ++v) qsum += q[v];
    if (qsum > 0.0)
      for (int v = 0; v < V; ++v) q[v] /= qsum;
  }
  *resampled = inverse_cdf(pt, u_final, final_margin);
  return -1;
}

// ---------------------------------------------------------------------------
// Sec. 3.2, deterministic drafting: the draft distribution of a drafted token x
// is the one-hot vector at x, so x is accepted with probability pt(x); on
// rejection the target becomes norm(max(0, pt - onehot(x))), i.e. x loses its
// mass and the rest is renormalised, and the next child is tested against that.
// Same arguments and results as verify_children (the candidate list plays no
// part: the drafts are not sampled).
// ---------------------------------------------------------------------------
int verify_children_deterministic(const std::vector<double>& p, const std::vector<int>& child,
                                  const std::vector<double>& u_acc, double u_final, int* resampled,
                                  std::vector<double>* accept_margins, double* final_margin) {
  const int V = (int)p.size();
  std::vector<double> pt(p);
  for (size_t j = 0; j < child.size(); ++j) {
    const int x = child[j];
    std::vector<double> q(V, 0.0);
    q[x] = 1.0;
    const bool accept = u_acc[j] * q[x] < pt[x];
    if (accept_margins) accept_margins->push_back(std::fabs(u_acc[j] - pt[x] / q[x]));
    if (accept) return (int)j;
    double rsum = 0.0;
    for (int v = 0; v < V; ++v) {
      pt[v] = std::max(0.0, pt[v] - q[v]);
      rsum += pt[v];
    }
    for (int v = 0; v < V; ++v) pt[v] /= rsum;
  }
  *resampled = inverse_cdf(pt, u_final, final_margin);
  return -1;
}

// Deterministic drafting: the m most probable candidates, most probable first
// (equal probabilities: lower token id first).  Returns indices into the list.
std::vector<int> most_probable(const std::vector<int>& id, const std::vector<double>& phi, int m, double* margin) {
  const int n = (int)id.size();
  std::vector<int> order(n);
  for (int i = 0; i < n; ++i) order[i] = i;
  std::sort(order.begin(), order.end(), [&](int a, int b) {
    if (phi[a] != phi[b]) return phi[a] > phi[b];
    return id[a] < id[b];
  });
  const int take = std::min(m, n);
  if (margin) {
    double gap = INFINITY;
    for (int r = 0; r < take && r + 1 < n; ++r) gap = std::min(gap, (phi[order[r]] - phi[order[r + 1]]) / phi[order[r]]);
    *margin = gap;
  }
  order.resize(take);
  return order;
}

// ---------------------------------------------------------------------------
// Sec. 4.2 Gumbel-Top-K: g_i = log phi_i - log(-log U_i); the m largest, in
// decreasing order (equal g: lower token id first).  Returns indices into the
// candidate list.
// ---------------------------------------------------------------------------
std::vector<int> gumbel_top(const std::vector<int>& id, const std::vector<double>& phi,
                            const std::vector<double>& U, int m, double* margin) {
  const int n = (int)id.size();
  std::vector<double> g(n);
  for (int i = 0; i < n; ++i) g[i] = std::log(phi[i]) - std::log(-std::log(U[i]));
  std::vector<int> order(n);
  for (int i = 0; i < n; ++i) order[i] = i;
  std::sort(order.begin(), order.end(), [&](int a, int b) {
    if (g[a] != g[b]) return g[a] > g[b];
    return id[a] < id[b];
  });
  const int take = std::min(m, n);
  if (margin) {
    double gap = INFINITY;
    for (int r = 0; r < take && r + 1 < n; ++r) {
      const double a = g[order[r]], b = g[order[r + 1]];
      gap = std::min(gap, (a - b) / std::max(1.0, std::max(std::fabs(a), std::fabs(b))));
    }
    *margin = gap;
  }
  order.resize(take);
  return order;
}

// ---------------------------------------------------------------------------
// Sec. 4.1 table entry and merge.
// ---------------------------------------------------------------------------
struct Entry {
  uint32_t count = 0;                         // how many distributions were averaged
  std::vector<std::pair<int, double>> items;  // (token id, mean probability), <= k
};

// new = old * c/(c+1) + fresh * 1/(c+1) over the union of ids (missing = 0),
// then the k most probable (equal probability: lower id).
void merge_entry(Entry& e, const std::vector<std::pair<int, double>>& fresh, int k, double* margin) {
  const double c = (double)e.count;
  const double w_old = c / (c + 1.0), w_new = 1.0 / (c + 1.0);
  std::map<int, double> merged;
  for (auto& it : e.items) merged[it.first] += it.second * w_old;
  for (auto& it : fresh) merged[it.first] += it.second * w_new;
  std::vector<std::pair<int, double>> all(merged.begin(), merged.end());
  std::sort(all.begin(), all.end(), [](const std::pair<int, double>& a, const std::pair<int, double>& b) {
    if (a.second != b.second) return a.second > b.second;
    return a.first < b.first;
  });
  if (margin) {
    *margin = INFINITY;
    if ((int)all.size() > k) {
      const double a = all[k - 1].second, b = all[k].second;
      *margin = a > 0.0 ? (a - b) / a : 0.0;
    }
  }
  if ((int)all.size() > k) all.resize(k);
  e.items = all;
  e.count += 1;
}

// ---------------------------------------------------------------------------
// The whole state of one decoder context.
// ---------------------------------------------------------------------------
struct Oracle {
  int B, N, V, K, n_max, dtype;
  int deterministic = 0;  // 1: deterministic drafting (Sec. 3.2), 0: stochastic (Sec. 4.2)
  int seq_base = 0;       // global index of sequence 0: the random-number counters use seq_base + b
  double T;
  uint64_t seed;
  std::vector<int> parent, depth;
  std::vector<std::vector<int>> children;
  int D = 0;

  std::map<std::vector<int>, Entry> table;  // key = the n context tokens, oldest first

  std::vector<std::vector<int>> tail;  // per sequence: the last <= n_max tokens
  std::vector<int64_t> len;            // per sequence: tokens so far (root's included)
  std::vector<std::vector<int>> tree;  // per sequence: token of every tree node, -1 = invalid
  std::vector<std::vector<std::vector<int>>> cand_id;      // [b][u]: snapshot of the list
  std::vector<std::vector<std::vector<double>>> cand_phi;  //         u's children were drawn from
  uint32_t step = 0;

  // results of the last verification, input of the update
  std::vector<std::vector<int>> emitted, path;
  std::vector<std::vector<std::vector<std::pair<int, double>>>> fresh;  // [b][j]: top-k of row path[j]
  bool pending = false;

  std::vector<MarginRec> margins;

  void add_margin(int kind, int b, int node, int aux, const std::vector<int>* key, double m) {
    MarginRec r;
    r.kind = kind; r.b = b; r.node = node; r.aux = aux; r.margin = m;
    for (int i = 0; i < 4; ++i) r.key[i] = -1;
    if (key)
      for (size_t i = 0; i < key->size() && i < 4; ++i) r.key[4 - key->size() + i] = (*key)[i];
    margins.push_back(r);
  }

  // ---- verification walk of one sequence (Sec. 3.2 + Sec. 4.2) -----------
  void verify_sequence(int b, const void* logits, std::vector<MarginRec>& local) {
    const size_t esize = dtype == 0 ? 4 : 2;
    // target distribution of every tree node of this sequence
    std::vector<std::vector<double>> P(N);
    for (int u = 0; u < N; ++u) {
      const char* row = (const char*)logits + ((size_t)b * N + u) * (size_t)V * esize;
      softmax_row(row, dtype, V, T, P[u], nullptr);
    }
    emitted[b].clear();
    path[b].clear();
    int u = 0;
    path[b].push_back(0);
    for (;;) {
      std::vector<int> drafted_nodes, drafted_tokens;
      for (int c : children[u])
        if (tree[b][c] >= 0) { drafted_nodes.push_back(c); drafted_tokens.push_back(tree[b][c]); }
      const double u_final = uniform_half_open(random_u24(seed, (uint32_t)(seq_base + b), step, u, SLOT_FINAL));
      MarginRec mr;
      mr.b = b; mr.node = u; for (int i = 0; i < 4; ++i) mr.key[i] = -1;
      if (drafted_nodes.empty()) {
        double fm;
        const int y = inverse_cdf(P[u], u_final, &fm);
        emitted[b].push_back(y);
        mr.kind = MARGIN_FINAL; mr.aux = y; mr.margin = fm; local.push_back(mr);
        break;
      }
      std::vector<double> u_acc(drafted_nodes.size());
      for (size_t j = 0; j < drafted_nodes.size(); ++j)
        u_acc[j] = uniform_half_open(random_u24(seed, (uint32_t)(seq_base + b), step, u, (uint32_t)j));
      int resampled = -1;
      std::vector<double> am;
      double fm = 1.0;
      const int acc = deterministic
                          ? verify_children_deterministic(P[u], drafted_tokens, u_acc, u_final, &resampled, &am, &fm)
                          : verify_children(P[u], cand_id[b][u], cand_phi[b][u], drafted_tokens, u_acc, u_final,
                                            &resampled, &am, &fm);
      for (size_t j = 0; j < am.size(); ++j) {
        mr.kind = MARGIN_ACCEPT; mr.aux = (int)j; mr.margin = am[j]; local.push_back(mr);
      }
      if (acc >= 0) {
        emitted[b].push_back(drafted_tokens[acc]);
        u = drafted_nodes[acc];
        path[b].push_back(u);
        continue;
      }
      emitted[b].push_back(resampled);
      mr.kind = MARGIN_FINAL; mr.aux = resampled; mr.margin = fm; local.push_back(mr);
      break;
    }
    // what the table will be fed: the compressed rows of the accepted path
    fresh[b].clear();
    for (int node : path[b]) {
      const char* row = (const char*)logits + ((size_t)b * N + node) * (size_t)V * esize;
      std::vector<std::pair<int, double>> items;
      for (int v : topk_ids(row, dtype, V, K)) items.push_back({v, P[node][v]});
      fresh[b].push_back(items);
    }
  }

  void verify(const void* logits) {
    step += 1;  // verification of the tree drafted in step s-1 runs in step s
    std::vector<std::vector<MarginRec>> local(B);
#pragma omp parallel for schedule(dynamic)
    for (int b = 0; b < B; ++b) verify_sequence(b, logits, local[b]);
    for (int b = 0; b < B; ++b) margins.insert(margins.end(), local[b].begin(), local[b].end());
    pending = true;
  }

  // ---- Sec. 4.1: feed one compressed row under every order ----------------
  // `window` holds the tokens that precede the predicted position, oldest
  // first (only its last n_max matter).
  void feed(const std::vector<int>& window, const std::vector<std::pair<int, double>>& items) {
    for (int n = 1; n <= n_max; ++n) {
      if ((int)window.size() < n) continue;
      std::vector<int> key(window.end() - n, window.end());
      double mg;
      merge_entry(table[key], items, K, &mg);
      if (mg < 1e-3) add_margin(MARGIN_MERGE, -1, -1, n, &key, mg);
    }
  }

  // Canonical order: sequence ascending, path position ascending, order
  // ascending; every update of a step precedes every lookup of that step.
  void update() {
    if (!pending) return;
    for (int b = 0; b < B; ++b) {
      std::vector<int> window(tail[b]);
      for (size_t j = 0; j < path[b].size(); ++j) {
        feed(window, fresh[b][j]);
        window.push_back(emitted[b][j]);
      }
      // the sequence grows by the emitted tokens
      if ((int)window.size() > n_max) window.erase(window.begin(), window.end() - n_max);
      tail[b] = window;
      len[b] += (int64_t)emitted[b].size();
    }
    pending = false;
  }

  // ---- Sec. 4.2: draft the next tree of one sequence -----------------------
  void draft_sequence(int b) {
    std::fill(tree[b].begin(), tree[b].end(), -1);
    tree[b][0] = tail[b].empty() ? -1 : tail[b].back();  // the root carries the last token
    for (int u = 0; u < N; ++u) {
      cand_id[b][u].clear();
      cand_phi[b][u].clear();
    }
    for (int u = 0; u < N; ++u) {  // nodes are numbered in breadth-first order
      const int m = (int)children[u].size();
      if (m == 0) continue;
      if (u != 0 && tree[b][u] < 0) continue;  // below an undrafted node nothing is drafted
      // the sequence as it would read if the path root..u were accepted
      std::vector<int> seq(tail[b]);
      std::vector<int> chain;
      for (int w = u; w != 0; w = parent[w]) chain.push_back(tree[b][w]);
      seq.insert(seq.end(), chain.rbegin(), chain.rend());
      const Entry* hit = nullptr;
      for (int n = n_max; n >= 1 && !hit; --n) {  // longest order first, first hit wins
        if ((int)seq.size() < n) continue;
        auto it = table.find(std::vector<int>(seq.end() - n, seq.end()));
        if (it != table.end()) hit = &it->second;
      }
      if (!hit) continue;
      std::vector<int> ids;
      std::vector<double> phis, U;
      for (auto& it : hit->items)
        if (it.second > 0.0) {
          ids.push_back(it.first);
          phis.push_back(it.second);
          U.push_back(uniform_open(random_u24(seed, (uint32_t)(seq_base + b), step, u, SLOT_GUMBEL | (uint32_t)it.first)));
        }
      double mg;
      std::vector<int> chosen = deterministic ? most_probable(ids, phis, m, &mg) : gumbel_top(ids, phis, U, m, &mg);
      if (!chosen.empty()) add_margin(MARGIN_GUMBEL, b, u, (int)chosen.size(), nullptr, mg);
      for (size_t r = 0; r < chosen.size(); ++r) tree[b][children[u][r]] = ids[chosen[r]];
      cand_id[b][u] = ids;
      cand_phi[b][u] = phis;
    }
  }

  void draft() {
    for (int b = 0; b < B; ++b) draft_sequence(b);
  }
};

}  // namespace

// ===========================================================================
// C interface (loaded with ctypes by the tests).
// ===========================================================================
extern "C" {

void so_philox(const uint32_t* ctr, const uint32_t* key, uint32_t* out) { philox4x32_10(ctr, key, out); }

double so_uniform(uint64_t seed, uint32_t b, uint32_t step, uint32_t node, uint32_t slot, int open) {
  const uint32_t u = random_u24(seed, b, step, node, slot);
  return open ? uniform_open(u) : uniform_half_open(u);
}

// One row: log-sum-exp of x/T, the top-k ids, their input values and their probabilities.
void so_row_stats(const void* row, int dtype, int V, double T, int k, double* lse, int32_t* ids,
                  double* values, double* probs, double* p_full) {
  std::vector<double> p;
  softmax_row(row, dtype, V, T, p, lse);
  std::vector<int> top = topk_ids(row, dtype, V, k);
  for (size_t i = 0; i < top.size(); ++i) {
    ids[i] = top[i];
    values[i] = element(row, dtype, top[i]);
    probs[i] = p[top[i]];
  }
  for (int i = (int)top.size(); i < k; ++i) { ids[i] = -1; values[i] = 0.0; probs[i] = 0.0; }
  if (p_full) std::memcpy(p_full, p.data(), sizeof(double) * V);
}

int so_inverse_cdf(const double* w, int V, double U, double* margin) {
  return inverse_cdf(std::vector<double>(w, w + V), U, margin);
}

// Verification of the children of one node with explicit uniforms.
// Returns accepted rank or -1; *resampled gets the resampled token.
int so_verify_children(const double* p, int V, const int32_t* cand_id, const double* cand_phi, int n_cand,
                       const int32_t* child, int n_child, const double* u_acc, double u_final,
                       int32_t* resampled) {
  std::vector<double> pv(p, p + V), phi(cand_phi, cand_phi + n_cand), ua(u_acc, u_acc + n_child);
  std::vector<int> ci(cand_id, cand_id + n_cand), ch(child, child + n_child);
  int res = -1;
  const int acc = verify_children(pv, ci, phi, ch, ua, u_final, &res, nullptr, nullptr);
  *resampled = res;
  return acc;
}

// Deterministic-drafting verification of the children of one node with explicit uniforms.
int so_verify_children_deterministic(const double* p, int V, const int32_t* child, int n_child, const double* u_acc,
                                     double u_final, int32_t* resampled) {
  std::vector<double> pv(p, p + V), ua(u_acc, u_acc + n_child);
  std::vector<int> ch(child, child + n_child);
  int res = -1;
  const int acc = verify_children_deterministic(pv, ch, ua, u_final, &res, nullptr, nullptr);
  *resampled = res;
  return acc;
}

// The m most probable candidates in order; writes the chosen token ids.
int so_most_probable(const int32_t* id, const double* phi, int n, int m, int32_t* chosen) {
  std::vector<int> ids(id, id + n);
  std::vector<double> ph(phi, phi + n);
  std::vector<int> c = most_probable(ids, ph, m, nullptr);
  for (size_t r = 0; r < c.size(); ++r) chosen[r] = ids[c[r]];
  return (int)c.size();
}

// Gumbel-Top-K with explicit uniforms in (0,1); writes the chosen token ids.
int so_gumbel_top(const int32_t* id, const double* phi, const double* U, int n, int m, int32_t* chosen) {
  std::vector<int> ids(id, id + n);
  std::vector<double> ph(phi, phi + n), uu(U, U + n);
  std::vector<int> c = gumbel_top(ids, ph, uu, m, nullptr);
  for (size_t r = 0; r < c.size(); ++r) chosen[r] = ids[c[r]];
  return (int)c.size();
}

void* so_create(int B, int N, int V, int topk, int order_max, int dtype, double T, uint64_t seed,
                const int32_t* parent) {
  Oracle* o = new Oracle;
  o->B = B; o->N = N; o->V = V; o->K = topk; o->n_max = order_max; o->dtype = dtype; o->T = T; o->seed = seed;
  o->parent.assign(parent, parent + N);
  o->depth.assign(N, 0);
  o->children.assign(N, {});
  for (int u = 1; u < N; ++u) {
    o->children[parent[u]].push_back(u);
    o->depth[u] = o->depth[parent[u]] + 1;
    o->D = std::max(o->D, o->depth[u]);
  }
  o->tail.assign(B, {});
  o->len.assign(B, 0);
  o->tree.assign(B, std::vector<int>(N, -1));
  o->cand_id.assign(B, std::vector<std::vector<int>>(N));
  o->cand_phi.assign(B, std::vector<std::vector<double>>(N));
  o->emitted.assign(B, {});
  o->path.assign(B, {});
  o->fresh.assign(B, {});
  return o;
}
void so_set_deterministic(void* h, int on) { ((Oracle*)h)->deterministic = on ? 1 : 0; }
// A batch split over several contexts: this context's sequence b is sequence seq_base + b of the batch.
void so_set_seq_base(void* h, int base) { ((Oracle*)h)->seq_base = base; }
void so_destroy(void* h) { delete (Oracle*)h; }
int so_depth(void* h) { return ((Oracle*)h)->D; }

// Start (or restart) the sequences: tail[b] = last tokens of the prompt, -1
// padded at the front.  The tables are kept (Sec. 5.1: the module persists
// across trajectories).  No tree is drafted yet.
void so_reset_sequences(void* h, const int32_t* tail, const int64_t* len) {
  Oracle* o = (Oracle*)h;
  for (int b = 0; b < o->B; ++b) {
    o->tail[b].clear();
    for (int i = 0; i < o->n_max; ++i)
      if (tail[b * o->n_max + i] >= 0) o->tail[b].push_back(tail[b * o->n_max + i]);
      else o->tail[b].clear();  // a gap: only the tokens after it form contexts
    o->len[b] = len[b];
    std::fill(o->tree[b].begin(), o->tree[b].end(), -1);
    o->tree[b][0] = o->tail[b].empty() ? -1 : o->tail[b].back();
    for (int u = 0; u < o->N; ++u) { o->cand_id[b][u].clear(); o->cand_phi[b][u].clear(); }
  }
  o->pending = false;
}

static void export_verify(Oracle* o, int32_t* emitted, int32_t* n_emitted) {
  const int W = o->D + 1;
  for (int b = 0; b < o->B; ++b) {
    n_emitted[b] = (int32_t)o->emitted[b].size();
    for (int j = 0; j < W; ++j) emitted[b * W + j] = j < (int)o->emitted[b].size() ? o->emitted[b][j] : -1;
  }
}
static void export_tree(Oracle* o, int32_t* tree) {
  for (int b = 0; b < o->B; ++b)
    for (int u = 0; u < o->N; ++u) tree[b * o->N + u] = o->tree[b][u];
}

void so_verify(void* h, const void* logits, int32_t* emitted, int32_t* n_emitted) {
  Oracle* o = (Oracle*)h;
  o->verify(logits);
  export_verify(o, emitted, n_emitted);
}
void so_update(void* h) { ((Oracle*)h)->update(); }
void so_draft(void* h, int32_t* tree) {
  Oracle* o = (Oracle*)h;
  o->draft();
  export_tree(o, tree);
}
void so_step(void* h, const void* logits, int32_t* emitted, int32_t* n_emitted, int32_t* tree) {
  Oracle* o = (Oracle*)h;
  o->verify(logits);
  export_verify(o, emitted, n_emitted);
  o->update();
  o->draft();
  export_tree(o, tree);
}

// Accepted path of the last verification: node indices, -1 padded, [B, D+1].
void so_get_path(void* h, int32_t* path) {
  Oracle* o = (Oracle*)h;
  const int W = o->D + 1;
  for (int b = 0; b < o->B; ++b)
    for (int j = 0; j < W; ++j) path[b * W + j] = j < (int)o->path[b].size() ? o->path[b][j] : -1;
}

// Bulk feed: row i carries a context window (last order_max tokens before the
// predicted position, -1 padded at the front) and a compressed distribution;
// rows are applied in index order, each under every order it is long enough for.
void so_update_bulk(void* h, const int32_t* ctx, const int32_t* ids, const float* probs, int64_t M) {
  Oracle* o = (Oracle*)h;
  for (int64_t i = 0; i < M; ++i) {
    std::vector<int> window;
    for (int t = 0; t < o->n_max; ++t)
      if (ctx[i * o->n_max + t] >= 0) window.push_back(ctx[i * o->n_max + t]);
      else window.clear();  // a gap: only the tokens after it form contexts
    std::vector<std::pair<int, double>> items;
    for (int t = 0; t < o->K; ++t)
      if (ids[i * o->K + t] >= 0) items.push_back({ids[i * o->K + t], (double)probs[i * o->K + t]});
    o->feed(window, items);
  }
}

int64_t so_table_size(void* h) { return (int64_t)((Oracle*)h)->table.size(); }
// Entries in map order.  keys: [M,4] padded with -1 at the front.
void so_table_dump(void* h, int32_t* keys, uint32_t* counts, int32_t* n_items, int32_t* ids, double* probs) {
  Oracle* o = (Oracle*)h;
  int64_t i = 0;
  for (auto& kv : o->table) {
    for (int t = 0; t < 4; ++t) keys[i * 4 + t] = -1;
    for (size_t t = 0; t < kv.first.size(); ++t) keys[i * 4 + 4 - kv.first.size() + t] = kv.first[t];
    counts[i] = kv.second.count;
    n_items[i] = (int32_t)kv.second.items.size();
    for (int t = 0; t < o->K; ++t) {
      const bool have = t < (int)kv.second.items.size();
      ids[i * o->K + t] = have ? kv.second.items[t].first : -1;
      probs[i * o->K + t] = have ? kv.second.items[t].second : 0.0;
    }
    ++i;
  }
}
// Look one context up (n tokens, oldest first).  Returns the item count or -1.
int so_table_get(void* h, const int32_t* key, int n, uint32_t* count, int32_t* ids, double* probs) {
  Oracle* o = (Oracle*)h;
  auto it = o->table.find(std::vector<int>(key, key + n));
  if (it == o->table.end()) return -1;
  *count = it->second.count;
  for (size_t t = 0; t < it->second.items.size(); ++t) {
    ids[t] = it->second.items[t].first;
    probs[t] = it->second.items[t].second;
  }
  return (int)it->second.items.size();
}

// Sequence state: tails [B,order_max] (-1 padded front), lengths, tree tokens
// [B,N], candidate snapshots [B,N,K] (ids -1 padded), step counter.
void so_get_state(void* h, int32_t* tail, int64_t* len, int32_t* tree, int32_t* cand_n, int32_t* cand_id,
                  double* cand_phi, uint32_t* step) {
  Oracle* o = (Oracle*)h;
  for (int b = 0; b < o->B; ++b) {
    const int have = (int)o->tail[b].size();
    for (int i = 0; i < o->n_max; ++i) {
      const int src = i - (o->n_max - have);
      tail[b * o->n_max + i] = src >= 0 ? o->tail[b][src] : -1;
    }
    len[b] = o->len[b];
    for (int u = 0; u < o->N; ++u) {
      tree[b * o->N + u] = o->tree[b][u];
      const int n = (int)o->cand_id[b][u].size();
      cand_n[b * o->N + u] = n;
      for (int t = 0; t < o->K; ++t) {
        cand_id[((size_t)b * o->N + u) * o->K + t] = t < n ? o->cand_id[b][u][t] : -1;
        cand_phi[((size_t)b * o->N + u) * o->K + t] = t < n ? o->cand_phi[b][u][t] : 0.0;
      }
    }
  }
  *step = o->step;
}

// Compressed rows of the last verification's accepted path: [B, D+1, K].
void so_get_fresh(void* h, int32_t* ids, double* probs) {
  Oracle* o = (Oracle*)h;
  const int W = o->D + 1;
  for (int b = 0; b < o->B; ++b)
    for (int j = 0; j < W; ++j)
      for (int t = 0; t < o->K; ++t) {
        const bool have = j < (int)o->fresh[b].size() && t < (int)o->fresh[b][j].size();
        ids[((size_t)b * W + j) * o->K + t] = have ? o->fresh[b][j][t].first : -1;
        probs[((size_t)b * W + j) * o->K + t] = have ? o->fresh[b][j][t].second : 0.0;
      }
}

int64_t so_margin_count(void* h) { return (int64_t)((Oracle*)h)->margins.size(); }
// Copies and clears the margin log.  Record layout: 8 int32 (kind, b, node,
// aux, key[4]) and one double.
void so_margin_take(void* h, int32_t* ints, double* margin) {
  Oracle* o = (Oracle*)h;
  for (size_t i = 0; i < o->margins.size(); ++i) {
    const MarginRec& r = o->margins[i];
    ints[i * 8 + 0] = r.kind; ints[i * 8 + 1] = r.b; ints[i * 8 + 2] = r.node; ints[i * 8 + 3] = r.aux;
    for (int t = 0; t < 4; ++t) ints[i * 8 + 4 + t] = r.key[t];
    margin[i] = r.margin;
  }
  o->margins.clear();
}

}  // extern "C"
