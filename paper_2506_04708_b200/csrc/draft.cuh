// Stochastic tree drafting (paper Sec. 4.2).  One thread block per sequence walks
// the static topology level by level; one warp per parent node:
//   - the contexts of order n_max..1 of the would-be sequence (tail + path tokens)
//     are probed at once, 8 lanes per order; the longest hit wins ("first
//     successful match", longest first);
//   - the hit's candidates (id, phi) sit one per lane; Gumbel-Top-K: each lane
//     forms g = log(phi) - log(-log U) with its own Philox uniform (keyed by the
//     token id) and its rank among the candidates; rank r < #children becomes the
//     child of draft rank r;
//   - the candidate list is kept as the draft distribution for the next verification.
#pragma once
#include "common.cuh"
#include "table.cuh"

namespace stand {

constexpr int K4_THREADS = 256;

struct DraftParams {
  const Slot* table;
  unsigned long long mask;
  int max_probe, B, N, K, n_max, D, V;
  unsigned long long seed;
  uint32_t step;
  const int* parent;       // [N]
  const int* first_child;  // [N]
  const int* n_children;   // [N]
  const int* level_start;  // [D+2]
  const int* tail;         // [B, n_max]
  int* tree;               // [B, N]
  int* tree_user;          // [B, N] or null
  int* cand_n;             // [B, N]
  int* cand_id;            // [B, N, K]
  float* cand_phi;         // [B, N, K]
  unsigned long long* stats;
  int deterministic;       // != 0: the children are the most probable candidates, no noise
  int seq_base;            // global index of sequence 0 (random-number counters use seq_base + b)
};

// Rank of this lane's candidate by g = log(phi) - log(-log U) in double precision (larger first, equal
// scores by lower id).  Called by all lanes of a warp; kept out of line: it runs for about one node in a hundred.
__device__ __noinline__ int gumbel_rank_double(bool valid, int id, float phi, uint32_t u24) {
  double g = 0.0;
  if (valid) {
    const double U = ((double)u24 + 0.5) * (1.0 / 16777216.0);
    g = log((double)phi) - log(-log(U));
  }
  int rank = 0;
  for (int j = 0; j < KMAX; ++j) {
    const double gj = __shfl_sync(FULL, g, j);
    const int idj = __shfl_sync(FULL, id, j);
    const bool vj = __shfl_sync(FULL, (int)valid, j) != 0;
    if (vj && (gj > g || (gj == g && idj < id))) ++rank;
  }
  return rank;
}

// Shared memory of one drafting block of NT threads.
template <int NT>
struct DraftShared {
  int tok[NODES_MAX], parent[NODES_MAX], fc[NODES_MAX], nch[NODES_MAX];
  int tail[ORDER_MAX], level[DEPTH_MAX + 2];
  Slot slot[NT / 32];        // per warp: the slot that won the lookup
  float g[NT / 32][KMAX];    // per warp: the candidates' perturbed scores and ids
  int gid[NT / 32][KMAX];
};

// The static topology into shared memory, and every node marked undrafted, by `nt` threads of the block numbered
// t = 0 .. nt - 1 (coalesced loads; the level loop touches shared memory only).  The topology never changes after
// stand_init, so this may run before any wait.
template <int NT>
__device__ __forceinline__ void draft_stage_topology(const DraftParams& p, DraftShared<NT>& sh, const int t, const int nt) {
  for (int u = t; u < p.N; u += nt) {
    sh.tok[u] = -1;
    sh.parent[u] = p.parent[u];
    sh.fc[u] = p.first_child[u];
    sh.nch[u] = p.n_children[u];
  }
  for (int i = t; i <= p.D + 1; i += nt) sh.level[i] = p.level_start[i];
}

// The next tree of sequence b by one block of NT threads (one warp per parent node of a level: trees with more
// than NT / 32 parents on a level take several rounds there).  WAIT: stop (griddepcontrol.wait) before the first
// read of what the previous kernel wrote; false when the caller has already ordered itself after that kernel.
// STAGED: the caller has filled sh's topology (draft_stage_topology) and sh.tail (the sequence's last tokens) and
// synchronised the block.
template <bool WAIT, int NT, bool STAGED>
__device__ __forceinline__ void draft_block(const DraftParams& p, const int b, DraftShared<NT>& sh) {
  int (&s_tok)[NODES_MAX] = sh.tok;
  int (&s_parent)[NODES_MAX] = sh.parent;
  int (&s_fc)[NODES_MAX] = sh.fc;
  int (&s_nch)[NODES_MAX] = sh.nch;
  int (&s_tail)[ORDER_MAX] = sh.tail;
  int (&s_level)[DEPTH_MAX + 2] = sh.level;
  Slot (&s_slot)[NT / 32] = sh.slot;
  float (&s_g)[NT / 32][KMAX] = sh.g;
  int (&s_gid)[NT / 32][KMAX] = sh.gid;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int N = p.N, K = p.K, n_max = p.n_max;
  pdl_trigger();
  if (!STAGED) {
    draft_stage_topology<NT>(p, sh, tid, NT);
    if (WAIT) pdl_wait();  // tails come from the verification, the table from the update
    if (tid < n_max) s_tail[tid] = p.tail[b * n_max + tid];
    __syncthreads();
  }
  if (tid == 0) s_tok[0] = s_tail[n_max - 1];  // the root carries the last token
  __syncthreads();

  for (int d = 0; d < p.D; ++d) {
    const int l0 = s_level[d], l1 = s_level[d + 1];
    for (int u = l0 + warp; u < l1; u += NT / 32) {
      const int m = s_nch[u];
      const long long row = (long long)b * N + u;
      if (m == 0) { if (lane == 0) p.cand_n[row] = 0; continue; }
      const bool drafted = u == 0 || s_tok[u] >= 0;
      if (!drafted) { if (lane == 0) p.cand_n[row] = 0; continue; }  // nothing is drafted below an undrafted node
      // last n_max tokens of the sequence as it reads if the path root..u is accepted
      int win[ORDER_MAX];
      {
        int filled = 0, w = u;
        while (w != 0 && filled < n_max) { win[n_max - 1 - filled] = s_tok[w]; ++filled; w = s_parent[w]; }
        for (int i = n_max - 1; filled < n_max; --i, ++filled) win[n_max - 1 - filled] = s_tail[i];
      }
      // one group of 8 lanes per order: all orders are probed at once
      const int grp = lane / GROUP;
      int key[4] = {-1, -1, -1, -1};
      bool ok = grp < n_max;
      if (ok) {
        const int n = grp + 1;
        for (int i = 0; i < n; ++i) {
          const int t = win[n_max - n + i];
          if (t < 0 || t >= p.V) ok = false;
          key[4 - n + i] = t;
        }
      }
      uint4 line[8];
      int src_lane;
      uint32_t slot = find_slot_group_fetch(p.table, p.mask, p.max_probe, key, ok, line, &src_lane);
      const unsigned found = __ballot_sync(FULL, slot != NO_SLOT);
      unsigned hits = 0;  // bit n-1: order n matched
      for (int gq = 0; gq < 32 / GROUP; ++gq)
        if ((found >> (gq * GROUP)) & 1u) hits |= 1u << gq;
      if (lane == 0) {
        atomicAdd(&p.stats[ST_LOOKUPS], 1ull);
        if (hits) atomicAdd(&p.stats[ST_HIT0 + (31 - __clz(hits))], 1ull);
      }
      if (hits == 0) { if (lane == 0) p.cand_n[row] = 0; continue; }
      const int winner = 31 - __clz(hits);  // the longest order that matched
      // the lane that probed the winning slot already holds its contents: hand them to the warp
      src_lane = __shfl_sync(FULL, src_lane, winner * GROUP);
      uint4* img = reinterpret_cast<uint4*>(&s_slot[warp]);
      if (lane == src_lane) {
#pragma unroll
        for (int t = 0; t < 8; ++t) img[t] = line[t];
      }
      __syncwarp();
      const Slot* s = &s_slot[warp];
      const int n_items = (int)s->n_items;
      int id = -1;
      float phi = 0.0f;
      if (lane < n_items && lane < K) { id = s->ids[lane]; phi = s->probs[lane]; }
      __syncwarp();
      const bool valid = id >= 0 && phi > 0.0f;
      // Perturbed scores in single precision first; they decide the order whenever every pair of
      // candidates is further apart than single precision can blur (1e-3 against errors of a few 1e-6).
      // Otherwise the scores are formed again in double precision.
      const uint32_t u24 = (valid && !p.deterministic) ? philox_u24(p.seed, (uint32_t)(p.seq_base + b), p.step, u, SLOT_GUMBEL | (uint32_t)id) : 0u;
      float gf = 0.0f;
      if (valid && p.deterministic) gf = phi;  // deterministic drafting (Sec. 3.2): rank by the stored probability itself
      else if (valid) {
        // L = -log U with U = (u24 + 1/2) / 2^24.  Below one half U is exact in fp32 and the hardware
        // logarithm serves; above, L = 2 atanh(v / (2 - v)) with the exact complement v = 1 - U <= 1/2.
        const float lo = -__logf(((float)u24 + 0.5f) * (1.0f / 16777216.0f));
        const float v = ((float)(16777216u - u24) - 0.5f) * (1.0f / 16777216.0f);
        const float t = __fdividef(v, 2.0f - v), t2 = t * t;
        const float hi = 2.0f * t * fmaf(t2, fmaf(t2, fmaf(t2, fmaf(t2, fmaf(t2, 1.0f / 11.0f, 1.0f / 9.0f), 1.0f / 7.0f), 0.2f), 1.0f / 3.0f), 1.0f);
        const float L = u24 < (1u << 23) ? lo : hi;
        gf = __logf(phi) - __logf(L);
      }
      // every lane reads the other scores from shared memory (independent loads; a chain of shuffles
      // would cost its full latency per candidate)
      if (lane < KMAX) { s_g[warp][lane] = gf; s_gid[warp][lane] = valid ? id : -1; }
      __syncwarp();
      int rank = 0;
      bool close = false;
      {
        // all scores are read first, then compared without short-circuit operators (those compile to a divergent
        // branch per candidate); lanes without a candidate compute along and are masked at the end
        float gj[KMAX];
        int idj[KMAX];
#pragma unroll
        for (int j = 0; j < KMAX; ++j) { gj[j] = s_g[warp][j]; idj[j] = s_gid[warp][j]; }
        int near = 0;
#pragma unroll
        for (int j = 0; j < KMAX; ++j) {
          const int live = idj[j] >= 0;
          rank += live & ((gj[j] > gf) | ((gj[j] == gf) & (idj[j] < id)));
          near |= live & (j != lane) & (fabsf(gj[j] - gf) < 1e-3f);
        }
        close = valid && near != 0;
        if (!valid) rank = 0;
      }
      __syncwarp();
      if (!p.deterministic && __any_sync(FULL, valid && close)) rank = gumbel_rank_double(valid, id, phi, u24);
      if (valid && rank < m) s_tok[s_fc[u] + rank] = id;
      const unsigned vmask = __ballot_sync(FULL, valid);
      if (valid) {
        const int pos = __popc(vmask & ((1u << lane) - 1u));
        p.cand_id[row * K + pos] = id;
        p.cand_phi[row * K + pos] = phi;
      }
      if (lane == 0) p.cand_n[row] = __popc(vmask);
    }
    __syncthreads();
  }
  // nodes of the deepest level have no children
  for (int u = s_level[p.D] + tid; u < N; u += NT) p.cand_n[(long long)b * N + u] = 0;
  for (int u = tid; u < N; u += NT) {
    const int t = s_tok[u];
    p.tree[(long long)b * N + u] = t;
    if (p.tree_user) p.tree_user[(long long)b * N + u] = t;
  }
}

__global__ void __launch_bounds__(K4_THREADS) draft_kernel(const DraftParams p) {
  __shared__ DraftShared<K4_THREADS> sh;
  draft_block<true, K4_THREADS, false>(p, (int)blockIdx.x, sh);
}

}  // namespace stand
