// Verification walk (paper Sec. 3.2 speculative sampling, applied to the tree
// drafted in Sec. 4.2).  One thread block per sequence.
//
//   phase 1 (all warps)  normaliser of every row of the sequence from the chunk
//                        pairs, and the target probability of every drafted
//                        candidate (a handful of gathered logits per node);
//   phase 2 (thread 0)   the walk: children in draft order, accept iff
//                        U * q(x) < p~(x); on rejection p~ <- norm(max(0, p~ - q)),
//                        x leaves q; off the candidate list p~ is the target scaled
//                        by a running factor, so the residual needs no pass over V;
//   phase 3 (all warps)  the one sampled token: inverse CDF in token order, coarse
//                        over chunk masses, then exact inside one 1024-entry chunk;
//   phase 4              the accepted rows compressed to top-k probabilities (the exact
//                        top-k is finished here, from the few chunks whose maximum
//                        can reach it) and the context windows for the N-gram
//                        update; sequence tails advance.
// Decisions are taken in double precision on top of the row pass's fp32 chunk sums.
#pragma once
#include "common.cuh"
#include "row_pass.cuh"

namespace stand {

constexpr int K2_THREADS = 256;

struct VerifyParams {
  const void* logits;
  int dtype, B, N, V, K, n_max, D, n_chunks;
  float c;
  unsigned long long seed;
  uint32_t step;
  const int* first_child;  // [N]
  const int* n_children;   // [N]
  const float2* pairs;     // [B*N, n_chunks] (sum, chunk max) from the row pass
  int* tail;               // [B, n_max]   advanced here
  long long* len;          // [B]          advanced here
  const int* tree;         // [B, N]
  const int* cand_n;       // [B, N]
  const int* cand_id;      // [B, N, K]
  const float* cand_phi;   // [B, N, K]
  int* emitted_user;       // [B, D+1] or null
  int* n_emitted_user;     // [B] or null
  int* emitted;            // [B, D+1]
  int* n_path;             // [B]
  int* path;               // [B, D+1]
  int* rec_ctx;            // [B, D+1, n_max]
  int* rec_ids;            // [B, D+1, K]
  float* rec_p;            // [B, D+1, K]
  unsigned long long* stats;
};

// Exclusive block scan of one double per thread (256 threads); returns the
// exclusive prefix, *total gets the block total.
__device__ __forceinline__ double block_scan_excl(double v, double* s_warp, double* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  double inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const double t = __shfl_up_sync(FULL, inc, o);
    if (lane >= o) inc += t;
  }
  __syncthreads();  // s_warp may still be read from a previous scan
  if (lane == 31) s_warp[warp] = inc;
  __syncthreads();
  double base = 0.0, tot = 0.0;
#pragma unroll
  for (int w = 0; w < K2_THREADS / 32; ++w) {
    const double t = s_warp[w];
    if (w < warp) base += t;
    tot += t;
  }
  *total = tot;
  return base + inc - v;
}

__global__ void __launch_bounds__(K2_THREADS) verify_kernel(const VerifyParams p) {
  __shared__ float s_off[NODES_MAX];
  __shared__ double s_Z[NODES_MAX];
  __shared__ double s_p[NODES_MAX][KMAX];  // target probability of candidate i of node u
  __shared__ double s_scan[K2_THREADS / 32];
  __shared__ int s_path[DEPTH_MAX + 1];
  __shared__ int s_emit[DEPTH_MAX + 1];
  __shared__ int s_m;         // accepted children (path has s_m + 1 nodes)
  __shared__ int s_nsup;      // candidates carrying an explicit residual value at the stop node
  __shared__ int s_sup_id[KMAX];
  __shared__ double s_sup_pt[KMAX];  // residual target on the candidates
  __shared__ double s_sup_p[KMAX];   // original target on the candidates
  __shared__ double s_scale;         // residual target off the candidates = scale * target
  __shared__ int s_pick, s_pick_last;
  __shared__ double s_base;
  __shared__ uint2 s_buf[K2_THREADS / 32][CAND_CAP];  // per-warp candidate buffers of the top-k selection
  __shared__ int s_cnt[K2_THREADS / 32];

  const int b = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int N = p.N, K = p.K;
  const double cd = (double)p.c;

  // ---- phase 1 -----------------------------------------------------------
  for (int u = warp; u < N; u += K2_THREADS / 32) {
    const long long row = (long long)b * N + u;
    const RowNorm nm = row_normaliser(p.pairs + row * p.n_chunks, p.n_chunks, p.c, lane);
    if (lane == 0) { s_off[u] = nm.off; s_Z[u] = nm.Z; }
    const int nc = p.cand_n[row];
    if (lane < nc) {
      const int id = p.cand_id[row * K + lane];
      const float x = load_logit(p.logits, p.dtype, row * (long long)p.V + id);
      s_p[u][lane] = exp2((double)x * cd - (double)nm.off) / nm.Z;
    }
  }
  __syncthreads();

  // ---- phase 2: the walk -----------------------------------------------------
  if (tid == 0) {
    int u = 0, m = 0;
    s_path[0] = 0;
    int nsup = 0;
    double scale = 1.0;
    for (;;) {
      const long long row = (long long)b * N + u;
      const int fc = p.first_child[u], nch = p.n_children[u];
      int drafted = 0;
      while (drafted < nch && p.tree[(long long)b * N + fc + drafted] >= 0) ++drafted;
      nsup = 0;
      scale = 1.0;
      if (drafted == 0) break;  // nothing drafted below u: sample from its target
      const int nc = p.cand_n[row];
      double q[KMAX], pt[KMAX];
      int cid[KMAX];
      double phis = 0.0;
      for (int i = 0; i < nc; ++i) {
        cid[i] = p.cand_id[row * K + i];
        q[i] = (double)p.cand_phi[row * K + i];
        phis += q[i];
        pt[i] = s_p[u][i];
      }
      for (int i = 0; i < nc; ++i) q[i] /= phis;
      int accepted = -1;
      for (int j = 0; j < drafted; ++j) {
        const int x = p.tree[(long long)b * N + fc + j];
        int ix = -1;
        for (int i = 0; i < nc; ++i)
          if (cid[i] == x) ix = i;
        const double U = (double)philox_u24(p.seed, b, p.step, u, (uint32_t)j) * (1.0 / 16777216.0);
        if (ix < 0 || U * q[ix] < pt[ix]) { accepted = j; break; }
        // rejected: residual target, x leaves the draft distribution
        double overlap = 0.0;
        for (int i = 0; i < nc; ++i) overlap += fmin(pt[i], q[i]);
        const double zr = 1.0 - overlap;
        for (int i = 0; i < nc; ++i) pt[i] = fmax(0.0, pt[i] - q[i]) / zr;
        scale /= zr;
        q[ix] = 0.0;
        double qs = 0.0;
        for (int i = 0; i < nc; ++i) qs += q[i];
        if (qs > 0.0)
          for (int i = 0; i < nc; ++i) q[i] /= qs;
      }
      if (accepted >= 0) {
        s_emit[m] = p.tree[(long long)b * N + fc + accepted];
        u = fc + accepted;
        ++m;
        s_path[m] = u;
        continue;
      }
      nsup = nc;
      for (int i = 0; i < nc; ++i) { s_sup_id[i] = cid[i]; s_sup_pt[i] = pt[i]; s_sup_p[i] = s_p[u][i]; }
      break;
    }
    s_m = m;
    s_nsup = nsup;
    s_scale = scale;
    s_pick = 0x7FFFFFFF;
    s_pick_last = -1;
  }
  __syncthreads();

  // ---- phase 3: one token by inverse CDF at the stop node ----------------------
  const int m = s_m;
  const int us = s_path[m];
  const long long rows = (long long)b * N + us;
  const int nsup = s_nsup;
  const double scale = s_scale;
  const float off = s_off[us];
  const double Z = s_Z[us];
  const double U = (double)philox_u24(p.seed, b, p.step, us, SLOT_FINAL) * (1.0 / 16777216.0);

  // coarse: mass of every chunk; thread t owns `per` consecutive chunks
  const int per = (p.n_chunks + K2_THREADS - 1) / K2_THREADS;  // <= 4 for V <= 2^20
  double cm[4];
  double mine = 0.0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    cm[i] = 0.0;
    const int ch = tid * per + i;
    if (i < per && ch < p.n_chunks) {
      const float2 pr = p.pairs[rows * p.n_chunks + ch];
      double mass = scale * (chunk_mass(pr, p.c, off) / Z);
      for (int s = 0; s < nsup; ++s)
        if (s_sup_id[s] / CHUNK == ch) mass += s_sup_pt[s] - scale * s_sup_p[s];
      cm[i] = fmax(mass, 0.0);
      mine += cm[i];
    }
  }
  double W;
  const double base = block_scan_excl(mine, s_scan, &W);
  const double target = U * W;
  {
    double cum = base;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int ch = tid * per + i;
      if (i < per && ch < p.n_chunks) {
        if (cm[i] > 0.0) {
          atomicMax(&s_pick_last, ch);
          if (target < cum + cm[i]) atomicMin(&s_pick, ch);
        }
        cum += cm[i];
      }
    }
  }
  __syncthreads();
  int chs = s_pick;
  if (chs == 0x7FFFFFFF) chs = s_pick_last;  // rounding pushed the target past the end
  if (chs < 0) chs = 0;
  {
    // mass before the chosen chunk
    const int owner = chs / per;
    if (tid == owner) {
      double cum = base;
      for (int i = 0; i < chs - owner * per; ++i) cum += cm[i];
      s_base = cum;
    }
  }
  __syncthreads();
  if (tid == 0) { s_pick = 0x7FFFFFFF; s_pick_last = -1; }
  // exact inside the chunk: thread t owns 4 consecutive entries
  double w[4];
  double wsum = 0.0;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const int v = chs * CHUNK + tid * 4 + e;
    w[e] = 0.0;
    if (v < p.V) {
      int s_hit = -1;
      for (int s = 0; s < nsup; ++s)
        if (s_sup_id[s] == v) s_hit = s;
      if (s_hit >= 0) w[e] = s_sup_pt[s_hit];
      else {
        const float x = load_logit(p.logits, p.dtype, rows * (long long)p.V + v);
        w[e] = scale * (exp2((double)x * cd - (double)off) / Z);
      }
    }
    wsum += w[e];
  }
  double tot;
  const double fb = block_scan_excl(wsum, s_scan, &tot);
  {
    double cum = s_base + fb;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int v = chs * CHUNK + tid * 4 + e;
      if (w[e] > 0.0) {
        atomicMax(&s_pick_last, v);
        if (target < cum + w[e]) atomicMin(&s_pick, v);
      }
      cum += w[e];
    }
  }
  __syncthreads();

  // ---- phase 4: outputs --------------------------------------------------------
  const int W1 = p.D + 1;
  if (tid == 0) {
    int y = s_pick;
    if (y == 0x7FFFFFFF) y = s_pick_last;
    if (y < 0) y = 0;
    s_emit[m] = y;
    // context windows of the accepted rows, then the advanced tail
    int win[ORDER_MAX];
    for (int i = 0; i < p.n_max; ++i) win[i] = p.tail[b * p.n_max + i];
    for (int j = 0; j <= m; ++j) {
      for (int i = 0; i < p.n_max; ++i) p.rec_ctx[((long long)b * W1 + j) * p.n_max + i] = win[i];
      for (int i = 0; i + 1 < p.n_max; ++i) win[i] = win[i + 1];
      win[p.n_max - 1] = s_emit[j];
    }
    for (int i = 0; i < p.n_max; ++i) p.tail[b * p.n_max + i] = win[i];
    p.len[b] += m + 1;
    p.n_path[b] = m + 1;
    if (p.n_emitted_user) p.n_emitted_user[b] = m + 1;
    atomicAdd(&p.stats[ST_EMITTED], (unsigned long long)(m + 1));
    if (b == 0) atomicAdd(&p.stats[ST_STEPS], 1ull);
  }
  __syncthreads();
  if (tid < W1) {
    const int e = tid <= m ? s_emit[tid] : -1;
    p.emitted[b * W1 + tid] = e;
    if (p.emitted_user) p.emitted_user[b * W1 + tid] = e;
    p.path[b * W1 + tid] = tid <= m ? s_path[tid] : -1;
  }
  // compressed rows of the accepted path: the exact top-k of each row, as probabilities
  for (int j = warp; j <= m; j += K2_THREADS / 32) {
    const int u = s_path[j];
    const long long row = (long long)b * N + u;
    const float o = s_off[u];
    const double z = s_Z[u];
    const int n = row_topk_warp(p.logits, p.dtype, row, p.V, p.pairs + row * p.n_chunks, p.n_chunks, K, s_buf[warp],
                                &s_cnt[warp], lane);
    if (lane < K) {
      const long long at = ((long long)b * W1 + j) * K + lane;
      if (lane < n) {
        const uint2 e = s_buf[warp][lane];
        p.rec_ids[at] = (int)e.y;
        p.rec_p[at] = (float)(exp2((double)__uint_as_float(e.x) * cd - (double)o) / z);
      } else {
        p.rec_ids[at] = -1;
        p.rec_p[at] = 0.0f;
      }
    }
    __syncwarp();
  }
}

}  // namespace stand
