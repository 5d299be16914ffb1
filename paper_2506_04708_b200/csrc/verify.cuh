// Verification walk (paper Sec. 3.2 speculative sampling, applied to the tree
// drafted in Sec. 4.2).  One thread block per sequence.
//
//   phase 0 (all warps)  the sequence's tree, candidate lists and topology are staged in
//                        shared memory with one round of coalesced loads;
//   phase 1 (all warps)  normaliser of every row of the sequence from the chunk
//                        pairs (8 lanes per row), and the target probability of every
//                        drafted candidate (one round of gathered logits);
//   phase 2 (warp 0)     the walk: children in draft order, accept iff
//                        U * q(x) < p~(x); on rejection p~ <- norm(max(0, p~ - q)),
//                        x leaves q; off the candidate list p~ is the target scaled
//                        by a running factor, so the residual needs no pass over V;
//   phase 3 (all warps)  the one sampled token: inverse CDF in token order, coarse
//                        over chunk masses, then exact inside one 1024-entry chunk;
//   phase 4              the accepted rows compressed to top-k probabilities (the exact
//                        top-k is finished here, from the few chunks whose maximum
//                        can reach it) and the context windows for the N-gram
//                        update; sequence tails advance.  Optionally stage 1 of the
//                        table update (context -> slot) for this sequence's records.
// Decisions are taken in double precision on top of the row pass's fp32 chunk sums.
#pragma once
#include "common.cuh"
#include "row_pass.cuh"
#include "table.cuh"

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
  unsigned long long* node_accepts;  // [N] how often each node lay on an accepted path
  int deterministic;       // != 0: deterministic drafting (every drafted token is a one-hot draft)
  int seq_base;            // global index of sequence 0 (random-number counters use seq_base + b)
  int fuse_locate;         // != 0: also run stage 1 of the N-gram update for this sequence's records
  UpdateParams upd;        // used when fuse_locate is set
};

// Barrier of the K2_THREADS threads that verify one sequence.  BAR 0: they are the whole block (the block
// barrier); BAR > 0: they are the first K2_THREADS threads of a wider block and meet on that named barrier.
template <int BAR>
__device__ __forceinline__ void verify_sync() {
  if (BAR == 0) __syncthreads();
  else asm volatile("bar.sync %0, %1;" ::"n"(BAR), "n"(K2_THREADS) : "memory");
}

// Exclusive scan of one double per thread over the K2_THREADS verifying threads; returns the exclusive prefix,
// *total gets the sum.
template <int BAR>
__device__ __forceinline__ double block_scan_excl(double v, double* s_warp, double* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  double inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const double t = __shfl_up_sync(FULL, inc, o);
    if (lane >= o) inc += t;
  }
  verify_sync<BAR>();  // s_warp may still be read from a previous scan
  if (lane == 31) s_warp[warp] = inc;
  verify_sync<BAR>();
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

constexpr int TOPK_ROWS = 4;       // path rows whose top-k is selected together
constexpr int TOPK_ITEMS = 1024;   // (row, chunk) work items per group of rows
constexpr int ROW_LANES = 8;       // lanes that share one row in the normaliser phase

// Dynamic shared memory of the verification kernel for a tree of N nodes.
inline size_t verify_smem_bytes(int N) {
  return (size_t)N * (KMAX * (sizeof(double) + sizeof(float) + sizeof(int)) + sizeof(double) + sizeof(float) + 4 * sizeof(int));
}

// Pushes the entries of chunk `ch` of a row that reach `floor` into buf (capacity cap; *cnt keeps
// counting past it, which the caller reads as overflow).  Called by all lanes of a warp.
__device__ __forceinline__ void push_chunk_candidates(const void* logits, int dtype, long long row, int V, int ch,
                                                      float floor, bool wide, uint2* buf, int* cnt, int cap, int lane) {
#pragma unroll
  for (int step = 0; step < 4; ++step) {
    float f[8];
    int idx[8];
    if (wide && dtype == 1) {
      const int i0 = ch * CHUNK + step * 256 + lane * 8;
      uint4 d = make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);
      if (i0 < V) d = __ldg(reinterpret_cast<const uint4*>((const unsigned short*)logits + row * (long long)V + i0));
      ElemTraits<1>::unpack(d, f);
#pragma unroll
      for (int e = 0; e < 8; ++e) idx[e] = i0 + e;
    } else if (wide) {
      const int i0 = ch * CHUNK + step * 256 + lane * 8;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        uint4 d = make_uint4(0xFF800000u, 0xFF800000u, 0xFF800000u, 0xFF800000u);
        if (i0 + 4 * h < V) d = __ldg(reinterpret_cast<const uint4*>((const float*)logits + row * (long long)V + i0 + 4 * h));
        f[4 * h] = __uint_as_float(d.x); f[4 * h + 1] = __uint_as_float(d.y);
        f[4 * h + 2] = __uint_as_float(d.z); f[4 * h + 3] = __uint_as_float(d.w);
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) idx[e] = i0 + e;
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        idx[e] = ch * CHUNK + step * 256 + e * 32 + lane;
        f[e] = idx[e] < V ? load_logit(logits, dtype, row * (long long)V + idx[e]) : -INFINITY;
      }
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      if (f[e] >= floor && idx[e] < V) {
        const int pos = atomicAdd(cnt, 1);
        const float canon = f[e] == 0.0f ? 0.0f : f[e];  // -0 and +0 are one value
        if (pos < cap) buf[pos] = make_uint2(__float_as_uint(canon), (uint32_t)idx[e]);
      }
    }
  }
}

// The same for rows whose entries can be read as aligned 16-byte vectors, split in two so that the loads
// of several chunks are in flight before any of them is examined.  DT: 0 float (8 vectors per lane and
// chunk), 1 bfloat16 (4 vectors).
template <int DT>
__device__ __forceinline__ void load_chunk_wide(const void* logits, long long row, int V, int ch, int lane,
                                                uint4 (&v)[DT == 1 ? 4 : 8]) {
  constexpr int NV = DT == 1 ? 4 : 8, VEC = DT == 1 ? 8 : 4;
  const uint32_t fill = DT == 1 ? 0xFF80FF80u : 0xFF800000u;
  const char* base = (const char*)logits + (size_t)row * (size_t)V * (DT == 1 ? 2 : 4);
#pragma unroll
  for (int k = 0; k < NV; ++k) {
    const int i0 = ch * CHUNK + (k * 32 + lane) * VEC;
    v[k] = i0 < V ? __ldg(reinterpret_cast<const uint4*>(base + (size_t)i0 * (DT == 1 ? 2 : 4))) : make_uint4(fill, fill, fill, fill);
  }
}
template <int DT>
__device__ __forceinline__ void push_chunk_wide(const uint4 (&v)[DT == 1 ? 4 : 8], int V, int ch, float floor, uint2* buf,
                                                int* cnt, int cap, int lane) {
  constexpr int NV = DT == 1 ? 4 : 8, VEC = DT == 1 ? 8 : 4;
#pragma unroll
  for (int k = 0; k < NV; ++k) {
    float f[VEC];
    ElemTraits<DT>::unpack(v[k], f);
    const int i0 = ch * CHUNK + (k * 32 + lane) * VEC;
    if (ElemTraits<DT>::vmax(v[k]) >= floor) {
#pragma unroll
      for (int e = 0; e < VEC; ++e) {
        if (f[e] >= floor && i0 + e < V) {
          const int pos = atomicAdd(cnt, 1);
          const float canon = f[e] == 0.0f ? 0.0f : f[e];  // -0 and +0 are one value
          if (pos < cap) buf[pos] = make_uint2(__float_as_uint(canon), (uint32_t)(i0 + e));
        }
      }
    }
  }
}
// Work items it, it + stride, ... of the list, two at a time.
template <int DT>
__device__ __forceinline__ void scan_items_wide(const void* logits, const int* path, long long row0, int V,
                                                const uint32_t* items, int nitems, int first, int stride,
                                                const float* floors, uint2 (*cand)[CAND_CAP], int* ncand, int lane) {
  constexpr int NV = DT == 1 ? 4 : 8;
  for (int it = first; it < nitems; it += 2 * stride) {
    const bool two = it + stride < nitems;
    const uint32_t a = items[it], c = items[two ? it + stride : it];
    const int ra = (int)(a >> 16), cha = (int)(a & 0xFFFFu), rc = (int)(c >> 16), chc = (int)(c & 0xFFFFu);
    uint4 va[NV], vc[NV];
    load_chunk_wide<DT>(logits, row0 + path[ra], V, cha, lane, va);
    if (two) load_chunk_wide<DT>(logits, row0 + path[rc], V, chc, lane, vc);
    push_chunk_wide<DT>(va, V, cha, floors[ra], cand[ra], &ncand[ra], CAND_CAP, lane);
    if (two) push_chunk_wide<DT>(vc, V, chc, floors[rc], cand[rc], &ncand[rc], CAND_CAP, lane);
  }
}

// The k-th largest of a row's chunk maxima (a lower bound of the row's k-th largest entry); -inf when
// the row has fewer than k chunks.  Called by all lanes of a warp.  Up to 256 chunks are held in
// registers as order-preserving integers and the largest is removed k - 1 times through the integer
// reduction unit; longer rows take the general loop.
__device__ __forceinline__ float kth_largest_chunk_max(const float2* pairs, int n_chunks, int k, int lane) {
  if (n_chunks < k) return -INFINITY;
  if (n_chunks <= 256) {
    uint32_t kv[8];  // 0 = no chunk (every real value maps above 0)
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int ch = lane + 32 * i;
      kv[i] = ch < n_chunks ? ordered_bits(__float_as_uint(pairs[ch].y)) : 0u;
    }
    uint32_t mx = 0u;
    for (int r = 0; r < k; ++r) {
      uint32_t lm = kv[0];
#pragma unroll
      for (int i = 1; i < 8; ++i) lm = max(lm, kv[i]);
      mx = warp_max_u32(lm);
      const int owner = 31 - (int)warp_max_u32(lm == mx ? 31u - (uint32_t)lane : 0u);  // the lowest lane that holds it
      if (lane == owner) {  // remove one instance
        bool gone = false;
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if (!gone && kv[i] == mx) { kv[i] = 0u; gone = true; }
      }
    }
    return __uint_as_float((mx & 0x80000000u) ? (mx ^ 0x80000000u) : ~mx);
  }
  unsigned long long below = ~0ull;
  for (int r = 0; r < k; ++r) {
    unsigned long long best = 0ull;
    for (int ch = lane; ch < n_chunks; ch += 32) {
      const unsigned long long key = select_key(__float_as_uint(pairs[ch].y), (uint32_t)ch);
      if (key < below && key > best) best = key;
    }
    below = warp_max_u64(best);
  }
  return key_value(below);
}

// Sum over the 16 lanes of a half-warp (both halves carry the same values); every lane gets it.
__device__ __forceinline__ double half_sum_d(double v) {
#pragma unroll
  for (int o = 8; o > 0; o >>= 1) v += __shfl_xor_sync(FULL, v, o);
  return v;
}

constexpr int HANDOFF_BAR = 2;  // named barrier on which a wider block's other threads wait for the walk's outputs

// Stage 1 of the table update for sequence b's records (8 lanes per record) by the threads K2_THREADS ..
// BLOCK_THREADS - 1 of a wider block, beside the verifying threads, which meanwhile compress the accepted rows: the
// contexts of the records need the emitted tokens only.  Positions past the path get "no slot".
template <int BLOCK_THREADS>
__device__ __forceinline__ void locate_beside_verify(const VerifyParams& p, const int b) {
  constexpr int HELPERS = BLOCK_THREADS - K2_THREADS;
  static_assert(HELPERS > 0 && HELPERS % 32 == 0, "whole warps");
  asm volatile("bar.sync %0, %1;" ::"n"(HANDOFF_BAR), "n"(BLOCK_THREADS) : "memory");  // context windows and path length are written
  if (!p.fuse_locate) return;
  const int W1 = p.D + 1, n_rec = W1 * p.n_max;
  const int ht = (int)threadIdx.x - K2_THREADS;
  for (int r0 = 0; r0 < n_rec; r0 += HELPERS / GROUP) {
    const int r = r0 + ht / GROUP;
    const bool in_range = r < n_rec;
    const int j = in_range ? r / p.n_max : 0;
    const int n = in_range ? r - j * p.n_max + 1 : 1;
    locate_record(p.upd, (long long)b * W1 + j, n, in_range);
  }
}

// The verification of sequence b by K2_THREADS threads: a whole block (BAR 0, BLOCK_THREADS = K2_THREADS), or
// threads 0 .. K2_THREADS - 1 of a block of BLOCK_THREADS threads, which then synchronise on named barrier BAR;
// the block's other threads call locate_beside_verify instead.
// s_tail_out (shared memory, may be null): also receives the sequence's advanced tail.
template <int BAR, int BLOCK_THREADS = K2_THREADS>
__device__ __forceinline__ void verify_block(const VerifyParams& p, const int b, int* s_tail_out = nullptr) {
  // per-node state, sized by the tree (verify_smem_bytes): target probabilities of the candidates, normaliser
  // reciprocals and offsets, the candidate lists, tree tokens and topology
  extern __shared__ __align__(16) unsigned char s_dyn[];
  double* s_p = reinterpret_cast<double*>(s_dyn);                 // [N][KMAX]
  double* s_invZ = s_p + (size_t)p.N * KMAX;                      // [N]
  float* s_off = reinterpret_cast<float*>(s_invZ + p.N);          // [N]
  float* s_cphi = s_off + p.N;                                    // [N][KMAX]
  int* s_cid = reinterpret_cast<int*>(s_cphi + (size_t)p.N * KMAX);  // [N][KMAX]
  int* s_tree = s_cid + (size_t)p.N * KMAX;                       // [N]
  int* s_cn = s_tree + p.N;
  int* s_fc = s_cn + p.N;
  int* s_nch = s_fc + p.N;
  __shared__ int s_tail[ORDER_MAX];
  __shared__ long long s_len;
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
  // top-k selection of up to TOPK_ROWS path rows at a time
  __shared__ uint32_t s_items[TOPK_ITEMS];  // (row slot << 16) | chunk: chunks that can hold a top-k entry
  __shared__ uint2 s_cand[TOPK_ROWS][CAND_CAP];
  __shared__ int s_ncand[TOPK_ROWS], s_nitems;
  __shared__ float s_floor[TOPK_ROWS];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int N = p.N, K = p.K;
  const double cd = (double)p.c;

  pdl_trigger();
  // ---- phase 0: stage the sequence's state.  It was written by the previous step, and this block cannot
  // have been scheduled before that step ended: the row pass releases its dependents only after its own wait ----
  for (int u = tid; u < N; u += K2_THREADS) {
    s_tree[u] = p.tree[(long long)b * N + u];
    s_cn[u] = p.cand_n[(long long)b * N + u];
    s_fc[u] = p.first_child[u];
    s_nch[u] = p.n_children[u];
  }
  for (int i = tid; i < N * K; i += K2_THREADS) {
    const int u = i / K, t = i - u * K;
    s_cid[(u) * KMAX + (t)] = p.cand_id[(long long)b * N * K + i];
    s_cphi[(u) * KMAX + (t)] = p.cand_phi[(long long)b * N * K + i];
  }
  if (tid < p.n_max) s_tail[tid] = p.tail[b * p.n_max + tid];
  if (tid == 32) s_len = p.len[b];  // read here so that the output phase does not wait for it
  verify_sync<BAR>();

  // ---- phase 1: the candidate logits are requested first (one round of gathers), the normalisers
  // (8 lanes per row) are formed while they travel ----
  // (trees of up to 128 nodes are covered by these six gathers per thread; larger ones gather again below)
  constexpr int GATHERS = 128 * KMAX / K2_THREADS;
  float gx[GATHERS];
#pragma unroll
  for (int k = 0; k < GATHERS; ++k) {
    const int i = tid + k * K2_THREADS;
    const int u = i / KMAX, t = i - u * KMAX;
    gx[k] = 0.0f;
    if (u < N && t < s_cn[u]) gx[k] = load_logit(p.logits, p.dtype, ((long long)b * N + u) * (long long)p.V + s_cid[(u) * KMAX + (t)]);
  }
  pdl_wait();  // the chunk pairs come from the row pass
  {
    const int gl = tid & (ROW_LANES - 1);
    for (int u0 = 0; u0 < N; u0 += K2_THREADS / ROW_LANES) {
      const int u = u0 + tid / ROW_LANES;
      const bool live = u < N;
      const float2* pairs = p.pairs + ((long long)b * N + (live ? u : 0)) * p.n_chunks;
      // the pairs are read in batches of independent loads (a loop of load-then-use would pay one
      // cache round trip per chunk)
      constexpr int BATCH = 8;
      float mm = -INFINITY;
      if (live)
        for (int c0 = gl; c0 < p.n_chunks; c0 += BATCH * ROW_LANES) {
          float y[BATCH];
#pragma unroll
          for (int k = 0; k < BATCH; ++k) {
            const int ch = c0 + k * ROW_LANES;
            y[k] = ch < p.n_chunks ? pairs[ch].y : -INFINITY;
          }
#pragma unroll
          for (int k = 0; k < BATCH; ++k) mm = fmaxf(mm, y[k]);
        }
#pragma unroll
      for (int o = ROW_LANES / 2; o > 0; o >>= 1) mm = fmaxf(mm, __shfl_xor_sync(FULL, mm, o));
      const float om = chunk_offset(mm, p.c);  // the offset grows with the maximum
      double z0 = 0.0, z1 = 0.0;
      if (live)
        for (int c0 = gl; c0 < p.n_chunks; c0 += BATCH * ROW_LANES) {
          float2 v[BATCH];
#pragma unroll
          for (int k = 0; k < BATCH; ++k) {
            const int ch = c0 + k * ROW_LANES;
            v[k] = ch < p.n_chunks ? pairs[ch] : make_float2(0.0f, -INFINITY);  // an empty chunk has no mass
          }
#pragma unroll
          for (int k = 0; k < BATCH; k += 2) {  // the same two running sums, in the same order, as one chunk at a time
            z0 += (double)chunk_mass_f(v[k], p.c, om);
            z1 += (double)chunk_mass_f(v[k + 1], p.c, om);
          }
        }
      double z = z0 + z1;
#pragma unroll
      for (int o = ROW_LANES / 2; o > 0; o >>= 1) z += __shfl_xor_sync(FULL, z, o);
      if (live && gl == 0) { s_off[u] = om; s_invZ[u] = 1.0 / z; }
    }
  }
  verify_sync<BAR>();
#pragma unroll
  for (int k = 0; k < GATHERS; ++k) {
    const int i = tid + k * K2_THREADS;
    const int u = i / KMAX, t = i - u * KMAX;
    if (u < N && t < s_cn[u]) s_p[(u) * KMAX + (t)] = exp2_d((double)gx[k] * cd - (double)s_off[u]) * s_invZ[u];
  }
  for (int i = tid + GATHERS * K2_THREADS; i < N * KMAX; i += K2_THREADS) {  // the rest of a large tree
    const int u = i / KMAX, t = i - u * KMAX;
    if (t < s_cn[u]) {
      const float x = load_logit(p.logits, p.dtype, ((long long)b * N + u) * (long long)p.V + s_cid[(u) * KMAX + (t)]);
      s_p[(u) * KMAX + (t)] = exp2_d((double)x * cd - (double)s_off[u]) * s_invZ[u];
    }
  }
  verify_sync<BAR>();

  // ---- phase 2: the walk, by warp 0 ------------------------------------------------------------
  // Lane i (and its mirror i + 16) carries candidate i of the current node.  Target and draft
  // distributions are kept unnormalised with their normalisers, so a rejection costs one 16-lane sum
  // and no division: with p~_i = ph_i / zr and q_i = qh_i / qn,
  //   accept x        iff  U * qh_x * zr < ph_x * qn
  //   after rejecting x:   ph_i <- max(0, ph_i * qn - qh_i * zr),  zr <- zr * qn - sum_i min(ph_i * qn, qh_i * zr),
  //                        qh_x <- 0,  qn <- qn - qh_x
  // and off the candidate list the residual target is the target times (product of the qn's) / zr.
  if (warp == 0) {
    const int li = lane & 15;
    int u = 0, m = 0;
    int nsup = 0;
    double scale = 1.0;
    if (lane == 0) s_path[0] = 0;
    for (;;) {
      const int fc = s_fc[u], nch = s_nch[u];
      // children are drafted in rank order: count the leading drafted ones
      const unsigned have = __ballot_sync(FULL, lane < nch && s_tree[fc + (lane < nch ? lane : 0)] >= 0);
      const int drafted = __ffs(~have) - 1;
      nsup = 0;
      scale = 1.0;
      if (drafted <= 0) break;  // nothing drafted below u: sample from its target
      const int nc = s_cn[u];
      const int cid = li < nc ? s_cid[(u) * KMAX + (li)] : -1;
      double ph = li < nc ? s_p[(u) * KMAX + (li)] : 0.0;
      double qh = li < nc ? (double)s_cphi[(u) * KMAX + (li)] : 0.0;
      double qn = half_sum_d(qh), zr = 1.0, pq = 1.0;
      // the uniforms of all children at once
      const double Uj = li < drafted ? (double)philox_u24(p.seed, (uint32_t)(p.seq_base + b), p.step, u, (uint32_t)li) * (1.0 / 16777216.0) : 0.0;
      int accepted = -1;
      for (int j = 0; j < drafted; ++j) {
        const int x = s_tree[fc + j];
        const unsigned hit = __ballot_sync(FULL, li < nc && cid == x) & 0xFFFFu;
        const int ix = hit ? 31 - __clz(hit) : -1;
        const double U = __shfl_sync(FULL, Uj, j & 15);
        const double qx = __shfl_sync(FULL, qh, ix < 0 ? 0 : ix);
        const double px = __shfl_sync(FULL, ph, ix < 0 ? 0 : ix);
        // A drafted token always comes from its parent's candidate list (stand_state_load clears any that does
        // not); should one be met all the same, it and its later siblings count as not drafted.
        if (ix < 0) break;
        if (p.deterministic) {
          // one-hot draft: accept iff U < p~(x); on rejection x loses its mass and the rest is renormalised
          if (U * zr < px) { accepted = j; break; }
          zr -= px;
          if (li == ix) ph = 0.0;
          continue;
        }
        if (U * qx * zr < px * qn) { accepted = j; break; }
        const double a = ph * qn, c2 = qh * zr;
        const double ov = half_sum_d(fmin(a, c2));
        pq *= qn;
        zr = zr * qn - ov;
        ph = fmax(0.0, a - c2);
        if (li == ix) qh = 0.0;
        qn -= qx;
      }
      if (accepted >= 0) {
        if (lane == 0) s_emit[m] = s_tree[fc + accepted];
        u = fc + accepted;
        ++m;
        if (lane == 0) s_path[m] = u;
        continue;
      }
      const double inv = 1.0 / zr;
      scale = pq * inv;
      nsup = nc;
      if (lane < nc) { s_sup_id[lane] = cid; s_sup_pt[lane] = ph * inv; s_sup_p[lane] = s_p[(u) * KMAX + (lane)]; }
      break;
    }
    if (lane == 0) {
      s_m = m;
      s_nsup = nsup;
      s_scale = scale;
      s_pick = 0x7FFFFFFF;
      s_pick_last = -1;
    }
  }
  verify_sync<BAR>();

  // ---- phase 3: one token by inverse CDF at the stop node ----------------------
  const int m = s_m;
  const int us = s_path[m];
  const long long rows = (long long)b * N + us;
  const int nsup = s_nsup;
  const double scale = s_scale;
  const float off = s_off[us];
  const double invZ = s_invZ[us];
  const double U = (double)philox_u24(p.seed, (uint32_t)(p.seq_base + b), p.step, us, SLOT_FINAL) * (1.0 / 16777216.0);

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
      double mass = scale * (chunk_mass(pr, p.c, off) * invZ);
      for (int s = 0; s < nsup; ++s)
        if (s_sup_id[s] / CHUNK == ch) mass += s_sup_pt[s] - scale * s_sup_p[s];
      cm[i] = fmax(mass, 0.0);
      mine += cm[i];
    }
  }
  double W;
  const double base = block_scan_excl<BAR>(mine, s_scan, &W);
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
  verify_sync<BAR>();
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
  verify_sync<BAR>();
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
        w[e] = scale * (exp2_d((double)x * cd - (double)off) * invZ);
      }
    }
    wsum += w[e];
  }
  double tot;
  const double fb = block_scan_excl<BAR>(wsum, s_scan, &tot);
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
  verify_sync<BAR>();

  // ---- phase 4: outputs --------------------------------------------------------
  const int W1 = p.D + 1;
  if (tid == 0) {
    int y = s_pick;
    if (y == 0x7FFFFFFF) y = s_pick_last;
    if (y < 0) y = 0;
    s_emit[m] = y;
    // context windows of the accepted rows, then the advanced tail
    int win[ORDER_MAX];
    for (int i = 0; i < p.n_max; ++i) win[i] = s_tail[i];
    for (int j = 0; j <= m; ++j) {
      for (int i = 0; i < p.n_max; ++i) p.rec_ctx[((long long)b * W1 + j) * p.n_max + i] = win[i];
      for (int i = 0; i + 1 < p.n_max; ++i) win[i] = win[i + 1];
      win[p.n_max - 1] = s_emit[j];
    }
    for (int i = 0; i < p.n_max; ++i) p.tail[b * p.n_max + i] = win[i];
    if (s_tail_out)
      for (int i = 0; i < p.n_max; ++i) s_tail_out[i] = win[i];
    p.len[b] = s_len + m + 1;
    p.n_path[b] = m + 1;
    if (p.n_emitted_user) p.n_emitted_user[b] = m + 1;
    atomicAdd(&p.stats[ST_EMITTED], (unsigned long long)(m + 1));
    if (b == 0) atomicAdd(&p.stats[ST_STEPS], 1ull);
  }
  verify_sync<BAR>();
  // a wider block's other threads take the records from here (they wait on this barrier; nobody waits for them)
  if (BLOCK_THREADS > K2_THREADS) asm volatile("bar.arrive %0, %1;" ::"n"(HANDOFF_BAR), "n"(BLOCK_THREADS) : "memory");
  if (tid < W1) {
    const int e = tid <= m ? s_emit[tid] : -1;
    p.emitted[b * W1 + tid] = e;
    if (p.emitted_user) p.emitted_user[b * W1 + tid] = e;
    p.path[b * W1 + tid] = tid <= m ? s_path[tid] : -1;
    if (tid <= m) atomicAdd(&p.node_accepts[s_path[tid]], 1ull);
  }
  // Compressed rows of the accepted path: the exact top-k of each row, as probabilities.  The k-th
  // largest chunk maximum bounds the k-th largest entry from below, so only the chunks whose maximum
  // reaches it (about k per row) are read again.  Up to TOPK_ROWS rows go through together: one warp
  // per row finds the bound and lists the row's chunks, all warps share the chunk reads, one warp
  // per row selects.
  const bool wide = p.dtype == 1 ? (((uintptr_t)p.logits & 15) == 0 && (p.V & 7) == 0)
                                 : (((uintptr_t)p.logits & 15) == 0 && (p.V & 3) == 0);
  for (int j0 = 0; j0 <= m; j0 += TOPK_ROWS) {
    const int nr = min(TOPK_ROWS, m + 1 - j0);
    if (tid < TOPK_ROWS) s_ncand[tid] = 0;
    if (tid == 0) s_nitems = 0;
    verify_sync<BAR>();
    if (warp < nr) {
      const float2* pairs = p.pairs + ((long long)b * N + s_path[j0 + warp]) * p.n_chunks;
      const float tau = kth_largest_chunk_max(pairs, p.n_chunks, K, lane);
      if (lane == 0) s_floor[warp] = tau;
      for (int ch = lane; ch < p.n_chunks; ch += 32)
        if (pairs[ch].y >= tau) {
          const int pos = atomicAdd(&s_nitems, 1);
          if (pos < TOPK_ITEMS) s_items[pos] = ((uint32_t)warp << 16) | (uint32_t)ch;
        }
    }
    verify_sync<BAR>();
    const bool items_over = s_nitems > TOPK_ITEMS;
    const int nitems = items_over ? 0 : s_nitems;
    if (wide && p.dtype == 1)
      scan_items_wide<1>(p.logits, s_path + j0, (long long)b * N, p.V, s_items, nitems, warp, K2_THREADS / 32, s_floor, s_cand,
                         s_ncand, lane);
    else if (wide)
      scan_items_wide<0>(p.logits, s_path + j0, (long long)b * N, p.V, s_items, nitems, warp, K2_THREADS / 32, s_floor, s_cand,
                         s_ncand, lane);
    else
      for (int it = warp; it < nitems; it += K2_THREADS / 32) {
        const uint32_t item = s_items[it];
        const int r = (int)(item >> 16), ch = (int)(item & 0xFFFFu);
        push_chunk_candidates(p.logits, p.dtype, (long long)b * N + s_path[j0 + r], p.V, ch, s_floor[r], false, s_cand[r],
                              &s_ncand[r], CAND_CAP, lane);
      }
    verify_sync<BAR>();
    if (warp < nr) {
      const int j = j0 + warp, u = s_path[j];
      const long long row = (long long)b * N + u;
      int n = s_ncand[warp];
      if (items_over || n > CAND_CAP) {
        // more entries reach the bound than the buffers hold (long runs of equal values): the streaming
        // selection copes with any input, one chunk at a time
        n = row_topk_warp(p.logits, p.dtype, row, p.V, p.pairs + row * p.n_chunks, p.n_chunks, K, s_cand[warp],
                          &s_ncand[warp], lane);
      } else if (n > 32) {
        compact_topk(s_cand[warp], &s_ncand[warp], n, K, lane, s_floor[warp]);
        n = n < K ? n : K;
      }
      // one candidate per lane: its rank among them decides its place in the record
      // (every lane counts the candidates that beat its own, reading them from shared memory)
      __syncwarp();
      const uint2 e = lane < n ? s_cand[warp][lane] : make_uint2(0u, 0u);
      const unsigned long long mine = select_key(e.x, e.y);
      int rank = 0;
      for (int t = 0; t < n; ++t) {
        const uint2 o = s_cand[warp][t];
        rank += select_key(o.x, o.y) > mine ? 1 : 0;  // ids are distinct, so are the keys
      }
      const int keep = n < K ? n : K;
      const long long at0 = ((long long)b * W1 + j) * K;
      if (lane < n && rank < K) {
        p.rec_ids[at0 + rank] = (int)e.y;
        p.rec_p[at0 + rank] = (float)(exp2_d((double)__uint_as_float(e.x) * cd - (double)s_off[u]) * s_invZ[u]);
      }
      if (lane >= keep && lane < K) { p.rec_ids[at0 + lane] = -1; p.rec_p[at0 + lane] = 0.0f; }
    }
    verify_sync<BAR>();
  }

  // ---- stage 1 of the table update for this sequence's records (8 lanes per record), unless the block's other
  // threads are doing it -----
  if (p.fuse_locate && BLOCK_THREADS == K2_THREADS) {
    const int n_rec = W1 * p.n_max;
    for (int r0 = 0; r0 < n_rec; r0 += K2_THREADS / GROUP) {
      const int r = r0 + tid / GROUP;
      const bool in_range = r < n_rec;
      const int j = in_range ? r / p.n_max : 0;
      const int n = in_range ? r - j * p.n_max + 1 : 1;
      locate_record(p.upd, (long long)b * W1 + j, n, in_range);
    }
  }
}

__global__ void __launch_bounds__(K2_THREADS, 2) verify_kernel(const VerifyParams p) { verify_block<0>(p, (int)blockIdx.x); }

// The same with a second set of warps that maps the update records to table slots beside the compression of the
// accepted rows.  One block per multiprocessor at its register use: for batches of at most that many sequences.
constexpr int K2_WIDE_THREADS = 2 * K2_THREADS;
__global__ void __launch_bounds__(K2_WIDE_THREADS, 1) verify_wide_kernel(const VerifyParams p) {
  if (threadIdx.x < K2_THREADS) verify_block<1, K2_WIDE_THREADS>(p, (int)blockIdx.x);
  else {
    pdl_trigger();
    pdl_wait();
    locate_beside_verify<K2_WIDE_THREADS>(p, (int)blockIdx.x);
  }
}

}  // namespace stand
