// Row pass: the one pass over the logits.  Temperature softmax statistics
// (paper Sec. 5: sampling at temperature T) and the per-row top-k that the
// N-gram module stores (Sec. 4.1), fused.
//
// Work unit = one warp streaming `cpu` consecutive 1024-entry chunks of one row.
// Per chunk the warp writes (sum_v 2^(x_v*c - o), o) with c = log2(e)/T and o an
// offset near the running maximum, so that a row's normaliser is rebuilt later
// as sum_c s_c * 2^(o_c - o*) and prefix sums over chunks serve the inverse-CDF
// sample.  Per unit the warp writes its k best (value, id) pairs; the per-row
// top-k is the merge of the unit lists.  HBM-bound: every logit is read exactly once
// with 16-byte loads that bypass L1; the next chunk is in flight while the
// current one is reduced.
#pragma once
#include "common.cuh"

namespace stand {

constexpr int K1_THREADS = 256;
constexpr int K1_WARPS = K1_THREADS / 32;
constexpr int COMPACT_AT = 64;              // candidate count that triggers a compaction
constexpr int CAND_CAP = COMPACT_AT + 256;  // a warp adds at most 32 lanes x 8 entries between checks

struct RowPassParams {
  const void* logits;
  long long rows;
  int V, n_chunks, cpu, upr;  // chunks per unit, units per row
  float c;                    // log2(e) / T
  int topk;
  float2* pairs;  // [rows, n_chunks]  (sum, offset)
  uint2* part;    // [rows, upr, topk] (value bits, id); id 0xFFFFFFFF = unused
};

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint4 ld_stream16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

template <int DT> struct ElemTraits;
template <> struct ElemTraits<0> {  // float
  static constexpr int VEC = 4, ESIZE = 4;
  static constexpr uint32_t NEG_INF_WORD = 0xFF800000u;
  __device__ static __forceinline__ void unpack(const uint4& d, float (&f)[4]) {
    f[0] = __uint_as_float(d.x); f[1] = __uint_as_float(d.y);
    f[2] = __uint_as_float(d.z); f[3] = __uint_as_float(d.w);
  }
  __device__ static __forceinline__ float vmax(const uint4& d) {
    return fmaxf(fmaxf(__uint_as_float(d.x), __uint_as_float(d.y)),
                 fmaxf(__uint_as_float(d.z), __uint_as_float(d.w)));
  }
};
template <> struct ElemTraits<1> {  // bfloat16, two per word, lower index in the low half
  static constexpr int VEC = 8, ESIZE = 2;
  static constexpr uint32_t NEG_INF_WORD = 0xFF80FF80u;
  __device__ static __forceinline__ void unpack(const uint4& d, float (&f)[8]) {
    f[0] = __uint_as_float(d.x << 16); f[1] = __uint_as_float(d.x & 0xFFFF0000u);
    f[2] = __uint_as_float(d.y << 16); f[3] = __uint_as_float(d.y & 0xFFFF0000u);
    f[4] = __uint_as_float(d.z << 16); f[5] = __uint_as_float(d.z & 0xFFFF0000u);
    f[6] = __uint_as_float(d.w << 16); f[7] = __uint_as_float(d.w & 0xFFFF0000u);
  }
  __device__ static __forceinline__ uint32_t max2(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
  }
  __device__ static __forceinline__ float vmax(const uint4& d) {
    const uint32_t m = max2(max2(d.x, d.y), max2(d.z, d.w));
    return fmaxf(__uint_as_float(m << 16), __uint_as_float(m & 0xFFFF0000u));
  }
};

// The NV 16-byte vectors of lane `lane` in chunk `chunk`: vector i covers entries
// chunk*1024 + i*32*VEC + lane*VEC .. +VEC.  Entries past V read as -inf.
template <int DT, bool ALIGNED>
__device__ __forceinline__ void load_chunk(const char* row, int V, int chunk, int lane,
                                           uint4 (&d)[CHUNK / (32 * ElemTraits<DT>::VEC)]) {
  using TR = ElemTraits<DT>;
  constexpr int VEC = TR::VEC, NV = CHUNK / (32 * VEC);
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int idx = chunk * CHUNK + i * 32 * VEC + lane * VEC;
    if (ALIGNED) {
      if (idx < V) d[i] = ld_stream16(row + (size_t)idx * TR::ESIZE);
      else d[i] = make_uint4(TR::NEG_INF_WORD, TR::NEG_INF_WORD, TR::NEG_INF_WORD, TR::NEG_INF_WORD);
    } else {
      uint32_t w[4];
      if (DT == 0) {
#pragma unroll
        for (int e = 0; e < 4; ++e)
          w[e] = idx + e < V ? __ldg((const uint32_t*)row + idx + e) : 0xFF800000u;
      } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const uint32_t lo = idx + 2 * e < V ? __ldg((const unsigned short*)row + idx + 2 * e) : 0xFF80u;
          const uint32_t hi = idx + 2 * e + 1 < V ? __ldg((const unsigned short*)row + idx + 2 * e + 1) : 0xFF80u;
          w[e] = lo | (hi << 16);
        }
      }
      d[i] = make_uint4(w[0], w[1], w[2], w[3]);
    }
  }
}

// Keeps the k best of the n buffered candidates at buf[0..k), best first; returns
// the new threshold (the k-th value, or -inf while fewer than k are known).
__device__ __forceinline__ float compact_topk(uint2* buf, int* cnt, int n, int k, int lane) {
  const int keep = n < k ? n : k;
  for (int r = 0; r < keep; ++r) {
    unsigned long long best = 0ull;
    int bpos = -1;
    for (int i = r + lane; i < n; i += 32) {
      const uint2 e = buf[i];
      const unsigned long long key = select_key(e.x, e.y);
      if (bpos < 0 || key > best) { best = key; bpos = i; }
    }
    const unsigned long long wbest = warp_max_u64(best);
    if (bpos >= 0 && best == wbest) {  // ids are distinct, so exactly one lane owns the winner
      const uint2 a = buf[bpos], b = buf[r];
      buf[r] = a;
      buf[bpos] = b;
    }
    __syncwarp();
  }
  if (lane == 0) *cnt = keep;
  __syncwarp();
  return keep == k ? __uint_as_float(buf[k - 1].x) : -INFINITY;
}

template <int DT, bool ALIGNED>
__global__ void __launch_bounds__(K1_THREADS) row_pass_kernel(const RowPassParams p) {
  using TR = ElemTraits<DT>;
  constexpr int VEC = TR::VEC, NV = CHUNK / (32 * VEC);
  __shared__ uint2 s_buf[K1_WARPS][CAND_CAP];
  __shared__ int s_cnt[K1_WARPS];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long unit = (long long)blockIdx.x * K1_WARPS + warp;
  if (unit >= p.rows * p.upr) return;  // warps are independent: no block-wide barrier below
  const long long row = unit / p.upr;
  const int split = (int)(unit - row * p.upr);
  const int c0 = split * p.cpu;
  const int c1 = min(c0 + p.cpu, p.n_chunks);
  const char* rowp = (const char*)p.logits + (size_t)row * (size_t)p.V * TR::ESIZE;
  uint2* buf = s_buf[warp];
  int* cnt = &s_cnt[warp];
  if (lane == 0) *cnt = 0;
  __syncwarp();

  const float c = p.c;
  const float span = 64.0f / c;  // re-centre when an entry exceeds the offset by 2^64
  float tau = -INFINITY;         // candidates must reach this value
  float off = 0.0f;              // current offset o (log2 domain)
  float guard = -INFINITY;       // entries above this value force a new offset
  bool first = true;

  uint4 cur[NV], nxt[NV];
  load_chunk<DT, ALIGNED>(rowp, p.V, c0, lane, cur);
  for (int ch = c0; ch < c1; ++ch) {
    if (ch + 1 < c1) load_chunk<DT, ALIGNED>(rowp, p.V, ch + 1, lane, nxt);

    float sum = 0.0f;
    bool over = first;
    float lane_max = -INFINITY;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      float f[VEC];
      TR::unpack(cur[i], f);
      const float vm = TR::vmax(cur[i]);
      lane_max = fmaxf(lane_max, vm);
      const bool hit = vm >= tau;
      over |= vm > guard;
      if (__any_sync(FULL, hit)) {  // rare after the first vectors of a unit
        if (hit) {
          const int idx0 = ch * CHUNK + i * 32 * VEC + lane * VEC;
#pragma unroll
          for (int e = 0; e < VEC; ++e) {
            if (f[e] >= tau && idx0 + e < p.V) {
              const int pos = atomicAdd(cnt, 1);
              const float canon = f[e] == 0.0f ? 0.0f : f[e];  // -0 and +0 are one value
              buf[pos] = make_uint2(__float_as_uint(canon), (uint32_t)(idx0 + e));
            }
          }
        }
        __syncwarp();
        const int n = *(volatile int*)cnt;
        if (n >= COMPACT_AT) tau = compact_topk(buf, cnt, n, p.topk, lane);
      }
#pragma unroll
      for (int e = 0; e < VEC; ++e) sum += ex2_approx(fmaf(f[e], c, -off));
    }
    if (__any_sync(FULL, over)) {
      // new offset from this chunk's maximum; redo the chunk's sum with it
      const float cm = warp_max_f(lane_max);
      off = cm == -INFINITY ? 0.0f : cm * c;
      guard = cm == -INFINITY ? -INFINITY : cm + span;
      first = false;
      sum = 0.0f;
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        float f[VEC];
        TR::unpack(cur[i], f);
#pragma unroll
        for (int e = 0; e < VEC; ++e) sum += ex2_approx(fmaf(f[e], c, -off));
      }
    }
    sum = warp_sum_f(sum);
    if (lane == 0) p.pairs[row * p.n_chunks + ch] = make_float2(sum, off);
#pragma unroll
    for (int i = 0; i < NV; ++i) cur[i] = nxt[i];
  }

  const int n = *(volatile int*)cnt;
  const int keep = n < p.topk ? n : p.topk;
  if (n > 0) compact_topk(buf, cnt, n, p.topk, lane);
  if (lane < p.topk) {
    p.part[(row * p.upr + split) * p.topk + lane] = lane < keep ? buf[lane] : make_uint2(0u, 0xFFFFFFFFu);
  }
}

// ---------------------------------------------------------------------------
// Per-row results from the unit partials (used by the context-free row-stats
// entry point; the verification kernel does the same for the rows it needs).
// ---------------------------------------------------------------------------
struct RowNorm {
  float off;  // o* = largest chunk offset
  double Z;   // sum_c s_c 2^(o_c - o*)
};

// All lanes of a warp call this; every lane gets the result.
__device__ __forceinline__ RowNorm row_normaliser(const float2* pairs, int n_chunks, int lane) {
  float om = -INFINITY;
  for (int c = lane; c < n_chunks; c += 32) {
    const float2 pr = pairs[c];
    if (pr.x > 0.0f) om = fmaxf(om, pr.y);
  }
  om = warp_max_f(om);
  double z = 0.0;
  for (int c = lane; c < n_chunks; c += 32) {
    const float2 pr = pairs[c];
    if (pr.x > 0.0f) z += (double)pr.x * exp2((double)pr.y - (double)om);
  }
  RowNorm r;
  r.off = om;
  r.Z = warp_sum_d(z);
  return r;
}

// k-th round of a merge of unit lists without marking: the largest key strictly
// below `below`.  All lanes call; every lane gets (key, value bits, id).
__device__ __forceinline__ unsigned long long next_best(const uint2* part, int n_entries, unsigned long long below,
                                                       int lane) {
  unsigned long long best = 0ull;
  for (int i = lane; i < n_entries; i += 32) {
    const uint2 e = part[i];
    if (e.y == 0xFFFFFFFFu) continue;
    const unsigned long long key = select_key(e.x, e.y);
    if (key < below && key > best) best = key;
  }
  return warp_max_u64(best);
}
// inverse of select_key
__device__ __forceinline__ uint32_t key_id(unsigned long long key) { return ~(uint32_t)key; }
__device__ __forceinline__ float key_value(unsigned long long key) {
  const uint32_t o = (uint32_t)(key >> 32);
  const uint32_t bits = (o & 0x80000000u) ? (o ^ 0x80000000u) : ~o;
  return __uint_as_float(bits);
}

struct RowFinalizeParams {
  const float2* pairs;
  const uint2* part;
  long long rows;
  int n_chunks, upr, topk;
  float c;
  float* lse;
  int* ids;
  float* values;
  float* probs;
};

__global__ void __launch_bounds__(256) row_finalize_kernel(const RowFinalizeParams p) {
  const int lane = threadIdx.x & 31;
  const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= p.rows) return;
  const RowNorm nm = row_normaliser(p.pairs + row * p.n_chunks, p.n_chunks, lane);
  if (lane == 0) p.lse[row] = (float)(((double)nm.off + log2(nm.Z)) * 0.6931471805599453);
  const uint2* part = p.part + row * p.upr * p.topk;
  unsigned long long below = ~0ull;
  for (int r = 0; r < p.topk; ++r) {
    const unsigned long long key = next_best(part, p.upr * p.topk, below, lane);
    if (lane == 0) {
      if (key == 0ull) {
        p.ids[row * p.topk + r] = -1;
        p.values[row * p.topk + r] = 0.0f;
        p.probs[row * p.topk + r] = 0.0f;
      } else {
        const float x = key_value(key);
        p.ids[row * p.topk + r] = (int)key_id(key);
        p.values[row * p.topk + r] = x;
        p.probs[row * p.topk + r] = (float)(exp2((double)x * (double)p.c - (double)nm.off) / nm.Z);
      }
    }
    if (key == 0ull) below = 0ull; else below = key;
  }
}

}  // namespace stand
