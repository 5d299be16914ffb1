// Row pass: the one pass over the logits (paper Sec. 5: sampling at temperature
// T, i.e. softmax of x / T).
//
// Per 1024-entry chunk of a row the pass writes (s, m): m = the chunk's largest
// input value and s = sum_v 2^(x_v * c - o) with c = log2(e) / T and the integer
// offset o = ceil(m * c).  A row's normaliser is rebuilt later as
// sum_chunks s * 2^(o - o*), exactly (integer exponents); prefix sums over chunks
// serve the inverse-CDF sample; and the chunk maxima bound the per-row top-k
// (Sec. 4.1) so tightly that it can be finished afterwards from about k chunks, for
// the few rows that need it (row_topk_warp below).
//
// The kernel is bound by HBM bandwidth: persistent CTAs (one per SM) walk a
// contiguous range of tiles (31 chunks for bf16, 16 for fp32: about 64 KB); one elected lane
// streams tiles into a ring of shared-memory stages with bulk asynchronous copies
// (TMA) that complete on mbarriers, marked evict-first in L2; each consumer warp
// takes one chunk of every tile.  The inner loop has no branches: packed bf16 max, packed fp32 FMA/ADD,
// one ex2 per entry.
#pragma once
#include "common.cuh"

namespace stand {

constexpr int K1_SMEM_DATA = 96 * 1024;  // ring bytes per SM = 2 * K1_SMEM_DATA, shared by the CTAs of an SM
constexpr int K1_CTAS = 1;               // persistent CTAs per SM
// Consumer warps per CTA = chunks per tile.  Measured on 1.9 - 2.1 GB: large bulk copies win (bf16: one CTA of 31
// consumer warps, 62 KB tiles, 6.81 TB/s; two CTAs of 16 warps, 32 KB tiles, 6.60; of 8 warps, 16 KB tiles, 6.2;
// fp32: 16 warps and 64 KB tiles 6.73 against 6.55 with 8 and 32 KB), as long as about 32 warps per SM keep the
// exp unit fed for bf16.  31 consumer warps + the producer warp fill a 1024-thread block.
template <int DT> struct K1Shape { static constexpr int CW = DT == 1 ? 31 : 16; };
template <int DT> constexpr int k1_stage_bytes() { return K1Shape<DT>::CW * CHUNK * (DT == 1 ? 2 : 4); }
template <int DT> constexpr int k1_smem_bytes() {
  return (2 * K1_SMEM_DATA / K1_CTAS / k1_stage_bytes<DT>()) * k1_stage_bytes<DT>();
}
constexpr unsigned SPIN_LIMIT = 1u << 22;                  // bounded waits: about a second, then the kernel gives up

constexpr int COMPACT_AT = 64;              // candidate count that triggers a compaction
constexpr int CAND_CAP = COMPACT_AT + 256;  // a warp adds at most 32 lanes x 8 entries between checks

// status word values written by a kernel that gave up waiting
constexpr int K1_ERR_FULL_WAIT = 1, K1_ERR_EMPTY_WAIT = 2;

struct RowPassParams {
  const void* logits;
  long long rows;
  int V, n_chunks;
  int tiles_per_row;
  long long total_tiles;
  float c;          // log2(e) / T
  float2* pairs;    // [rows, n_chunks]  (sum, chunk max)
  int* status;      // device word, set non-zero if a bounded wait ran out (may be null)
  unsigned empty_wait_limit;  // polls the producer spends on one free-stage wait (SPIN_LIMIT unless a test lowers it)
};

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Offset of a chunk with maximum m: the integer o = ceil(m * c); 0 for an all -inf chunk.
__device__ __forceinline__ float chunk_offset(float m, float c) {
  return m == -INFINITY ? 0.0f : ceilf(__fmul_rn(m, c));
}

// ---- packed fp32 pairs (sm_100: two fp32 lanes per instruction) ----------------
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(unsigned long long v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ unsigned long long add2(unsigned long long a, unsigned long long b) {
  unsigned long long d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}

// Warp maximum of a float through the integer reduction unit.
__device__ __forceinline__ float warp_max_redux(float v) {
  const uint32_t key = ordered_bits(__float_as_uint(v));
  uint32_t m;
  asm volatile("redux.sync.max.u32 %0, %1, 0xffffffff;" : "=r"(m) : "r"(key));
  const uint32_t bits = (m & 0x80000000u) ? (m ^ 0x80000000u) : ~m;
  return __uint_as_float(bits);
}

template <int DT> struct ElemTraits;
template <> struct ElemTraits<0> {  // float
  static constexpr int VEC = 4, ESIZE = 4;
  static constexpr uint32_t NEG_INF_WORD = 0xFF800000u;
  __device__ static __forceinline__ float vmax(const uint4& d) {
    return fmaxf(fmaxf(__uint_as_float(d.x), __uint_as_float(d.y)),
                 fmaxf(__uint_as_float(d.z), __uint_as_float(d.w)));
  }
  // sum2 += 2^(x * c - o) for the 4 entries of d
  __device__ static __forceinline__ void accumulate(const uint4& d, unsigned long long c2, unsigned long long no2,
                                                    unsigned long long& sum2) {
    float a, b;
    unpack2(fma2(pack2(__uint_as_float(d.x), __uint_as_float(d.y)), c2, no2), a, b);
    sum2 = add2(sum2, pack2(ex2_approx(a), ex2_approx(b)));
    unpack2(fma2(pack2(__uint_as_float(d.z), __uint_as_float(d.w)), c2, no2), a, b);
    sum2 = add2(sum2, pack2(ex2_approx(a), ex2_approx(b)));
  }
  __device__ static __forceinline__ void unpack(const uint4& d, float (&f)[4]) {
    f[0] = __uint_as_float(d.x); f[1] = __uint_as_float(d.y);
    f[2] = __uint_as_float(d.z); f[3] = __uint_as_float(d.w);
  }
};
template <> struct ElemTraits<1> {  // bfloat16, two per word, lower index in the low half
  static constexpr int VEC = 8, ESIZE = 2;
  static constexpr uint32_t NEG_INF_WORD = 0xFF80FF80u;
  __device__ static __forceinline__ uint32_t vmax_packed(const uint4& d) {
    return max_bf16x2(max_bf16x2(d.x, d.y), max_bf16x2(d.z, d.w));
  }
  __device__ static __forceinline__ float unpack_max(uint32_t m) {
    return fmaxf(__uint_as_float(m << 16), __uint_as_float(m & 0xFFFF0000u));
  }
  __device__ static __forceinline__ float vmax(const uint4& d) { return unpack_max(vmax_packed(d)); }
  __device__ static __forceinline__ void word(uint32_t w, unsigned long long c2, unsigned long long no2,
                                              unsigned long long& sum2) {
    float a, b;
    unpack2(fma2(pack2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u)), c2, no2), a, b);
    sum2 = add2(sum2, pack2(ex2_approx(a), ex2_approx(b)));
  }
  __device__ static __forceinline__ void accumulate(const uint4& d, unsigned long long c2, unsigned long long no2,
                                                    unsigned long long& sum2) {
    word(d.x, c2, no2, sum2); word(d.y, c2, no2, sum2); word(d.z, c2, no2, sum2); word(d.w, c2, no2, sum2);
  }
  __device__ static __forceinline__ void unpack(const uint4& d, float (&f)[8]) {
    f[0] = __uint_as_float(d.x << 16); f[1] = __uint_as_float(d.x & 0xFFFF0000u);
    f[2] = __uint_as_float(d.y << 16); f[3] = __uint_as_float(d.y & 0xFFFF0000u);
    f[4] = __uint_as_float(d.z << 16); f[5] = __uint_as_float(d.z & 0xFFFF0000u);
    f[6] = __uint_as_float(d.w << 16); f[7] = __uint_as_float(d.w & 0xFFFF0000u);
  }
};

// (sum, max) of one chunk held as NV 16-byte vectors per lane; all lanes get the result.
template <int DT, int NV>
__device__ __forceinline__ float2 reduce_chunk(const uint4 (&v)[NV], float c) {
  using TR = ElemTraits<DT>;
  float lane_max;
  if (DT == 1) {
    uint32_t m = ElemTraits<1>::vmax_packed(v[0]);
#pragma unroll
    for (int i = 1; i < NV; ++i) m = max_bf16x2(m, ElemTraits<1>::vmax_packed(v[i]));
    lane_max = ElemTraits<1>::unpack_max(m);
  } else {
    lane_max = TR::vmax(v[0]);
#pragma unroll
    for (int i = 1; i < NV; ++i) lane_max = fmaxf(lane_max, TR::vmax(v[i]));
  }
  const float cm = warp_max_redux(lane_max);
  const float off = chunk_offset(cm, c);
  const unsigned long long c2 = pack2(c, c), no2 = pack2(-off, -off);
  unsigned long long sum2 = pack2(0.0f, 0.0f);
#pragma unroll
  for (int i = 0; i < NV; ++i) TR::accumulate(v[i], c2, no2, sum2);
  float a, b;
  unpack2(sum2, a, b);
  return make_float2(warp_sum_f(a + b), cm);
}

// ---- mbarrier / bulk-copy primitives ---------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait; false if the limit ran out or another thread of the CTA already gave up.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, const volatile int* abort_flag,
                                                  unsigned limit = SPIN_LIMIT) {
  for (unsigned spin = 0; spin < limit; ++spin) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
  }
  return false;
}
__device__ __forceinline__ unsigned long long l2_evict_first_policy() {
  unsigned long long pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ unsigned long long l2_evict_last_policy() {
  unsigned long long pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
// Store of one (sum, max) pair that asks L2 to keep the line: the pairs (a few MB) are read by the
// verification kernel right afterwards and overwritten by the next step, so they need never travel to
// DRAM.  Written back in the shadow of the logit stream they cost 10 us per 1.87 GB pass (measured:
// 272 us with plain stores, 262 us with this hint or with no stores at all): every write-back burst
// turns the DRAM bus around.
__device__ __forceinline__ void store_pair_keep(float2* dst, float2 v, unsigned long long policy) {
  asm volatile("st.global.L2::cache_hint.v2.f32 [%0], {%1, %2}, %3;" ::"l"(dst), "f"(v.x), "f"(v.y), "l"(policy) : "memory");
}
// global -> shared bulk copy (16-byte aligned addresses, size a multiple of 16), completes on `bar`
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar,
                                          unsigned long long policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy)
      : "memory");
}

// ---------------------------------------------------------------------------------
// The streaming kernel.  Requires a 16-byte aligned base and V * sizeof(elem) a
// multiple of 16 (the host checks and falls back to row_pass_plain_kernel).
// ---------------------------------------------------------------------------------
template <int DT, int CW, int CTAS>  // CW consumer warps = chunks per tile; CTAS CTAs per SM share the ring budget
__global__ void __launch_bounds__((CW + 1) * 32, CTAS) row_pass_kernel(const RowPassParams p) {
  using TR = ElemTraits<DT>;
  constexpr int VEC = TR::VEC, NV = CHUNK / (32 * VEC);
  constexpr int STAGE_BYTES = CW * CHUNK * TR::ESIZE;
  constexpr int STAGES = (2 * K1_SMEM_DATA / CTAS) / STAGE_BYTES;
  static_assert(STAGES >= 2, "ring too small");
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ __align__(8) unsigned long long s_full[STAGES], s_empty[STAGES];
  __shared__ volatile int s_abort;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long t0 = (long long)blockIdx.x * p.total_tiles / gridDim.x;
  const long long t1 = (long long)(blockIdx.x + 1) * p.total_tiles / gridDim.x;
  const int n_tiles = (int)(t1 - t0);
  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_addr(&s_full[s]), 1);
      mbar_init(smem_addr(&s_empty[s]), CW);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  pdl_wait();  // chained after the previous step: nothing is read or written before that step has ended
  // Only now may the next kernel of this step be scheduled.  It reads sequence state (trees, candidate lists,
  // tails) before its own wait, and its wait covers this grid only, not the step before: released earlier, it
  // could run while the previous step's last kernel is still writing that state.
  pdl_trigger();
  const size_t row_bytes = (size_t)p.V * TR::ESIZE;
  // tile coordinates advance without divisions
  long long row = t0 / p.tiles_per_row;
  int t = (int)(t0 - row * p.tiles_per_row);

  if (warp == CW) {
    // ---- producer: one lane keeps the ring full ------------------------------------
    if (lane == 0) {
      const unsigned long long policy = l2_evict_first_policy();
      int issued = 0, s = 0;
      uint32_t parity = 1;  // waiting for the phase before the first one succeeds at once
      const char* src_row = (const char*)p.logits + (size_t)row * row_bytes;
      for (int i = 0; i < n_tiles; ++i) {
        if (!mbar_wait_bounded(smem_addr(&s_empty[s]), parity, &s_abort, p.empty_wait_limit)) {
          if (!s_abort && p.status) atomicExch(p.status, K1_ERR_EMPTY_WAIT);
          s_abort = 1;
          break;
        }
        const size_t at = (size_t)t * STAGE_BYTES;
        const uint32_t bytes = (uint32_t)(row_bytes - at < (size_t)STAGE_BYTES ? row_bytes - at : (size_t)STAGE_BYTES);
        const uint32_t bar = smem_addr(&s_full[s]);
        mbar_expect_tx(bar, bytes);
        bulk_load(smem_addr(smem + (size_t)s * STAGE_BYTES), src_row + at, bytes, bar, policy);
        issued = i + 1;
        if (++t == p.tiles_per_row) { t = 0; src_row += row_bytes; }
        if (++s == STAGES) { s = 0; parity ^= 1u; }
      }
      if (s_abort) {
        // leave no copy in flight behind: wait (bounded) for the stages that were issued last
        for (int i = issued > STAGES ? issued - STAGES : 0; i < issued; ++i) {
          const uint32_t bar = smem_addr(&s_full[i % STAGES]);
          for (unsigned spin = 0; spin < SPIN_LIMIT && !mbar_try_wait(bar, (uint32_t)(i / STAGES) & 1u); ++spin) {}
        }
      }
    }
    return;
  }

  // ---- consumers: warp w takes chunk w of every tile -----------------------------------
  const float c = p.c;
  const unsigned long long keep = l2_evict_last_policy();
  int s = 0;
  uint32_t parity = 0;
  float2* out = p.pairs + row * p.n_chunks;
  for (int i = 0; i < n_tiles; ++i) {
    const bool landed = mbar_wait_bounded(smem_addr(&s_full[s]), parity, &s_abort);
    if (!__all_sync(FULL, landed)) {  // warp-uniform: the lanes leave together
      if (lane == 0) {
        if (!s_abort && p.status) atomicExch(p.status, K1_ERR_FULL_WAIT);
        s_abort = 1;
      }
      break;
    }
    const int chunk = t * CW + warp;
    if (chunk < p.n_chunks) {
      const uint4* src = reinterpret_cast<const uint4*>(smem + (size_t)s * STAGE_BYTES + (size_t)warp * CHUNK * TR::ESIZE);
      uint4 v[NV];
#pragma unroll
      for (int k = 0; k < NV; ++k) v[k] = src[k * 32 + lane];
      if ((chunk + 1) * CHUNK > p.V) {  // the row's ragged last chunk: entries past V count as -inf
#pragma unroll
        for (int k = 0; k < NV; ++k)
          if (chunk * CHUNK + (k * 32 + lane) * VEC >= p.V)
            v[k] = make_uint4(TR::NEG_INF_WORD, TR::NEG_INF_WORD, TR::NEG_INF_WORD, TR::NEG_INF_WORD);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_addr(&s_empty[s]));  // the data is in registers: hand the stage back early
      const float2 r = reduce_chunk<DT, NV>(v, c);
      if (lane == 0) store_pair_keep(out + chunk, r, keep);
    } else {
      if (lane == 0) mbar_arrive(smem_addr(&s_empty[s]));
    }
    if (++t == p.tiles_per_row) { t = 0; out += p.n_chunks; }
    if (++s == STAGES) { s = 0; parity ^= 1u; }
  }
}

// Small launches: every chunk is read by a warp of its own, straight from global memory with 16-byte loads
// (same alignment requirement as the streaming kernel).  While the whole launch fits the GPU's resident warps a
// few times over, most of its loads are in flight at once and the pass costs little more than one memory
// round trip plus the transfer, where the streaming kernel's few blocks would still be filling their rings.
// Measured alone, back to back (us per launch, streaming / direct): 64 rows of 151,936 bf16 10.2 / 7.0; 128 rows
// 12.9 / 10.3; 512 rows 29.2 / 28.9; 1,024 rows 50.7 / 55.3: the streaming kernel wins from about ten waves on.
#ifndef STAND_DIRECT_WAVES
#define STAND_DIRECT_WAVES 8  // launches of up to this many waves of resident warps take the direct kernel
#endif
constexpr int DIRECT_WARPS = 8;           // warps (chunks) per block of the direct kernel
constexpr int DIRECT_WARPS_PER_SM = 48;   // resident at its register use

__device__ __forceinline__ uint4 load_stream16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

template <int DT>
__global__ void __launch_bounds__(DIRECT_WARPS * 32) row_pass_direct_kernel(const RowPassParams p) {
  using TR = ElemTraits<DT>;
  constexpr int VEC = TR::VEC, NV = CHUNK / (32 * VEC);
  const int lane = threadIdx.x & 31;
  const long long unit = (long long)blockIdx.x * DIRECT_WARPS + (threadIdx.x >> 5);
  pdl_wait();     // chained after the previous step: nothing is read or written before that step has ended
  pdl_trigger();  // and only then may the next kernel of this step be scheduled (see the streaming kernel)
  if (unit >= p.rows * p.n_chunks) return;
  const long long row = unit / p.n_chunks;
  const int chunk = (int)(unit - row * p.n_chunks);
  const char* src = (const char*)p.logits + ((size_t)row * (size_t)p.V + (size_t)chunk * CHUNK) * TR::ESIZE;
  uint4 v[NV];
#pragma unroll
  for (int k = 0; k < NV; ++k) {  // V is a multiple of the vector length: a vector lies inside the row or past it
    const int e = (k * 32 + lane) * VEC;
    v[k] = chunk * CHUNK + e < p.V ? load_stream16(src + (size_t)e * TR::ESIZE)
                                   : make_uint4(TR::NEG_INF_WORD, TR::NEG_INF_WORD, TR::NEG_INF_WORD, TR::NEG_INF_WORD);
  }
  const float2 r = reduce_chunk<DT, NV>(v, p.c);
  if (lane == 0) store_pair_keep(p.pairs + unit, r, l2_evict_last_policy());
}

// Fallback for rows that are not 16-byte aligned: one warp per (row, chunk), scalar loads.
template <int DT>
__global__ void __launch_bounds__(256) row_pass_plain_kernel(const RowPassParams p) {
  const int lane = threadIdx.x & 31;
  const long long unit = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (unit >= p.rows * p.n_chunks) return;
  const long long row = unit / p.n_chunks;
  const int chunk = (int)(unit - row * p.n_chunks);
  float x[CHUNK / 32];
  float lane_max = -INFINITY;
#pragma unroll
  for (int j = 0; j < CHUNK / 32; ++j) {
    const int v = chunk * CHUNK + j * 32 + lane;
    x[j] = v < p.V ? load_logit(p.logits, DT, row * (long long)p.V + v) : -INFINITY;
    lane_max = fmaxf(lane_max, x[j]);
  }
  const float cm = warp_max_redux(lane_max);
  const float off = chunk_offset(cm, p.c);
  float sum = 0.0f;
#pragma unroll
  for (int j = 0; j < CHUNK / 32; ++j) sum += ex2_approx(fmaf(x[j], p.c, -off));
  sum = warp_sum_f(sum);
  if (lane == 0) p.pairs[unit] = make_float2(sum, cm);
}

// ---------------------------------------------------------------------------
// Per-row results from the chunk pairs.
// ---------------------------------------------------------------------------
struct RowNorm {
  float off;  // o* = largest chunk offset (an integer)
  double Z;   // sum_c s_c 2^(o_c - o*)
};

// All lanes of a warp call this; every lane gets the result.
__device__ __forceinline__ RowNorm row_normaliser(const float2* pairs, int n_chunks, float c, int lane);

// Mass of one chunk relative to the row offset `off` (before division by Z): s * 2^(o - off), exact in
// fp32 (a power-of-two scaling; terms below 2^-126 of the row's largest flush to zero).
__device__ __forceinline__ float chunk_mass_f(float2 pr, float c, float off) {
  const int k = (int)(chunk_offset(pr.y, c) - off);
  const float pw = k >= -126 ? __int_as_float((k + 127) << 23) : 0.0f;
  return pr.x > 0.0f ? pr.x * pw : 0.0f;
}
__device__ __forceinline__ double chunk_mass(float2 pr, float c, float off) { return (double)chunk_mass_f(pr, c, off); }

// All lanes of a warp call this; every lane gets the result.  The row offset is the offset of the largest
// chunk maximum (the offset grows with the maximum).
__device__ __forceinline__ RowNorm row_normaliser(const float2* pairs, int n_chunks, float c, int lane) {
  float mm = -INFINITY;
  for (int ch = lane; ch < n_chunks; ch += 32) mm = fmaxf(mm, pairs[ch].y);
  mm = warp_max_f(mm);
  const float om = chunk_offset(mm, c);
  double z = 0.0;
  for (int ch = lane; ch < n_chunks; ch += 32) z += (double)chunk_mass_f(pairs[ch], c, om);
  RowNorm r;
  r.off = om;
  r.Z = warp_sum_d(z);
  return r;
}

// Keeps the k best of the n buffered candidates at buf[0..k), best first; returns
// the new threshold (the k-th value, or `floor` while fewer than k are known).
__device__ __forceinline__ float compact_topk(uint2* buf, int* cnt, int n, int k, int lane, float floor) {
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
  return keep == k ? fmaxf(floor, __uint_as_float(buf[k - 1].x)) : floor;
}

// inverse of select_key
__device__ __forceinline__ uint32_t key_id(unsigned long long key) { return ~(uint32_t)key; }
__device__ __forceinline__ float key_value(unsigned long long key) {
  const uint32_t o = (uint32_t)(key >> 32);
  const uint32_t bits = (o & 0x80000000u) ? (o ^ 0x80000000u) : ~o;
  return __uint_as_float(bits);
}

// Sec. 4.1: the k entries of one row that the table keeps, by (value descending, id
// ascending), exact.  The k-th largest chunk maximum is a lower bound of the k-th
// largest entry (k different chunks hold an entry at least that large), so only
// chunks whose maximum reaches it can hold a top-k entry: about k of them are read
// again.  Called by all lanes of a warp; buf/cnt are the warp's own shared memory
// (CAND_CAP entries).  On return buf[0..n) holds the entries, best first; returns n.
__device__ __forceinline__ int row_topk_warp(const void* logits, int dtype, long long row, int V, const float2* pairs,
                                             int n_chunks, int k, uint2* buf, int* cnt, int lane) {
  // the k-th largest chunk maximum (chunk index breaks ties, so keys are distinct)
  float tau = -INFINITY;
  if (n_chunks >= k) {
    unsigned long long below = ~0ull;
    for (int r = 0; r < k; ++r) {
      unsigned long long best = 0ull;
      for (int ch = lane; ch < n_chunks; ch += 32) {
        const unsigned long long key = select_key(__float_as_uint(pairs[ch].y), (uint32_t)ch);
        if (key < below && key > best) best = key;
      }
      below = warp_max_u64(best);
    }
    tau = key_value(below);
  }
  const float floor = tau;
  if (lane == 0) *cnt = 0;
  __syncwarp();
  const bool wide = dtype == 1 ? (((uintptr_t)logits & 15) == 0 && (V & 7) == 0)
                               : (((uintptr_t)logits & 15) == 0 && (V & 3) == 0);
  for (int c0 = 0; c0 < n_chunks; c0 += 32) {
    const int mych = c0 + lane;
    unsigned todo = __ballot_sync(FULL, mych < n_chunks && pairs[mych < n_chunks ? mych : 0].y >= floor);
    while (todo) {
      const int ch = c0 + __ffs(todo) - 1;
      todo &= todo - 1;
      // 1024 entries, 32 per lane, in 4 steps of 8 (at most 256 pushes between compaction checks)
#pragma unroll 1
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
          if (f[e] >= tau && idx[e] < V) {
            const int pos = atomicAdd(cnt, 1);
            const float canon = f[e] == 0.0f ? 0.0f : f[e];  // -0 and +0 are one value
            buf[pos] = make_uint2(__float_as_uint(canon), (uint32_t)idx[e]);
          }
        }
        __syncwarp();
        const int n = *(volatile int*)cnt;
        if (n >= COMPACT_AT) tau = compact_topk(buf, cnt, n, k, lane, floor);
      }
    }
  }
  const int n = *(volatile int*)cnt;
  if (n > 0) compact_topk(buf, cnt, n, k, lane, floor);
  return n < k ? n : k;
}

struct RowFinalizeParams {
  const void* logits;
  int dtype, V;
  const float2* pairs;
  const int* status;  // non-zero: the row pass gave up on a wait, its pairs are not to be trusted
  long long rows;
  int n_chunks, topk;
  float c;
  float* lse;
  int* ids;
  float* values;
  float* probs;
};

constexpr int FIN_WARPS = 4;
__global__ void __launch_bounds__(FIN_WARPS * 32) row_finalize_kernel(const RowFinalizeParams p) {
  __shared__ uint2 s_buf[FIN_WARPS][CAND_CAP];
  __shared__ int s_cnt[FIN_WARPS];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const long long row = (long long)blockIdx.x * FIN_WARPS + warp;
  if (row >= p.rows) return;
  if (*p.status != 0) {  // report the failure in-band: NaN and no entries
    if (lane == 0) p.lse[row] = __int_as_float(0x7FC00000);
    if (lane < p.topk) {
      p.ids[row * p.topk + lane] = -1;
      p.values[row * p.topk + lane] = 0.0f;
      p.probs[row * p.topk + lane] = 0.0f;
    }
    return;
  }
  const float2* pairs = p.pairs + row * p.n_chunks;
  const RowNorm nm = row_normaliser(pairs, p.n_chunks, p.c, lane);
  if (lane == 0) p.lse[row] = (float)(((double)nm.off + log2(nm.Z)) * 0.6931471805599453);
  const int n = row_topk_warp(p.logits, p.dtype, row, p.V, pairs, p.n_chunks, p.topk, s_buf[warp], &s_cnt[warp], lane);
  if (lane < p.topk) {
    const long long at = row * p.topk + lane;
    if (lane < n) {
      const uint2 e = s_buf[warp][lane];
      const float x = __uint_as_float(e.x);
      p.ids[at] = (int)e.y;
      p.values[at] = x;
      p.probs[at] = (float)(exp2_d((double)x * (double)p.c - (double)nm.off) / nm.Z);
    } else {
      p.ids[at] = -1;
      p.values[at] = 0.0f;
      p.probs[at] = 0.0f;
    }
  }
}

}  // namespace stand
