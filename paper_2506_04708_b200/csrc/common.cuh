// Shared device helpers of the STAND CUDA library (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <math.h>

namespace stand {

constexpr unsigned FULL = 0xFFFFFFFFu;
constexpr int CHUNK = 1024;  // vocabulary entries per chunk: one (sum, offset) pair each
constexpr int KMAX = 12;     // STAND_MAX_TOPK
constexpr int ORDER_MAX = 4; // STAND_MAX_ORDER
constexpr int NODES_MAX = 640;  // STAND_MAX_NODES
constexpr int DEPTH_MAX = 32;
constexpr int VOCAB_MAX = 1 << 20;  // STAND_MAX_VOCAB

constexpr uint32_t SLOT_FINAL = 0x40000000u;
constexpr uint32_t SLOT_GUMBEL = 0x80000000u;
constexpr uint32_t NO_SLOT = 0xFFFFFFFFu;

// indices into the device statistics block (uint64 each)
enum Stat {
  ST_STEPS = 0, ST_EMITTED, ST_RECORDS, ST_INSERTS, ST_DROPS, ST_BAD_TOKENS, ST_LOOKUPS,
  ST_HIT0, ST_HIT1, ST_HIT2, ST_HIT3, ST_MAX_PROBE, ST_COUNT = 16
};

// ---------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al. 2011), counter = (sequence, step, node, slot),
// key = seed.  Returns the top 24 bits of output word 0.
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t philox_u24(unsigned long long seed, uint32_t b, uint32_t step, uint32_t node,
                                               uint32_t slot) {
  uint32_t c0 = b, c1 = step, c2 = node, c3 = slot;
  uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return c0 >> 8;
}

// ---------------------------------------------------------------------------
// Programmatic dependent launch: a kernel of the step lets the next one start being scheduled at once
// (pdl_trigger) and the next one stops before it reads anything the previous one wrote (pdl_wait, which
// returns once the previous grid has completed and its writes are visible).  Both are no-ops in a kernel
// that was launched without the attribute.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---------------------------------------------------------------------------
// warp helpers
// ---------------------------------------------------------------------------
__device__ __forceinline__ float warp_max_f(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(FULL, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum_f(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(FULL, v, o);
  return v;
}
__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(FULL, v, o);
  return v;
}
__device__ __forceinline__ uint32_t warp_max_u32(uint32_t v) {
  uint32_t m;
  asm volatile("redux.sync.max.u32 %0, %1, 0xffffffff;" : "=r"(m) : "r"(v));
  return m;
}
// 64-bit maximum as two passes through the integer reduction unit: high words, then the low words of
// the lanes that hold the largest high word.
__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v) {
  const uint32_t hi = (uint32_t)(v >> 32), lo = (uint32_t)v;
  const uint32_t mh = warp_max_u32(hi);
  const uint32_t ml = warp_max_u32(hi == mh ? lo : 0u);
  return ((unsigned long long)mh << 32) | ml;
}

// ---------------------------------------------------------------------------
// Short double-precision helpers for the serial parts of the step (a library exp2 or scalbn costs
// several times as many dependent instructions).
// ---------------------------------------------------------------------------
// 2^k exactly; 0 below the normal range (such terms are far below one ulp of any sum they enter).
__device__ __forceinline__ double pow2_int(int k) {
  if (k < -1022) return 0.0;
  if (k > 1023) k = 1023;
  return __longlong_as_double((long long)(k + 1023) << 52);
}
// 2^t for t <= ~1000, relative error below 1e-14: t = n + f, |f| <= 1/2, Taylor series of 2^f to degree 11.
__device__ __forceinline__ double exp2_d(double t) {
  if (!(t > -1100.0)) return 0.0;
  const int n = __double2int_rn(t);
  const double f = (t - (double)n) * 0.6931471805599453094;
  double r = 1.0 / 39916800.0;
  r = fma(r, f, 1.0 / 3628800.0);
  r = fma(r, f, 1.0 / 362880.0);
  r = fma(r, f, 1.0 / 40320.0);
  r = fma(r, f, 1.0 / 5040.0);
  r = fma(r, f, 1.0 / 720.0);
  r = fma(r, f, 1.0 / 120.0);
  r = fma(r, f, 1.0 / 24.0);
  r = fma(r, f, 1.0 / 6.0);
  r = fma(r, f, 0.5);
  r = fma(r, f, 1.0);
  r = fma(r, f, 1.0);
  return r * pow2_int(n);
}

// Order-preserving map float bits -> uint32 (larger float = larger integer).
__device__ __forceinline__ uint32_t ordered_bits(uint32_t bits) {
  return bits ^ ((uint32_t)((int32_t)bits >> 31) | 0x80000000u);
}
// Selection key of a (value, id) pair: larger value first, equal values by lower id.
__device__ __forceinline__ unsigned long long select_key(uint32_t value_bits, uint32_t id) {
  return ((unsigned long long)ordered_bits(value_bits) << 32) | (uint32_t)~id;
}

// One logit as float.  dtype 0: float, 1: bfloat16 (upper half of a float).
__device__ __forceinline__ float load_logit(const void* base, int dtype, long long index) {
  if (dtype == 0) return __ldg((const float*)base + index);
  const unsigned short h = __ldg((const unsigned short*)base + index);
  return __uint_as_float((uint32_t)h << 16);
}

}  // namespace stand
