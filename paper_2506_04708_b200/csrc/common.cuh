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
constexpr int NODES_MAX = 128;
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
__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const unsigned long long w = __shfl_xor_sync(FULL, v, o);
    v = w > v ? w : v;
  }
  return v;
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
