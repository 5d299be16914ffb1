// Logit-based N-gram module (paper Sec. 4.1) as one open-addressing hash table in
// device memory.  A slot is one 128-byte line: the context (up to 4 tokens, -1
// padded at the front, so the order is the number of tokens), the number of
// distributions averaged so far, and up to 12 (token id, mean probability) pairs.
// A context is claimed lock-free with a single 16-byte compare-and-swap on the key.
//
// "Efficient logit approximation": a repeat of a context seen c times is merged as
// old * c/(c+1) + new * 1/(c+1) over the union of ids (missing = 0) and cut to the
// top-k again.  The merge is not commutative, so same-step updates of one context
// are applied in record order by the record with the lowest index.
#pragma once
#include "common.cuh"

namespace stand {

struct __align__(128) Slot {
  int key[4];         // -1,-1,-1,-1 = empty
  uint32_t count;     // distributions averaged
  uint32_t n_items;   // stored pairs
  uint32_t pad[2];
  int ids[KMAX];
  float probs[KMAX];
};
static_assert(sizeof(Slot) == 128, "one slot is one 128-byte line");

__device__ __forceinline__ unsigned long long hash_key(const int (&k)[4]) {
  unsigned long long h = 0x9E3779B97F4A7C15ull;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    h ^= (unsigned long long)(uint32_t)k[i];
    h *= 0xFF51AFD7ED558CCDull;
    h ^= h >> 29;
  }
  h *= 0xC4CEB9FE1A85EC53ull;
  h ^= h >> 32;
  return h;
}

__device__ __forceinline__ ulonglong2 cas128(void* addr, ulonglong2 expected, ulonglong2 desired) {
  ulonglong2 old;
  asm volatile(
      "{\n\t.reg .b128 e, d, o;\n\t"
      "mov.b128 e, {%2, %3};\n\t"
      "mov.b128 d, {%4, %5};\n\t"
      "atom.relaxed.gpu.global.cas.b128 o, [%6], e, d;\n\t"
      "mov.b128 {%0, %1}, o;\n\t}"
      : "=l"(old.x), "=l"(old.y)
      : "l"(expected.x), "l"(expected.y), "l"(desired.x), "l"(desired.y), "l"(addr)
      : "memory");
  return old;
}

__device__ __forceinline__ ulonglong2 pack_key(const int (&k)[4]) {
  ulonglong2 r;
  r.x = (unsigned long long)(uint32_t)k[0] | ((unsigned long long)(uint32_t)k[1] << 32);
  r.y = (unsigned long long)(uint32_t)k[2] | ((unsigned long long)(uint32_t)k[3] << 32);
  return r;
}

// Finds the slot of `key`, claiming an empty one if the key is new.  Bounded
// linear probing; NO_SLOT when the limit is reached.
__device__ __forceinline__ uint32_t find_or_insert(Slot* table, unsigned long long mask, int max_probe,
                                                   const int (&key)[4], unsigned long long* stats) {
  const ulonglong2 mine = pack_key(key);
  const ulonglong2 empty = make_ulonglong2(~0ull, ~0ull);
  unsigned long long h = hash_key(key);
  for (int i = 0; i < max_probe; ++i) {
    const unsigned long long s = (h + (unsigned long long)i) & mask;
    const ulonglong2 old = cas128(&table[s], empty, mine);
    const bool claimed = old.x == empty.x && old.y == empty.y;
    if (claimed || (old.x == mine.x && old.y == mine.y)) {
      if (i > 0) atomicMax(&stats[ST_MAX_PROBE], (unsigned long long)i);
      return (uint32_t)s;
    }
  }
  atomicAdd(&stats[ST_DROPS], 1ull);
  return NO_SLOT;
}

// Read-only lookup (no writer may be active).
__device__ __forceinline__ uint32_t find_slot(const Slot* table, unsigned long long mask, int max_probe,
                                              const int (&key)[4]) {
  unsigned long long h = hash_key(key);
  for (int i = 0; i < max_probe; ++i) {
    const unsigned long long s = (h + (unsigned long long)i) & mask;
    const int4 k = *reinterpret_cast<const int4*>(table[s].key);
    if (k.x == key[0] && k.y == key[1] && k.z == key[2] && k.w == key[3]) return (uint32_t)s;
    if (k.x == -1 && k.y == -1 && k.z == -1 && k.w == -1) return NO_SLOT;
  }
  return NO_SLOT;
}

__global__ void table_clear_kernel(Slot* table, unsigned long long n_slots) {
  // one thread per 16 bytes: 8 per slot
  const unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_slots * 8) return;
  uint4* w = reinterpret_cast<uint4*>(table) + i;
  *w = (i & 7) == 0 ? make_uint4(~0u, ~0u, ~0u, ~0u) : make_uint4(0u, 0u, 0u, 0u);
}

// ---------------------------------------------------------------------------
// Update, stage 1: record r = (row, order n) -> slot.  Rows are compressed
// distributions with a context window of n_max tokens; for the step path row =
// (sequence, path position) and only the first n_path[sequence] positions count.
// ---------------------------------------------------------------------------
struct UpdateParams {
  Slot* table;
  unsigned long long mask;
  int max_probe, V, K, n_max;
  long long n_rows;
  const int* rec_ctx;   // [n_rows, n_max]
  const int* rec_ids;   // [n_rows, K]
  const float* rec_p;   // [n_rows, K]
  const int* n_path;    // [n_rows / width] or null (all rows count)
  int width;            // rows per sequence when n_path is given
  uint32_t* rec_slot;   // [n_rows * n_max]
  unsigned long long* stats;
};

__global__ void __launch_bounds__(256) update_locate_kernel(const UpdateParams p) {
  const long long r = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= p.n_rows * p.n_max) return;
  const long long row = r / p.n_max;
  const int n = (int)(r - row * p.n_max) + 1;
  uint32_t slot = NO_SLOT;
  bool live = true;
  if (p.n_path) live = (int)(row % p.width) < p.n_path[row / p.width];
  if (live) {
    int key[4] = {-1, -1, -1, -1};
    bool ok = true;
    for (int i = 0; i < n; ++i) {
      const int t = p.rec_ctx[row * p.n_max + (p.n_max - n + i)];
      if (t < 0) ok = false;           // context shorter than n: this order is skipped
      else if (t >= p.V) { ok = false; atomicAdd(&p.stats[ST_BAD_TOKENS], 1ull); }
      key[4 - n + i] = t;
    }
    if (ok) slot = find_or_insert(p.table, p.mask, p.max_probe, key, p.stats);
  }
  p.rec_slot[r] = slot;
}

// One merge of a compressed row into a slot image held in registers/local memory.
__device__ __forceinline__ void merge_into(int (&ids)[KMAX], float (&probs)[KMAX], uint32_t& count, uint32_t& n_items,
                                           const int* f_ids, const float* f_p, int K) {
  int mid[2 * KMAX];
  double mval[2 * KMAX];
  int n = 0;
  const double c = (double)count;
  const double w_old = c / (c + 1.0), w_new = 1.0 / (c + 1.0);
  for (uint32_t i = 0; i < n_items; ++i) { mid[n] = ids[i]; mval[n] = __dmul_rn((double)probs[i], w_old); ++n; }
  for (int i = 0; i < K; ++i) {
    const int id = f_ids[i];
    if (id < 0) continue;
    const double add = __dmul_rn((double)f_p[i], w_new);
    int at = -1;
    for (int j = 0; j < n; ++j)
      if (mid[j] == id) at = j;
    if (at >= 0) mval[at] = __dadd_rn(mval[at], add);
    else { mid[n] = id; mval[n] = add; ++n; }
  }
  // the k most probable, equal probabilities by lower id
  const int keep = n < K ? n : K;
  for (int r = 0; r < keep; ++r) {
    int best = r;
    for (int j = r + 1; j < n; ++j)
      if (mval[j] > mval[best] || (mval[j] == mval[best] && mid[j] < mid[best])) best = j;
    const int ti = mid[r]; mid[r] = mid[best]; mid[best] = ti;
    const double tv = mval[r]; mval[r] = mval[best]; mval[best] = tv;
    ids[r] = mid[r];
    probs[r] = (float)mval[r];
  }
  n_items = (uint32_t)keep;
  count += 1;
}

// Update, stage 2: the lowest-index record of every slot applies all records of
// that slot in index order (the canonical order of same-step updates).
__global__ void __launch_bounds__(256) update_apply_kernel(const UpdateParams p) {
  const long long n_rec = p.n_rows * p.n_max;
  const long long r = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= n_rec) return;
  const uint32_t slot = p.rec_slot[r];
  if (slot == NO_SLOT) return;
  for (long long i = 0; i < r; ++i)
    if (__ldg(&p.rec_slot[i]) == slot) return;  // an earlier record leads this slot
  Slot* s = &p.table[slot];
  int ids[KMAX];
  float probs[KMAX];
  uint32_t count = s->count, n_items = s->n_items;
  for (int i = 0; i < KMAX; ++i) { ids[i] = s->ids[i]; probs[i] = s->probs[i]; }
  const bool fresh_slot = count == 0;
  unsigned long long applied = 0;
  for (long long i = r; i < n_rec; ++i) {
    if (i != r && __ldg(&p.rec_slot[i]) != slot) continue;
    const long long row = i / p.n_max;
    merge_into(ids, probs, count, n_items, p.rec_ids + row * p.K, p.rec_p + row * p.K, p.K);
    ++applied;
  }
  s->count = count;
  s->n_items = n_items;
  for (int i = 0; i < KMAX; ++i) { s->ids[i] = i < (int)n_items ? ids[i] : 0; s->probs[i] = i < (int)n_items ? probs[i] : 0.0f; }
  atomicAdd(&p.stats[ST_RECORDS], applied);
  if (fresh_slot) atomicAdd(&p.stats[ST_INSERTS], 1ull);
}

// ---------------------------------------------------------------------------
// Export / import.
// ---------------------------------------------------------------------------
__global__ void table_dump_kernel(const Slot* table, unsigned long long n_slots, int K, int* keys, uint32_t* counts,
                                  int* n_items, int* ids, float* probs, unsigned long long cap,
                                  unsigned long long* total) {
  const unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_slots) return;
  const Slot* s = &table[i];
  if (s->key[3] < 0 || s->count == 0) return;
  const unsigned long long at = atomicAdd(total, 1ull);
  if (at >= cap) return;
  for (int t = 0; t < 4; ++t) keys[at * 4 + t] = s->key[t];
  counts[at] = s->count;
  n_items[at] = (int)s->n_items;
  for (int t = 0; t < K; ++t) {
    ids[at * K + t] = t < (int)s->n_items ? s->ids[t] : -1;
    probs[at * K + t] = t < (int)s->n_items ? s->probs[t] : 0.0f;
  }
}

__global__ void table_load_kernel(Slot* table, unsigned long long mask, int max_probe, int K, const int* keys,
                                  const uint32_t* counts, const int* n_items, const int* ids, const float* probs,
                                  unsigned long long M, unsigned long long* stats) {
  const unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= M) return;
  int key[4];
  for (int t = 0; t < 4; ++t) key[t] = keys[i * 4 + t];
  const uint32_t slot = find_or_insert(table, mask, max_probe, key, stats);
  if (slot == NO_SLOT) return;
  Slot* s = &table[slot];
  s->count = counts[i];
  const int n = n_items[i] < K ? n_items[i] : K;
  s->n_items = (uint32_t)n;
  for (int t = 0; t < KMAX; ++t) {
    s->ids[t] = t < n ? ids[i * K + t] : 0;
    s->probs[t] = t < n ? probs[i * K + t] : 0.0f;
  }
}

}  // namespace stand
