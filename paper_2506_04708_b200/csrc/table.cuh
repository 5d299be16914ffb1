// Logit-based N-gram module (paper Sec. 4.1) as one open-addressing hash table in
// device memory.  A slot is one 128-byte line: the context (up to 4 tokens, -1
// padded at the front, so the order is the number of tokens), the number of
// distributions averaged so far, and up to 12 (token id, mean probability) pairs.
//
// Probing: double hashing (odd stride over a power-of-two table), so probe
// lengths stay short at high load and do not cluster.  A lookup is made by a
// group of 8 lanes that read 8 probe positions at once: nearly every lookup costs
// one memory round trip.  A context is claimed lock-free with a single 16-byte
// compare-and-swap on the key; entries are never removed, so a key lives at the
// first position of its probe sequence that was free when it arrived.
//
// "Efficient logit approximation": a repeat of a context seen c times is merged as
// old * c/(c+1) + new * 1/(c+1) over the union of ids (missing = 0) and cut to the
// top-k again.  The merge is not commutative, so same-step updates of one context
// are applied in record order: stage 1 notes per slot the lowest record that maps
// to it and how many do; in stage 2 the warp of that record applies them all.
#pragma once
#include "common.cuh"

namespace stand {

constexpr int GROUP = 8;               // lanes that probe together
constexpr uint32_t NO_REC = 0xFFFFFFFFu;

struct __align__(128) Slot {
  int key[4];         // -1,-1,-1,-1 = empty
  uint32_t count;     // distributions averaged
  uint32_t n_items;   // stored pairs
  uint32_t lead;      // during an update: lowest row whose record maps here; NO_REC otherwise
  uint32_t pend;      // during an update: how many records map here; 0 otherwise
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

// Probe i of a key sits at (start + i * stride) & mask; stride is odd, so the
// sequence visits every slot of a power-of-two table.
struct ProbeSeq {
  unsigned long long start, stride;
};
__device__ __forceinline__ ProbeSeq probe_seq(const int (&key)[4], unsigned long long mask) {
  const unsigned long long h = hash_key(key);
  ProbeSeq p;
  p.start = h & mask;
  p.stride = ((h >> 40) | 1ull) & mask;
  if (p.stride == 0) p.stride = 1;
  return p;
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

// One 16-byte key read as a single access, safe against a concurrent cas128.
__device__ __forceinline__ ulonglong2 ld_key_relaxed(const void* addr) {
  ulonglong2 v;
  asm volatile(
      "{\n\t.reg .b128 t;\n\t"
      "ld.relaxed.gpu.global.b128 t, [%2];\n\t"
      "mov.b128 {%0, %1}, t;\n\t}"
      : "=l"(v.x), "=l"(v.y)
      : "l"(addr)
      : "memory");
  return v;
}

__device__ __forceinline__ ulonglong2 pack_key(const int (&k)[4]) {
  ulonglong2 r;
  r.x = (unsigned long long)(uint32_t)k[0] | ((unsigned long long)(uint32_t)k[1] << 32);
  r.y = (unsigned long long)(uint32_t)k[2] | ((unsigned long long)(uint32_t)k[3] << 32);
  return r;
}

// Finds the slot of `key`, claiming a free one if the key is new.  Called by ALL 32
// lanes of a warp; the 8 lanes of a group share one key (`live` false: the group
// has no work and only takes part in the votes).  Bounded: at most max_probe
// positions are tried, then the update is dropped and NO_SLOT returned.
__device__ __forceinline__ uint32_t find_or_insert_group(Slot* table, unsigned long long mask, int max_probe,
                                                         const int (&key)[4], bool live, unsigned long long* stats) {
  const int lane = threadIdx.x & 31, gl = lane & (GROUP - 1), gbase = lane & ~(GROUP - 1);
  const ulonglong2 mine = pack_key(key);
  const ulonglong2 empty = make_ulonglong2(~0ull, ~0ull);
  const ProbeSeq ps = probe_seq(key, mask);
  uint32_t result = NO_SLOT;
  bool done = !live;
  for (int base = 0; __any_sync(FULL, !done); base += GROUP) {
    if (!done && base >= max_probe) {
      done = true;
      if (gl == 0) atomicAdd(&stats[ST_DROPS], 1ull);
    }
    const int i = base + gl;
    const unsigned long long s = (ps.start + (unsigned long long)i * ps.stride) & mask;
    int st = 0;  // 0: another key, 1: this key, 2: free
    if (!done && i < max_probe) {
      const ulonglong2 k = ld_key_relaxed(&table[s]);
      st = (k.x == mine.x && k.y == mine.y) ? 1 : ((k.x == empty.x && k.y == empty.y) ? 2 : 0);
    }
    // settle the positions of this batch in probe order
    for (;;) {
      const unsigned votes = __ballot_sync(FULL, !done && st != 0);
      const unsigned mine_votes = (votes >> gbase) & ((1u << GROUP) - 1u);
      const bool active = !done && mine_votes != 0;
      if (!__any_sync(FULL, active)) break;
      const int first = mine_votes ? __ffs(mine_votes) - 1 : 0;
      int outcome = 0;  // 1: settled at this position, 2: lost the position to another key
      if (active && gl == first) {
        if (st == 1) outcome = 1;
        else {
          const ulonglong2 old = cas128(&table[s], empty, mine);
          const bool ok = (old.x == empty.x && old.y == empty.y) || (old.x == mine.x && old.y == mine.y);
          outcome = ok ? 1 : 2;
        }
      }
      outcome = __shfl_sync(FULL, outcome, gbase + first);
      const unsigned long long s_first = __shfl_sync(FULL, s, gbase + first);
      if (active) {
        if (outcome == 1) {
          result = (uint32_t)s_first;
          done = true;
          if (gl == 0 && base + first > 0) atomicMax(&stats[ST_MAX_PROBE], (unsigned long long)(base + first));
        } else if (gl == first) {
          st = 0;
        }
      }
    }
  }
  return result;
}

// Read-only lookup by a group of 8 lanes (no writer may be active).  Called by ALL
// 32 lanes of a warp, as above.
__device__ __forceinline__ uint32_t find_slot_group(const Slot* table, unsigned long long mask, int max_probe,
                                                    const int (&key)[4], bool live) {
  const int lane = threadIdx.x & 31, gl = lane & (GROUP - 1), gbase = lane & ~(GROUP - 1);
  const ProbeSeq ps = probe_seq(key, mask);
  uint32_t result = NO_SLOT;
  bool done = !live;
  for (int base = 0; __any_sync(FULL, !done); base += GROUP) {
    if (base >= max_probe) done = true;
    const int i = base + gl;
    const unsigned long long s = (ps.start + (unsigned long long)i * ps.stride) & mask;
    int st = 0;
    if (!done && i < max_probe) {
      const int4 k = *reinterpret_cast<const int4*>(table[s].key);
      st = (k.x == key[0] && k.y == key[1] && k.z == key[2] && k.w == key[3]) ? 1
           : ((k.x == -1 && k.y == -1 && k.z == -1 && k.w == -1) ? 2 : 0);
    }
    const unsigned votes = __ballot_sync(FULL, !done && st != 0);
    const unsigned mine_votes = (votes >> gbase) & ((1u << GROUP) - 1u);
    const int first = mine_votes ? __ffs(mine_votes) - 1 : 0;
    const int st_first = __shfl_sync(FULL, st, gbase + first);
    const unsigned long long s_first = __shfl_sync(FULL, s, gbase + first);
    if (!done && mine_votes != 0) {
      if (st_first == 1) result = (uint32_t)s_first;
      done = true;  // the key, or a free position before it: absent
    }
  }
  return result;
}

// Read-only lookup that also brings the whole 128-byte slot: every probing lane reads its slot's eight
// 16-byte words at once, so a hit costs one memory round trip instead of two (key, then contents).
// Returns the slot index or NO_SLOT; *src_lane is the lane that holds the matching slot in `line`.
// Called by ALL 32 lanes of a warp, 8 lanes per key.
__device__ __forceinline__ uint32_t find_slot_group_fetch(const Slot* table, unsigned long long mask, int max_probe,
                                                          const int (&key)[4], bool live, uint4 (&line)[8], int* src_lane) {
  const int lane = threadIdx.x & 31, gl = lane & (GROUP - 1), gbase = lane & ~(GROUP - 1);
  const ProbeSeq ps = probe_seq(key, mask);
  uint32_t result = NO_SLOT;
  *src_lane = gbase;
  bool done = !live;
  for (int base = 0; __any_sync(FULL, !done); base += GROUP) {
    if (base >= max_probe) done = true;
    const int i = base + gl;
    const unsigned long long s = (ps.start + (unsigned long long)i * ps.stride) & mask;
    int st = 0;
    if (!done && i < max_probe) {
      const uint4* w = reinterpret_cast<const uint4*>(&table[s]);
#pragma unroll
      for (int t = 0; t < 8; ++t) line[t] = w[t];
      const uint4 k = line[0];
      st = ((int)k.x == key[0] && (int)k.y == key[1] && (int)k.z == key[2] && (int)k.w == key[3]) ? 1
           : ((k.x & k.y & k.z & k.w) == 0xFFFFFFFFu ? 2 : 0);
    }
    const unsigned votes = __ballot_sync(FULL, !done && st != 0);
    const unsigned mine_votes = (votes >> gbase) & ((1u << GROUP) - 1u);
    const int first = mine_votes ? __ffs(mine_votes) - 1 : 0;
    const int st_first = __shfl_sync(FULL, st, gbase + first);
    const unsigned long long s_first = __shfl_sync(FULL, s, gbase + first);
    if (!done && mine_votes != 0) {
      if (st_first == 1) { result = (uint32_t)s_first; *src_lane = gbase + first; }
      done = true;  // the key, or a free position before it: absent
    }
  }
  return result;
}

__global__ void table_clear_kernel(Slot* table, unsigned long long n_slots) {
  // one thread per 16 bytes: 8 per slot
  const unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_slots * 8) return;
  uint4* w = reinterpret_cast<uint4*>(table) + i;
  const int part = (int)(i & 7);
  *w = part == 0 ? make_uint4(~0u, ~0u, ~0u, ~0u) : (part == 1 ? make_uint4(0u, 0u, NO_REC, 0u) : make_uint4(0u, 0u, 0u, 0u));
}

// ---------------------------------------------------------------------------
// Update, stage 1: record (row, order n) -> slot.  Rows are compressed
// distributions with a context window of n_max tokens; for the step path row =
// (sequence, path position) and only the first n_path[sequence] positions count.
// One group of 8 lanes per record.  rec_slot is laid out [n_max][n_rows], so the
// records that can share a slot (same order) are contiguous.
// ---------------------------------------------------------------------------
struct UpdateParams {
  Slot* table;
  unsigned long long mask;
  int max_probe, V, K, n_max;
  long long n_rows;
  const int* rec_ctx;   // [n_rows, n_max]   rows ctx_stride words apart
  const int* rec_ids;   // [n_rows, K]       rows item_stride words apart
  const float* rec_p;   // [n_rows, K]       rows item_stride words apart
  int ctx_stride, item_stride;  // n_max and K for separate arrays; the row length for rows packed as (ctx, ids, probs)
  const int* n_path;    // [n_rows / width] or null (all rows count)
  int width;            // rows per sequence when n_path is given
  uint32_t* rec_slot;   // [n_max, n_rows]
  unsigned long long* stats;
};

// The locate step of one record; called by all lanes of a warp, 8 lanes per record.  check_path false: the
// row is known to lie on its sequence's accepted path (n_path need not have been written yet).
__device__ __forceinline__ void locate_record(const UpdateParams& p, long long row, int n, bool in_range, bool check_path = true) {
  const int gl = threadIdx.x & (GROUP - 1);
  int key[4] = {-1, -1, -1, -1};
  bool ok = in_range;
  if (ok && check_path && p.n_path) ok = (int)(row % p.width) < p.n_path[row / p.width];
  if (ok) {
    for (int i = 0; i < n; ++i) {
      const int t = p.rec_ctx[row * p.ctx_stride + (p.n_max - n + i)];
      if (t < 0) ok = false;  // context shorter than n: this order is skipped
      else if (t >= p.V) {
        ok = false;
        if (gl == 0) atomicAdd(&p.stats[ST_BAD_TOKENS], 1ull);
      }
      key[4 - n + i] = t;
    }
  }
  const uint32_t slot = find_or_insert_group(p.table, p.mask, p.max_probe, key, ok, p.stats);
  if (in_range && gl == 0) {
    p.rec_slot[(long long)(n - 1) * p.n_rows + row] = slot;
    if (slot != NO_SLOT) {
      atomicMin(&p.table[slot].lead, (uint32_t)row);
      atomicAdd(&p.table[slot].pend, 1u);
    }
  }
}

__global__ void __launch_bounds__(256) update_locate_kernel(const UpdateParams p) {
  pdl_trigger();
  pdl_wait();  // the rows may come from the kernel before this one
  const long long g = ((long long)blockIdx.x * blockDim.x + threadIdx.x) / GROUP;  // record index
  const bool in_range = g < p.n_rows * p.n_max;
  const long long row = in_range ? g / p.n_max : 0;
  const int n = in_range ? (int)(g - row * p.n_max) + 1 : 1;
  locate_record(p, row, n, in_range);
}

// ---------------------------------------------------------------------------
// One merge of a compressed row into a slot image in shared memory, by a whole
// warp.  Lanes 0..11 carry the stored pairs, lanes 16..27 the fresh ones; equal
// ids are paired, every lane ranks its pair among all of them by (probability
// descending, id ascending), and the K best are written back.
// ---------------------------------------------------------------------------
struct SlotImage {
  uint32_t count, n_items;
  int ids[KMAX];
  float probs[KMAX];
  // working area of a merge: the pairs of all 32 lanes (id < 0: no pair)
  double m_val[32];
  int m_id[32];
};

// Lanes exchange their pairs through shared memory rather than shuffles: a lane reads the other pairs
// with independent loads, which a single warp overlaps, where a chain of shuffles costs its full
// latency each (measured: 3,000 cycles per merge with shuffles and match_any).  The loops below have constant
// trip counts and read before they compare, so that the loads of a phase are issued together.
// The fresh row arrives in registers: lane 16 + t carries entry t (fid < 0: none).
__device__ __forceinline__ void merge_warp(SlotImage* img, int fid, float fp, int K, int lane) {
  // weights c / (c + 1) and 1 / (c + 1): single-precision reciprocal refined by one Newton step in double (relative
  // error about 4e-15; a double division would put some two hundred dependent cycles into every merge of a chain)
  const double c = (double)img->count, c1 = c + 1.0;
  const double r0 = (double)__frcp_rn((float)c1);
  const double w_new = r0 * (2.0 - c1 * r0), w_old = c * w_new;
  const int n_items = (int)img->n_items;
  int id = -1;
  double val = 0.0;
  if (lane < KMAX) {
    if (lane < n_items) { id = img->ids[lane]; val = __dmul_rn((double)img->probs[lane], w_old); }
  } else if (lane >= 16 && lane < 16 + K) {
    if (fid >= 0) { id = fid; val = __dmul_rn((double)fp, w_new); }
  }
  img->m_id[lane] = id;
  img->m_val[lane] = val;
  __syncwarp();
  // a fresh id that is already stored: the stored pair absorbs it, the fresh lane drops out.  Every lane reads the
  // ids of the other half (stored lanes the fresh ones and the other way round) with independent loads first.
  {
    const int base = lane < 16 ? 16 : 0;
    int other[KMAX];
#pragma unroll
    for (int t = 0; t < KMAX; ++t) other[t] = img->m_id[base + t];
    int match = -1;
#pragma unroll
    for (int t = 0; t < KMAX; ++t)
      if (other[t] == id) match = t;  // ids of one half are distinct: at most one match
    if (id >= 0 && match >= 0) {
      if (lane < 16) val = __dadd_rn(val, img->m_val[16 + match]);
      else id = -1;
    }
  }
  __syncwarp();
  img->m_id[lane] = id;
  img->m_val[lane] = val;
  __syncwarp();
  // rank of this lane's pair among all pairs by (value descending, id ascending); eight pairs are read at a time.
  // The values are non-negative doubles, which order like their bit patterns read as integers: the comparisons
  // run on the integer units.
  int rank = 0;
  const long long vbits = __double_as_longlong(val);
  const long long* m_bits = reinterpret_cast<const long long*>(img->m_val);
  static_assert(KMAX == 12, "pairs sit at 0..11 (stored) and 16..27 (fresh)");
#pragma unroll
  for (int j0 = 0; j0 < 32; j0 += 16) {
#pragma unroll
    for (int h = 0; h < KMAX; h += 6) {
      int idj[6];
      long long vj[6];
#pragma unroll
      for (int t = 0; t < 6; ++t) { idj[t] = img->m_id[j0 + h + t]; vj[t] = m_bits[j0 + h + t]; }
#pragma unroll
      for (int t = 0; t < 6; ++t)  // no short-circuit operators: they compile to divergent branches, one pair at a time
        rank += (int)((idj[t] >= 0) & ((vj[t] > vbits) | ((vj[t] == vbits) & (idj[t] < id))));
    }
  }
  const int n_valid = __popc(__ballot_sync(FULL, id >= 0));
  if (id >= 0 && rank < K) { img->ids[rank] = id; img->probs[rank] = (float)val; }
  if (lane == 0) { img->n_items = (uint32_t)(n_valid < K ? n_valid : K); img->count += 1; }
  __syncwarp();
}

// Update, stage 2: one warp per record.  The warp of the lowest row of a slot
// applies all records of that slot in row order (the canonical order of same-step
// updates) and closes the slot's update fields.
constexpr int APPLY_WARPS = 8;
// Entry t of compressed row i for lane 16 + t (other lanes: none).
__device__ __forceinline__ void load_fresh(const UpdateParams& p, long long i, int lane, int& fid, float& fp) {
  fid = -1;
  fp = 0.0f;
  if (lane >= 16 && lane < 16 + p.K) {
    fid = p.rec_ids[i * p.item_stride + (lane - 16)];
    fp = p.rec_p[i * p.item_stride + (lane - 16)];
  }
}

// Record g (order-major index) by one warp; img is the warp's working image of the slot.
__device__ __forceinline__ void apply_record(const UpdateParams& p, const long long g, SlotImage* img, const int lane) {
  if (g >= p.n_rows * p.n_max) return;
  // order-major, so that the warps of a block work on neighbouring rows of one order
  const int n = (int)(g / p.n_rows) + 1;
  const long long row = g - (long long)(n - 1) * p.n_rows;
  const uint32_t* seg = p.rec_slot + (long long)(n - 1) * p.n_rows;
  // one round trip: the record's slot, its compressed row, and the first window of later records
  const uint32_t slot = seg[row];
  int fid;
  float fp;
  load_fresh(p, row, lane, fid, fp);
  constexpr int WIN = 4;
  long long i0 = (row + 1) & ~31ll;
  uint32_t got[WIN];
#pragma unroll
  for (int w = 0; w < WIN; ++w) {
    const long long i = i0 + 32 * w + lane;
    got[w] = (i > row && i < p.n_rows) ? seg[i] : NO_SLOT;
  }
  if (slot == NO_SLOT) return;
  // second round trip: the whole 128-byte slot, one word per lane (key 0-3, count, n_items, lead, pend, ids, probs)
  uint32_t* line = reinterpret_cast<uint32_t*>(&p.table[slot]);
  const uint32_t word = line[lane];
  if (__shfl_sync(FULL, word, 6) != (uint32_t)row) return;  // another record leads this slot
  const uint32_t pending = __shfl_sync(FULL, word, 7);
  if (lane == 4) img->count = word;
  if (lane == 5) img->n_items = word;
  if (lane >= 8 && lane < 8 + KMAX) img->ids[lane - 8] = (int)word;
  if (lane >= 8 + KMAX) img->probs[lane - 8 - KMAX] = __uint_as_float(word);
  __syncwarp();
  const bool fresh_slot = img->count == 0;
  merge_warp(img, fid, fp, p.K, lane);
  uint32_t applied = 1;
  // the other records of this slot, in row order; four 32-wide windows of rec_slot are in flight at once, and the
  // compressed row of the next record is requested before the current one is merged
  while (applied < pending && i0 < p.n_rows) {
#pragma unroll
    for (int w = 0; w < WIN; ++w) {
      unsigned hits = __ballot_sync(FULL, got[w] == slot);
      if (hits) load_fresh(p, i0 + 32 * w + __ffs(hits) - 1, lane, fid, fp);
      while (hits) {
        hits &= hits - 1;
        const int cfid = fid;
        const float cfp = fp;
        if (hits) load_fresh(p, i0 + 32 * w + __ffs(hits) - 1, lane, fid, fp);
        merge_warp(img, cfid, cfp, p.K, lane);
        ++applied;
      }
    }
    i0 += 32 * WIN;
    if (applied < pending && i0 < p.n_rows) {
#pragma unroll
      for (int w = 0; w < WIN; ++w) {
        const long long i = i0 + 32 * w + lane;
        got[w] = i < p.n_rows ? seg[i] : NO_SLOT;
      }
    }
  }
  // the slot goes back as one line: update fields closed, entries past n_items zeroed
  const int n_items = (int)img->n_items;
  uint32_t out = word;  // key words unchanged
  if (lane == 4) out = img->count;
  if (lane == 5) out = img->n_items;
  if (lane == 6) out = NO_REC;
  if (lane == 7) out = 0u;
  if (lane >= 8 && lane < 8 + KMAX) out = lane - 8 < n_items ? (uint32_t)img->ids[lane - 8] : 0u;
  if (lane >= 8 + KMAX) out = lane - 8 - KMAX < n_items ? __float_as_uint(img->probs[lane - 8 - KMAX]) : 0u;
  line[lane] = out;
  if (lane == 0) {
    atomicAdd(&p.stats[ST_RECORDS], (unsigned long long)applied);
    if (fresh_slot) atomicAdd(&p.stats[ST_INSERTS], 1ull);
  }
}

__global__ void __launch_bounds__(APPLY_WARPS * 32) update_apply_kernel(const UpdateParams p) {
  __shared__ SlotImage s_img[APPLY_WARPS];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  pdl_trigger();
  pdl_wait();  // records and slot marks come from stage 1
  apply_record(p, (long long)blockIdx.x * APPLY_WARPS + warp, &s_img[warp], lane);
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

// One group of 8 lanes per entry.
__global__ void __launch_bounds__(256) table_load_kernel(Slot* table, unsigned long long mask, int max_probe, int K,
                                                         const int* keys, const uint32_t* counts, const int* n_items,
                                                         const int* ids, const float* probs, unsigned long long M,
                                                         unsigned long long* stats) {
  const unsigned long long i = ((unsigned long long)blockIdx.x * blockDim.x + threadIdx.x) / GROUP;
  const int gl = threadIdx.x & (GROUP - 1);
  const bool live = i < M;
  int key[4] = {-1, -1, -1, -1};
  if (live)
    for (int t = 0; t < 4; ++t) key[t] = keys[i * 4 + t];
  const uint32_t slot = find_or_insert_group(table, mask, max_probe, key, live, stats);
  if (!live || slot == NO_SLOT || gl != 0) return;
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
