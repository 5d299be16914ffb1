/* STAND speculative-sampling hot path for NVIDIA B200 (sm_100a): C interface.
 *
 * One decoding step passes once over the target logits of every draft-tree
 * node (B sequences x N tree nodes x V vocabulary entries) and then
 *   1. verifies the drafted tree by speculative sampling (paper Sec. 3.2 and
 *      Sec. 4.2 "Stochastic tree drafting"),
 *   2. feeds the accepted rows into the logit-based N-gram module (Sec. 4.1),
 *   3. drafts the next tree from that module with Gumbel-Top-K (Sec. 4.2).
 * The target model is not part of this library: logits are an input.
 *
 * Conventions
 *   - Pointers named dev_* are DEVICE pointers, host_* are HOST pointers.  The
 *     caller owns every buffer it passes, including the workspace; the library
 *     keeps the workspace pointer until stand_destroy.
 *   - `cu_stream` is a cudaStream_t passed as void* (NULL = default stream).
 *     Calls that take a stream only enqueue work and return; they do not
 *     synchronise unless stated.
 *   - Return value: STAND_OK (0) or a negative STAND_E_* code.  Problems found
 *     on the device (table full, probe limit, token id out of range) never trap:
 *     they are counted and reported by stand_get_stats.
 *   - Layouts are row-major, innermost dimension contiguous.
 *   - Tree: node 0 is the root and carries the last token of the sequence;
 *     parent[u] < u; nodes are numbered breadth-first so that the children of a
 *     node are consecutive and ordered by draft rank.  Row (b,u) of the logits
 *     is the target distribution of the token that FOLLOWS node u.
 *   - Randomness: Philox4x32-10, key = seed, counter = (sequence, step, node,
 *     slot), first output word, top 24 bits.  Slot j < 2^30: accept test of the
 *     child of rank j; 0x40000000: the final sample of a walk; 0x80000000|t:
 *     Gumbel noise of candidate token t.
 */
#ifndef STAND_H_
#define STAND_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define STAND_MAX_TOPK 12   /* entries kept per context (one 128-byte table slot) */
#define STAND_MAX_ORDER 4   /* N-gram orders 1..4 (Sec. 4.1) */
#define STAND_MAX_NODES 640 /* tree nodes per sequence (Algorithm 1's initial tree has 625) */
#define STAND_MAX_DEPTH 32
#define STAND_MAX_VOCAB (1 << 20)

#define STAND_DTYPE_F32 0
#define STAND_DTYPE_BF16 1

#define STAND_OK 0
#define STAND_E_ARG (-1)       /* invalid argument or configuration */
#define STAND_E_WORKSPACE (-2) /* workspace missing, misaligned or too small */
#define STAND_E_CUDA (-3)      /* a CUDA runtime call failed */
#define STAND_E_STATE (-4)     /* call not valid in the current state */
#define STAND_E_TOO_LARGE (-5) /* problem does not fit the library's built-in scratch buffer */

typedef struct stand_ctx stand_ctx;

typedef struct {
  int32_t B;           /* sequences, >= 1 */
  int32_t N;           /* tree nodes per sequence, root included, 1..STAND_MAX_NODES */
  int32_t V;           /* vocabulary size, 2..STAND_MAX_VOCAB */
  int32_t topk;        /* entries kept per context, 1..STAND_MAX_TOPK */
  int32_t order_max;   /* N-gram orders 1..order_max, <= STAND_MAX_ORDER */
  int32_t dtype;       /* STAND_DTYPE_* of the logits */
  float temperature;   /* > 0 (Sec. 5: all sampling at temperature T) */
  int32_t max_probe;   /* hash-table probe limit, >= 1 (0 = default 96) */
  uint64_t seed;
  uint64_t table_slots;   /* power of two, >= 2; one slot = 128 bytes */
  const int32_t* parent;  /* HOST, [N]; parent[0] = -1; read during stand_init only */
  int32_t deterministic;   /* 0: stochastic drafting (Sec. 4.2); 1: deterministic drafting (Sec. 3.2): the children of a
                              node are its most probable candidates in order, each verified as a one-hot draft */
  int32_t host_staging;    /* != 0: reserve a logits staging buffer for stand_step_host */
  int32_t seq_base;        /* global index of this context's sequence 0, >= 0.  The random-number counters use
                              seq_base + b, so a batch split over several contexts draws what the whole batch would */
  int32_t reserved;        /* must be 0 */
} stand_config;

typedef struct {
  uint64_t steps;           /* verifications run */
  uint64_t emitted_tokens;  /* tokens emitted (accepted + sampled) */
  uint64_t records;         /* (context, order) updates applied */
  uint64_t inserts;         /* new contexts created */
  uint64_t drops;           /* updates lost: probe limit reached / table full */
  uint64_t bad_tokens;      /* token ids outside [0, V) met on the device */
  uint64_t lookups;         /* drafting lookups (one per tree node with children) */
  uint64_t lookup_hits[STAND_MAX_ORDER]; /* hits by order-1 */
  uint64_t max_probe_seen;  /* longest probe sequence */
  uint64_t wait_timeouts;   /* non-zero: a bounded wait inside a kernel ran out (results of that step are invalid) */
} stand_stats;

/* Bytes of device workspace a configuration needs; 0 if the configuration is invalid. */
size_t stand_workspace_bytes(const stand_config* cfg);

/* Creates a context in caller-owned device memory (256-byte aligned, at least
 * stand_workspace_bytes).  Clears the N-gram tables, uploads the topology and
 * synchronises the device once.  The sequences start empty: call
 * stand_reset_sequences before the first step. */
int stand_init(const stand_config* cfg, void* dev_workspace, size_t bytes, stand_ctx** out);

/* Frees the host-side context.  Device memory stays with the caller. */
int stand_destroy(stand_ctx* ctx);

/* (Re)starts all sequences.  dev_tail [B, order_max] int32: the last tokens of each
 * prompt, -1 padded at the front; dev_len [B] int64: tokens so far.  The N-gram
 * tables are kept: the module persists across trajectories (Sec. 5.1).  The draft
 * tree is cleared, so the next verification samples one token from the root row. */
int stand_reset_sequences(stand_ctx* ctx, const int32_t* dev_tail, const int64_t* dev_len, void* cu_stream);

/* Sec. 3.2 + Sec. 4.2: one pass over dev_logits [B, N, V] (temperature softmax
 * statistics and per-row top-k), then the verification walk of every sequence:
 * drafted children are tested in draft order with the speculative-sampling ratio
 * (recursive rejection, residual target, rejected token removed from the draft
 * distribution); at the stop node one token is drawn by inverse CDF in token order.
 * Writes dev_emitted [B, D+1] int32 (-1 padded; D = tree depth) and dev_n_emitted
 * [B] int32, advances the sequences and the step counter, and records the
 * accepted rows for stand_ngram_update. */
int stand_verify_tree(stand_ctx* ctx, const void* dev_logits, int32_t* dev_emitted, int32_t* dev_n_emitted,
                      void* cu_stream);

/* Sec. 4.1: feeds the rows accepted by the last verification into the tables,
 * under every order 1..order_max whose context is available: a new context stores
 * the row's top-k probabilities with count 1; a known one is averaged with weights
 * c/(c+1) and 1/(c+1) (missing ids = 0), cut to the top-k, count c+1.  Updates are
 * applied in (sequence, path position, order) order.  STAND_E_STATE if there is no
 * pending verification. */
int stand_ngram_update(stand_ctx* ctx, void* cu_stream);

/* Sec. 4.1 without logits: M rows, each a context window (dev_ctx [M, order_max],
 * the tokens before the predicted position, -1 padded at the front) and a
 * compressed distribution (dev_ids [M, topk], -1 = unused; dev_probs [M, topk]);
 * applied in row order, each under every order it is long enough for. */
int stand_ngram_update_bulk(stand_ctx* ctx, const int32_t* dev_ctx, const int32_t* dev_ids, const float* dev_probs,
                            int64_t M, void* cu_stream);

/* Sec. 4.1 when the sequences of one N-gram module are split over several contexts (one per GPU): the
 * accepted rows of the last verification in the layout stand_ngram_update_bulk takes.  Writes B * (D+1)
 * rows in (sequence, path position) order: dev_ctx [B*(D+1), order_max], dev_ids / dev_probs
 * [B*(D+1), topk].  Positions past a sequence's accepted path get an all -1 context, ids -1 and
 * probabilities 0; a bulk update skips them.  Every context then applies the rows of all contexts,
 * concatenated in the order of their seq_base, with stand_ngram_update_bulk: each table ends up as the
 * table of one context that held all the sequences.  STAND_E_STATE without a pending verification. */
int stand_export_records(stand_ctx* ctx, int32_t* dev_ctx, int32_t* dev_ids, float* dev_probs, void* cu_stream);

/* The same exchange with one buffer per context: row r of dev_rows [B*(D+1), order_max + 2*topk] int32 holds the
 * context window, then the ids, then the probabilities (float bit patterns) of row r as stand_export_records
 * writes them, so the rows of all contexts travel in ONE gather; stand_ngram_update_packed applies M such rows
 * in row order, exactly as stand_ngram_update_bulk applies the three arrays. */
int stand_export_records_packed(stand_ctx* ctx, int32_t* dev_rows, void* cu_stream);
int stand_ngram_update_packed(stand_ctx* ctx, const int32_t* dev_rows, int64_t M, void* cu_stream);

/* Drops the pending verification's own update (its rows reach the tables through
 * stand_ngram_update_bulk instead).  Host only.  STAND_E_STATE if no verification is pending. */
int stand_skip_update(stand_ctx* ctx);

/* Sec. 4.2: drafts the next tree of every sequence.  Breadth-first over the static
 * topology; for a node with children the contexts of order order_max..1 are looked
 * up, the first hit gives up to topk candidates (id, phi); the children are the
 * candidates with the largest log(phi) - log(-log U) (Gumbel-Top-K), in that order.
 * Nodes that cannot be drafted get -1.  Writes dev_tree_tokens [B, N] int32 (may be
 * NULL) and keeps the tree and the candidate lists for the next verification. */
int stand_draft_tree(stand_ctx* ctx, int32_t* dev_tree_tokens, void* cu_stream);

/* All kernels of the hot path are launched with programmatic stream serialisation: each may be scheduled while
 * the kernel before it in the stream is draining, and stops (griddepcontrol.wait) before it reads anything that
 * kernel may have written, whichever kernel it is; the stage calls above therefore chain like the fused step.
 *
 * verify -> update -> draft on one stream, no host synchronisation: two kernel launches for up to 16
 * sequences (the row pass, then verification, update and drafting in one block, or in one thread-block
 * cluster with a block per sequence), four for larger batches. */
int stand_step(stand_ctx* ctx, const void* dev_logits, int32_t* dev_emitted, int32_t* dev_n_emitted,
               int32_t* dev_tree_tokens, void* cu_stream);

/* The same step for callers whose buffers live in HOST memory: copies host_logits
 * [B, N, V] to the staging buffer (needs cfg.host_staging), runs the step, copies
 * the three results back and synchronises the stream before returning. */
int stand_step_host(stand_ctx* ctx, const void* host_logits, int32_t* host_emitted, int32_t* host_n_emitted,
                    int32_t* host_tree_tokens, void* cu_stream);

/* The row pass on its own (Sec. 5 temperature softmax, Sec. 4.1 top-k), without a
 * context: for each of `rows` rows of dev_logits [rows, V] writes the log-sum-exp of
 * x/T (dev_lse [rows] float), and the top-k entries by (value descending, id
 * ascending): dev_ids [rows, topk] int32, dev_values [rows, topk] float (input
 * values), dev_probs [rows, topk] float (softmax probabilities).  dev_scratch must
 * hold stand_row_stats_scratch_bytes bytes, 256-byte aligned.  Inputs are -inf or
 * finite with |x| * log2(e) / T < 2^24 (beyond that the fp32 exponent offsets lose their
 * integer precision); the same holds for every entry point that takes logits.  If a bounded wait inside the kernel runs out (never seen; it guards against a
 * hang), every dev_lse entry is NaN and every id -1. */
size_t stand_row_stats_scratch_bytes(int64_t rows, int32_t V, int32_t dtype, int32_t topk);
int stand_row_stats(const void* dev_logits, int64_t rows, int32_t V, int32_t dtype, float temperature, int32_t topk,
                    void* dev_scratch, size_t scratch_bytes, float* dev_lse, int32_t* dev_ids, float* dev_values,
                    float* dev_probs, void* cu_stream);

/* stand_row_stats for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this entry point exists for the library's users, not for the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a region
 * that must not synchronise the device or grow its memory footprint (a serving loop
 * with a fixed memory budget, a plugin that is handed buffers by its host and has no
 * allocator of its own, a latency-critical path where an allocation could stall on
 * other streams).  Such a caller still owns the input and the four outputs; only the
 * scratch memory that stand_row_stats asks for is replaced by a buffer that is part
 * of the library image: STAND_STATIC_SCRATCH_BYTES of device memory, held by every
 * GPU that loads the library from load until the process exits.
 *
 * Same arguments, results and layouts as stand_row_stats, minus the scratch pair.
 * Differences:
 *   - Shapes whose scratch need (stand_row_stats_scratch_bytes) exceeds
 *     STAND_STATIC_SCRATCH_BYTES are refused with STAND_E_TOO_LARGE; nothing is
 *     launched.
 *   - The first call on a device looks up the buffer's device address (once per
 *     device, for the device that is current at the call) and caches it.  Make that
 *     first call outside any stream capture.
 *   - All calls on a device share the one buffer, and it keeps the previous call's
 *     contents.  Each call clears the one word that must start at zero and overwrites
 *     every other scratch entry it later reads; but two calls whose kernels overlap on the GPU (different
 *     streams without an ordering between them) race on it.  Order such calls.
 *   - No cudaMalloc, cudaFree or other allocating routine is called, here or below. */
#define STAND_STATIC_SCRATCH_BYTES (8u << 20)
int stand_row_stats_static(const void* dev_logits, int64_t rows, int32_t V, int32_t dtype, float temperature,
                           int32_t topk, float* dev_lse, int32_t* dev_ids, float* dev_values, float* dev_probs,
                           void* cu_stream);

/* Synchronises the stream the context last used and copies the counters. */
int stand_get_stats(stand_ctx* ctx, stand_stats* host_out);

/* Results of the last verification, for inspection: accepted path dev_path [B, D+1]
 * (node indices, -1 padded) and the compressed rows that will be fed to the tables,
 * dev_ids / dev_probs [B, D+1, topk].  Any pointer may be NULL. */
int stand_last_path(stand_ctx* ctx, int32_t* dev_path, int32_t* dev_ids, float* dev_probs, void* cu_stream);
int32_t stand_tree_depth(const stand_ctx* ctx);

/* Table export/import.  Device arrays: keys [cap, 4] int32 (-1 padded at the front),
 * counts [cap] uint32, n_items [cap] int32, ids [cap, topk] int32, probs [cap, topk]
 * float.  dump writes at most `cap` entries in arbitrary order and the total number
 * of contexts to dev_total [1] uint64.  load inserts M entries (clear != 0 empties
 * the tables first). */
int stand_table_dump(stand_ctx* ctx, int32_t* dev_keys, uint32_t* dev_counts, int32_t* dev_n_items, int32_t* dev_ids,
                     float* dev_probs, uint64_t cap, uint64_t* dev_total, void* cu_stream);
int stand_table_load(stand_ctx* ctx, const int32_t* dev_keys, const uint32_t* dev_counts, const int32_t* dev_n_items,
                     const int32_t* dev_ids, const float* dev_probs, uint64_t M, int32_t clear, void* cu_stream);

/* Sequence state export/import (checkpoint/resume): tails [B, order_max], lengths
 * [B] int64, tree tokens [B, N], candidate lists cand_n [B, N], cand_id / cand_phi
 * [B, N, topk], and the step counter (host).  load discards a pending verification and checks the tree
 * against the candidate lists: a drafted node whose token is outside the vocabulary, missing from its parent's
 * candidate list (the draft distribution its verification divides by) or below an undrafted parent is cleared
 * (-1) and counted in stand_stats.bad_tokens; candidate counts are clamped to [0, topk]. */
int stand_state_dump(stand_ctx* ctx, int32_t* dev_tail, int64_t* dev_len, int32_t* dev_tree, int32_t* dev_cand_n,
                     int32_t* dev_cand_id, float* dev_cand_phi, uint32_t* host_step, void* cu_stream);
int stand_state_load(stand_ctx* ctx, const int32_t* dev_tail, const int64_t* dev_len, const int32_t* dev_tree,
                     const int32_t* dev_cand_n, const int32_t* dev_cand_id, const float* dev_cand_phi,
                     uint32_t step, void* cu_stream);

/* Timing hook for benchmarks: when both events (cudaEvent_t as void*) are non-NULL, every later
 * verification records ev_before on the stream just before the row-pass kernel and ev_after just
 * after it, so the caller can time that kernel alone.  NULL, NULL switches the hook off. */
int stand_profile_row_pass(stand_ctx* ctx, void* ev_before, void* ev_after);

/* Sec. 4.2 "Data-driven draft tree optimization", the measuring half: how often each node of the static
 * tree lay on the accepted path since stand_init (or the last reset).  Synchronises the stream the context
 * last used, copies N counters to host_counts and, if reset != 0, clears them.  The root is on every path,
 * so host_counts[0] = sequences x steps. */
int stand_node_accepts(stand_ctx* ctx, uint64_t* host_counts, int32_t reset);

/* The selecting half: keeps the `keep` nodes with the highest counts (equal counts: the lower index), the
 * root included.  A node is never accepted more often than its parent, so the kept set is closed under
 * parents.  Host only.  Writes the parent array of the smaller tree to host_parent_out [keep], in the same
 * breadth-first numbering convention, and to host_old_index [keep] (may be NULL) the node each kept node
 * was.  STAND_E_ARG if keep < 1, keep > n or the input is not a valid tree. */
int stand_prune_tree(const int32_t* host_parent, int32_t n, const uint64_t* host_counts, int32_t keep,
                     int32_t* host_parent_out, int32_t* host_old_index);

/* App. A.1, Algorithm 1: the initial tree that the optimisation starts from.  Nodes are created level by
 * level for `levels` levels below the root (20 in the paper: 625 nodes); a node of depth 0 gets 8 children,
 * of depth 1 max(8 - 2 * order, 1), deeper ones max(ceil((siblings - 1) / (0.7 * order + 1)), floor) with
 * floor 2 at depths 2 and 3 and 0 below, where `order` is the node's rank among its siblings and
 * `siblings` its parent's child count; the first node of every level gets at least 3.  Host only.  Writes
 * the first min(capacity, total) nodes in creation order (a prefix is closed under parents) to
 * host_parent / host_depth / host_order (the last two may be NULL) and the total to *total_nodes. */
int stand_initial_tree(int32_t levels, int32_t* host_parent, int32_t* host_depth, int32_t* host_order, int32_t capacity,
                       int32_t* total_nodes);

/* Timing hook for benchmarks: events [5] (cudaEvent_t as void*, any may be NULL) are recorded on the
 * stream by every later step at: before the row pass, after it, after the verification walk, after the
 * table update, after drafting.  A NULL array switches the hook off. */
int stand_profile_stages(stand_ctx* ctx, void* const* events);

/* Failure handling of the streaming kernel, made testable.  Every wait inside the kernels is bounded; when one
 * runs out the kernel records it, lets its copies in flight land and returns, and the host sees
 * stand_stats.wait_timeouts (or NaN / -1 results from stand_row_stats): the GPU context stays usable.  This
 * call sets, for the whole process, how many polls the kernel's loader spends waiting for a free stage of its
 * shared-memory ring: 1 .. 2^22 (the default, about a second); 0 makes its very first wait give up before
 * anything was copied, which is how the tests reach the failure path; a negative value restores the default.
 * Larger values are clamped: a wait cannot be made unbounded. */
int stand_set_wait_limit(int64_t polls);

/* How many kernels the library has launched through this context so far. */
uint64_t stand_launch_count(const stand_ctx* ctx);

const char* stand_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* STAND_H_ */
