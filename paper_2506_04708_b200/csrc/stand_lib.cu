// C interface of the STAND CUDA library: context, workspace layout, launches.
// Declarations and the meaning of every argument: include/stand.h.
#include "../../include/stand.h"

#include <cuda_runtime.h>
#include <atomic>
#include <new>
#include <vector>
#include <stdio.h>
#include <string.h>

#include "common.cuh"
#include "draft.cuh"
#include "row_pass.cuh"
#include "table.cuh"
#include "tail.cuh"
#include "verify.cuh"

using namespace stand;

namespace {

constexpr int BULK_ROWS = 16384;  // rows per batch of the bulk update

struct Layout {
  size_t table, topo, tail, len, tree, cand_n, cand_id, cand_phi, pairs, emitted, n_path, path, rec_ctx, rec_ids,
      rec_p, rec_slot, stats, accepts, status, staging, total;
};

inline size_t align_up(size_t x) { return (x + 255) & ~(size_t)255; }

struct Derived {
  int D, n_chunks;
  int parent[NODES_MAX], first_child[NODES_MAX], n_children[NODES_MAX], depth[NODES_MAX], level_start[DEPTH_MAX + 2];
};

bool derive(const stand_config* c, Derived* d) {
  if (!c) return false;
  if (c->B < 1 || c->N < 1 || c->N > STAND_MAX_NODES || c->V < 2 || c->V > STAND_MAX_VOCAB) return false;
  if (c->topk < 1 || c->topk > STAND_MAX_TOPK || c->order_max < 1 || c->order_max > STAND_MAX_ORDER) return false;
  if (c->dtype != STAND_DTYPE_F32 && c->dtype != STAND_DTYPE_BF16) return false;
  if (!(c->temperature > 0.0f) || c->max_probe < 0 || (c->deterministic != 0 && c->deterministic != 1)) return false;
  if (c->seq_base < 0 || (long long)c->seq_base + c->B > 0x7FFFFFFFll || c->reserved != 0) return false;
  if (c->table_slots < 2 || (c->table_slots & (c->table_slots - 1)) != 0 || c->table_slots > (1ull << 32) - 2) return false;
  if (!c->parent || c->parent[0] != -1) return false;
  if ((long long)c->B * c->N > (1ll << 31) / 4) return false;
  memset(d, 0, sizeof(*d));
  d->parent[0] = -1;
  d->D = 0;
  for (int u = 0; u < c->N; ++u) d->first_child[u] = -1;
  for (int u = 1; u < c->N; ++u) {
    const int par = c->parent[u];
    if (par < 0 || par >= u) return false;
    if (u > 1 && par < c->parent[u - 1]) return false;  // breadth-first numbering, siblings contiguous
    d->parent[u] = par;
    d->depth[u] = d->depth[par] + 1;
    if (d->depth[u] < d->depth[u - 1]) return false;
    if (d->depth[u] > STAND_MAX_DEPTH) return false;
    if (d->first_child[par] < 0) d->first_child[par] = u;
    d->n_children[par] += 1;
    if (d->depth[u] > d->D) d->D = d->depth[u];
  }
  for (int u = 0; u < c->N; ++u)
    if (d->first_child[u] < 0) d->first_child[u] = 0;
  for (int l = 0; l <= d->D + 1; ++l) d->level_start[l] = c->N;
  for (int u = c->N - 1; u >= 0; --u) d->level_start[d->depth[u]] = u;
  d->n_chunks = (c->V + CHUNK - 1) / CHUNK;
  return true;
}

size_t esize_of(int dtype) { return dtype == STAND_DTYPE_F32 ? 4 : 2; }

void layout_of(const stand_config* c, const Derived* d, Layout* L) {
  const size_t B = c->B, N = c->N, K = c->topk, W = d->D + 1, n = c->order_max;
  size_t rec_rows = B * W;
  if (rec_rows < (size_t)BULK_ROWS) rec_rows = BULK_ROWS;
  size_t at = 0;
  auto take = [&](size_t bytes) { const size_t here = at; at = align_up(at + bytes); return here; };
  L->table = take((size_t)c->table_slots * sizeof(Slot));
  L->topo = take((4 * NODES_MAX + DEPTH_MAX + 2) * sizeof(int));
  L->tail = take(B * n * 4);
  L->len = take(B * 8);
  L->tree = take(B * N * 4);
  L->cand_n = take(B * N * 4);
  L->cand_id = take(B * N * K * 4);
  L->cand_phi = take(B * N * K * 4);
  L->pairs = take(B * N * (size_t)d->n_chunks * sizeof(float2));
  L->emitted = take(B * W * 4);
  L->n_path = take(B * 4);
  L->path = take(B * W * 4);
  L->rec_ctx = take(B * W * n * 4);
  L->rec_ids = take(B * W * K * 4);
  L->rec_p = take(B * W * K * 4);
  L->rec_slot = take(rec_rows * n * 4);
  L->stats = take(ST_COUNT * 8);
  L->accepts = take(NODES_MAX * 8);
  L->status = take(64);
  L->staging = take(c->host_staging ? B * N * (size_t)c->V * esize_of(c->dtype) : 0);
  L->total = at;
}

}  // namespace

struct stand_ctx {
  stand_config cfg;
  Derived d;
  Layout L;
  char* ws;
  uint32_t step;
  bool pending;
  bool located;  // the pending verification already mapped its records to slots
  uint64_t launches;
  cudaStream_t last_stream;
  int max_probe;
  int tail_form;  // 0: three kernels; 1: one block (single sequence); 2: one cluster of B blocks
  float c;  // log2(e) / T
  cudaEvent_t ev_before, ev_after;  // optional timing hook around the row pass
  cudaEvent_t ev_stage[5];          // optional timing hook at the stage boundaries of a step

  template <typename T> T* at(size_t off) const { return reinterpret_cast<T*>(ws + off); }
  int* topo_parent() const { return at<int>(L.topo); }
  int* topo_first_child() const { return at<int>(L.topo) + NODES_MAX; }
  int* topo_n_children() const { return at<int>(L.topo) + 2 * NODES_MAX; }
  int* topo_depth() const { return at<int>(L.topo) + 3 * NODES_MAX; }
  int* topo_level_start() const { return at<int>(L.topo) + 4 * NODES_MAX; }
};

namespace {

int cuda_ok(cudaError_t e) { return e == cudaSuccess ? STAND_OK : STAND_E_CUDA; }
int launch_ok() { return cuda_ok(cudaGetLastError()); }

float log2e_over_T(float T) { return (float)(1.4426950408889634 / (double)T); }

bool rows_aligned(const void* base, int V, int dtype) {
  const size_t es = esize_of(dtype);
  return ((uintptr_t)base % 16 == 0) && (((size_t)V * es) % 16 == 0);
}

template <typename P>
int launch_dependent(void (*kernel)(P), unsigned grid, unsigned block, cudaStream_t st, const P& params, size_t smem = 0);

// The streaming kernel needs more dynamic shared memory than the default limit: raise it once per device.
constexpr int MAX_DEVICES = 64;
std::atomic<unsigned> g_empty_wait_limit{SPIN_LIMIT};  // stand_set_wait_limit
std::atomic<int> g_k1_ready[MAX_DEVICES];
std::atomic<int> g_sm_count[MAX_DEVICES];

int prepare_device(int* sm_count) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return STAND_E_CUDA;
  if (dev < 0 || dev >= MAX_DEVICES) return STAND_E_ARG;
  if (!g_k1_ready[dev].load(std::memory_order_acquire)) {
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return STAND_E_CUDA;
    if (cudaFuncSetAttribute(row_pass_kernel<0, K1Shape<0>::CW, K1_CTAS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             k1_smem_bytes<0>()) != cudaSuccess)
      return STAND_E_CUDA;
    if (cudaFuncSetAttribute(row_pass_kernel<1, K1Shape<1>::CW, K1_CTAS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             k1_smem_bytes<1>()) != cudaSuccess)
      return STAND_E_CUDA;
    // large trees keep their per-node state in more shared memory than the default limit
    if (cudaFuncSetAttribute(verify_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)verify_smem_bytes(NODES_MAX)) !=
        cudaSuccess)
      return STAND_E_CUDA;
    if (cudaFuncSetAttribute(tail_single_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)verify_smem_bytes(NODES_MAX)) !=
            cudaSuccess ||
        cudaFuncSetAttribute(verify_wide_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)verify_smem_bytes(NODES_MAX)) !=
            cudaSuccess)
      return STAND_E_CUDA;
    if (cudaFuncSetAttribute(tail_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)verify_smem_bytes(NODES_MAX)) !=
            cudaSuccess ||
        cudaFuncSetAttribute(tail_cluster_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess)
      return STAND_E_CUDA;
    g_sm_count[dev].store(sms, std::memory_order_relaxed);
    g_k1_ready[dev].store(1, std::memory_order_release);
  }
  *sm_count = g_sm_count[dev].load(std::memory_order_relaxed);
  return STAND_OK;
}

int launch_row_pass(const void* logits, long long rows, int V, int dtype, int n_chunks, float c, float2* pairs, int* status,
                    cudaStream_t st, bool chain = false) {
  RowPassParams rp;
  rp.logits = logits; rp.rows = rows; rp.V = V; rp.n_chunks = n_chunks; rp.c = c; rp.pairs = pairs; rp.status = status;
  rp.empty_wait_limit = g_empty_wait_limit.load(std::memory_order_relaxed);
  const int tile_chunks = dtype == STAND_DTYPE_BF16 ? K1Shape<1>::CW : K1Shape<0>::CW;
  rp.tiles_per_row = (n_chunks + tile_chunks - 1) / tile_chunks;
  rp.total_tiles = rows * rp.tiles_per_row;
  if (rows <= 0 || rows * n_chunks > 0x7FFFFFFFll * 8) return STAND_E_ARG;
  if (rows_aligned(logits, V, dtype)) {
    int sms = 0;
    const int rc = prepare_device(&sms);
    if (rc) return rc;
    const long long units = rows * n_chunks;
    if (units <= (long long)STAND_DIRECT_WAVES * DIRECT_WARPS_PER_SM * sms) {  // small: one warp per chunk, everything in flight at once
      const unsigned blocks = (unsigned)((units + DIRECT_WARPS - 1) / DIRECT_WARPS);
      if (chain) {
        if (dtype == STAND_DTYPE_BF16) return launch_dependent(row_pass_direct_kernel<1>, blocks, DIRECT_WARPS * 32u, st, rp);
        return launch_dependent(row_pass_direct_kernel<0>, blocks, DIRECT_WARPS * 32u, st, rp);
      }
      if (dtype == STAND_DTYPE_BF16) row_pass_direct_kernel<1><<<blocks, DIRECT_WARPS * 32, 0, st>>>(rp);
      else row_pass_direct_kernel<0><<<blocks, DIRECT_WARPS * 32, 0, st>>>(rp);
      return launch_ok();
    }
    const long long want = (long long)K1_CTAS * sms;  // each CTA walks a contiguous range of tiles
    const unsigned grid = (unsigned)(rp.total_tiles < want ? rp.total_tiles : want);
    if (chain) {  // may be scheduled while the previous step's last kernel drains; waits for it before any access
      if (dtype == STAND_DTYPE_BF16)
        return launch_dependent(row_pass_kernel<1, K1Shape<1>::CW, K1_CTAS>, grid, (K1Shape<1>::CW + 1) * 32, st, rp,
                                (size_t)k1_smem_bytes<1>());
      return launch_dependent(row_pass_kernel<0, K1Shape<0>::CW, K1_CTAS>, grid, (K1Shape<0>::CW + 1) * 32, st, rp,
                              (size_t)k1_smem_bytes<0>());
    }
    if (dtype == STAND_DTYPE_BF16)
      row_pass_kernel<1, K1Shape<1>::CW, K1_CTAS><<<grid, (K1Shape<1>::CW + 1) * 32, k1_smem_bytes<1>(), st>>>(rp);
    else
      row_pass_kernel<0, K1Shape<0>::CW, K1_CTAS><<<grid, (K1Shape<0>::CW + 1) * 32, k1_smem_bytes<0>(), st>>>(rp);
  } else {
    const unsigned blocks = (unsigned)((rows * n_chunks + 7) / 8);
    if (dtype == STAND_DTYPE_BF16) row_pass_plain_kernel<1><<<blocks, 256, 0, st>>>(rp);
    else row_pass_plain_kernel<0><<<blocks, 256, 0, st>>>(rp);
  }
  return launch_ok();
}

// Launch with programmatic stream serialisation: the kernel may be scheduled while its predecessor in the
// stream is still running; it calls pdl_wait() before it touches the predecessor's results.
template <typename P>
int launch_dependent(void (*kernel)(P), unsigned grid, unsigned block, cudaStream_t st, const P& params, size_t smem) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cuda_ok(cudaLaunchKernelEx(&cfg, kernel, params));
}

// The same, as one thread-block cluster of `grid` blocks.
template <typename P>
int launch_dependent_cluster(void (*kernel)(P), unsigned grid, unsigned block, cudaStream_t st, const P& params, size_t smem) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = grid;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cuda_ok(cudaLaunchKernelEx(&cfg, kernel, params));
}

// Can one cluster of B tail blocks run on this device?  (Asked once, at stand_init.)
bool cluster_tail_fits(int B, size_t smem) {
  if (B < 2 || B > TAIL_CLUSTER_MAX) return false;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)B);
  cfg.blockDim = dim3(TAIL_THREADS);
  cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)B;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int clusters = 0;
  if (cudaOccupancyMaxActiveClusters(&clusters, tail_cluster_kernel, &cfg) != cudaSuccess) {
    cudaGetLastError();  // not an error of the library: the batch takes the three-kernel form
    return false;
  }
  return clusters >= 1;
}

UpdateParams update_params(stand_ctx* x, long long n_rows, const int* ctxw, const int* ids, const float* probs,
                           const int* n_path, int width, int packed_stride = 0) {
  const stand_config& c = x->cfg;
  UpdateParams u;
  u.table = x->at<Slot>(x->L.table); u.mask = c.table_slots - 1; u.max_probe = x->max_probe; u.V = c.V; u.K = c.topk;
  u.n_max = c.order_max; u.n_rows = n_rows; u.rec_ctx = ctxw; u.rec_ids = ids; u.rec_p = probs; u.n_path = n_path;
  u.ctx_stride = packed_stride ? packed_stride : c.order_max;
  u.item_stride = packed_stride ? packed_stride : c.topk;
  u.width = width; u.rec_slot = x->at<uint32_t>(x->L.rec_slot); u.stats = x->at<unsigned long long>(x->L.stats);
  return u;
}

UpdateParams step_update_params(stand_ctx* x) {
  const int W = x->d.D + 1;
  return update_params(x, (long long)x->cfg.B * W, x->at<int>(x->L.rec_ctx), x->at<int>(x->L.rec_ids),
                       x->at<float>(x->L.rec_p), x->at<int>(x->L.n_path), W);
}

VerifyParams verify_params(stand_ctx* x, const void* logits, int32_t* emitted, int32_t* n_emitted, bool fuse_locate) {
  const stand_config& c = x->cfg;
  VerifyParams v;
  v.logits = logits; v.dtype = c.dtype; v.B = c.B; v.N = c.N; v.V = c.V; v.K = c.topk; v.n_max = c.order_max;
  v.D = x->d.D; v.n_chunks = x->d.n_chunks; v.c = x->c; v.seed = c.seed; v.step = x->step;
  v.first_child = x->topo_first_child(); v.n_children = x->topo_n_children();
  v.pairs = x->at<float2>(x->L.pairs);
  v.tail = x->at<int>(x->L.tail); v.len = x->at<long long>(x->L.len); v.tree = x->at<int>(x->L.tree);
  v.cand_n = x->at<int>(x->L.cand_n); v.cand_id = x->at<int>(x->L.cand_id); v.cand_phi = x->at<float>(x->L.cand_phi);
  v.emitted_user = emitted; v.n_emitted_user = n_emitted;
  v.emitted = x->at<int>(x->L.emitted); v.n_path = x->at<int>(x->L.n_path); v.path = x->at<int>(x->L.path);
  v.rec_ctx = x->at<int>(x->L.rec_ctx); v.rec_ids = x->at<int>(x->L.rec_ids); v.rec_p = x->at<float>(x->L.rec_p);
  v.stats = x->at<unsigned long long>(x->L.stats);
  v.node_accepts = x->at<unsigned long long>(x->L.accepts);
  v.deterministic = c.deterministic;
  v.seq_base = c.seq_base;
  v.fuse_locate = fuse_locate ? 1 : 0;
  v.upd = step_update_params(x);
  return v;
}

DraftParams draft_params(stand_ctx* x, int32_t* tree_user) {
  const stand_config& c = x->cfg;
  DraftParams d;
  d.table = x->at<Slot>(x->L.table); d.mask = c.table_slots - 1; d.max_probe = x->max_probe; d.B = c.B; d.N = c.N;
  d.K = c.topk; d.n_max = c.order_max; d.D = x->d.D; d.V = c.V; d.seed = c.seed; d.step = x->step;
  d.parent = x->topo_parent(); d.first_child = x->topo_first_child(); d.n_children = x->topo_n_children();
  d.level_start = x->topo_level_start(); d.tail = x->at<int>(x->L.tail); d.tree = x->at<int>(x->L.tree);
  d.tree_user = tree_user; d.cand_n = x->at<int>(x->L.cand_n); d.cand_id = x->at<int>(x->L.cand_id);
  d.cand_phi = x->at<float>(x->L.cand_phi); d.stats = x->at<unsigned long long>(x->L.stats);
  d.deterministic = c.deterministic;
  d.seq_base = c.seq_base;
  return d;
}

// fuse_locate: the verification kernel also maps this step's records to table slots (stage 1 of the update).
int run_verify(stand_ctx* x, const void* logits, int32_t* emitted, int32_t* n_emitted, bool fuse_locate, cudaStream_t st) {
  const stand_config& c = x->cfg;
  if (x->ev_before) cudaEventRecord(x->ev_before, st);
  if (x->ev_stage[0]) cudaEventRecord(x->ev_stage[0], st);
  int rc = launch_row_pass(logits, (long long)c.B * c.N, c.V, c.dtype, x->d.n_chunks, x->c, x->at<float2>(x->L.pairs),
                           x->at<int>(x->L.status), st, !x->ev_before && !x->ev_stage[0]);
  if (rc) return rc;
  if (x->ev_after) cudaEventRecord(x->ev_after, st);
  if (x->ev_stage[1]) cudaEventRecord(x->ev_stage[1], st);
  x->launches += 1;
  x->step += 1;  // the tree drafted in step s-1 is verified in step s
  const VerifyParams v = verify_params(x, logits, emitted, n_emitted, fuse_locate);
  // with no timing events between the launches the kernels chain programmatically
  const bool chain = !x->ev_after && !x->ev_stage[1];
  const size_t vsm = verify_smem_bytes(c.N);
  // a batch that leaves every block a multiprocessor of its own takes the wide form (the extra warps locate the records)
  int sms = 0;
  rc = prepare_device(&sms);
  if (rc) return rc;
  const bool wide = fuse_locate && c.B <= sms;
  if (chain) rc = wide ? launch_dependent(verify_wide_kernel, (unsigned)c.B, K2_WIDE_THREADS, st, v, vsm)
                       : launch_dependent(verify_kernel, (unsigned)c.B, K2_THREADS, st, v, vsm);
  else if (wide) { verify_wide_kernel<<<c.B, K2_WIDE_THREADS, vsm, st>>>(v); rc = launch_ok(); }
  else { verify_kernel<<<c.B, K2_THREADS, vsm, st>>>(v); rc = launch_ok(); }
  if (rc) return rc;
  if (x->ev_stage[2]) cudaEventRecord(x->ev_stage[2], st);
  x->launches += 1;
  x->pending = true;
  x->located = fuse_locate;
  return STAND_OK;
}

int run_update_rows(stand_ctx* x, const UpdateParams& u, bool located, cudaStream_t st) {
  const long long n_rec = u.n_rows * u.n_max;
  int rc;
  // both stages stop (griddepcontrol.wait) before they read anything, so they may be scheduled while the kernel
  // before them in the stream drains, whichever kernel that is
  const bool chain = !x->ev_stage[2];
  if (!located) {
    const unsigned locate_blocks = (unsigned)((n_rec * GROUP + 255) / 256);
    if (chain) rc = launch_dependent(update_locate_kernel, locate_blocks, 256u, st, u);
    else { update_locate_kernel<<<locate_blocks, 256, 0, st>>>(u); rc = launch_ok(); }
    if (rc) return rc;
    x->launches += 1;
  }
  const unsigned apply_blocks = (unsigned)((n_rec + APPLY_WARPS - 1) / APPLY_WARPS);
  if (chain) rc = launch_dependent(update_apply_kernel, apply_blocks, APPLY_WARPS * 32, st, u);
  else { update_apply_kernel<<<apply_blocks, APPLY_WARPS * 32, 0, st>>>(u); rc = launch_ok(); }
  if (rc) return rc;
  x->launches += 1;
  return STAND_OK;
}

int run_update(stand_ctx* x, cudaStream_t st) {
  const int rc = run_update_rows(x, step_update_params(x), x->located, st);
  if (rc == STAND_OK) { x->pending = false; x->located = false; }
  if (x->ev_stage[3]) cudaEventRecord(x->ev_stage[3], st);
  return rc;
}

int run_draft(stand_ctx* x, int32_t* tree_user, bool chained, cudaStream_t st) {
  const stand_config& c = x->cfg;
  const DraftParams d = draft_params(x, tree_user);
  int rc;
  if (chained && !x->ev_stage[3]) rc = launch_dependent(draft_kernel, (unsigned)c.B, K4_THREADS, st, d);
  else { draft_kernel<<<c.B, K4_THREADS, 0, st>>>(d); rc = launch_ok(); }
  if (rc == STAND_OK) x->launches += 1;
  if (x->ev_stage[4]) cudaEventRecord(x->ev_stage[4], st);
  return rc;
}

bool timing_hooks(const stand_ctx* x) {
  if (x->ev_before || x->ev_after) return true;
  for (int i = 0; i < 5; ++i)
    if (x->ev_stage[i]) return true;
  return false;
}

// One whole step on a stream.  A single sequence and a small batch take two launches (row pass, then the
// whole tail in one block or one cluster); larger batches take four.
int run_step(stand_ctx* x, const void* logits, int32_t* emitted, int32_t* n_emitted, int32_t* tree_user, cudaStream_t st) {
  const stand_config& c = x->cfg;
  if (x->tail_form != 0 && !timing_hooks(x)) {
    int rc = launch_row_pass(logits, (long long)c.B * c.N, c.V, c.dtype, x->d.n_chunks, x->c, x->at<float2>(x->L.pairs),
                             x->at<int>(x->L.status), st, true);
    if (rc) return rc;
    x->step += 1;
    TailParams t;
    t.v = verify_params(x, logits, emitted, n_emitted, true);
    t.d = draft_params(x, tree_user);
    if (x->tail_form == 1) rc = launch_dependent(tail_single_kernel, 1u, TAIL_THREADS, st, t, verify_smem_bytes(c.N));
    else rc = launch_dependent_cluster(tail_cluster_kernel, (unsigned)c.B, TAIL_THREADS, st, t, verify_smem_bytes(c.N));
    if (rc) return rc;
    x->launches += 2;
    x->pending = false;
    x->located = false;
    return STAND_OK;
  }
  int rc = run_verify(x, logits, emitted, n_emitted, true, st);
  if (rc) return rc;
  rc = run_update(x, st);
  if (rc) return rc;
  return run_draft(x, tree_user, true, st);
}

__global__ void reset_tree_kernel(int B, int N, int n_max, const int* tail, int* tree, int* cand_n) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (long long)B * N) return;
  const int b = (int)(i / N), u = (int)(i % N);
  tree[i] = u == 0 ? tail[b * n_max + n_max - 1] : -1;
  cand_n[i] = 0;
}

// After a state import: a drafted node must carry a token of the vocabulary that its parent's candidate list
// holds (that list is the draft distribution the verification divides by), under a drafted parent.  A node
// that does not is cleared and counted; candidate counts are clamped to the list's capacity.
__global__ void validate_state_kernel(int B, int N, int K, int V, const int* parent, int* tree, int* cand_n, const int* cand_id,
                                      unsigned long long* stats) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (long long)B * N) return;
  const int b = (int)(i / N), v = (int)(i % N);
  int cn = cand_n[i];
  if (cn < 0 || cn > K) { cn = cn < 0 ? 0 : K; cand_n[i] = cn; }
  if (v == 0) return;
  const int tok = tree[i];
  if (tok < 0) return;
  const int par = parent[v];
  const long long pi = (long long)b * N + par;
  bool ok = tok < V && (par == 0 || tree[pi] >= 0);
  if (ok) {
    int pn = cand_n[pi];
    pn = pn < 0 ? 0 : (pn > K ? K : pn);
    bool listed = false;
    for (int t = 0; t < pn; ++t) listed |= cand_id[pi * K + t] == tok;
    ok = listed;
  }
  if (!ok) {
    tree[i] = -1;
    atomicAdd(&stats[ST_BAD_TOKENS], 1ull);
  }
}

// The records of the last verification as rows for a bulk update: positions past a sequence's accepted
// path get an all -1 context (a bulk update skips such a row), ids -1 and probabilities 0.
struct ExportParams {
  int B, W, n_max, K;
  const int* n_path;
  const int* rec_ctx;
  const int* rec_ids;
  const float* rec_p;
  int* out_ctx;
  int* out_ids;
  float* out_p;
  int ctx_stride, item_stride;
};

// Output rows are ctx_stride / item_stride words apart (n_max and K for three separate arrays, the row length for
// packed rows).
__global__ void export_records_entry(const ExportParams q) {
  const int B = q.B, W = q.W, n_max = q.n_max, K = q.K, ctx_stride = q.ctx_stride, item_stride = q.item_stride;
  const int* n_path = q.n_path;
  const int* rec_ctx = q.rec_ctx;
  const int* rec_ids = q.rec_ids;
  const float* rec_p = q.rec_p;
  int* out_ctx = q.out_ctx;
  int* out_ids = q.out_ids;
  float* out_p = q.out_p;
  pdl_trigger();
  pdl_wait();  // the records come from the verification kernel before this one
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;  // one thread per (row, entry)
  const int per_row = n_max + K;
  if (i >= (long long)B * W * per_row) return;
  const long long row = i / per_row;
  const int e = (int)(i - row * per_row);
  const bool live = (int)(row % W) < n_path[row / W];
  if (e < n_max) out_ctx[row * ctx_stride + e] = live ? rec_ctx[row * n_max + e] : -1;
  else {
    const int k = e - n_max;
    out_ids[row * item_stride + k] = live ? rec_ids[row * K + k] : -1;
    out_p[row * item_stride + k] = live ? rec_p[row * K + k] : 0.0f;
  }
}

}  // namespace

extern "C" {

size_t stand_workspace_bytes(const stand_config* cfg) {
  Derived d;
  if (!derive(cfg, &d)) return 0;
  Layout L;
  layout_of(cfg, &d, &L);
  return L.total;
}

int stand_init(const stand_config* cfg, void* dev_workspace, size_t bytes, stand_ctx** out) {
  if (!out) return STAND_E_ARG;
  *out = nullptr;
  Derived d;
  if (!derive(cfg, &d)) return STAND_E_ARG;
  Layout L;
  layout_of(cfg, &d, &L);
  if (!dev_workspace || ((uintptr_t)dev_workspace & 255) != 0 || bytes < L.total) return STAND_E_WORKSPACE;
  {
    int sms = 0;
    const int prc = prepare_device(&sms);  // kernel attributes of this device, once
    if (prc) return prc;
  }
  stand_ctx* x = new (std::nothrow) stand_ctx;
  if (!x) return STAND_E_ARG;
  x->cfg = *cfg;
  x->cfg.parent = nullptr;  // the host array is not kept
  x->d = d;
  x->L = L;
  x->ws = (char*)dev_workspace;
  x->step = 0;
  x->pending = false;
  x->located = false;
  x->launches = 0;
  x->last_stream = 0;
  x->max_probe = cfg->max_probe > 0 ? cfg->max_probe : 96;
  x->tail_form = cfg->B == 1 ? 1 : (cluster_tail_fits(cfg->B, verify_smem_bytes(cfg->N)) ? 2 : 0);
  x->ev_before = nullptr;
  x->ev_after = nullptr;
  for (int i = 0; i < 5; ++i) x->ev_stage[i] = nullptr;
  x->c = log2e_over_T(cfg->temperature);

  int topo[4 * NODES_MAX + DEPTH_MAX + 2];
  memset(topo, 0, sizeof(topo));
  memcpy(topo, d.parent, sizeof(d.parent));
  memcpy(topo + NODES_MAX, d.first_child, sizeof(d.first_child));
  memcpy(topo + 2 * NODES_MAX, d.n_children, sizeof(d.n_children));
  memcpy(topo + 3 * NODES_MAX, d.depth, sizeof(d.depth));
  memcpy(topo + 4 * NODES_MAX, d.level_start, sizeof(d.level_start));
  int rc = cuda_ok(cudaMemcpy(x->ws + L.topo, topo, sizeof(topo), cudaMemcpyHostToDevice));
  if (rc == STAND_OK) {
    const unsigned long long n16 = (unsigned long long)cfg->table_slots * 8;
    table_clear_kernel<<<(unsigned)((n16 + 255) / 256), 256>>>(x->at<Slot>(L.table), cfg->table_slots);
    rc = launch_ok();
  }
  // everything after the table starts at zero, tails at -1
  if (rc == STAND_OK) rc = cuda_ok(cudaMemset(x->ws + L.tail, 0xFF, L.len - L.tail));
  if (rc == STAND_OK) rc = cuda_ok(cudaMemset(x->ws + L.len, 0, L.staging - L.len));
  if (rc == STAND_OK) rc = cuda_ok(cudaMemset(x->ws + L.tree, 0xFF, L.cand_n - L.tree));
  if (rc == STAND_OK) rc = cuda_ok(cudaDeviceSynchronize());
  if (rc != STAND_OK) { delete x; return rc; }
  x->launches += 1;
  *out = x;
  return STAND_OK;
}

int stand_destroy(stand_ctx* ctx) {
  if (!ctx) return STAND_E_ARG;
  delete ctx;
  return STAND_OK;
}

int stand_reset_sequences(stand_ctx* x, const int32_t* dev_tail, const int64_t* dev_len, void* cu_stream) {
  if (!x || !dev_tail || !dev_len) return STAND_E_ARG;
  cudaStream_t st = (cudaStream_t)cu_stream;
  x->last_stream = st;
  const stand_config& c = x->cfg;
  int rc = cuda_ok(cudaMemcpyAsync(x->ws + x->L.tail, dev_tail, (size_t)c.B * c.order_max * 4, cudaMemcpyDeviceToDevice, st));
  if (rc) return rc;
  rc = cuda_ok(cudaMemcpyAsync(x->ws + x->L.len, dev_len, (size_t)c.B * 8, cudaMemcpyDeviceToDevice, st));
  if (rc) return rc;
  const long long n = (long long)c.B * c.N;
  reset_tree_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(c.B, c.N, c.order_max, x->at<int>(x->L.tail),
                                                                 x->at<int>(x->L.tree), x->at<int>(x->L.cand_n));
  rc = launch_ok();
  if (rc) return rc;
  x->launches += 1;
  x->pending = false;
  x->located = false;
  return STAND_OK;
}

int stand_verify_tree(stand_ctx* x, const void* dev_logits, int32_t* dev_emitted, int32_t* dev_n_emitted, void* cu_stream) {
  if (!x || !dev_logits) return STAND_E_ARG;
  x->last_stream = (cudaStream_t)cu_stream;
  if (x->pending && x->located) return STAND_E_STATE;  // slots are marked for an update that has not run
  return run_verify(x, dev_logits, dev_emitted, dev_n_emitted, false, (cudaStream_t)cu_stream);
}

int stand_ngram_update(stand_ctx* x, void* cu_stream) {
  if (!x) return STAND_E_ARG;
  if (!x->pending) return STAND_E_STATE;
  x->last_stream = (cudaStream_t)cu_stream;
  return run_update(x, (cudaStream_t)cu_stream);
}

int stand_ngram_update_bulk(stand_ctx* x, const int32_t* dev_ctx, const int32_t* dev_ids, const float* dev_probs, int64_t M,
                            void* cu_stream) {
  if (!x || M < 0 || (M > 0 && (!dev_ctx || !dev_ids || !dev_probs))) return STAND_E_ARG;
  cudaStream_t st = (cudaStream_t)cu_stream;
  x->last_stream = st;
  const stand_config& c = x->cfg;
  for (int64_t at = 0; at < M; at += BULK_ROWS) {
    const long long n = M - at < BULK_ROWS ? M - at : BULK_ROWS;
    const int rc = run_update_rows(x, update_params(x, n, dev_ctx + at * c.order_max, dev_ids + at * c.topk,
                                                    dev_probs + at * c.topk, nullptr, 1), false, st);
    if (rc) return rc;
  }
  return STAND_OK;
}

static int export_records(stand_ctx* x, int32_t* out_ctx, int32_t* out_ids, float* out_p, int ctx_stride, int item_stride,
                          cudaStream_t st) {
  if (!x->pending) return STAND_E_STATE;
  x->last_stream = st;
  const stand_config& c = x->cfg;
  const int W = x->d.D + 1;
  const long long n = (long long)c.B * W * (c.order_max + c.topk);
  ExportParams e;
  e.B = c.B; e.W = W; e.n_max = c.order_max; e.K = c.topk; e.n_path = x->at<int>(x->L.n_path);
  e.rec_ctx = x->at<int>(x->L.rec_ctx); e.rec_ids = x->at<int>(x->L.rec_ids); e.rec_p = x->at<float>(x->L.rec_p);
  e.out_ctx = out_ctx; e.out_ids = out_ids; e.out_p = out_p; e.ctx_stride = ctx_stride; e.item_stride = item_stride;
  const int rc = launch_dependent(export_records_entry, (unsigned)((n + 255) / 256), 256u, st, e);
  if (rc == STAND_OK) x->launches += 1;
  return rc;
}

int stand_export_records(stand_ctx* x, int32_t* dev_ctx, int32_t* dev_ids, float* dev_probs, void* cu_stream) {
  if (!x || !dev_ctx || !dev_ids || !dev_probs) return STAND_E_ARG;
  return export_records(x, dev_ctx, dev_ids, dev_probs, x->cfg.order_max, x->cfg.topk, (cudaStream_t)cu_stream);
}

int stand_export_records_packed(stand_ctx* x, int32_t* dev_rows, void* cu_stream) {
  if (!x || !dev_rows) return STAND_E_ARG;
  const int n = x->cfg.order_max, K = x->cfg.topk, stride = n + 2 * K;
  return export_records(x, dev_rows, dev_rows + n, reinterpret_cast<float*>(dev_rows + n + K), stride, stride, (cudaStream_t)cu_stream);
}

int stand_ngram_update_packed(stand_ctx* x, const int32_t* dev_rows, int64_t M, void* cu_stream) {
  if (!x || M < 0 || (M > 0 && !dev_rows)) return STAND_E_ARG;
  cudaStream_t st = (cudaStream_t)cu_stream;
  x->last_stream = st;
  const int n = x->cfg.order_max, K = x->cfg.topk, stride = n + 2 * K;
  for (int64_t at = 0; at < M; at += BULK_ROWS) {
    const long long rows = M - at < BULK_ROWS ? M - at : BULK_ROWS;
    const int32_t* base = dev_rows + at * stride;
    const int rc = run_update_rows(x, update_params(x, rows, base, base + n, reinterpret_cast<const float*>(base + n + K), nullptr, 1,
                                                    stride), false, st);
    if (rc) return rc;
  }
  return STAND_OK;
}

int stand_skip_update(stand_ctx* x) {
  if (!x) return STAND_E_ARG;
  if (!x->pending || x->located) return STAND_E_STATE;  // located: slots are already marked for the update
  x->pending = false;
  return STAND_OK;
}

int stand_draft_tree(stand_ctx* x, int32_t* dev_tree_tokens, void* cu_stream) {
  if (!x) return STAND_E_ARG;
  x->last_stream = (cudaStream_t)cu_stream;
  return run_draft(x, dev_tree_tokens, true, (cudaStream_t)cu_stream);
}

int stand_step(stand_ctx* x, const void* dev_logits, int32_t* dev_emitted, int32_t* dev_n_emitted, int32_t* dev_tree_tokens,
               void* cu_stream) {
  if (!x || !dev_logits) return STAND_E_ARG;
  cudaStream_t st = (cudaStream_t)cu_stream;
  x->last_stream = st;
  if (x->pending && x->located) return STAND_E_STATE;
  return run_step(x, dev_logits, dev_emitted, dev_n_emitted, dev_tree_tokens, st);
}

int stand_step_host(stand_ctx* x, const void* host_logits, int32_t* host_emitted, int32_t* host_n_emitted,
                    int32_t* host_tree_tokens, void* cu_stream) {
  if (!x || !host_logits) return STAND_E_ARG;
  if (!x->cfg.host_staging) return STAND_E_STATE;
  cudaStream_t st = (cudaStream_t)cu_stream;
  x->last_stream = st;
  const stand_config& c = x->cfg;
  const size_t bytes = (size_t)c.B * c.N * c.V * esize_of(c.dtype);
  int rc = cuda_ok(cudaMemcpyAsync(x->ws + x->L.staging, host_logits, bytes, cudaMemcpyHostToDevice, st));
  if (rc) return rc;
  rc = run_step(x, x->ws + x->L.staging, nullptr, nullptr, nullptr, st);
  if (rc) return rc;
  const size_t W = x->d.D + 1;
  if (host_emitted) rc = cuda_ok(cudaMemcpyAsync(host_emitted, x->ws + x->L.emitted, c.B * W * 4, cudaMemcpyDeviceToHost, st));
  if (rc) return rc;
  if (host_n_emitted) rc = cuda_ok(cudaMemcpyAsync(host_n_emitted, x->ws + x->L.n_path, (size_t)c.B * 4, cudaMemcpyDeviceToHost, st));
  if (rc) return rc;
  if (host_tree_tokens) rc = cuda_ok(cudaMemcpyAsync(host_tree_tokens, x->ws + x->L.tree, (size_t)c.B * c.N * 4, cudaMemcpyDeviceToHost, st));
  if (rc) return rc;
  return cuda_ok(cudaStreamSynchronize(st));
}

size_t stand_row_stats_scratch_bytes(int64_t rows, int32_t V, int32_t dtype, int32_t topk) {
  if (rows < 1 || V < 2 || V > STAND_MAX_VOCAB || topk < 1 || topk > STAND_MAX_TOPK) return 0;
  if (dtype != STAND_DTYPE_F32 && dtype != STAND_DTYPE_BF16) return 0;
  const size_t n_chunks = (V + CHUNK - 1) / CHUNK;
  // a status word, then one (sum, max) pair per chunk
  return 256 + align_up((size_t)rows * n_chunks * sizeof(float2));
}

int stand_row_stats(const void* dev_logits, int64_t rows, int32_t V, int32_t dtype, float temperature, int32_t topk,
                    void* dev_scratch, size_t scratch_bytes, float* dev_lse, int32_t* dev_ids, float* dev_values,
                    float* dev_probs, void* cu_stream) {
  const size_t need = stand_row_stats_scratch_bytes(rows, V, dtype, topk);
  if (need == 0 || !dev_logits || !dev_lse || !dev_ids || !dev_values || !dev_probs || !(temperature > 0.0f)) return STAND_E_ARG;
  if (!dev_scratch || ((uintptr_t)dev_scratch & 255) != 0 || scratch_bytes < need) return STAND_E_WORKSPACE;
  cudaStream_t st = (cudaStream_t)cu_stream;
  const int n_chunks = (V + CHUNK - 1) / CHUNK;
  int* status = (int*)dev_scratch;
  float2* pairs = (float2*)((char*)dev_scratch + 256);
  const float c = log2e_over_T(temperature);
  int rc = cuda_ok(cudaMemsetAsync(status, 0, sizeof(int), st));  // the scratch may hold an earlier call's status
  if (rc) return rc;
  rc = launch_row_pass(dev_logits, rows, V, dtype, n_chunks, c, pairs, status, st);
  if (rc) return rc;
  RowFinalizeParams f;
  f.logits = dev_logits; f.dtype = dtype; f.V = V; f.pairs = pairs; f.status = status; f.rows = rows; f.n_chunks = n_chunks;
  f.topk = topk; f.c = c; f.lse = dev_lse; f.ids = dev_ids; f.values = dev_values; f.probs = dev_probs;
  row_finalize_kernel<<<(unsigned)((rows + FIN_WARPS - 1) / FIN_WARPS), FIN_WARPS * 32, 0, st>>>(f);
  return launch_ok();
}

// Scratch of stand_row_stats_static.  In host code this name is only a handle for
// cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[STAND_STATIC_SCRATCH_BYTES];
constexpr int STATIC_MAX_DEVICES = 64;
static std::atomic<void*> g_static_scratch_addr[STATIC_MAX_DEVICES];

int stand_row_stats_static(const void* dev_logits, int64_t rows, int32_t V, int32_t dtype, float temperature,
                           int32_t topk, float* dev_lse, int32_t* dev_ids, float* dev_values, float* dev_probs,
                           void* cu_stream) {
  const size_t need = stand_row_stats_scratch_bytes(rows, V, dtype, topk);
  // the same argument checks, in the same order, as stand_row_stats: an invalid call is an invalid call at any size
  if (need == 0 || !dev_logits || !dev_lse || !dev_ids || !dev_values || !dev_probs || !(temperature > 0.0f)) return STAND_E_ARG;
  if (need > (size_t)STAND_STATIC_SCRATCH_BYTES) return STAND_E_TOO_LARGE;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return STAND_E_CUDA;
  if (dev < 0 || dev >= STATIC_MAX_DEVICES) return STAND_E_ARG;
  void* scratch = g_static_scratch_addr[dev].load(std::memory_order_acquire);
  if (!scratch) {
    // first call on this device: resolve the buffer's address in this device's copy of the image
    if (cudaGetSymbolAddress(&scratch, g_static_scratch) != cudaSuccess || !scratch) return STAND_E_CUDA;
    g_static_scratch_addr[dev].store(scratch, std::memory_order_release);
  }
  return stand_row_stats(dev_logits, rows, V, dtype, temperature, topk, scratch, (size_t)STAND_STATIC_SCRATCH_BYTES, dev_lse,
                         dev_ids, dev_values, dev_probs, cu_stream);
}

int stand_get_stats(stand_ctx* x, stand_stats* host_out) {
  if (!x || !host_out) return STAND_E_ARG;
  int rc = cuda_ok(cudaStreamSynchronize(x->last_stream));
  if (rc) return rc;
  unsigned long long s[ST_COUNT];
  rc = cuda_ok(cudaMemcpy(s, x->ws + x->L.stats, sizeof(s), cudaMemcpyDeviceToHost));
  if (rc) return rc;
  host_out->steps = s[ST_STEPS];
  host_out->emitted_tokens = s[ST_EMITTED];
  host_out->records = s[ST_RECORDS];
  host_out->inserts = s[ST_INSERTS];
  host_out->drops = s[ST_DROPS];
  host_out->bad_tokens = s[ST_BAD_TOKENS];
  host_out->lookups = s[ST_LOOKUPS];
  for (int i = 0; i < STAND_MAX_ORDER; ++i) host_out->lookup_hits[i] = s[ST_HIT0 + i];
  host_out->max_probe_seen = s[ST_MAX_PROBE];
  int status = 0;
  rc = cuda_ok(cudaMemcpy(&status, x->ws + x->L.status, sizeof(int), cudaMemcpyDeviceToHost));
  if (rc) return rc;
  host_out->wait_timeouts = (uint64_t)(status != 0);
  return STAND_OK;
}

int stand_last_path(stand_ctx* x, int32_t* dev_path, int32_t* dev_ids, float* dev_probs, void* cu_stream) {
  if (!x) return STAND_E_ARG;
  cudaStream_t st = (cudaStream_t)cu_stream;
  x->last_stream = st;
  const stand_config& c = x->cfg;
  const size_t W = x->d.D + 1;
  int rc = STAND_OK;
  if (dev_path) rc = cuda_ok(cudaMemcpyAsync(dev_path, x->ws + x->L.path, c.B * W * 4, cudaMemcpyDeviceToDevice, st));
  if (rc == STAND_OK && dev_ids) rc = cuda_ok(cudaMemcpyAsync(dev_ids, x->ws + x->L.rec_ids, c.B * W * c.topk * 4, cudaMemcpyDeviceToDevice, st));
  if (rc == STAND_OK && dev_probs) rc = cuda_ok(cudaMemcpyAsync(dev_probs, x->ws + x->L.rec_p, c.B * W * c.topk * 4, cudaMemcpyDeviceToDevice, st));
  return rc;
}

int32_t stand_tree_depth(const stand_ctx* x) { return x ? x->d.D : -1; }

int stand_table_dump(stand_ctx* x, int32_t* dev_keys, uint32_t* dev_counts, int32_t* dev_n_items, int32_t* dev_ids,
                     float* dev_probs, uint64_t cap, uint64_t* dev_total, void* cu_stream) {
  if (!x || !dev_total || (cap > 0 && (!dev_keys || !dev_counts || !dev_n_items || !dev_ids || !dev_probs))) return STAND_E_ARG;
  cudaStream_t st = (cudaStream_t)cu_stream;
  x->last_stream = st;
  int rc = cuda_ok(cudaMemsetAsync(dev_total, 0, 8, st));
  if (rc) return rc;
  const unsigned long long n = x->cfg.table_slots;
  table_dump_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(x->at<Slot>(x->L.table), n, x->cfg.topk, dev_keys, dev_counts,
                                                                 dev_n_items, dev_ids, dev_probs, cap,
                                                                 (unsigned long long*)dev_total);
  rc = launch_ok();
  if (rc == STAND_OK) x->launches += 1;
  return rc;
}

int stand_table_load(stand_ctx* x, const int32_t* dev_keys, const uint32_t* dev_counts, const int32_t* dev_n_items,
                     const int32_t* dev_ids, const float* dev_probs, uint64_t M, int32_t clear, void* cu_stream) {
  if (!x || (M > 0 && (!dev_keys || !dev_counts || !dev_n_items || !dev_ids || !dev_probs))) return STAND_E_ARG;
  cudaStream_t st = (cudaStream_t)cu_stream;
  x->last_stream = st;
  int rc = STAND_OK;
  if (clear) {
    const unsigned long long n16 = (unsigned long long)x->cfg.table_slots * 8;
    table_clear_kernel<<<(unsigned)((n16 + 255) / 256), 256, 0, st>>>(x->at<Slot>(x->L.table), x->cfg.table_slots);
    rc = launch_ok();
    if (rc) return rc;
    x->launches += 1;
  }
  if (M > 0) {
    table_load_kernel<<<(unsigned)((M * GROUP + 255) / 256), 256, 0, st>>>(x->at<Slot>(x->L.table), x->cfg.table_slots - 1, x->max_probe,
                                                                   x->cfg.topk, dev_keys, dev_counts, dev_n_items, dev_ids,
                                                                   dev_probs, M, x->at<unsigned long long>(x->L.stats));
    rc = launch_ok();
    if (rc == STAND_OK) x->launches += 1;
  }
  return rc;
}

int stand_state_dump(stand_ctx* x, int32_t* dev_tail, int64_t* dev_len, int32_t* dev_tree, int32_t* dev_cand_n,
                     int32_t* dev_cand_id, float* dev_cand_phi, uint32_t* host_step, void* cu_stream) {
  if (!x) return STAND_E_ARG;
  cudaStream_t st = (cudaStream_t)cu_stream;
  x->last_stream = st;
  const stand_config& c = x->cfg;
  const size_t BN = (size_t)c.B * c.N;
  int rc = STAND_OK;
  auto cp = [&](void* dst, size_t off, size_t bytes) {
    if (rc == STAND_OK && dst) rc = cuda_ok(cudaMemcpyAsync(dst, x->ws + off, bytes, cudaMemcpyDeviceToDevice, st));
  };
  cp(dev_tail, x->L.tail, (size_t)c.B * c.order_max * 4);
  cp(dev_len, x->L.len, (size_t)c.B * 8);
  cp(dev_tree, x->L.tree, BN * 4);
  cp(dev_cand_n, x->L.cand_n, BN * 4);
  cp(dev_cand_id, x->L.cand_id, BN * c.topk * 4);
  cp(dev_cand_phi, x->L.cand_phi, BN * c.topk * 4);
  if (host_step) *host_step = x->step;
  return rc;
}

int stand_state_load(stand_ctx* x, const int32_t* dev_tail, const int64_t* dev_len, const int32_t* dev_tree,
                     const int32_t* dev_cand_n, const int32_t* dev_cand_id, const float* dev_cand_phi, uint32_t step,
                     void* cu_stream) {
  if (!x || !dev_tail || !dev_len || !dev_tree || !dev_cand_n || !dev_cand_id || !dev_cand_phi) return STAND_E_ARG;
  cudaStream_t st = (cudaStream_t)cu_stream;
  x->last_stream = st;
  const stand_config& c = x->cfg;
  const size_t BN = (size_t)c.B * c.N;
  int rc = STAND_OK;
  auto cp = [&](size_t off, const void* src, size_t bytes) {
    if (rc == STAND_OK) rc = cuda_ok(cudaMemcpyAsync(x->ws + off, src, bytes, cudaMemcpyDeviceToDevice, st));
  };
  cp(x->L.tail, dev_tail, (size_t)c.B * c.order_max * 4);
  cp(x->L.len, dev_len, (size_t)c.B * 8);
  cp(x->L.tree, dev_tree, BN * 4);
  cp(x->L.cand_n, dev_cand_n, BN * 4);
  cp(x->L.cand_id, dev_cand_id, BN * c.topk * 4);
  cp(x->L.cand_phi, dev_cand_phi, BN * c.topk * 4);
  if (rc == STAND_OK) {
    validate_state_kernel<<<(unsigned)((BN + 255) / 256), 256, 0, st>>>(c.B, c.N, c.topk, c.V, x->topo_parent(), x->at<int>(x->L.tree),
                                                                       x->at<int>(x->L.cand_n), x->at<int>(x->L.cand_id),
                                                                       x->at<unsigned long long>(x->L.stats));
    rc = launch_ok();
    if (rc == STAND_OK) x->launches += 1;
  }
  if (rc == STAND_OK) { x->step = step; x->pending = false; x->located = false; }
  return rc;
}

int stand_profile_row_pass(stand_ctx* x, void* ev_before, void* ev_after) {
  if (!x || ((ev_before == nullptr) != (ev_after == nullptr))) return STAND_E_ARG;
  x->ev_before = (cudaEvent_t)ev_before;
  x->ev_after = (cudaEvent_t)ev_after;
  return STAND_OK;
}

int stand_node_accepts(stand_ctx* x, uint64_t* host_counts, int32_t reset) {
  if (!x || !host_counts) return STAND_E_ARG;
  int rc = cuda_ok(cudaStreamSynchronize(x->last_stream));
  if (rc) return rc;
  rc = cuda_ok(cudaMemcpy(host_counts, x->ws + x->L.accepts, (size_t)x->cfg.N * 8, cudaMemcpyDeviceToHost));
  if (rc == STAND_OK && reset) rc = cuda_ok(cudaMemset(x->ws + x->L.accepts, 0, (size_t)x->cfg.N * 8));
  return rc;
}

int stand_prune_tree(const int32_t* host_parent, int32_t n, const uint64_t* host_counts, int32_t keep,
                     int32_t* host_parent_out, int32_t* host_old_index) {
  if (!host_parent || !host_counts || !host_parent_out || n < 1 || keep < 1 || keep > n || host_parent[0] != -1) return STAND_E_ARG;
  for (int32_t u = 1; u < n; ++u)
    if (host_parent[u] < 0 || host_parent[u] >= u) return STAND_E_ARG;
  // a node is kept if fewer than `keep` nodes come before it in (count descending, index ascending) order
  std::vector<char> kept((size_t)n, 0);
  std::vector<int32_t> new_index((size_t)n, -1);
  for (int32_t u = 0; u < n; ++u) {
    int32_t before = 0;
    for (int32_t w = 0; w < n; ++w)
      if (host_counts[w] > host_counts[u] || (host_counts[w] == host_counts[u] && w < u)) ++before;
    kept[u] = before < keep ? 1 : 0;
  }
  if (!kept[0]) return STAND_E_ARG;  // the root is on every path: counts that rank it out are not acceptance counts
  int32_t at = 0;
  for (int32_t u = 0; u < n; ++u) {  // the old numbering is breadth-first with siblings together: so is the new one
    if (!kept[u]) continue;
    if (u > 0 && !kept[host_parent[u]]) return STAND_E_ARG;  // counts that grow towards the leaves: not acceptance counts
    new_index[u] = at;
    host_parent_out[at] = u == 0 ? -1 : new_index[host_parent[u]];
    if (host_old_index) host_old_index[at] = u;
    ++at;
  }
  return at == keep ? STAND_OK : STAND_E_ARG;
}

int stand_initial_tree(int32_t levels, int32_t* host_parent, int32_t* host_depth, int32_t* host_order, int32_t capacity,
                       int32_t* total_nodes) {
  if (levels < 0 || levels > 64 || !total_nodes || capacity < 0 || (capacity > 0 && !host_parent)) return STAND_E_ARG;
  struct Node { int32_t parent, depth, order, n_children; };
  std::vector<Node> nodes;
  nodes.push_back({-1, 0, 0, 0});
  size_t level_begin = 0, level_end = 1;  // the nodes of the current level are nodes[level_begin, level_end)
  for (int32_t l = 0; l < levels; ++l) {
    for (size_t at = level_begin; at < level_end; ++at) {
      const Node me = nodes[at];
      int64_t n;
      if (me.depth == 0) n = 8;
      else if (me.depth == 1) n = 8 - 2 * me.order > 1 ? 8 - 2 * me.order : 1;
      else {
        // ceil((siblings - 1) / (0.7 * order + 1)) in integers: ceil(10 (siblings - 1) / (7 order + 10))
        const int64_t num = 10 * (int64_t)(nodes[me.parent].n_children - 1), den = 7 * (int64_t)me.order + 10;
        n = (num + den - 1) / den;
        const int64_t floor = (me.depth == 2 || me.depth == 3) ? 2 : 0;
        if (n < floor) n = floor;
      }
      if (at == level_begin && n < 3) n = 3;
      if (nodes.size() + (size_t)n > (1u << 24)) return STAND_E_ARG;
      nodes[at].n_children = (int32_t)n;
      for (int32_t k = 0; k < (int32_t)n; ++k) nodes.push_back({(int32_t)at, me.depth + 1, k, 0});
    }
    level_begin = level_end;
    level_end = nodes.size();
  }
  *total_nodes = (int32_t)nodes.size();
  const size_t out = nodes.size() < (size_t)capacity ? nodes.size() : (size_t)capacity;
  for (size_t i = 0; i < out; ++i) {
    host_parent[i] = nodes[i].parent;
    if (host_depth) host_depth[i] = nodes[i].depth;
    if (host_order) host_order[i] = nodes[i].order;
  }
  return STAND_OK;
}

int stand_profile_stages(stand_ctx* x, void* const* events) {
  if (!x) return STAND_E_ARG;
  for (int i = 0; i < 5; ++i) x->ev_stage[i] = events ? (cudaEvent_t)events[i] : nullptr;
  return STAND_OK;
}

uint64_t stand_launch_count(const stand_ctx* x) { return x ? x->launches : 0; }

int stand_set_wait_limit(int64_t polls) {
  g_empty_wait_limit.store(polls < 0 || polls > (int64_t)SPIN_LIMIT ? SPIN_LIMIT : (unsigned)polls, std::memory_order_relaxed);
  return STAND_OK;
}

const char* stand_strerror(int code) {
  switch (code) {
    case STAND_OK: return "ok";
    case STAND_E_ARG: return "invalid argument or configuration";
    case STAND_E_WORKSPACE: return "workspace missing, misaligned or too small";
    case STAND_E_CUDA: return "a CUDA runtime call failed";
    case STAND_E_STATE: return "call not valid in the current state";
    case STAND_E_TOO_LARGE: return "problem does not fit the built-in scratch buffer";
    default: return "unknown error code";
  }
}

}  // extern "C"
