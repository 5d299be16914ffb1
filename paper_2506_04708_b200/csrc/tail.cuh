// Step tail without kernel boundaries: verification, table update and drafting in one thread block (a single
// sequence) or one thread-block cluster (a small batch).
#pragma once
#include "common.cuh"
#include "draft.cuh"
#include "table.cuh"
#include "verify.cuh"

namespace stand {

// A whole step's tail without kernel boundaries, for a single sequence (one block) or a small batch (one
// block per sequence, all blocks in ONE thread-block cluster): verification with stage 1 of the update,
// stage 2 of the update, drafting.  Where the batch form relies on a kernel boundary ("every sequence has
// located its records", "the table is up to date") this form has a block barrier, or the hardware barrier
// of the cluster, whose release/acquire pair also orders the blocks' global-memory writes.
// The block is TAIL_THREADS wide: its first K2_THREADS threads verify (on a named barrier of their own); the others
// map the update records to table slots as soon as the walk has emitted its tokens, beside the compression of the
// accepted rows; all of them then apply the records and draft, where more warps mean fewer rounds (one warp per
// record, one warp per parent node of a tree level).
constexpr int TAIL_THREADS = 512;
constexpr int TAIL_CLUSTER_MAX = 16;  // largest cluster the hardware offers (beyond 8 it has to be asked for)
static_assert(TAIL_THREADS >= K2_THREADS && TAIL_THREADS % 32 == 0, "the verifying threads are part of the block");
struct TailParams {
  VerifyParams v;  // fuse_locate set; v.upd describes this step's records
  DraftParams d;
};

template <bool CLUSTER>
__device__ __forceinline__ void tail_barrier() {
  if (CLUSTER) asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
  else __syncthreads();
}

template <bool CLUSTER>
__device__ __forceinline__ void tail_body(const TailParams& p, const int b) {
  constexpr int WARPS = TAIL_THREADS / 32;
  __shared__ SlotImage s_img[WARPS];
  __shared__ DraftShared<TAIL_THREADS> s_draft;
  if (threadIdx.x < K2_THREADS) verify_block<1, TAIL_THREADS>(p.v, b, s_draft.tail);
  else {
    pdl_trigger();
    draft_stage_topology<TAIL_THREADS>(p.d, s_draft, (int)threadIdx.x - K2_THREADS, TAIL_THREADS - K2_THREADS);  // for later
    pdl_wait();
    locate_beside_verify<TAIL_THREADS>(p.v, b);
  }
  tail_barrier<CLUSTER>();  // records, slot marks and the advanced tails of all sequences are visible
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // this block applies the records of its own sequence; only the rows of the accepted path carry any:
  // (row, order) pairs of the first n_path rows.  (A slot's records are applied by the warp that holds its
  // lowest row, whichever block that is: the canonical order does not depend on who runs what.)
  const int W1 = p.v.D + 1;
  const int live_rows = p.v.n_path[b];
  const int n_rec = live_rows * p.v.upd.n_max;
  for (int r = warp; r < n_rec; r += WARPS) {
    const int n = r / live_rows, row = r - n * live_rows;
    apply_record(p.v.upd, (long long)n * p.v.upd.n_rows + (long long)b * W1 + row, &s_img[warp], lane);
  }
  tail_barrier<CLUSTER>();  // the table is up to date
  draft_block<false, TAIL_THREADS, true>(p.d, b, s_draft);  // topology staged above, the tail left by the verification
}

__global__ void __launch_bounds__(TAIL_THREADS) tail_single_kernel(const TailParams p) { tail_body<false>(p, 0); }
// Launched as one cluster of B blocks (cluster dimension = grid dimension = B <= TAIL_CLUSTER_MAX).
__global__ void __launch_bounds__(TAIL_THREADS) tail_cluster_kernel(const TailParams p) { tail_body<true>(p, (int)blockIdx.x); }

}  // namespace stand
