// Single-sequence step tail: verification, table update and drafting in one thread block.
#pragma once
#include "common.cuh"
#include "draft.cuh"
#include "table.cuh"
#include "verify.cuh"

namespace stand {

// A whole step's tail for ONE sequence in one block: verification (with stage 1 of the update), stage 2 of
// the update, drafting.  With a single sequence every ordering the three kernels get from their launch
// boundaries is a block barrier here, which saves two kernel boundaries on the latency path.
static_assert(K2_THREADS == K4_THREADS && K2_THREADS == APPLY_WARPS * 32, "one block shape for the three stages");
struct TailParams {
  VerifyParams v;  // fuse_locate set; v.upd describes this step's records
  DraftParams d;
};
__global__ void __launch_bounds__(K2_THREADS) tail_single_kernel(const TailParams p) {
  __shared__ SlotImage s_img[APPLY_WARPS];
  verify_block(p.v, 0);
  __syncthreads();  // records, slot marks and the advanced tail are visible to the whole block
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // only the rows of the accepted path carry records: (row, order) pairs of the first n_path rows
  const int live_rows = p.v.n_path[0];
  const int n_rec = live_rows * p.v.upd.n_max;
  for (int r = warp; r < n_rec; r += APPLY_WARPS) {
    const int n = r / live_rows, row = r - n * live_rows;
    apply_record(p.v.upd, (long long)n * p.v.upd.n_rows + row, &s_img[warp], lane);
  }
  __syncthreads();  // the table is up to date
  draft_block<false>(p.d, 0);
}

}  // namespace stand
