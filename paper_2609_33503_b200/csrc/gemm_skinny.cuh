// Internal: projections of 5 to 128 rows (the query's own tokens): one 128 x 128 output tile per thread-block cluster,
// K split over the cluster's blocks, partial tiles summed through distributed shared memory (gemm_skinny_sm100.cu).
#pragma once
#include "common.cuh"

namespace relaxkv {

constexpr int kSkinnyMaxRows = 128;

// Where the columns of y = x W^T go: segment i takes columns [col0[i], col0[i + 1]) and is a row-major matrix of that
// width of its own (+ an optional residual of the same shape).  Segment widths are multiples of 8.
struct SkinnyOut {
  uint16_t* y[3];
  const uint16_t* residual[3];
  int col0[4];
  int n;
};

// Column tiles of an n_out-wide projection.
int skinny_tiles(int n_out);

// x [n_rows <= 128, n_in], weight [n_out, n_in].  Arguments are validated by the caller.
relaxkv_status launch_gemm_skinny(const void* x, const void* weight, const SkinnyOut& outs, int n_rows, int n_out, int n_in,
                                  cudaStream_t stream);

}  // namespace relaxkv
