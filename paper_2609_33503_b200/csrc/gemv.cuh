// Internal: the streaming kernel for projections of one to four rows (a decode token); relaxkv_linear and
// relaxkv_linear_swiglu route there by the row count.
#pragma once
#include "common.cuh"

namespace relaxkv {

constexpr int kGemvMaxRows = 4;

// y [n_rows, n_out] = x [n_rows, n_in] weight^T (+ residual).  swiglu != 0: weight is the gate/up-tiled matrix
// [n_out, n_in] of relaxkv_linear_swiglu and y is [n_rows, n_out / 2].  Arguments are validated by the caller.
relaxkv_status launch_gemv(const void* x, const void* weight, const void* residual, void* y, int n_rows, int n_out,
                           int n_in, int swiglu, cudaStream_t stream);

// The same for several weight matrices stacked along the output features (weight [n_out, n_in], n_out = the sum of the
// segments' widths): segment i = features [col0[i], col0[i + 1]) goes to its own row-major buffer y[i] of that width.
struct GemvOut {
  uint16_t* y[3];
  int col0[4];
  int n;
};
relaxkv_status launch_gemv_segments(const void* x, const void* weight, const GemvOut& outs, int n_rows, int n_out, int n_in,
                                    cudaStream_t stream);

}  // namespace relaxkv
