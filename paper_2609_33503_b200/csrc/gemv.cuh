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

}  // namespace relaxkv
