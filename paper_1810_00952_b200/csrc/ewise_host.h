// Host-side launch helpers of the memory-bound kernels that other groups reuse
// (the dense / conv2d gradient groups need dZ = dy (.) act'(y) and its column sums).
#pragma once
#include "common.h"

namespace relay {

// number of row slices (and therefore of partial rows) a column sum over [rows, cols] uses
int colsum_slices(int64_t rows, int64_t cols, int32_t storage);

// dz = dy (.) act'(y) over a [rows, cols] view; if db != nullptr also db[c] = sum_r dz[r,c]
// (fp32).  `partials` must hold colsum_slices(...) * cols floats when db is wanted.
// cols must be a multiple of 8 (bf16) / 4 (f32).
relay_status_t launch_act_grad(int32_t storage, const void *dy, const void *y, void *dz, float *db, float *partials,
                               int64_t rows, int64_t cols, int act, cudaStream_t st);

// out[c] = sum_r in[r,c] for a bf16 [rows, cols] tensor (cols a multiple of 8); `partials` holds
// colsum_slices(rows, cols, RELAY_BF16) * cols floats
relay_status_t launch_colsum_bf16(const void *in, int64_t rows, int64_t cols, float *partials, float *out, cudaStream_t st);

relay_status_t launch_colsum_finalize(const float *partial, int n_slices, int64_t cols, float scale, float *out,
                                      cudaStream_t st);

}  // namespace relay

namespace relay {
// dz = dy (.) act'(y) and (if db) db = column sums of dz for ANY [rows, cols] (falls back to
// scalar kernels when a row is not a whole number of 16-byte vectors).
relay_status_t act_grad_any(int32_t dt, const void *dy, const void *y, void *dz, float *db, float *partials, int64_t rows,
                            int64_t cols, int act, cudaStream_t st);
}  // namespace relay
