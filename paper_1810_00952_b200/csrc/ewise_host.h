// Host-side launch helpers of the memory-bound kernels that other groups reuse
// (the dense / conv2d gradient groups need dZ = dy (.) act'(y) and its column sums).
#pragma once
#include <string>

#include "common.h"

namespace relay {

struct TypedProgram;

// Collapsed 2-D view [rows, cols] of a group: every input is full-shape, constant down the rows, or a scalar, all in one
// float storage type, with whole 16-byte vectors per row (ok = false otherwise).
struct View2D { bool ok; int64_t rows, cols; int kind[RELAY_MAX_INPUTS]; int32_t storage; };
View2D view2d(const TypedProgram &tp);

// Vectorised evaluator for programs without a pre-compiled body (ewise_vm.cu): plan on the host, then launch.
struct VmPlan { bool ok = false; int n_sum = 0; alignas(8) unsigned char storage[1024]; };
bool vm_plan(const TypedProgram &tp, const View2D &v, const int32_t *out_values, const bool *colsum, int n_out, VmPlan *plan);
int vm_grid_slices(const View2D &v, int n_slices_wanted);
relay_status_t vm_launch(const VmPlan &plan, const View2D &v, const relay_tensor_t *const *inputs, int n_in, const relay_tensor_t *const *outputs,
                         int n_out, float *partials, int n_slices, cudaStream_t st);
// Bodies compiled at run time for the same class of groups (ewise_jit.cu).  jit_get: the kernel for this group (compiled on first
// use, cached), or nullptr when there is no run-time compiler on this machine, it is switched off, or the group is outside the
// class: the caller then takes the interpreter.  out_dtype[k]: storage type of result k; partials: [n_sum][n_slices][cols].
bool jit_usable();
bool jit_set_cached_only(bool on);   // this thread: use only bodies compiled already (returns the previous setting)
bool jit_in_class(const TypedProgram &tp, const View2D &v, const int32_t *out_values, int n_out);
const void *jit_get(const TypedProgram &tp, const View2D &v, const int32_t *out_values, const int32_t *out_dtype, const bool *colsum, int n_out);
int jit_n_slices(const View2D &v, bool any_sum);
int jit_compile_only(const TypedProgram &tp, const View2D &v, const int32_t *out_values, const int32_t *out_dtype, const bool *colsum, int n_out,
                     std::string *src, std::string *log);
relay_status_t jit_launch(const void *kernel, const View2D &v, const relay_tensor_t *const *inputs, int n_in, const relay_tensor_t *const *outputs,
                          int n_out, float *partials, int n_slices, cudaStream_t st);
// finalises n_out column sums whose partials lie one after another ([k][n_slices][cols]); scale[k] multiplies sum k (null: 1)
relay_status_t launch_colsum_finalize_n(const float *partial, int n_slices, int64_t cols, const float *scale, float *const *out, int n_out,
                                        cudaStream_t st);

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
