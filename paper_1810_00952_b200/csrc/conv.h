// Shapes of one conv2d instance and the kernel tiers that run it.
#pragma once
#include "common.h"

namespace relay {

struct ConvDims {
    int64_t Nb = 0, C = 0, H = 0, W = 0, O = 0, R = 0, S = 0, P = 0, Q = 0;
    int32_t stride = 1, pad = 0, dt = RELAY_F32;
    bool nhwc = false;                // x, y, dy, dx are (N,H,W,C) tensors; the kernels below work on NCHW
};

// layout change: out[b][s][r] = in[b][r][s] for `batch` matrices of R x S elements of 2 or 4 bytes
// (NCHW -> NHWC: R = C, S = H*W;  NHWC -> NCHW: R = H*W, S = C)
relay_status_t launch_layout_change(int32_t dt, const void *in, void *out, int64_t batch, int64_t R, int64_t S, cudaStream_t st);

// general (SIMT) tier: any stride / pad / window, implicit GEMM with gathers in the tile loaders (conv_igemm.cu);
// the weight gradient is split along its sum and needs conv_dw_partial_bytes(d) of fp32 partials
relay_status_t launch_conv_fwd_direct(const ConvDims &d, const void *x, const void *w, const void *b, int32_t b_dt, int act,
                                      void *y, cudaStream_t st);
relay_status_t launch_conv_dx_direct(const ConvDims &d, const void *dz, const void *w, void *dx, cudaStream_t st);
size_t conv_dw_partial_bytes(const ConvDims &d);
relay_status_t launch_conv_dw_direct(const ConvDims &d, const void *dz, const void *x, void *dw, float *partials, cudaStream_t st);
relay_status_t launch_conv_db(const ConvDims &d, const void *dz, float *db, cudaStream_t st);

// implicit-GEMM tensor-core tier (3x3, stride 1, pad 1, bf16)
bool conv_tc_eligible(const ConvDims &d);
size_t conv_tc_fwd_workspace(const ConvDims &d);
size_t conv_tc_grad_workspace(const ConvDims &d);
// `x_is_nhwc`: x is already in the kernel's own activation layout, the repack pass is skipped (y is NCHW either way)
// `y_nhwc` (optional): the result is wanted as [Nb][H][W][O]; `y` is then an NCHW temporary that the call may or may not use
relay_status_t launch_conv_fwd_tc(const ConvDims &d, const void *x, bool x_is_nhwc, const void *w, const void *b, int32_t b_dt, int act,
                                  void *y, void *ws, cudaStream_t st, void *y_nhwc = nullptr);
// whole gradient group: dZ = dy (.) act'(y) (kept in NHWC), db, dx (if wanted), dw
// `nhwc_in`: x, y, dy are NHWC already (no repack passes; `nhwc_partials` holds the column-sum partials of db) and the
// input gradient is wanted in `dx_nhwc`; `dx` is then an NCHW temporary that the call may or may not use
relay_status_t launch_conv_grad_tc(const ConvDims &d, const void *x, const void *w, const void *y, const void *dy, int act, void *dx,
                                   void *dw, float *db, void *ws, cudaStream_t st, bool nhwc_in = false, float *nhwc_partials = nullptr,
                                   void *dx_nhwc = nullptr);

}  // namespace relay
