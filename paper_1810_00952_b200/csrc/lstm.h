// Persistent tensor-core kernel for the recurrent half of the LSTM sequence.
#pragma once
#include <cuda_bf16.h>

#include "common.h"

namespace relay {

// B <= 128, H a multiple of 64 and <= 1024 (the block's slice of W_hh must fit in shared memory),
// H / 16 blocks co-resident on the device
bool lstm_tc_eligible(int64_t T, int64_t B, int64_t H);
size_t lstm_tc_workspace(int64_t B, int64_t H);
// launch_lstm_tc_prepare packs W_hh into the blocks' slices and clears the step counters (both in `ws`); it reads nothing that
// the input projection writes, so the caller enqueues it BEFORE that contraction, whose set-up then overlaps its tail.
relay_status_t launch_lstm_tc_prepare(int64_t B, int64_t H, const void *w_hh, void *ws, cudaStream_t st);
// zx: [T*B][4H] fp32 (input projection + bias); runs all T steps.  `timing` (optional, device, 8 entries): block 0 leaves
// cycle counts summed over the steps: [0] step loop, [1] epilogue warp waiting for the accumulator, [2] epilogue (TMEM
// read, gates, publish), [3] loader waiting on the grid barrier, [4] loader issuing the step's copies, [5] issuer
// waiting for the step's first stage, [6] issuer from there to the step's last commit, [7] T
relay_status_t launch_lstm_tc(int64_t T, int64_t B, int64_t H, const float *zx, const void *w_hh, const float *h0, const float *c0,
                              float *h_all, float *c_final, void *ws, cudaStream_t st, long long *timing = nullptr);

// The dependent steps of the gradient program, last to first, as one persistent kernel of thread-block clusters: needs
// lstm_tc_eligible(T, B, H) and room for all its clusters at once.  gates: [T*B][4H] activated gates, c_all: [T*B][H],
// dz: [T*B][4H] (written), counter: 1024 bytes of device scratch.  *launched = false (and RELAY_OK) when the shape or
// the device does not take it: nothing was enqueued then.
relay_status_t launch_lstm_grad_cluster(int64_t T, int64_t B, int64_t H, const float *gates, const float *c_all, const float *c0,
                                        const float *dh_all, const float *dc_final, const void *w_hh, __nv_bfloat16 *dz, float *dh0,
                                        float *dc0, unsigned int *counter, cudaStream_t st, bool *launched);

#ifdef __CUDACC__
__device__ __forceinline__ float lstm_tanh_fast(float x) { return 1.0f - __fdividef(2.0f, 1.0f + __expf(2.0f * x)); }
// The gate derivatives of one (row, unit) at one step.  dh: partial of h_t; dc: carried partial of c_t
// (in: from step t+1, out: for step t-1); dz: partials of the pre-activations i | f | g | o.
__device__ __forceinline__ void lstm_gate_grads(float ig, float fg, float gg, float og, float c_t, float c_prev, float dh, float &dc,
                                                float (&dz)[4])
{
    const float tc = lstm_tanh_fast(c_t);
    const float d_o = dh * tc;
    const float dct = fmaf(dh * og, 1.0f - tc * tc, dc);
    dz[0] = dct * gg * ig * (1.0f - ig);
    dz[1] = dct * c_prev * fg * (1.0f - fg);
    dz[2] = dct * ig * (1.0f - gg * gg);
    dz[3] = d_o * og * (1.0f - og);
    dc = dct * fg;
}
#endif

}  // namespace relay
