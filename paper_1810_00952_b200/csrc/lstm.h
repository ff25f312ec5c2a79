// Persistent tensor-core kernel for the recurrent half of the LSTM sequence.
#pragma once
#include "common.h"

namespace relay {

// B <= 128, H a multiple of 64 and <= 1024 (the block's slice of W_hh must fit in shared memory),
// H / 16 blocks co-resident on the device
bool lstm_tc_eligible(int64_t T, int64_t B, int64_t H);
size_t lstm_tc_workspace(int64_t B, int64_t H);
// zx: [T*B][4H] fp32 (input projection + bias); runs all T steps.  `timing` (optional, device, 8 entries): block 0 leaves
// cycle counts summed over the steps: [0] step loop, [1] epilogue warp waiting for the accumulator, [2] epilogue (TMEM
// read, gates, publish), [3] loader waiting on the grid barrier, [4] loader issuing the step's copies, [5] issuer
// waiting for the step's first stage, [6] issuer from there to the step's last commit, [7] T
relay_status_t launch_lstm_tc(int64_t T, int64_t B, int64_t H, const float *zx, const void *w_hh, const float *h0, const float *c0,
                              float *h_all, float *c_final, void *ws, cudaStream_t st, long long *timing = nullptr);

}  // namespace relay
