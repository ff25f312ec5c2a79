// LSTM cell applied over a sequence (host entry point and the step kernels).
//
// Plan: (1) one batched contraction zx[t,b,:] = x[t,b,:] W_ih + bias for all T*B rows (tensor
// bound, independent of the recurrence); (2) the T dependent steps, each adding the recurrent
// product bf16(h) W_hh and applying the gates.  c_final doubles as the running cell state;
// h_all[t-1] is the running hidden state.
#include "ewise_kernels.cuh"
#include "gemm.h"
#include "lstm.h"

namespace relay {

constexpr int kRowsPerBlock = 8;   // batch rows that share one pass over W_hh
constexpr int kChunk = 128;        // k-extent of h staged in shared memory at a time

// one step: block = 256 hidden units x kRowsPerBlock batch rows
__global__ void __launch_bounds__(256) lstm_step_kernel(const float *__restrict__ zx_t,          // [B, 4H] (bias included)
                                                         const __nv_bfloat16 *__restrict__ w_hh,  // [H, 4H]
                                                         const float *__restrict__ h_prev,        // [B, H]
                                                         float *__restrict__ c,                   // [B, H] in/out
                                                         float *__restrict__ h_out,               // [B, H]
                                                         int64_t B, int64_t H)
{
    __shared__ float hs[kRowsPerBlock][kChunk];
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t b0 = (int64_t)blockIdx.y * kRowsPerBlock;
    const bool live = j < H;
    float acc[kRowsPerBlock][4];
#pragma unroll
    for (int r = 0; r < kRowsPerBlock; ++r)
#pragma unroll
        for (int g = 0; g < 4; ++g) acc[r][g] = 0.0f;

    for (int64_t k0 = 0; k0 < H; k0 += kChunk) {
        for (int e = threadIdx.x; e < kRowsPerBlock * kChunk; e += blockDim.x) {
            int r = e / kChunk, kk = e % kChunk;
            int64_t b = b0 + r, k = k0 + kk;
            hs[r][kk] = (b < B && k < H) ? round_bf16(h_prev[b * H + k]) : 0.0f;   // the recurrent product reads bf16(h)
        }
        __syncthreads();
        if (live) {
            const int kmax = (int)min((int64_t)kChunk, H - k0);
            for (int kk = 0; kk < kmax; ++kk) {
                const __nv_bfloat16 *wr = w_hh + (k0 + kk) * 4 * H + j;
                float wv[4];
#pragma unroll
                for (int g = 0; g < 4; ++g) wv[g] = __bfloat162float(wr[g * H]);
#pragma unroll
                for (int r = 0; r < kRowsPerBlock; ++r) {
                    const float hv = hs[r][kk];
#pragma unroll
                    for (int g = 0; g < 4; ++g) acc[r][g] = fmaf(hv, wv[g], acc[r][g]);
                }
            }
        }
        __syncthreads();
    }
    if (!live) return;
#pragma unroll
    for (int r = 0; r < kRowsPerBlock; ++r) {
        const int64_t b = b0 + r;
        if (b >= B) break;
        const float *z = zx_t + b * 4 * H + j;
        const float ig = sigmoid_<false>(z[0] + acc[r][0]);
        const float fg = sigmoid_<false>(z[H] + acc[r][1]);
        const float gg = tanhf(z[2 * H] + acc[r][2]);
        const float og = sigmoid_<false>(z[3 * H] + acc[r][3]);
        const float cn = fmaf(fg, c[b * H + j], ig * gg);
        c[b * H + j] = cn;
        h_out[b * H + j] = og * tanhf(cn);
    }
}

struct LstmDims { int64_t T, B, I, H; };

static relay_status_t check_lstm(const relay_tensor_t *x, const relay_tensor_t *w_ih, const relay_tensor_t *w_hh, LstmDims *d)
{
    relay_tensor_t ht, ct;
    RELAY_TRY(relay_infer_lstm(x, w_ih, w_hh, &ht, &ct));
    d->T = x->shape[0]; d->B = x->shape[1]; d->I = x->shape[2]; d->H = w_hh->shape[0];
    return RELAY_OK;
}

static size_t lstm_zx_bytes(const LstmDims &d) { return align_up((size_t)d.T * d.B * 4 * d.H * sizeof(float), 1024); }
static size_t lstm_ws(const LstmDims &d)
{
    return lstm_zx_bytes(d) + (lstm_tc_eligible(d.T, d.B, d.H) ? lstm_tc_workspace(d.B, d.H) : 0);
}

}  // namespace relay

using namespace relay;

extern "C" size_t relay_workspace_bytes_lstm(const relay_tensor_t *x, const relay_tensor_t *w_ih, const relay_tensor_t *w_hh)
{
    LstmDims d;
    if (!x || !w_ih || !w_hh || check_lstm(x, w_ih, w_hh, &d) != RELAY_OK) return 0;
    return lstm_ws(d);
}

static relay_status_t lstm_seq(const relay_tensor_t *x, const relay_tensor_t *w_ih, const relay_tensor_t *w_hh, const relay_tensor_t *b,
                               const relay_tensor_t *h0, const relay_tensor_t *c0, const relay_tensor_t *h_all, const relay_tensor_t *c_final,
                               void *ws, size_t ws_bytes, void *stream, long long *timing)
{
    clear_error();
    const relay_tensor_t *all[8] = {x, w_ih, w_hh, b, h0, c0, h_all, c_final};
    const char *names[8] = {"x", "w_ih", "w_hh", "b", "h0", "c0", "h_all", "c_final"};
    for (int i = 0; i < 8; ++i) RELAY_TRY(check_not_null(all[i], names[i]));
    LstmDims d;
    RELAY_TRY(check_lstm(x, w_ih, w_hh, &d));
    for (int i = 3; i < 8; ++i) RELAY_TRY(check_type(all[i], names[i]));
    RELAY_TRY(check_rank(b, 1, "b"));
    RELAY_TRY(check_rank(h0, 2, "h0"));
    RELAY_TRY(check_rank(c0, 2, "c0"));
    RELAY_TRY(check_rank(h_all, 3, "h_all"));
    RELAY_TRY(check_rank(c_final, 2, "c_final"));
    for (int i = 3; i < 8; ++i) RELAY_TRY(check_dtype(all[i], RELAY_F32, names[i]));
    RELAY_TRY(check_shape(b, {4 * d.H}, "b"));
    RELAY_TRY(check_shape(h0, {d.B, d.H}, "h0"));
    RELAY_TRY(check_shape(c0, {d.B, d.H}, "c0"));
    RELAY_TRY(check_shape(h_all, {d.T, d.B, d.H}, "h_all"));
    RELAY_TRY(check_shape(c_final, {d.B, d.H}, "c_final"));
    for (int i = 0; i < 8; ++i) RELAY_TRY(check_data(all[i], names[i]));
    RELAY_TRY(check_no_overlap(all + 6, 2, all, 6));
    RELAY_TRY(check_workspace(ws, ws_bytes, lstm_ws(d)));
    cudaStream_t st = (cudaStream_t)stream;
    if (d.B == 0 || d.H == 0) return RELAY_OK;
    const bool tc = d.T > 0 && lstm_tc_eligible(d.T, d.B, d.H);
    // the per-step kernels carry the cell state in c_final; the persistent kernel keeps it in registers and writes c_final itself
    if (!tc) RELAY_CUDA(cudaMemcpyAsync(c_final->data, c0->data, nbytes(c0), cudaMemcpyDeviceToDevice, st));
    if (d.T == 0) return RELAY_OK;
    if (tc) RELAY_TRY(launch_lstm_tc_prepare(d.B, d.H, w_hh->data, (char *)ws + lstm_zx_bytes(d), st));

    // (1) zx = x W_ih + b for all T*B rows
    float *zx = (float *)ws;
    GemmDesc g;
    g.M = d.T * d.B; g.N = 4 * d.H; g.K = d.I;
    g.a = x->data; g.a_sm = d.I; g.a_sk = 1;
    g.b = w_ih->data; g.b_sk = 4 * d.H; g.b_sn = 1;
    g.c = zx; g.ldc = 4 * d.H;
    g.in_dtype = RELAY_BF16; g.out_dtype = RELAY_F32;
    g.bias = b->data; g.bias_dtype = RELAY_F32;
    g.act = RELAY_ACT_NONE;
    RELAY_TRY(launch_gemm(g, st));

    // (2) the dependent steps: one persistent kernel when the shape fits it, else one launch per step
    if (tc)
        return launch_lstm_tc(d.T, d.B, d.H, zx, w_hh->data, (const float *)h0->data, (const float *)c0->data, (float *)h_all->data,
                              (float *)c_final->data, (char *)ws + lstm_zx_bytes(d), st, timing);
    if (timing) return fail(RELAY_ERR_UNSUPPORTED, "phase cycles are counted by the persistent kernel only; this shape runs one launch per step");
    dim3 grid((unsigned)((d.H + 255) / 256), (unsigned)((d.B + kRowsPerBlock - 1) / kRowsPerBlock));
    float *hall = (float *)h_all->data;
    for (int64_t t = 0; t < d.T; ++t) {
        const float *h_prev = t == 0 ? (const float *)h0->data : hall + (t - 1) * d.B * d.H;
        lstm_step_kernel<<<grid, 256, 0, st>>>(zx + t * d.B * 4 * d.H, (const __nv_bfloat16 *)w_hh->data, h_prev,
                                               (float *)c_final->data, hall + t * d.B * d.H, d.B, d.H);
        RELAY_TRY(check_launch("lstm_step"));
    }
    return RELAY_OK;
}

extern "C" relay_status_t relay_lstm_cell_seq(const relay_tensor_t *x, const relay_tensor_t *w_ih, const relay_tensor_t *w_hh,
                                              const relay_tensor_t *b, const relay_tensor_t *h0, const relay_tensor_t *c0,
                                              const relay_tensor_t *h_all, const relay_tensor_t *c_final, void *ws, size_t ws_bytes,
                                              void *stream)
{
    return lstm_seq(x, w_ih, w_hh, b, h0, c0, h_all, c_final, ws, ws_bytes, stream, nullptr);
}

extern "C" relay_status_t relay_debug_lstm_phase_cycles(const relay_tensor_t *x, const relay_tensor_t *w_ih, const relay_tensor_t *w_hh,
                                                        const relay_tensor_t *b, const relay_tensor_t *h0, const relay_tensor_t *c0,
                                                        const relay_tensor_t *h_all, const relay_tensor_t *c_final, void *ws, size_t ws_bytes,
                                                        int64_t *cycles, void *stream)
{
    clear_error();
    RELAY_TRY(check_not_null(cycles, "cycles"));
    if (((uintptr_t)cycles & 7) != 0) return fail(RELAY_ERR_ALIGN, "cycles: not 8-byte aligned");
    RELAY_CUDA(cudaMemsetAsync(cycles, 0, 8 * sizeof(int64_t), (cudaStream_t)stream));
    return lstm_seq(x, w_ih, w_hh, b, h0, c0, h_all, c_final, ws, ws_bytes, stream, (long long *)cycles);
}
