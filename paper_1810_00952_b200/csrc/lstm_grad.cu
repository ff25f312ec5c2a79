// Gradient program of the LSTM sequence (Section 4.2 of the paper: reverse mode, here through the
// recursion over time).
//
// Plan:
//   (1) batched, independent of the recursion: hq[t] = bf16(h_{t-1}) from the saved h_all, one contraction
//       Z = [x | hq] [W_ih ; W_hh] + b for all T*B rows (fp32), then one sweep over time that turns Z into
//       the activated gates in place and stores every cell state c_t;
//   (2) the T dependent steps, last to first: dh = dh_all[t] + dz_{t+1} W_hh^T, the gate derivatives, and
//       dz_t (bf16) written into dZ[t]: one persistent kernel of thread-block clusters when the shape fits it
//       (lstm_grad_tc.cu), else one launch per step;
//   (3) batched again: dx = dZ W_ih^T, dW_ih = x^T dZ, dW_hh = hq^T dZ (tensor-core contractions), db = column
//       sums of dZ.
// dz is rounded to bf16 before any contraction reads it (it is the bf16 operand of four of them).
#include <algorithm>

#include "ewise_host.h"
#include "ewise_kernels.cuh"
#include "gemm.h"
#include "lstm.h"

namespace relay {

namespace {

__device__ __forceinline__ float sigm(float x) { return __fdividef(1.0f, 1.0f + __expf(-x)); }
__device__ __forceinline__ float tanh_fast(float x) { return lstm_tanh_fast(x); }

// a[t*B+b][0..I) = x[t,b,:],  a[t*B+b][I..I+H) = bf16(h_{t-1}[b,:])   (h_{-1} = h0)
// VEC = 8: one thread moves 8 consecutive elements (I and H multiples of 8); VEC = 1: any shape
template <int VEC>
__global__ void __launch_bounds__(256) lstm_cat_kernel(const __nv_bfloat16 *__restrict__ x, const float *__restrict__ h0,
                                                        const float *__restrict__ h_all, __nv_bfloat16 *__restrict__ a, int64_t T,
                                                        int64_t B, int64_t I, int64_t H)
{
    const int64_t W = I + H, total = T * B * W / VEC;
    pdl_wait();
    for (int64_t v = (int64_t)blockIdx.x * 256 + threadIdx.x; v < total; v += (int64_t)gridDim.x * 256) {
        const int64_t e = v * VEC;
        const int64_t row = e / W, col = e % W;
        if (col < I) {
            if (VEC == 8) *reinterpret_cast<uint4 *>(a + e) = ld_stream(x + row * I + col);
            else a[e] = x[row * I + col];
        } else {
            const int64_t t = row / B, b = row % B;
            const float *src = (t == 0 ? h0 + b * H : h_all + ((t - 1) * B + b) * H) + (col - I);
            if (VEC == 8) {
                float f[8];
                const float4 lo = *reinterpret_cast<const float4 *>(src), hi = *reinterpret_cast<const float4 *>(src + 4);
                f[0] = lo.x; f[1] = lo.y; f[2] = lo.z; f[3] = lo.w; f[4] = hi.x; f[5] = hi.y; f[6] = hi.z; f[7] = hi.w;
                *reinterpret_cast<uint4 *>(a + e) = pack(f);
            } else {
                a[e] = __float2bfloat16_rn(*src);
            }
        }
    }
}

// one thread per (batch row, hidden unit): over time, z -> activated gates in place, c_all[t] = c_t.
// Only c carries from step to step: the loads of four steps are issued together so that their latency is paid once.
// ACTIVATED: z already holds the activated gates (the contraction's epilogue applied them); only c_t is left to do, from
// i, f and g, and nothing is written back to z.
template <bool ACTIVATED>
__global__ void __launch_bounds__(256) lstm_cell_sweep_kernel(float *__restrict__ z, const float *__restrict__ c0,
                                                               float *__restrict__ c_all, int64_t T, int64_t B, int64_t H)
{
    const int64_t idx = (int64_t)blockIdx.x * 256 + threadIdx.x;
    pdl_wait();
    if (idx >= B * H) return;
    const int64_t b = idx / H, u = idx % H;
    float c = c0[idx];
    constexpr int U = ACTIVATED ? 8 : 4;
    for (int64_t t0 = 0; t0 < T; t0 += U) {
        float zi[U], zf[U], zg[U], zo[ACTIVATED ? 1 : U];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            if (t0 + k < T) {
                const float *zr = z + ((t0 + k) * B + b) * 4 * H + u;
                zi[k] = zr[0]; zf[k] = zr[H]; zg[k] = zr[2 * H];
                if (!ACTIVATED) zo[k] = zr[3 * H];
            }
        }
#pragma unroll
        for (int k = 0; k < U; ++k) {
            if (t0 + k < T) {
                if (ACTIVATED) {
                    c = fmaf(zf[k], c, zi[k] * zg[k]);
                } else {
                    float *zr = z + ((t0 + k) * B + b) * 4 * H + u;
                    const float ig = sigm(zi[k]), fg = sigm(zf[k]), gg = tanh_fast(zg[k]), og = sigm(zo[ACTIVATED ? 0 : k]);
                    c = fmaf(fg, c, ig * gg);
                    zr[0] = ig; zr[H] = fg; zr[2 * H] = gg; zr[3 * H] = og;
                }
                c_all[((t0 + k) * B + b) * H + u] = c;
            }
        }
    }
}

// One step for any shape: thread per (batch row, hidden unit); the recurrent partial is a plain dot product
// over the 4H columns of dz_{t+1}.  `last` = the extra pass that only produces dh0.
__global__ void __launch_bounds__(256) lstm_grad_step_kernel(const float *__restrict__ gates_t, const float *__restrict__ c_t,
                                                              const float *__restrict__ c_prev, const float *__restrict__ dh_t,
                                                              const __nv_bfloat16 *__restrict__ dz_next,   // [B,4H] or nullptr
                                                              const __nv_bfloat16 *__restrict__ w_hh,      // [H,4H]
                                                              float *__restrict__ dc,                      // [B,H] in/out
                                                              __nv_bfloat16 *__restrict__ dz_t,            // [B,4H] out
                                                              float *__restrict__ dh0, int64_t B, int64_t H, int last)
{
    const int64_t idx = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (idx >= B * H) return;
    const int64_t b = idx / H, u = idx % H;
    float rec = 0.0f;
    if (dz_next != nullptr) {
        const __nv_bfloat16 *dr = dz_next + b * 4 * H, *wr = w_hh + u * 4 * H;
        for (int64_t k = 0; k < 4 * H; ++k) rec = fmaf(__bfloat162float(dr[k]), __bfloat162float(wr[k]), rec);
    }
    if (last) { if (dh0) dh0[idx] = rec; return; }
    const float *gr = gates_t + b * 4 * H + u;
    float dz[4], dcv = dc[idx];
    lstm_gate_grads(gr[0], gr[H], gr[2 * H], gr[3 * H], c_t[idx], c_prev[idx], dh_t[idx] + rec, dcv, dz);
    dc[idx] = dcv;
#pragma unroll
    for (int g = 0; g < 4; ++g) dz_t[b * 4 * H + g * H + u] = __float2bfloat16_rn(dz[g]);
}

// out[c] = sum_r in[r,c] for rows that are not whole 16-byte vectors
__global__ void __launch_bounds__(128) colsum_any_kernel(const __nv_bfloat16 *__restrict__ in, int64_t rows, int64_t cols, float *__restrict__ out)
{
    const int64_t c = (int64_t)blockIdx.x * 128 + threadIdx.x;
    if (c >= cols) return;
    float s = 0.0f;
    for (int64_t r = 0; r < rows; ++r) s += __bfloat162float(in[r * cols + c]);
    out[c] = s;
}

struct GradDims { int64_t T, B, I, H; };

struct GradPlan {
    size_t gates, c_all, dz, a_cat, w_cat, dc, partials, counters, total;
    bool tc;
    int n_slices;
};

size_t up(size_t v) { return align_up(v, 1024); }

GradPlan plan_of(const GradDims &d)
{
    GradPlan p{};
    const size_t rows = (size_t)d.T * d.B, G = 4 * (size_t)d.H;
    size_t off = 0;
    p.gates = off; off += up(rows * G * sizeof(float));
    p.c_all = off; off += up(rows * d.H * sizeof(float));
    p.dz = off; off += up(rows * G * 2);
    p.a_cat = off; off += up(rows * (size_t)(d.I + d.H) * 2);
    p.w_cat = off; off += up((size_t)(d.I + d.H) * G * 2);
    p.dc = off; off += up((size_t)d.B * d.H * sizeof(float));
    p.n_slices = (G % 8 == 0 && rows > 0) ? colsum_slices((int64_t)rows, (int64_t)G, RELAY_BF16) : 0;
    p.partials = off; off += up((size_t)p.n_slices * G * sizeof(float));
    p.counters = off; off += 1024;
    p.total = off;
    p.tc = lstm_tc_eligible(d.T, d.B, d.H);
    return p;
}

relay_status_t check_lstm_dims(const relay_tensor_t *x, const relay_tensor_t *w_ih, const relay_tensor_t *w_hh, GradDims *d)
{
    relay_tensor_t ht, ct;
    RELAY_TRY(relay_infer_lstm(x, w_ih, w_hh, &ht, &ct));
    d->T = x->shape[0]; d->B = x->shape[1]; d->I = x->shape[2]; d->H = w_hh->shape[0];
    return RELAY_OK;
}

relay_status_t run_steps_any(const GradDims &d, const GradPlan &pl, char *ws, const void *w_hh, const float *c0, const float *dh_all,
                             const float *dc_final, float *dh0, float *dc0, cudaStream_t st)
{
    float *dc = (float *)(ws + pl.dc);
    const size_t bh = (size_t)d.B * d.H;
    if (dc_final) RELAY_CUDA(cudaMemcpyAsync(dc, dc_final, bh * sizeof(float), cudaMemcpyDeviceToDevice, st));
    else RELAY_CUDA(cudaMemsetAsync(dc, 0, bh * sizeof(float), st));
    const float *gates = (const float *)(ws + pl.gates), *c_all = (const float *)(ws + pl.c_all);
    __nv_bfloat16 *dz = (__nv_bfloat16 *)(ws + pl.dz);
    const unsigned grid = (unsigned)((bh + 255) / 256);
    const size_t G = 4 * (size_t)d.H;
    for (int64_t t = d.T - 1; t >= 0; --t) {
        lstm_grad_step_kernel<<<grid, 256, 0, st>>>(gates + (size_t)t * d.B * G, c_all + (size_t)t * bh, t > 0 ? c_all + (size_t)(t - 1) * bh : c0,
                                                    dh_all + (size_t)t * bh, t < d.T - 1 ? dz + (size_t)(t + 1) * d.B * G : nullptr,
                                                    (const __nv_bfloat16 *)w_hh, dc, dz + (size_t)t * d.B * G, nullptr, d.B, d.H, 0);
        RELAY_TRY(check_launch("lstm_grad_step"));
    }
    if (dh0) {
        lstm_grad_step_kernel<<<grid, 256, 0, st>>>(nullptr, nullptr, nullptr, nullptr, dz, (const __nv_bfloat16 *)w_hh, dc, nullptr, dh0, d.B, d.H, 1);
        RELAY_TRY(check_launch("lstm_grad_step"));
    }
    if (dc0) RELAY_CUDA(cudaMemcpyAsync(dc0, dc, bh * sizeof(float), cudaMemcpyDeviceToDevice, st));
    return RELAY_OK;
}

}  // namespace
}  // namespace relay

using namespace relay;

extern "C" size_t relay_workspace_bytes_lstm_grad(const relay_tensor_t *x, const relay_tensor_t *w_ih, const relay_tensor_t *w_hh)
{
    GradDims d;
    if (!x || !w_ih || !w_hh || check_lstm_dims(x, w_ih, w_hh, &d) != RELAY_OK) return 0;
    return plan_of(d).total;
}

extern "C" relay_status_t relay_lstm_cell_seq_grad(const relay_tensor_t *x, const relay_tensor_t *w_ih, const relay_tensor_t *w_hh,
                                                   const relay_tensor_t *b, const relay_tensor_t *h0, const relay_tensor_t *c0,
                                                   const relay_tensor_t *h_all, const relay_tensor_t *dh_all,
                                                   const relay_tensor_t *dc_final, const relay_tensor_t *dx, const relay_tensor_t *dw_ih,
                                                   const relay_tensor_t *dw_hh, const relay_tensor_t *db, const relay_tensor_t *dh0,
                                                   const relay_tensor_t *dc0, void *ws, size_t ws_bytes, void *stream)
{
    clear_error();
    const relay_tensor_t *need[10] = {x, w_ih, w_hh, b, h0, c0, h_all, dh_all, dw_ih, dw_hh};
    const char *need_name[10] = {"x", "w_ih", "w_hh", "b", "h0", "c0", "h_all", "dh_all", "dw_ih", "dw_hh"};
    for (int i = 0; i < 10; ++i) RELAY_TRY(check_not_null(need[i], need_name[i]));
    GradDims d;
    RELAY_TRY(check_lstm_dims(x, w_ih, w_hh, &d));
    // f32 tensors: name, rank, shape
    struct F { const relay_tensor_t *t; const char *name; int rank; int64_t s0, s1, s2; };
    const F f32s[9] = {{b, "b", 1, 4 * d.H, 0, 0},          {h0, "h0", 2, d.B, d.H, 0},       {c0, "c0", 2, d.B, d.H, 0},
                       {h_all, "h_all", 3, d.T, d.B, d.H},  {dh_all, "dh_all", 3, d.T, d.B, d.H}, {dc_final, "dc_final", 2, d.B, d.H, 0},
                       {db, "db", 1, 4 * d.H, 0, 0},        {dh0, "dh0", 2, d.B, d.H, 0},     {dc0, "dc0", 2, d.B, d.H, 0}};
    const F bf16s[3] = {{dx, "dx", 3, d.T, d.B, d.I}, {dw_ih, "dw_ih", 2, d.I, 4 * d.H, 0}, {dw_hh, "dw_hh", 2, d.H, 4 * d.H, 0}};
    for (const F &f : f32s) if (f.t) { RELAY_TRY(check_type(f.t, f.name)); RELAY_TRY(check_rank(f.t, f.rank, f.name)); }
    for (const F &f : bf16s) if (f.t) { RELAY_TRY(check_type(f.t, f.name)); RELAY_TRY(check_rank(f.t, f.rank, f.name)); }
    for (const F &f : f32s) if (f.t) RELAY_TRY(check_dtype(f.t, RELAY_F32, f.name));
    for (const F &f : bf16s) if (f.t) RELAY_TRY(check_dtype(f.t, RELAY_BF16, f.name));
    auto shape_ok = [](const F &f) -> relay_status_t {
        if (f.rank == 1) return check_shape(f.t, {f.s0}, f.name);
        if (f.rank == 2) return check_shape(f.t, {f.s0, f.s1}, f.name);
        return check_shape(f.t, {f.s0, f.s1, f.s2}, f.name);
    };
    for (const F &f : f32s) if (f.t) RELAY_TRY(shape_ok(f));
    for (const F &f : bf16s) if (f.t) RELAY_TRY(shape_ok(f));
    const relay_tensor_t *ins[9] = {x, w_ih, w_hh, b, h0, c0, h_all, dh_all, dc_final};
    const relay_tensor_t *outs[6] = {dx, dw_ih, dw_hh, db, dh0, dc0};
    for (int i = 0; i < 9; ++i) if (ins[i]) RELAY_TRY(check_data(ins[i], "input"));
    for (int i = 0; i < 6; ++i) if (outs[i]) RELAY_TRY(check_data(outs[i], "output"));
    RELAY_TRY(check_no_overlap(outs, 6, ins, 9));
    const GradPlan pl = plan_of(d);
    RELAY_TRY(check_workspace(ws, ws_bytes, pl.total));

    cudaStream_t st = (cudaStream_t)stream;
    const size_t bh = (size_t)d.B * d.H;
    if (d.T == 0 || d.B == 0 || d.H == 0) {
        // nothing flows through time: the weights get the zero tensor (Fig. 5 Type-Zero), the initial state gets
        // what the final state was given
        if (numel(dw_ih)) RELAY_CUDA(cudaMemsetAsync(dw_ih->data, 0, nbytes(dw_ih), st));
        if (numel(dw_hh)) RELAY_CUDA(cudaMemsetAsync(dw_hh->data, 0, nbytes(dw_hh), st));
        if (db && numel(db)) RELAY_CUDA(cudaMemsetAsync(db->data, 0, nbytes(db), st));
        if (dh0 && bh) RELAY_CUDA(cudaMemsetAsync(dh0->data, 0, bh * sizeof(float), st));
        if (dc0 && bh) {
            if (dc_final) RELAY_CUDA(cudaMemcpyAsync(dc0->data, dc_final->data, bh * sizeof(float), cudaMemcpyDeviceToDevice, st));
            else RELAY_CUDA(cudaMemsetAsync(dc0->data, 0, bh * sizeof(float), st));
        }
        return RELAY_OK;
    }

    char *base = (char *)ws;
    const int64_t rows = d.T * d.B, G = 4 * d.H, W = d.I + d.H;
    __nv_bfloat16 *a_cat = (__nv_bfloat16 *)(base + pl.a_cat), *w_cat = (__nv_bfloat16 *)(base + pl.w_cat);
    __nv_bfloat16 *dz = (__nv_bfloat16 *)(base + pl.dz);
    float *gates = (float *)(base + pl.gates), *c_all = (float *)(base + pl.c_all);

    // (1) recompute the forward values the reverse sweep reads
    {
        const bool vec = d.I % 8 == 0 && d.H % 8 == 0;
        const unsigned grid = (unsigned)std::max<int64_t>(1, std::min<int64_t>((rows * W / (vec ? 8 : 1) + 255) / 256, 148 * 32));
        if (vec) RELAY_CUDA(launch_pdl(lstm_cat_kernel<8>, dim3(grid), dim3(256), 0, st, (const __nv_bfloat16 *)x->data, (const float *)h0->data,
                                       (const float *)h_all->data, a_cat, d.T, d.B, d.I, d.H));
        else RELAY_CUDA(launch_pdl(lstm_cat_kernel<1>, dim3(grid), dim3(256), 0, st, (const __nv_bfloat16 *)x->data, (const float *)h0->data,
                                   (const float *)h_all->data, a_cat, d.T, d.B, d.I, d.H));
        RELAY_TRY(check_launch("lstm_cat"));
        RELAY_CUDA(cudaMemcpyAsync(w_cat, w_ih->data, (size_t)d.I * G * 2, cudaMemcpyDeviceToDevice, st));
        RELAY_CUDA(cudaMemcpyAsync(w_cat + (size_t)d.I * G, w_hh->data, (size_t)d.H * G * 2, cudaMemcpyDeviceToDevice, st));
        GemmDesc g;
        g.M = rows; g.N = G; g.K = W;
        g.a = a_cat; g.a_sm = W; g.a_sk = 1;
        g.b = w_cat; g.b_sk = G; g.b_sn = 1;
        g.c = gates; g.ldc = G;
        g.in_dtype = RELAY_BF16; g.out_dtype = RELAY_F32;
        g.bias = b->data; g.bias_dtype = RELAY_F32; g.act = RELAY_ACT_NONE;
        // where the two-SM contraction kernel takes the shape its epilogue applies the gate activations, and the sweep that
        // follows only forms c_t: it then reads three of the four gates and writes no gate back (134 MB instead of 302 MB
        // at T = 128, B = 64, H = 1024)
        int dev = 0, sms = 0;
        RELAY_CUDA(cudaGetDevice(&dev));
        RELAY_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        const bool fused_gates = d.H % 32 == 0 && gemm_tc_eligible(g) && gemm_tc2_eligible(g, sms);
        if (fused_gates) {
            g.gate_block = d.H;
            RELAY_TRY(launch_gemm_tc2(g, sms, st));
            RELAY_CUDA(launch_pdl(lstm_cell_sweep_kernel<true>, dim3((unsigned)((bh + 255) / 256)), dim3(256), 0, st, gates, (const float *)c0->data,
                                  c_all, d.T, d.B, d.H));
        } else {
            RELAY_TRY(launch_gemm(g, st));
            RELAY_CUDA(launch_pdl(lstm_cell_sweep_kernel<false>, dim3((unsigned)((bh + 255) / 256)), dim3(256), 0, st, gates, (const float *)c0->data,
                                  c_all, d.T, d.B, d.H));
        }
        RELAY_TRY(check_launch("lstm_cell_sweep"));
    }

    // (2) the dependent steps, last to first
    const float *dcf = dc_final ? (const float *)dc_final->data : nullptr;
    float *dh0p = dh0 ? (float *)dh0->data : nullptr, *dc0p = dc0 ? (float *)dc0->data : nullptr;
    bool clustered = false;
    if (pl.tc) RELAY_TRY(launch_lstm_grad_cluster(d.T, d.B, d.H, gates, c_all, (const float *)c0->data, (const float *)dh_all->data, dcf, w_hh->data, dz,
                                                  dh0p, dc0p, (unsigned int *)(base + pl.counters), st, &clustered));
    if (!clustered) RELAY_TRY(run_steps_any(d, pl, base, w_hh->data, (const float *)c0->data, (const float *)dh_all->data, dcf, dh0p, dc0p, st));

    // (3) the batched contractions over all T*B rows of dZ
    if (dx && d.I > 0) {
        GemmDesc g;
        g.M = rows; g.N = d.I; g.K = G;
        g.a = dz; g.a_sm = G; g.a_sk = 1;
        g.b = w_ih->data; g.b_sk = 1; g.b_sn = G;
        g.c = dx->data; g.ldc = d.I;
        g.in_dtype = RELAY_BF16; g.out_dtype = RELAY_BF16;
        RELAY_TRY(launch_gemm(g, st));
    }
    for (int which = 0; which < 2; ++which) {
        const relay_tensor_t *out = which == 0 ? dw_ih : dw_hh;
        const int64_t M = which == 0 ? d.I : d.H;
        if (M == 0) continue;
        GemmDesc g;
        g.M = M; g.N = G; g.K = rows;
        g.a = a_cat + (which == 0 ? 0 : d.I); g.a_sm = 1; g.a_sk = W;
        g.b = dz; g.b_sk = G; g.b_sn = 1;
        g.c = out->data; g.ldc = G;
        g.in_dtype = RELAY_BF16; g.out_dtype = RELAY_BF16;
        RELAY_TRY(launch_gemm(g, st));
    }
    if (db) {
        if (pl.n_slices > 0) {
            RELAY_TRY(launch_colsum_bf16(dz, rows, G, (float *)(base + pl.partials), (float *)db->data, st));
        } else {
            colsum_any_kernel<<<(unsigned)((G + 127) / 128), 128, 0, st>>>(dz, rows, G, (float *)db->data);
            RELAY_TRY(check_launch("colsum_any"));
        }
    }
    return RELAY_OK;
}
