// Gradient program of the LSTM sequence (Section 4.2 of the paper: reverse mode, here through the
// recursion over time).
//
// Plan:
//   (1) batched, independent of the recursion: hq[t] = bf16(h_{t-1}) from the saved h_all, one contraction
//       Z = [x | hq] [W_ih ; W_hh] + b for all T*B rows (fp32), then one sweep over time that turns Z into
//       the activated gates in place and stores every cell state c_t;
//   (2) the T dependent steps, last to first: dh = dh_all[t] + dz_{t+1} W_hh^T, the gate derivatives, and
//       dz_t (bf16) written into dZ[t]: one persistent cooperative kernel when the shape fits it (the
//       block's slice of W_hh stays in shared memory, dz_{t+1} is streamed by TMA, tcgen05 does the
//       product), else one launch per step;
//   (3) batched again: dx = dZ W_ih^T, dW_ih = x^T dZ, dW_hh = hq^T dZ (tensor-core contractions), db = column
//       sums of dZ.
// dz is rounded to bf16 before any contraction reads it (it is the bf16 operand of four of them).
#include <cooperative_groups.h>

#include <algorithm>

#include "ewise_host.h"
#include "ewise_kernels.cuh"
#include "gemm.h"
#include "lstm.h"
#include "tc_common.cuh"

namespace relay {

relay_status_t make_tmap_2d_bf16(CUtensorMap *m, const void *base, uint64_t inner, uint64_t outer, uint64_t row_stride,
                                 uint32_t box_inner, uint32_t box_outer);

namespace {

__device__ __forceinline__ float sigm(float x) { return __fdividef(1.0f, 1.0f + __expf(-x)); }
__device__ __forceinline__ float tanh_fast(float x) { return 1.0f - __fdividef(2.0f, 1.0f + __expf(2.0f * x)); }

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
__global__ void __launch_bounds__(256) lstm_cell_sweep_kernel(float *__restrict__ z, const float *__restrict__ c0,
                                                               float *__restrict__ c_all, int64_t T, int64_t B, int64_t H)
{
    const int64_t idx = (int64_t)blockIdx.x * 256 + threadIdx.x;
    pdl_wait();
    if (idx >= B * H) return;
    const int64_t b = idx / H, u = idx % H;
    float c = c0[idx];
    constexpr int U = 4;
    for (int64_t t0 = 0; t0 < T; t0 += U) {
        float zi[U], zf[U], zg[U], zo[U];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            if (t0 + k < T) {
                const float *zr = z + ((t0 + k) * B + b) * 4 * H + u;
                zi[k] = zr[0]; zf[k] = zr[H]; zg[k] = zr[2 * H]; zo[k] = zr[3 * H];
            }
        }
#pragma unroll
        for (int k = 0; k < U; ++k) {
            if (t0 + k < T) {
                float *zr = z + ((t0 + k) * B + b) * 4 * H + u;
                const float ig = sigm(zi[k]), fg = sigm(zf[k]), gg = tanh_fast(zg[k]), og = sigm(zo[k]);
                c = fmaf(fg, c, ig * gg);
                zr[0] = ig; zr[H] = fg; zr[2 * H] = gg; zr[3 * H] = og;
                c_all[((t0 + k) * B + b) * H + u] = c;
            }
        }
    }
}

// The gate derivatives of one (row, unit) at one step.  dh: partial of h_t; dc: carried partial of c_t
// (in: from step t+1, out: for step t-1).
__device__ __forceinline__ void gate_grads(float ig, float fg, float gg, float og, float c_t, float c_prev, float dh, float &dc,
                                           float (&dz)[4])
{
    const float tc = tanh_fast(c_t);
    const float d_o = dh * tc;
    const float dct = fmaf(dh * og, 1.0f - tc * tc, dc);
    dz[0] = dct * gg * ig * (1.0f - ig);
    dz[1] = dct * c_prev * fg * (1.0f - fg);
    dz[2] = dct * ig * (1.0f - gg * gg);
    dz[3] = d_o * og * (1.0f - og);
    dc = dct * fg;
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
    gate_grads(gr[0], gr[H], gr[2 * H], gr[3 * H], c_t[idx], c_prev[idx], dh_t[idx] + rec, dcv, dz);
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

// ---- the dependent steps as one persistent cooperative kernel -----------------------------------------------
// Block (grp, blk) owns 16 hidden units and the batch rows of group grp.  Per step s = 1 .. T it needs
// dh_rec[row, unit] = sum_col dz_{T-s}[row, col] * W_hh[unit, col] over all 4H columns: its 16 rows of W_hh
// (16 x 4H bf16, at most 128 KB) stay in shared memory, dz of the group's rows is streamed from the dZ array
// (L2) through a ring by TMA, issuer warps run tcgen05.mma (D[row, 16 units] in TMEM).  The epilogue warp
// owning a row adds dh_all, applies the gate derivatives, writes bf16(dz_t) of its 64 gate columns into
// dZ[t] and arrives on the group's grid barrier; the carried dc stays in registers.
constexpr int UNITS = 16;
constexpr int BK = 64, MAX_STAGES = 32;
constexpr int A_TILE = 128 * BK * 2;             // what one MMA reads as its A operand: 128 rows x 64 k
constexpr int RING_BYTES = 96 * 1024;
constexpr int W_KB = UNITS * BK * 2;             // one k-block of the resident W slice
// As in the forward kernel, ring stages are only as far apart as the rows a group really has: the MMA's rows
// beyond the group's are whatever follows in shared memory, and the accumulator rows they produce are never read.
constexpr int N_ISS = 4;                         // MMA-issuing threads (one lane each of warps 4, 6, 7, 8), one accumulator each
constexpr int NUM_THREADS = 512;                 // warps 0-3 and 12-15 epilogue, warp 4 W loader + issuer 0, warps 5 and 9 dz loaders, warps 6-8 issuers 1-3
constexpr int TMEM_COLS = N_ISS * UNITS;
// Issuing a tcgen05.mma of N = 16 costs the issuing warp tens of cycles even with warp-uniform operands (about 130
// from a single divergent lane), far more than the tensor pipe needs for it.  So a ring stage holds N_ISS k-blocks (one barrier round per stage), each
// issuer takes one k-block of every stage into its own accumulator, and the epilogue adds the accumulators up.

struct GradParams {
    int T, B, H, n_blocks, k_blocks;
    int rows_per_group, n_epi;
    int rows_per_warp;               // 32 (M = 128 MMAs), or 16 with M = 64 MMAs for groups of at most 64 rows (half the A rows read)
    int tile_stride, n_stages;       // bytes between the k-block tiles of the ring (a stage is N_ISS tiles); stages in the ring
    int n_load;                      // loader threads (1 or 2): they take the stages of a step in turn
    const float *gates;              // [T*B][4H] activated gates i | f | g | o
    const float *c_all, *c0;         // [T*B][H], [B][H]
    const float *dh_all;             // [T*B][H]
    const float *dc_final;           // [B][H] or nullptr
    __nv_bfloat16 *dz;               // [T*B][4H]
    float *dh0, *dc0;                // [B][H] or nullptr
    unsigned int *counter;
    int *err;
};

__device__ __forceinline__ unsigned int ld_acquire(const unsigned int *p)
{
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release_add(unsigned int *p, unsigned int v)
{
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void load8(const float *p, float (&v)[UNITS / 2])
{
#pragma unroll
    for (int i = 0; i < UNITS / 2; i += 4) {
        const float4 q = *reinterpret_cast<const float4 *>(p + i);
        v[i] = q.x; v[i + 1] = q.y; v[i + 2] = q.z; v[i + 3] = q.w;
    }
}
__device__ __forceinline__ void load16(const float *p, float (&v)[UNITS])
{
#pragma unroll
    for (int i = 0; i < UNITS; i += 4) {
        const float4 q = *reinterpret_cast<const float4 *>(p + i);
        v[i] = q.x; v[i + 1] = q.y; v[i + 2] = q.z; v[i + 3] = q.w;
    }
}

__global__ void __launch_bounds__(NUM_THREADS, 1)
lstm_grad_persistent_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_dz, const GradParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *a_s = smem;                                           // [n_stages][rows of the group x 128 B], RING_BYTES
    uint8_t *w_s = smem + RING_BYTES;                              // [k_blocks][16 rows x 128 B]
    uint64_t *bars = reinterpret_cast<uint64_t *>(w_s + max(p.k_blocks * W_KB, A_TILE));
    uint64_t *full = bars, *empty = bars + MAX_STAGES, *w_full = bars + 2 * MAX_STAGES, *tmem_full = bars + 2 * MAX_STAGES + 1;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * MAX_STAGES + 2);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;   // provably warp-uniform
    const int blk = blockIdx.x % p.n_blocks, grp = blockIdx.x / p.n_blocks;
    const int j0 = blk * UNITS;
    const int b_lo = grp * p.rows_per_group;
    const int nb = min(p.rows_per_group, p.B - b_lo);
    unsigned int *counter = p.counter + grp * 32;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.n_stages; ++s) { tc::mbar_init(&full[s], 1); tc::mbar_init(&empty[s], N_ISS); }
        tc::mbar_init(w_full, 1);
        tc::mbar_init(tmem_full, N_ISS);
        *abort_flag = 0;
        tc::fence_barrier_init();
        tc::prefetch_tmap(&tm_w);
        tc::prefetch_tmap(&tm_dz);
    }
    for (int i = threadIdx.x; i < RING_BYTES / 16; i += NUM_THREADS) reinterpret_cast<uint4 *>(a_s)[i] = make_uint4(0, 0, 0, 0);
    tc::fence_proxy_async();
    if (warp == 4) { tc::tmem_alloc(tmem_slot, TMEM_COLS); tc::tmem_relinquish(); }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp < 4 || warp >= 12) {
      const int ew = warp & 3, half = warp >= 12 ? 1 : 0;
      if (ew < p.n_epi) {
        // ------------------------------ epilogue: one batch row per lane, 8 of the block's 16 units per warp ------------------------------
        // Two warps share a TMEM lane quarter (warps w and 12 + w) and take 8 units each: one warp alone issues its
        // instructions only every few cycles, and this part is on the critical path of every step.
        // M = 128: accumulator row r sits in TMEM lane r.  M = 64: rows 16w .. 16w+15 sit in lanes 32w .. 32w+15, so warp w
        // owns 16 rows in its first 16 lanes.
        constexpr int HU = UNITS / 2;
        const int u0 = j0 + half * HU;
        const int b = b_lo + ew * p.rows_per_warp + lane;
        const bool live = lane < p.rows_per_warp && ew * p.rows_per_warp + lane < nb;
        float dc[HU], c_cur[HU];
#pragma unroll
        for (int i = 0; i < HU; ++i) { dc[i] = 0.0f; c_cur[i] = 0.0f; }
        if (live) {
            if (p.dc_final) load8(p.dc_final + (size_t)b * p.H + u0, dc);
            load8(p.c_all + ((size_t)(p.T - 1) * p.B + b) * p.H + u0, c_cur);
        }
        for (int s = 0; s <= p.T; ++s) {
            const int t = p.T - 1 - s;
            // what does not depend on the recurrent product is fetched while it runs
            float gt[4][HU], c_prev[HU], dh[HU];
            if (live && s < p.T) {
                const float *grow = p.gates + ((size_t)t * p.B + b) * 4 * p.H + u0;
#pragma unroll
                for (int g = 0; g < 4; ++g) load8(grow + (size_t)g * p.H, gt[g]);
                load8(t > 0 ? p.c_all + ((size_t)(t - 1) * p.B + b) * p.H + u0 : p.c0 + (size_t)b * p.H + u0, c_prev);
                load8(p.dh_all + ((size_t)t * p.B + b) * p.H + u0, dh);
            }
            if (s > 0) {
                int ok = 1;
                if (lane == 0) ok = tc::mbar_wait(tmem_full, (s - 1) & 1, abort_flag, p.err, tc::ERR_WAIT_TMEM_FULL) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                tc::tc_fence_after_sync();
                uint32_t d[N_ISS][HU];                                                // the four issuers' partial sums of this warp's units
                const uint32_t taddr = tmem_base + ((uint32_t)(ew * 32) << 16) + half * HU;
#pragma unroll
                for (int a = 0; a < N_ISS; ++a) tc::tmem_ld_32x8(taddr + a * UNITS, d[a]);
                tc::tmem_ld_wait();
                tc::tc_fence_before_sync();
                float rec[HU];
#pragma unroll
                for (int i = 0; i < HU; ++i)
                    rec[i] = (__uint_as_float(d[0][i]) + __uint_as_float(d[1][i])) + (__uint_as_float(d[2][i]) + __uint_as_float(d[3][i]));
                if (s == p.T) {
                    if (live && p.dh0) {
                        float4 *o = reinterpret_cast<float4 *>(p.dh0 + (size_t)b * p.H + u0);
#pragma unroll
                        for (int i = 0; i < HU; i += 4) o[i / 4] = make_float4(rec[i], rec[i + 1], rec[i + 2], rec[i + 3]);
                    }
                    break;
                }
#pragma unroll
                for (int i = 0; i < HU; ++i) dh[i] += rec[i];
            }
            if (live) {
                float dzv[4][HU];
#pragma unroll
                for (int i = 0; i < HU; ++i) {
                    float q[4];
                    gate_grads(gt[0][i], gt[1][i], gt[2][i], gt[3][i], c_cur[i], c_prev[i], dh[i], dc[i], q);
                    dzv[0][i] = q[0]; dzv[1][i] = q[1]; dzv[2][i] = q[2]; dzv[3][i] = q[3];
                    c_cur[i] = c_prev[i];
                }
                __nv_bfloat16 *drow = p.dz + ((size_t)t * p.B + b) * 4 * p.H + u0;
#pragma unroll
                for (int g = 0; g < 4; ++g)
                    *reinterpret_cast<uint4 *>(drow + (size_t)g * p.H) =
                        make_uint4(pack2(dzv[g][0], dzv[g][1]), pack2(dzv[g][2], dzv[g][3]), pack2(dzv[g][4], dzv[g][5]), pack2(dzv[g][6], dzv[g][7]));
            }
            // dZ[t] is read by TMA (async proxy) in the other blocks: fence the generic stores for it; the warp barrier orders
            // the warp's stores before lane 0's release, which is cumulative
            asm volatile("fence.proxy.async.global;" ::: "memory");
            __syncwarp();
            if (lane == 0) red_release_add(counter, 1u);
        }
        if (live && p.dc0) {
            float4 *o = reinterpret_cast<float4 *>(p.dc0 + (size_t)b * p.H + u0);
#pragma unroll
            for (int i = 0; i < HU; i += 4) o[i / 4] = make_float4(dc[i], dc[i + 1], dc[i + 2], dc[i + 3]);
        }
      }
    } else if (warp == 5 || warp == 9) {
        // ------------------------------ dz loaders: dZ[T-s] rows of the group -> ring, by TMA ------------------------------
        // (two loader warps take the stages of a step in turn)
        const int ld = warp == 5 ? 0 : 1;
        if (ld < p.n_load) {                                           // warp-uniform loop, an elected lane issues
            int st = ld;
            uint32_t phase = 0;
            bool ok = true;
            const uint32_t stage_bytes = (uint32_t)(N_ISS * p.rows_per_group * 128);
            for (int s = 1; s <= p.T && ok; ++s) {
                // grid barrier: every block of the group has written its columns of dZ[T-s] (lane 0 polls, the warp follows)
                const unsigned int target = (unsigned int)(2 * p.n_epi * p.n_blocks) * (unsigned int)s;   // two epilogue warps per 16 or 32 rows
                if (lane == 0) {
                    const long long t0 = clock64();
                    unsigned spins = 0;
                    while (ld_acquire(counter) < target) {
                        if ((++spins & 255u) == 0 && (*abort_flag || clock64() - t0 > tc::kWaitLimitCycles)) {
                            if (!*abort_flag) { *abort_flag = 1; atomicCAS(p.err, 0, tc::ERR_WAIT_STEP); }
                            ok = false;
                            break;
                        }
                    }
                }
                __syncwarp();                                           // lane 0's acquire is ordered before the other lanes' accesses
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
                asm volatile("fence.proxy.async.global;" ::: "memory");   // every lane: whichever lane is elected issues the copies
                const int row0 = (p.T - s) * p.B + b_lo;
                for (int kb = ld * N_ISS; kb < p.k_blocks; kb += p.n_load * N_ISS) {
                    ok = __all_sync(0xffffffffu, tc::mbar_wait(&empty[st], phase ^ 1, abort_flag, p.err, tc::ERR_WAIT_EMPTY));
                    if (!ok) break;
                    uint8_t *dst = a_s + (size_t)st * N_ISS * p.tile_stride;
                    if (tc::elect_one()) {
                        tc::mbar_expect_tx(&full[st], stage_bytes);
#pragma unroll
                        for (int i = 0; i < N_ISS; ++i) tc::tma_load_2d(dst + (size_t)i * p.tile_stride, &tm_dz, &full[st], (kb + i) * BK, row0);
                    }
                    __syncwarp();
                    st += p.n_load;
                    if (st >= p.n_stages) { st -= p.n_stages; phase ^= 1; }
                }
            }
        }
    } else if (warp == 4 || (warp >= 6 && warp <= 8)) {
        // ------------------------------ MMA issuers (warp 4 also loads the W slice) ------------------------------
        // The whole warp runs the loop with warp-uniform values and one elected lane issues (mma_bf16_elect).
        {
            const int iss = warp == 4 ? 0 : warp - 5;                 // warps 4, 6, 7, 8 -> issuers 0..3
            if (iss == 0 && lane == 0) {
                tc::mbar_expect_tx(w_full, (uint32_t)(p.k_blocks * W_KB));
                for (int kb = 0; kb < p.k_blocks; ++kb) tc::tma_load_2d(w_s + (size_t)kb * W_KB, &tm_w, w_full, kb * BK, j0);
            }
            __syncwarp();
            bool ok = __all_sync(0xffffffffu, tc::mbar_wait(w_full, 0, abort_flag, p.err, tc::ERR_WAIT_FULL));
            const uint32_t idesc = tc::instr_desc_bf16(p.rows_per_warp == 16 ? 64 : 128, UNITS, false, false);
            // descriptors differ from the first one only in the start-address field (16-byte units): one add per MMA
            const uint64_t desc_a0 = tc::smem_desc(tc::smem_u32(a_s) + (uint32_t)(iss * p.tile_stride), 16, 1024);
            const uint64_t desc_b0 = tc::smem_desc(tc::smem_u32(w_s) + (uint32_t)(iss * W_KB), 16, 1024);
            const uint32_t a_stage = (uint32_t)(N_ISS * p.tile_stride) >> 4, b_stage = (uint32_t)(N_ISS * W_KB) >> 4;
            const uint32_t d_tmem = tmem_base + iss * UNITS;
            int st = 0;
            uint32_t phase = 0, a_off = 0;
            for (int s = 1; s <= p.T && ok; ++s) {
                uint32_t b_off = 0;
                for (int kb = 0; kb < p.k_blocks; kb += N_ISS) {       // this issuer's k-block of the stage: kb + iss
                    // every lane waits; the vote reconverges the warp (the lanes leave the wait at different times)
                    ok = __all_sync(0xffffffffu, tc::mbar_wait(&full[st], phase, abort_flag, p.err, tc::ERR_WAIT_FULL));
                    if (!ok) break;
                    tc::tc_fence_after_sync();
                    const uint64_t da = desc_a0 + a_off, db = desc_b0 + b_off;
                    const uint32_t acc = kb != 0;
#pragma unroll
                    for (int kk = 0; kk < BK / 16; ++kk) tc::mma_bf16_elect(d_tmem, da + 2 * kk, db + 2 * kk, idesc, acc | (kk != 0));
                    tc::mma_commit_elect(&empty[st]);
                    a_off += a_stage; b_off += b_stage;
                    if (++st == p.n_stages) { st = 0; phase ^= 1; a_off = 0; }
                }
                if (ok) tc::mma_commit_elect(tmem_full);
            }
        }
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    if (warp == 4) { tc::tc_fence_after_sync(); tc::tmem_dealloc(tmem_base, TMEM_COLS); }
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

relay_status_t run_steps_tc(const GradDims &d, const GradPlan &pl, char *ws, const void *w_hh, const float *c0, const float *dh_all,
                            const float *dc_final, float *dh0, float *dc0, cudaStream_t st)
{
    unsigned int *counter = (unsigned int *)(ws + pl.counters);
    RELAY_CUDA(cudaMemsetAsync(counter, 0, 1024, st));
    const int n_blocks = (int)(d.H / UNITS);
    int dev = 0, sms = 148;
    RELAY_CUDA(cudaGetDevice(&dev));
    RELAY_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    int groups = std::max(1, std::min({sms / n_blocks, (int)(d.B / 8), 8}));
    const int rows_per_group = (int)((d.B + groups - 1) / groups);
    groups = (int)((d.B + rows_per_group - 1) / rows_per_group);
    CUtensorMap tm_w, tm_dz;
    RELAY_TRY(make_tmap_2d_bf16(&tm_w, w_hh, (uint64_t)(4 * d.H), (uint64_t)d.H, (uint64_t)(4 * d.H), BK, UNITS));
    RELAY_TRY(make_tmap_2d_bf16(&tm_dz, ws + pl.dz, (uint64_t)(4 * d.H), (uint64_t)(d.T * d.B), (uint64_t)(4 * d.H), BK,
                                (uint32_t)rows_per_group));
    GradParams p{};
    p.T = (int)d.T; p.B = (int)d.B; p.H = (int)d.H; p.n_blocks = n_blocks; p.k_blocks = (int)(4 * d.H / BK);
    p.rows_per_group = rows_per_group;
    p.rows_per_warp = rows_per_group <= 64 ? 16 : 32;
    p.n_epi = (rows_per_group + p.rows_per_warp - 1) / p.rows_per_warp;
    p.gates = (const float *)(ws + pl.gates); p.c_all = (const float *)(ws + pl.c_all); p.c0 = c0;
    p.dh_all = dh_all; p.dc_final = dc_final; p.dz = (__nv_bfloat16 *)(ws + pl.dz); p.dh0 = dh0; p.dc0 = dc0;
    p.counter = counter;
    p.err = device_error_word();
    if (!p.err) return fail(RELAY_ERR_CUDA, "no device error word");
    p.tile_stride = (int)align_up((size_t)rows_per_group * 128, 1024);
    p.n_stages = std::min(MAX_STAGES, RING_BYTES / (N_ISS * p.tile_stride));
    // two loaders when the stages of a step split evenly between them (each then walks the ring in steps of two)
    p.n_load = ((p.k_blocks / N_ISS) % 2 == 0 && p.n_stages % 2 == 0) ? 2 : 1;
    // what follows the ring is at least one A tile long, so the rows an MMA reads past the last stage stay inside the allocation
    const size_t smem = 1024 + (size_t)RING_BYTES + std::max<size_t>((size_t)p.k_blocks * W_KB, A_TILE) + 1024;
    RELAY_CUDA(cudaFuncSetAttribute(lstm_grad_persistent_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    void *args[] = {(void *)&tm_w, (void *)&tm_dz, (void *)&p};
    RELAY_CUDA(cudaLaunchCooperativeKernel((const void *)lstm_grad_persistent_kernel, dim3(n_blocks * groups), dim3(NUM_THREADS), args, smem, st));
    count_launch();
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
        RELAY_TRY(launch_gemm(g, st));
        RELAY_CUDA(launch_pdl(lstm_cell_sweep_kernel, dim3((unsigned)((bh + 255) / 256)), dim3(256), 0, st, gates, (const float *)c0->data,
                              c_all, d.T, d.B, d.H));
        RELAY_TRY(check_launch("lstm_cell_sweep"));
    }

    // (2) the dependent steps, last to first
    const float *dcf = dc_final ? (const float *)dc_final->data : nullptr;
    float *dh0p = dh0 ? (float *)dh0->data : nullptr, *dc0p = dc0 ? (float *)dc0->data : nullptr;
    if (pl.tc) RELAY_TRY(run_steps_tc(d, pl, base, w_hh->data, (const float *)c0->data, (const float *)dh_all->data, dcf, dh0p, dc0p, st));
    else RELAY_TRY(run_steps_any(d, pl, base, w_hh->data, (const float *)c0->data, (const float *)dh_all->data, dcf, dh0p, dc0p, st));

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
