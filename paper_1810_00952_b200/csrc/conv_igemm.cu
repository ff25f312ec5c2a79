// General conv2d tier (SIMT): every stride / padding / window size, both float types.  The three
// contractions of a conv2d group are run as implicit GEMMs on 64 x 64 output tiles, k-blocks of 16, with the
// operand gathers done by the tile loaders (no im2col buffer; smaller tiles for small grids and few channels):
//
//   forward          Y[(n,p,q), o]   = sum over (c,r,s) of  X[n, c, p*st-pad+r, q*st-pad+s] * W[o, (c,r,s)]
//   input gradient   dX[(n,i,j), c]  = sum over (o,r,s) of  dZ[n, o, (i+pad-r)/st, (j+pad-s)/st] * W[o, c, r, s]
//   weight gradient  dW[o, (c,r,s)]  = sum over (n,p,q) of  dZ[n, o, p, q] * X[n, c, p*st-pad+r, q*st-pad+s]
//
// Index decompositions are hoisted: a loader thread keeps the part of the index that does not change from
// k-block to k-block in registers.  The loads of k-block i+1 are issued before the arithmetic of k-block i.
// The weight gradient, whose output is small and whose sum is long, is split along k over the grid; the
// slices' fp32 partials are added in slice order by a second kernel (no atomics: reruns are bit-identical).
// Accumulation as in the SIMT dense kernel (simt_acc.cuh).
#include <algorithm>
#include <climits>
#include <type_traits>

#include "conv.h"
#include "ewise_kernels.cuh"
#include "simt_acc.cuh"

namespace relay {

namespace {

constexpr int BK = 16;       // k-block depth; a block tile is (16 * TMR) x (16 * TN), a thread tile TMR x TN
enum { FWD = 0, DX = 1, DW = 2 };

template <typename T> __device__ __forceinline__ float ldf(const T *p, int64_t i)
{
    if constexpr (sizeof(T) == 2) return __bfloat162float(p[i]);
    else return p[i];
}
template <typename T> __device__ __forceinline__ void stf(T *p, int64_t i, float v)
{
    if constexpr (sizeof(T) == 2) p[i] = __float2bfloat16_rn(v);
    else p[i] = v;
}

struct IgemmArgs {
    int Nb, C, H, W, O, R, S, P, Q, stride, pad;
    int64_t Mg, Ng, Kg;        // GEMM extents of this mode
    int k_per_slice;           // DW: k range of one grid.z slice (multiple of BK); else Kg rounded up
    const void *a, *b;         // FWD: x, w;  DX: dz, w;  DW: dz, x
    void *out;                 // FWD: y;  DX: dx;  DW: fp32 partials [slice][O][C*R*S]
    const void *bias;
    int bias_bf16, act;
};

// (c, r, s) of a flattened window index moved on by `step`: carries, a division only when a carry happens
__device__ __forceinline__ void advance(int &c, int &r, int &s, int step, int R, int S)
{
    s += step;
    if (s >= S) {
        const int q = s / S;
        s -= q * S;
        r += q;
        if (r >= R) {
            const int q2 = r / R;
            r -= q2 * R;
            c += q2;
        }
    }
}

// TMR x TN outputs per thread: 4 x 4 in general; FWD and DX also come with 2 or 1 rows (more blocks when the grid
// would leave SMs idle) and with 2 or 1 columns (few output channels: less arithmetic on padding)
template <typename T, int MODE, bool FAST, bool STRIDE1, int TMR, int TN>
__global__ void __launch_bounds__(256, 2) conv_igemm_kernel(const IgemmArgs g)
{
    static_assert(MODE != DW || (TMR == 4 && TN == 4), "the weight gradient uses the 64 x 64 tile");
    constexpr int BM = 16 * TMR, BN = 16 * TN;
    constexpr int LDA = TMR, LDB = TN;                  // loader slots per thread: BM * BK / 256, BN * BK / 256
    constexpr int KSTEP = 256 / BM;                     // FWD, DX: k distance between a thread's A slots
    // the operand whose values per thread are the same across a half-warp is read as one vector
    __shared__ __align__(16) float As[BK][BM + 4];
    __shared__ __align__(16) float Bs[BK][BN + 4];
    const T *A = (const T *)g.a;
    const T *B = (const T *)g.b;
    const int tid = threadIdx.x;
    const int64_t m0 = (int64_t)blockIdx.x * BM, n0 = (int64_t)blockIdx.y * BN;
    const int64_t k_begin = (int64_t)blockIdx.z * g.k_per_slice;
    const int64_t k_end = min(g.Kg, k_begin + (int64_t)g.k_per_slice);
    const int RS = g.R * g.S, PQ = g.P * g.Q, HW = g.H * g.W;
    const int stride = STRIDE1 ? 1 : g.stride;
    constexpr bool WIDE = sizeof(T) == 4;
    using Acc = typename std::conditional<WIDE, PairSum, float>::type;
    Acc acc[TMR][TN] = {};
    // output rows / columns of this thread: lanes run along the axis that is contiguous in memory
    // (pixels for FWD and DX, the flattened (c,r,s) index for DW)
    const int lane_m = MODE == DW ? tid / 16 : tid % 16, lane_n = MODE == DW ? tid % 16 : tid / 16;

    // ---- loader state that does not depend on the k-block ---------------------------------------------
    // FWD, DX: A slot i holds (row mm = tid % BM, k-offset kk = tid / BM + KSTEP i): the row's pixel is decomposed once.
    // DW:      A and B slot i hold (k-offset kk = tid % 16, row / column tid / 16 + 16 i): k is decomposed once per
    //          k-block, the B column's (c,r,s) once per slot.
    int a_img = 0, a_y = 0, a_x = 0;          // FWD: (n, p*st-pad, q*st-pad);  DX: (n, i+pad, j+pad)
    bool a_row_ok = false;
    if (MODE != DW) {
        const int64_t m = m0 + tid % BM;
        a_row_ok = m < g.Mg;
        if (a_row_ok) {
            const int per = MODE == FWD ? PQ : HW, wdt = MODE == FWD ? g.Q : g.W;
            a_img = (int)(m / per);
            const int rem = (int)(m % per);
            a_y = rem / wdt; a_x = rem % wdt;
            if (MODE == FWD) { a_y = a_y * stride - g.pad; a_x = a_x * stride - g.pad; }
            else { a_y += g.pad; a_x += g.pad; }
        }
    }
    int64_t b_off[LDB];                         // DW: (c*H + r - pad)*W + s - pad of the slot's column
    int b_dy[LDB], b_dx[LDB];                   // DW: r - pad, s - pad (INT_MIN marks a column out of range)
    if (MODE == DW) {
#pragma unroll
        for (int i = 0; i < LDB; ++i) {
            const int64_t n = n0 + tid / BK + 16 * i;
            b_dy[i] = INT_MIN; b_dx[i] = 0; b_off[i] = 0;
            if (n < g.Ng) {
                const int c = (int)(n / RS), rs = (int)(n % RS);
                b_dy[i] = rs / g.S - g.pad; b_dx[i] = rs % g.S - g.pad;
                b_off[i] = ((int64_t)c * g.H + b_dy[i]) * g.W + b_dx[i];
            }
        }
    }

    float ra[LDA], rb[LDB];
    auto load_tiles = [&](int64_t k0) {
        if (MODE == FWD) {
            // slot 0's k is decomposed by division, the other slots follow by carries
            const int64_t kf = k0 + tid / BM;
            int c = (int)(kf / RS), r, sx;
            { const int rs = (int)(kf % RS); r = rs / g.S; sx = rs % g.S; }
#pragma unroll
            for (int i = 0; i < LDA; ++i) {
                float v = 0.0f;
                if (a_row_ok && kf + KSTEP * i < k_end) {
                    const int yy = a_y + r, xx = a_x + sx;
                    if (yy >= 0 && yy < g.H && xx >= 0 && xx < g.W) v = ldf(A, (((int64_t)a_img * g.C + c) * g.H + yy) * g.W + xx);
                }
                ra[i] = v;
                advance(c, r, sx, KSTEP, g.R, g.S);
            }
            const int64_t k = k0 + tid % BK;
#pragma unroll
            for (int i = 0; i < LDB; ++i) {
                const int64_t n = n0 + tid / BK + 16 * i;
                rb[i] = (n < g.Ng && k < k_end) ? ldf(B, n * g.Kg + k) : 0.0f;
            }
        } else if (MODE == DX) {
            const int64_t kf = k0 + tid / BM;
            int o = (int)(kf / RS), r, sx;
            { const int rs = (int)(kf % RS); r = rs / g.S; sx = rs % g.S; }
#pragma unroll
            for (int i = 0; i < LDA; ++i) {
                float v = 0.0f;
                if (a_row_ok && kf + KSTEP * i < k_end) {
                    const int yn = a_y - r, xn = a_x - sx;
                    if (STRIDE1) {
                        if (yn >= 0 && xn >= 0 && yn < g.P && xn < g.Q) v = ldf(A, (((int64_t)a_img * g.O + o) * g.P + yn) * g.Q + xn);
                    } else if (yn >= 0 && xn >= 0 && yn % stride == 0 && xn % stride == 0) {
                        const int p = yn / stride, q = xn / stride;
                        if (p < g.P && q < g.Q) v = ldf(A, (((int64_t)a_img * g.O + o) * g.P + p) * g.Q + q);
                    }
                }
                ra[i] = v;
                advance(o, r, sx, KSTEP, g.R, g.S);
            }
            const int64_t k = k0 + tid % BK;
            const int ob = (int)(k / RS), rsb = (int)(k % RS);
#pragma unroll
            for (int i = 0; i < LDB; ++i) {
                const int64_t c = n0 + tid / BK + 16 * i;
                rb[i] = (c < g.Ng && k < k_end) ? ldf(B, ((int64_t)ob * g.C + c) * RS + rsb) : 0.0f;
            }
        } else {
            const int64_t k = k0 + tid % BK;
            const bool k_ok = k < k_end;
            int img = 0, p = 0, q = 0;
            if (k_ok) {
                img = (int)(k / PQ);
                const int pq = (int)(k % PQ);
                p = pq / g.Q; q = pq % g.Q;
            }
#pragma unroll
            for (int i = 0; i < LDA; ++i) {
                const int64_t o = m0 + tid / BK + 16 * i;
                ra[i] = (k_ok && o < g.Mg) ? ldf(A, ((int64_t)img * g.O + o) * PQ + (int64_t)p * g.Q + q) : 0.0f;
            }
            const int y0 = p * stride, x0 = q * stride;
            const int64_t base = (int64_t)img * g.C * HW + (int64_t)y0 * g.W + x0;
#pragma unroll
            for (int i = 0; i < LDB; ++i) {
                float v = 0.0f;
                if (k_ok && b_dy[i] != INT_MIN) {
                    const int yy = y0 + b_dy[i], xx = x0 + b_dx[i];
                    if (yy >= 0 && yy < g.H && xx >= 0 && xx < g.W) v = ldf(B, base + b_off[i]);
                }
                rb[i] = v;
            }
        }
    };

    if (k_begin < k_end) load_tiles(k_begin);
    for (int64_t k0 = k_begin; k0 < k_end; k0 += BK) {
#pragma unroll
        for (int i = 0; i < LDA; ++i) {
            if (MODE == DW) As[tid % BK][tid / BK + 16 * i] = ra[i];
            else As[tid / BM + KSTEP * i][tid % BM] = ra[i];
        }
#pragma unroll
        for (int i = 0; i < LDB; ++i) Bs[tid % BK][tid / BK + 16 * i] = rb[i];
        __syncthreads();
        if (k0 + BK < k_end) load_tiles(k0 + BK);
        float part[TMR][TN] = {};
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float av[TMR], bv[TN];
            if (MODE == DW) {
                const float4 a4 = *reinterpret_cast<const float4 *>(&As[kk][4 * lane_m]);
                av[0] = a4.x; av[1] = a4.y; av[2] = a4.z; av[3] = a4.w;
#pragma unroll
                for (int j = 0; j < TN; ++j) bv[j] = Bs[kk][lane_n + 16 * j];
            } else {
#pragma unroll
                for (int i = 0; i < TMR; ++i) av[i] = As[kk][lane_m + 16 * i];
                if constexpr (TN == 4) {
                    const float4 b4 = *reinterpret_cast<const float4 *>(&Bs[kk][4 * lane_n]);
                    bv[0] = b4.x; bv[1] = b4.y; bv[2] = b4.z; bv[3] = b4.w;
                } else if constexpr (TN == 2) {
                    const float2 b2 = *reinterpret_cast<const float2 *>(&Bs[kk][2 * lane_n]);
                    bv[0] = b2.x; bv[1] = b2.y;
                } else {
                    bv[0] = Bs[kk][lane_n];
                }
            }
#pragma unroll
            for (int i = 0; i < TMR; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) {
                    if constexpr (WIDE) part[i][j] = fmaf(av[i], bv[j], part[i][j]);
                    else acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
                }
        }
        if constexpr (WIDE) {
#pragma unroll
            for (int i = 0; i < TMR; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) acc[i][j].add(part[i][j]);
        }
        __syncthreads();
    }

    // ---- store ---------------------------------------------------------------------------------------------
#pragma unroll
    for (int i = 0; i < TMR; ++i) {
        const int64_t m = m0 + (MODE == DW ? 4 * lane_m + i : lane_m + 16 * i);
        if (m >= g.Mg) continue;
        int64_t row_base = 0;      // FWD: offset of y[n, 0, p, q];  DX: offset of dx[n, 0, i, j]
        if (MODE == FWD) row_base = (m / PQ) * (int64_t)g.O * PQ + m % PQ;
        if (MODE == DX) row_base = (m / HW) * (int64_t)g.C * HW + m % HW;
#pragma unroll
        for (int j = 0; j < TN; ++j) {
            const int64_t n = n0 + (MODE == DW ? lane_n + 16 * j : TN * lane_n + j);
            if (n >= g.Ng) continue;
            float bv = 0.0f;
            if (MODE == FWD && g.bias) bv = g.bias_bf16 ? __bfloat162float(((const __nv_bfloat16 *)g.bias)[n]) : ((const float *)g.bias)[n];
            float z;
            if constexpr (WIDE) z = (float)(acc[i][j].value() + (double)bv);
            else z = acc[i][j] + bv;
            if (MODE == FWD) stf((T *)g.out, row_base + n * PQ, act_fwd<FAST>(z, g.act));
            else if (MODE == DX) stf((T *)g.out, row_base + n * HW, z);
            else ((float *)g.out)[((int64_t)blockIdx.z * g.Mg + m) * g.Ng + n] = z;
        }
    }
}

// dw[e] = sum over slices of part[slice][e], in a fixed order: one warp per element, lane l adds the slices
// l, l + 32, ... (independent loads, one round trip), then the lanes are combined by a fixed shuffle tree
template <typename T>
__global__ void __launch_bounds__(256) conv_dw_reduce_kernel(const float *__restrict__ part, int n_slices, int64_t total, T *__restrict__ dw)
{
    const int lane = threadIdx.x & 31;
    const int64_t e = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (e >= total) return;
    PairSum s;
    for (int z = lane; z < n_slices; z += 32) s.add(part[(int64_t)z * total + e]);
#pragma unroll
    for (int k = 16; k > 0; k >>= 1) {
        const float oh = __shfl_down_sync(0xffffffffu, s.hi, k), ol = __shfl_down_sync(0xffffffffu, s.lo, k);
        s.add(oh);
        s.lo += ol;
    }
    if (lane == 0) stf(dw, e, (float)s.value());
}

IgemmArgs base_args(const ConvDims &d)
{
    IgemmArgs g{};
    g.Nb = (int)d.Nb; g.C = (int)d.C; g.H = (int)d.H; g.W = (int)d.W; g.O = (int)d.O; g.R = (int)d.R; g.S = (int)d.S;
    g.P = (int)d.P; g.Q = (int)d.Q; g.stride = d.stride; g.pad = d.pad;
    return g;
}

bool fits_int(const ConvDims &d)
{
    const int64_t lim = (1ll << 31) - 1;
    return d.Nb <= lim && d.C <= lim && d.O <= lim && d.H * d.W <= lim && d.P * d.Q <= lim && d.C * d.R * d.S <= lim &&
           d.O * d.R * d.S <= lim && d.Nb * d.P * d.Q <= (1ll << 40) && d.Nb * d.H * d.W <= (1ll << 40);
}

relay_status_t grid_of(const IgemmArgs &g, int bm, int bn, int slices, dim3 *grid)
{
    const int64_t gx = (g.Mg + bm - 1) / bm, gy = (g.Ng + bn - 1) / bn;
    if (gx > 2147483647ll || gy > 65535 || slices > 65535) return fail(RELAY_ERR_UNSUPPORTED, "conv2d: extent exceeds the grid limit");
    *grid = dim3((unsigned)gx, (unsigned)gy, (unsigned)slices);
    return RELAY_OK;
}

// slices of the weight gradient's sum: enough blocks for two per SM, at least four k-blocks per slice
int dw_slices(const ConvDims &d)
{
    const int64_t tiles = ((d.O + 63) / 64) * ((d.C * d.R * d.S + 63) / 64);
    const int64_t Kg = d.Nb * d.P * d.Q;
    const int64_t by_work = std::max<int64_t>(1, Kg / (4 * BK));
    return (int)std::max<int64_t>(1, std::min<int64_t>(std::min<int64_t>(by_work, 4096), (2 * 148 + tiles - 1) / tiles));
}

template <int MODE, int TMR, int TN>
void launch_tile(const ConvDims &d, const IgemmArgs &g, dim3 grid, cudaStream_t st)
{
    const bool bf = d.dt == RELAY_BF16, s1 = d.stride == 1;
    if (bf && s1) conv_igemm_kernel<__nv_bfloat16, MODE, true, true, TMR, TN><<<grid, 256, 0, st>>>(g);
    else if (bf) conv_igemm_kernel<__nv_bfloat16, MODE, true, false, TMR, TN><<<grid, 256, 0, st>>>(g);
    else if (s1) conv_igemm_kernel<float, MODE, false, true, TMR, TN><<<grid, 256, 0, st>>>(g);
    else conv_igemm_kernel<float, MODE, false, false, TMR, TN><<<grid, 256, 0, st>>>(g);
}

// FWD and DX: the tile is as wide as the output channels need (16, 32 or 64 columns) and as tall (64, 32 or 16 rows)
// as still gives every SM a block: with few warps on an SM a block's time goes to waiting for its own
// shared-memory reads, so while SMs are idle more and lighter blocks finish sooner
template <int MODE, int TN>
relay_status_t launch_rows(const ConvDims &d, const IgemmArgs &g, cudaStream_t st)
{
    const int64_t cols = (g.Ng + 16 * TN - 1) / (16 * TN);
    auto blocks = [&](int bm) { return ((g.Mg + bm - 1) / bm) * cols; };
    dim3 grid;
    if (blocks(64) >= 148) { RELAY_TRY(grid_of(g, 64, 16 * TN, 1, &grid)); launch_tile<MODE, 4, TN>(d, g, grid, st); }
    else if (blocks(32) >= 148) { RELAY_TRY(grid_of(g, 32, 16 * TN, 1, &grid)); launch_tile<MODE, 2, TN>(d, g, grid, st); }
    else { RELAY_TRY(grid_of(g, 16, 16 * TN, 1, &grid)); launch_tile<MODE, 1, TN>(d, g, grid, st); }
    return RELAY_OK;
}

template <int MODE>
relay_status_t launch_rows_cols(const ConvDims &d, const IgemmArgs &g, cudaStream_t st)
{
    if (g.Ng <= 16) return launch_rows<MODE, 1>(d, g, st);
    if (g.Ng <= 32) return launch_rows<MODE, 2>(d, g, st);
    return launch_rows<MODE, 4>(d, g, st);
}

}  // namespace

size_t conv_dw_partial_bytes(const ConvDims &d)
{
    return align_up((size_t)dw_slices(d) * (size_t)(d.O * d.C * d.R * d.S) * sizeof(float), 256);
}

relay_status_t launch_conv_fwd_direct(const ConvDims &d, const void *x, const void *w, const void *b, int32_t b_dt, int act,
                                      void *y, cudaStream_t st)
{
    if (d.Nb * d.O * d.P * d.Q == 0) return RELAY_OK;
    if (!fits_int(d)) return fail(RELAY_ERR_UNSUPPORTED, "conv2d: extents beyond the general tier's index range");
    IgemmArgs g = base_args(d);
    g.Mg = d.Nb * d.P * d.Q; g.Ng = d.O; g.Kg = d.C * d.R * d.S;
    g.k_per_slice = (int)((g.Kg + BK - 1) / BK * BK);
    g.a = x; g.b = w; g.out = y; g.bias = b; g.bias_bf16 = b_dt == RELAY_BF16; g.act = act;
    RELAY_TRY(launch_rows_cols<FWD>(d, g, st));
    return check_launch("conv_igemm_fwd");
}

relay_status_t launch_conv_dx_direct(const ConvDims &d, const void *dz, const void *w, void *dx, cudaStream_t st)
{
    if (d.Nb * d.C * d.H * d.W == 0) return RELAY_OK;
    if (!fits_int(d)) return fail(RELAY_ERR_UNSUPPORTED, "conv2d: extents beyond the general tier's index range");
    IgemmArgs g = base_args(d);
    g.Mg = d.Nb * d.H * d.W; g.Ng = d.C; g.Kg = d.O * d.R * d.S;
    g.k_per_slice = (int)((g.Kg + BK - 1) / BK * BK);
    g.a = dz; g.b = w; g.out = dx;
    RELAY_TRY(launch_rows_cols<DX>(d, g, st));
    return check_launch("conv_igemm_dx");
}

relay_status_t launch_conv_dw_direct(const ConvDims &d, const void *dz, const void *x, void *dw, float *partials, cudaStream_t st)
{
    const int64_t total = d.O * d.C * d.R * d.S;
    if (total == 0) return RELAY_OK;
    if (!fits_int(d)) return fail(RELAY_ERR_UNSUPPORTED, "conv2d: extents beyond the general tier's index range");
    IgemmArgs g = base_args(d);
    g.Mg = d.O; g.Ng = d.C * d.R * d.S; g.Kg = d.Nb * d.P * d.Q;
    const int want = dw_slices(d);
    g.k_per_slice = (int)(((g.Kg + want - 1) / want + BK - 1) / BK * BK);
    const int slices = g.Kg == 0 ? 1 : (int)((g.Kg + g.k_per_slice - 1) / g.k_per_slice);     // <= want
    g.a = dz; g.b = x; g.out = partials;
    dim3 grid;
    RELAY_TRY(grid_of(g, 64, 64, slices, &grid));
    launch_tile<DW, 4, 4>(d, g, grid, st);
    RELAY_TRY(check_launch("conv_igemm_dw"));
    const unsigned rb = (unsigned)((total + 7) / 8);
    if (d.dt == RELAY_BF16) conv_dw_reduce_kernel<<<rb, 256, 0, st>>>(partials, slices, total, (__nv_bfloat16 *)dw);
    else conv_dw_reduce_kernel<<<rb, 256, 0, st>>>(partials, slices, total, (float *)dw);
    return check_launch("conv_dw_reduce");
}

}  // namespace relay
