// Memory-bound groups: fused broadcast-elementwise (relay_fused_ewise) and fused
// elementwise + reduce (relay_fused_reduce).
//
// Two tiers of kernels, both on the GPU:
//   * pre-compiled bodies over a collapsed 2-D view [rows, cols]: 128-bit loads/stores, operands
//     that are broadcast down the rows kept in registers, several rows in flight per thread,
//     column sums as per-thread accumulators -> shared-memory combine -> per-slice partials ->
//     a second fixed-order pass (deterministic, no float atomics);
//   * a generic evaluator that interprets any well-typed program for any broadcast pattern and
//     any axes mask (one element per thread; one warp or one block per reduced result).
#include <algorithm>
#include <cstring>
#include <string>

#include "ewise_host.h"
#include "ewise_kernels.cuh"
#include "ewise_prog.h"

namespace relay {

// =================================================================================================
// kernels
// =================================================================================================
constexpr int kTX = 32, kTY = 8;

// CL > 1: the kernel is launched in clusters of CL blocks along y, the row slices of one column strip.  The slices'
// partial column sums then never leave the chip: every block leaves its partials in its own shared memory, and after a
// cluster barrier block r of the cluster adds up, in slice order, the CL partials of its share of the strip's columns
// through distributed shared memory and writes the final sums (A.final[k], times A.scale[k]).  No second launch and no
// scratch memory; the order is fixed, so reruns are bit-identical.
constexpr int kColsumCluster = 8;

// TX lanes of 16 bytes side by side in a row (the block covers TX * V columns), 256 / TX rows per pass, UN passes of loads
// in flight per thread.
template <typename Body, typename T, bool FAST, int CL = 1, int TX = 32, int UN = 4>
__global__ void __launch_bounds__(256, Body::NIN >= 4 ? 2 : 3) ewise2d_kernel(const Args2D<Body::NIN, Body::NOUT> A)
{
    constexpr int V = VecN<T>::N, NIN = Body::NIN, NOUT = Body::NOUT;
    constexpr int kTX = TX, kTY = 256 / TX, kUnroll = UN;
    const int tx = threadIdx.x, ty = threadIdx.y;
    const int64_t col0 = ((int64_t)blockIdx.x * kTX + tx) * V;
    pdl_wait();
    const bool active = col0 < A.cols;

    float fixed[NIN][V];  // operands that do not change from row to row
#pragma unroll
    for (int i = 0; i < NIN; ++i) {
        if (Body::kind(i) == KIND_ROWVEC && active) {
            unpack(ld_stream((const T *)A.in[i] + col0), fixed[i]);
        } else if (Body::kind(i) == KIND_SCALAR) {
            float s;
            if constexpr (sizeof(T) == 2) s = __bfloat162float(*(const __nv_bfloat16 *)A.in[i]);
            else s = *(const float *)A.in[i];
#pragma unroll
            for (int v = 0; v < V; ++v) fixed[i][v] = s;
        } else {
#pragma unroll
            for (int v = 0; v < V; ++v) fixed[i][v] = 0.0f;
        }
    }

    float acc[NOUT][V];
#pragma unroll
    for (int k = 0; k < NOUT; ++k)
#pragma unroll
        for (int v = 0; v < V; ++v) acc[k][v] = 0.0f;

    const int64_t r0 = (int64_t)blockIdx.y * A.rows_per_slice;
    const int64_t r1 = min(A.rows, r0 + (int64_t)A.rows_per_slice);

    if (active) {
        for (int64_t r = r0 + ty; r < r1; r += kTY * kUnroll) {
            uint4 raw[kUnroll][NIN];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const int64_t rr = r + u * kTY;
#pragma unroll
                for (int i = 0; i < NIN; ++i)
                    if (Body::kind(i) == KIND_FULL && rr < r1) raw[u][i] = ld_stream((const T *)A.in[i] + rr * A.cols + col0);
            }
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const int64_t rr = r + u * kTY;
                if (rr >= r1) break;
                float vin[NIN][V];
#pragma unroll
                for (int i = 0; i < NIN; ++i) {
                    if (Body::kind(i) == KIND_FULL) unpack(raw[u][i], vin[i]);
                    else {
#pragma unroll
                        for (int v = 0; v < V; ++v) vin[i][v] = fixed[i][v];
                    }
                }
                float vout[NOUT][V];
#pragma unroll
                for (int v = 0; v < V; ++v) {
                    float ein[NIN], eout[NOUT];
#pragma unroll
                    for (int i = 0; i < NIN; ++i) ein[i] = vin[i][v];
                    Body::template apply<FAST>(ein, eout, A.aux);
#pragma unroll
                    for (int k = 0; k < NOUT; ++k) vout[k][v] = eout[k];
                }
#pragma unroll
                for (int k = 0; k < NOUT; ++k) {
                    if (Body::col_sum(k)) {
#pragma unroll
                        for (int v = 0; v < V; ++v) acc[k][v] += vout[k][v];
                    }
                    if (A.out[k] != nullptr) st_stream((T *)A.out[k] + rr * A.cols + col0, pack(vout[k]));
                }
            }
        }
    }

    // combine the kTY row-threads of each column, in ty order, and publish one partial per slice
    constexpr bool any_sum = []() { bool s = false; for (int k = 0; k < NOUT; ++k) s = s || Body::col_sum(k); return s; }();
    if constexpr (any_sum) {
        __shared__ float sm[kTY][kTX * V + 1];
        __shared__ float mine[CL > 1 ? NOUT : 1][kTX * V];      // CL > 1: this block's partials, read by its cluster
#pragma unroll
        for (int k = 0; k < NOUT; ++k) {
            if (!Body::col_sum(k)) continue;
#pragma unroll
            for (int v = 0; v < V; ++v) sm[ty][tx * V + v] = acc[k][v];
            __syncthreads();
            if (ty == 0) {
#pragma unroll
                for (int v = 0; v < V; ++v) {
                    float s = 0.0f;
#pragma unroll
                    for (int j = 0; j < kTY; ++j) s += sm[j][tx * V + v];
                    if constexpr (CL > 1) mine[k][tx * V + v] = active ? s : 0.0f;
                    else if (active && A.partial[k] != nullptr && relay_in_bounds(&A.partial[k][(int64_t)blockIdx.y * A.cols + col0 + v], 4))
                        A.partial[k][(int64_t)blockIdx.y * A.cols + col0 + v] = s;
                }
            }
            __syncthreads();
        }
        if constexpr (CL > 1) {
            asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
            uint32_t rank;
            asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
            constexpr int share = kTX * V / CL;                     // columns of the strip that this block finishes
            const int t = ty * kTX + tx;
            if (t < share) {
                const int c = (int)rank * share + t;
                const int64_t col = (int64_t)blockIdx.x * (kTX * V) + c;
#pragma unroll
                for (int k = 0; k < NOUT; ++k) {
                    if (!Body::col_sum(k) || A.final[k] == nullptr) continue;
                    float s = 0.0f;
#pragma unroll
                    for (int j = 0; j < CL; ++j) {
                        uint32_t remote;
                        float v;
                        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"((uint32_t)__cvta_generic_to_shared(&mine[k][c])), "r"(j));
                        asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
                        s += v;
                    }
                    if (col < A.cols && relay_in_bounds(&A.final[k][col], 4)) A.final[k][col] = s * A.scale[k];
                }
            }
            // no block may exit (and give up its shared memory) while another still reads it
            asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
        }
    }
}

// second pass of a column sum: thread (tx, ty) adds the partials of slices ty, ty+TY, ... of its column in
// slice order, then the TY row-threads are combined in ty order (fixed order, so reruns are bit-identical).
// grid.y indexes the summed result k: partials at partial + k * n_slices * cols, output out[k].
struct FinalizeOuts { float *out[RELAY_MAX_OUTPUTS]; float scale[RELAY_MAX_OUTPUTS]; };
template <int TY>
__global__ void __launch_bounds__(32 * TY) colsum_finalize_kernel(const float *__restrict__ partial, int n_slices, int64_t cols,
                                                                  const FinalizeOuts outs)
{
    __shared__ float sm[TY][33];
    const int tx = threadIdx.x, ty = threadIdx.y;
    pdl_wait();
    const int64_t c = (int64_t)blockIdx.x * 32 + tx;
    const float *p = partial + (size_t)blockIdx.y * n_slices * cols;
    float s = 0.0f;
    if (c < cols)
        for (int j = ty; j < n_slices; j += TY)
            if (relay_in_bounds(&p[(int64_t)j * cols + c], 4)) s += p[(int64_t)j * cols + c];
    sm[ty][tx] = s;
    __syncthreads();
    if (ty == 0 && c < cols) {
        float t = 0.0f;
#pragma unroll
        for (int j = 0; j < TY; ++j) t += sm[j][tx];
        if (relay_in_bounds(&outs.out[blockIdx.y][c], 4)) outs.out[blockIdx.y][c] = t * outs.scale[blockIdx.y];
    }
}

// reduction over the last axis of a [rows, cols] tensor: one warp per row, 128-bit loads.
// max / argmax work on whole vectors: the maximum of a 16-byte vector is taken with packed comparisons on the
// stored type (exact: comparing needs no arithmetic), and only a vector that beats the lane's running maximum is
// kept (its raw bits and its index); the first element that attains the maximum is looked up once, at the end.
// A lane meets its vectors in increasing column order and replaces only on strictly greater, so the kept vector
// is the lane's first one holding the maximum: ties go to the lowest index.
__device__ __forceinline__ float vec_max(const uint4 &r, const __nv_bfloat16 *)
{
    const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162 *>(&r.x), b = *reinterpret_cast<const __nv_bfloat162 *>(&r.y);
    const __nv_bfloat162 c = *reinterpret_cast<const __nv_bfloat162 *>(&r.z), d = *reinterpret_cast<const __nv_bfloat162 *>(&r.w);
    const __nv_bfloat162 m = __hmax2(__hmax2(a, b), __hmax2(c, d));
    return fmaxf(__low2float(m), __high2float(m));
}
__device__ __forceinline__ float vec_max(const uint4 &r, const float *)
{
    return fmaxf(fmaxf(__uint_as_float(r.x), __uint_as_float(r.y)), fmaxf(__uint_as_float(r.z), __uint_as_float(r.w)));
}

template <typename T, int RED>
__global__ void __launch_bounds__(256) rowreduce_kernel(const T *__restrict__ in, int64_t rows, int64_t cols, float scale,
                                                         void *__restrict__ out)
{
    constexpr int V = VecN<T>::N;
    constexpr int U = 8;                 // 16-byte loads in flight per lane
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= rows) return;
    const T *p = in + row * cols;
    const int64_t nvec = cols / V;
    float best = RED == RELAY_RED_SUM ? 0.0f : -INFINITY;
    uint4 best_raw = make_uint4(0, 0, 0, 0);
    int64_t best_vec = 0;
    for (int64_t j = lane; j < nvec; j += 32 * U) {
        uint4 raw[U];
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (j + u * 32 < nvec) raw[u] = ld_stream(p + (j + u * 32) * V);
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (j + u * 32 >= nvec) break;
            if (RED == RELAY_RED_SUM) {
                float f[V];
                unpack(raw[u], f);
                float s = 0.0f;
#pragma unroll
                for (int v = 0; v < V; ++v) s += f[v];
                best += s;
            } else {
                const float m = vec_max(raw[u], (const T *)nullptr);
                if (m > best) { best = m; best_raw = raw[u]; best_vec = j + u * 32; }
            }
        }
    }
    int64_t pos = 0;
    if (RED == RELAY_RED_ARGMAX) {
        float f[V];
        unpack(best_raw, f);
        int first = 0;
#pragma unroll
        for (int v = V - 1; v >= 0; --v)
            if (f[v] == best) first = v;
        pos = best_vec * V + first;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        float ob = __shfl_xor_sync(0xffffffffu, best, o);
        if (RED == RELAY_RED_SUM) best += ob;
        else if (RED == RELAY_RED_MAX) best = fmaxf(best, ob);
        else {
            int64_t op = __shfl_xor_sync(0xffffffffu, pos, o);
            if (ob > best || (ob == best && op < pos)) { best = ob; pos = op; }
        }
    }
    if (lane == 0) {
        if (RED == RELAY_RED_ARGMAX) { if (relay_in_bounds((int64_t *)out + row, 8)) ((int64_t *)out)[row] = pos; }
        else if (relay_in_bounds((float *)out + row, 4)) ((float *)out)[row] = best * scale;
    }
}

struct DevOutputs {
    int32_t n_out;
    int32_t value[RELAY_MAX_OUTPUTS];
    int32_t dtype[RELAY_MAX_OUTPUTS];
    void *ptr[RELAY_MAX_OUTPUTS];
};

__global__ void __launch_bounds__(256) ewise_generic_kernel(const DevProgram P, const DevOutputs O, int64_t total)
{
    Val vals[kDevMaxValues];
    int64_t idx[RELAY_MAX_RANK];
    for (int64_t lin = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; lin < total; lin += (int64_t)gridDim.x * blockDim.x) {
        unravel(lin, P.rank, P.shape, idx);
        eval_program(P, idx, vals);
        for (int k = 0; k < O.n_out; ++k) store_value(O.ptr[k], lin, O.dtype[k], vals[O.value[k]]);
    }
}

struct DevReduce {
    int32_t red_op, value, n_kept, n_red;
    int32_t kept_axis[RELAY_MAX_RANK], red_axis[RELAY_MAX_RANK];
    int64_t kept_elems, red_elems;
    void *out;
    float scale;
    int32_t group;  // threads that share one result: 32 (a warp) or 256 (the block)
    // n_split > 1 (group 256 only): the reduced extent of every result is cut into n_split runs of `chunk` elements, one block
    // each, which leave (value, position) in part_val / part_pos[result * n_split + run] for reduce_split_finish_kernel
    int32_t n_split;
    int64_t chunk;
    float *part_val;
    long long *part_pos;
};

__device__ __forceinline__ void combine(int red_op, float &best, int64_t &pos, float ob, int64_t op)
{
    if (red_op == RELAY_RED_SUM || red_op == RELAY_RED_MEAN) best += ob;
    else if (ob > best || (ob == best && op < pos)) { best = ob; pos = op; }
}

// one warp (group 32) or one block (group 256) per reduced result; fixed combine order
__global__ void __launch_bounds__(256) reduce_generic_kernel(const DevProgram P, const DevReduce R)
{
    __shared__ float sbest[8];
    __shared__ long long spos[8];
    Val vals[kDevMaxValues];
    int64_t idx[RELAY_MAX_RANK];
    const int lane_in_group = threadIdx.x % R.group;
    const int groups_per_block = blockDim.x / R.group;
    const int64_t unit = (int64_t)blockIdx.x * groups_per_block + threadIdx.x / R.group;
    const int64_t kept = R.n_split > 1 ? unit / R.n_split : unit;
    const int64_t run = R.n_split > 1 ? unit % R.n_split : 0;
    const int64_t j0 = run * R.chunk, j1 = R.n_split > 1 ? min(R.red_elems, j0 + R.chunk) : R.red_elems;
    const bool live = kept < R.kept_elems;
    const bool is_sum = R.red_op == RELAY_RED_SUM || R.red_op == RELAY_RED_MEAN;
    float best = is_sum ? 0.0f : -INFINITY;
    int64_t pos = 0;
    if (live) {
        int64_t rem = kept;
        for (int i = R.n_kept - 1; i >= 0; --i) {
            int ax = R.kept_axis[i];
            idx[ax] = rem % P.shape[ax];
            rem /= P.shape[ax];
        }
        for (int64_t j = j0 + lane_in_group; j < j1; j += R.group) {
            int64_t rj = j;
            for (int i = R.n_red - 1; i >= 0; --i) {
                int ax = R.red_axis[i];
                idx[ax] = rj % P.shape[ax];
                rj /= P.shape[ax];
            }
            eval_program(P, idx, vals);
            float v = vals[R.value].f;
            if (is_sum) best += v;
            else if (v > best) { best = v; pos = j; }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        float ob = __shfl_xor_sync(0xffffffffu, best, o);
        int64_t op = __shfl_xor_sync(0xffffffffu, pos, o);
        combine(R.red_op, best, pos, ob, op);
    }
    if (R.group > 32) {
        const int warp = threadIdx.x >> 5;
        if ((threadIdx.x & 31) == 0) { sbest[warp] = best; spos[warp] = pos; }
        __syncthreads();
        if (threadIdx.x == 0) {
            best = sbest[0]; pos = spos[0];
            for (int w = 1; w < (int)(blockDim.x >> 5); ++w) combine(R.red_op, best, pos, sbest[w], spos[w]);
        }
    }
    if (live && lane_in_group == 0) {
        if (R.n_split > 1) {
            if (relay_in_bounds(R.part_val + unit, 4)) R.part_val[unit] = best;
            if (relay_in_bounds(R.part_pos + unit, 8)) R.part_pos[unit] = pos;
        } else if (R.red_op == RELAY_RED_ARGMAX) { if (relay_in_bounds((int64_t *)R.out + kept, 8)) ((int64_t *)R.out)[kept] = pos; }
        else if (relay_in_bounds((float *)R.out + kept, 4)) ((float *)R.out)[kept] = best * R.scale;
    }
}

// second pass of a split reduction: one thread per result combines its runs in run order (sums in fp64: the runs are few)
__global__ void __launch_bounds__(128) reduce_split_finish_kernel(const DevReduce R)
{
    const int64_t kept = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (kept >= R.kept_elems) return;
    const bool is_sum = R.red_op == RELAY_RED_SUM || R.red_op == RELAY_RED_MEAN;
    double sum = 0.0;
    float best = -INFINITY;
    int64_t pos = 0;
    for (int s = 0; s < R.n_split; ++s) {
        const int64_t u = kept * R.n_split + s;
        if (!relay_in_bounds(R.part_val + u, 4) || !relay_in_bounds(R.part_pos + u, 8)) continue;
        const float v = R.part_val[u];
        if (is_sum) sum += (double)v;
        else if (v > best) { best = v; pos = R.part_pos[u]; }      // runs are in index order: the first maximum stays
    }
    if (R.red_op == RELAY_RED_ARGMAX) { if (relay_in_bounds((int64_t *)R.out + kept, 8)) ((int64_t *)R.out)[kept] = pos; }
    else if (relay_in_bounds((float *)R.out + kept, 4)) ((float *)R.out)[kept] = is_sum ? (float)(sum * (double)R.scale) : best;
}

// =================================================================================================
// host: canonical form of a program value, used to pick a pre-compiled body
// =================================================================================================
static bool commutative(int op)
{
    return op == RELAY_OP_ADD || op == RELAY_OP_MUL || op == RELAY_OP_MAX || op == RELAY_OP_MIN || op == RELAY_OP_EQ || op == RELAY_OP_NE;
}

// Expression tree of a value written as text, operands of commutative operators sorted, so
// that two programs that compute the same expression compare equal whatever their let order.
static std::string canon(const TypedProgram &tp, int v, int depth = 0)
{
    if (depth > 24) return "?";
    char buf[64];
    if (v < tp.n_in) { snprintf(buf, sizeof buf, "i%d:%d", v, tp.dtype[v]); return buf; }
    const relay_instr_t &in = tp.instr[v - tp.n_in];
    if (in.op == RELAY_OP_CONST) { snprintf(buf, sizeof buf, "k%.9g:%d", in.imm, in.dtype); return buf; }
    std::string args[3];
    int n = 0;
    if (in.a >= 0) args[n++] = canon(tp, in.a, depth + 1);
    if (in.b >= 0) args[n++] = canon(tp, in.b, depth + 1);
    if (in.c >= 0) args[n++] = canon(tp, in.c, depth + 1);
    if (commutative(in.op) && n == 2 && args[1] < args[0]) std::swap(args[0], args[1]);
    snprintf(buf, sizeof buf, "o%d:%d(", in.op, in.dtype);
    std::string s = buf;
    for (int i = 0; i < n; ++i) { if (i) s += ","; s += args[i]; if (s.size() > 4096) return "?"; }
    return s + ")";
}

// canonical text of the benchmark groups' values, produced from the same typed-program machinery
static void build(TypedProgram &tp, int n_in, int32_t in_dt)
{
    tp = TypedProgram();
    tp.n_in = n_in;
    for (int i = 0; i < n_in; ++i) tp.dtype[i] = in_dt;
}
static int emit(TypedProgram &tp, int op, int a, int b, int c, int dt, double imm = 0.0)
{
    relay_instr_t &in = tp.instr[tp.n_instr];
    in.op = op; in.a = a; in.b = b; in.c = c; in.dtype = dt; in.imm = imm; in.reserved = 0;
    tp.dtype[tp.n_in + tp.n_instr] = dt;
    tp.n_values = tp.n_in + tp.n_instr + 1;
    return tp.n_in + tp.n_instr++;
}

struct KnownFwd { std::string out; };
struct KnownGrad { std::string dx, da, db; };

static KnownFwd known_tanh_affine_fwd(int32_t st)
{
    TypedProgram p; build(p, 3, st);
    const int F = RELAY_F32;
    int x = emit(p, RELAY_OP_CAST, 0, -1, -1, F), a = emit(p, RELAY_OP_CAST, 1, -1, -1, F), b = emit(p, RELAY_OP_CAST, 2, -1, -1, F);
    int u = emit(p, RELAY_OP_ADD, emit(p, RELAY_OP_MUL, a, x, -1, F), b, -1, F);
    int o = emit(p, RELAY_OP_ADD, emit(p, RELAY_OP_TANH, u, -1, -1, F), x, -1, F);
    return KnownFwd{canon(p, emit(p, RELAY_OP_CAST, o, -1, -1, st))};
}
static KnownGrad known_tanh_affine_grad(int32_t st)
{
    TypedProgram p; build(p, 4, st);
    const int F = RELAY_F32;
    int d = emit(p, RELAY_OP_CAST, 0, -1, -1, F), x = emit(p, RELAY_OP_CAST, 1, -1, -1, F);
    int a = emit(p, RELAY_OP_CAST, 2, -1, -1, F), b = emit(p, RELAY_OP_CAST, 3, -1, -1, F);
    int t = emit(p, RELAY_OP_TANH, emit(p, RELAY_OP_ADD, emit(p, RELAY_OP_MUL, a, x, -1, F), b, -1, F), -1, -1, F);
    int one = emit(p, RELAY_OP_CONST, -1, -1, -1, F, 1.0);
    int s = emit(p, RELAY_OP_SUB, one, emit(p, RELAY_OP_SQ, t, -1, -1, F), -1, F);
    int g = emit(p, RELAY_OP_ADD, emit(p, RELAY_OP_MUL, a, s, -1, F), one, -1, F);
    int dx = emit(p, RELAY_OP_CAST, emit(p, RELAY_OP_MUL, d, g, -1, F), -1, -1, st);
    int ds = emit(p, RELAY_OP_MUL, d, s, -1, F);
    int da = emit(p, RELAY_OP_MUL, ds, x, -1, F);
    return KnownGrad{canon(p, dx), canon(p, da), canon(p, ds)};
}

// =================================================================================================
// host: launches
// =================================================================================================
static void fill_dev_program(const TypedProgram &tp, const relay_tensor_t *const *inputs, DevProgram *P)
{
    memset(P, 0, sizeof(*P));
    P->n_in = tp.n_in; P->n_instr = tp.n_instr; P->rank = tp.rank;
    for (int d = 0; d < tp.rank; ++d) P->shape[d] = tp.shape[d];
    for (int i = 0; i < tp.n_in; ++i) {
        int64_t stride = 1;
        for (int d = tp.rank - 1; d >= 0; --d) {
            P->in_stride[i][d] = tp.in_shape[i][d] == 1 ? 0 : stride;
            stride *= tp.in_shape[i][d];
        }
        P->in_ptr[i] = inputs[i]->data;
        P->in_dtype[i] = (int8_t)inputs[i]->dtype;
    }
    for (int j = 0; j < tp.n_instr; ++j) {
        P->op[j] = (int8_t)tp.instr[j].op; P->a[j] = (int8_t)tp.instr[j].a; P->b[j] = (int8_t)tp.instr[j].b;
        P->c[j] = (int8_t)tp.instr[j].c; P->dt[j] = (int8_t)tp.instr[j].dtype; P->imm[j] = tp.instr[j].imm;
    }
}

View2D view2d(const TypedProgram &tp)
{
    View2D v{};
    v.ok = false;
    if (tp.rank < 1 || tp.n_in < 1 || tp.total == 0) return v;
    v.cols = tp.shape[tp.rank - 1];
    v.rows = tp.total / v.cols;
    v.storage = tp.dtype[0];
    if (!is_float(v.storage)) return v;
    const int vec = v.storage == RELAY_BF16 ? 8 : 4;
    if (v.cols % vec != 0) return v;
    for (int i = 0; i < tp.n_in; ++i) {
        if (tp.dtype[i] != v.storage) return v;
        bool full = true, lead1 = true;
        for (int d = 0; d < tp.rank; ++d) {
            if (tp.in_shape[i][d] != tp.shape[d]) full = false;
            if (d < tp.rank - 1 && tp.in_shape[i][d] != 1) lead1 = false;
        }
        if (full) v.kind[i] = KIND_FULL;
        else if (lead1 && tp.in_shape[i][tp.rank - 1] == v.cols) v.kind[i] = KIND_ROWVEC;
        else if (lead1 && tp.in_shape[i][tp.rank - 1] == 1) v.kind[i] = KIND_SCALAR;
        else return v;
    }
    v.ok = true;
    return v;
}

template <typename Body>
static bool kinds_match(const View2D &v)
{
    for (int i = 0; i < Body::NIN; ++i)
        if (v.kind[i] != Body::kind(i)) return false;
    return true;
}

int colsum_slices(int64_t rows, int64_t cols, int32_t storage)
{
    const int vec = storage == RELAY_BF16 ? 8 : 4;
    const int64_t gx = (cols + (int64_t)kTX * vec - 1) / (kTX * vec);
    // about 8 blocks of 256 threads per SM in total, but at least 32 rows per slice
    int64_t want = std::max<int64_t>(1, (148 * 8) / gx);
    int64_t max_by_rows = std::max<int64_t>(1, rows / 32);
    return (int)std::max<int64_t>(1, std::min(want, max_by_rows));
}

template <typename Body>
relay_status_t launch_body2d(int32_t storage, const Args2D<Body::NIN, Body::NOUT> &A0, int n_slices, cudaStream_t st,
                             const char *what)
{
    Args2D<Body::NIN, Body::NOUT> A = A0;
    const int vec = storage == RELAY_BF16 ? 8 : 4;
    dim3 block(kTX, kTY);
    dim3 grid((unsigned)((A.cols + (int64_t)kTX * vec - 1) / (kTX * vec)), (unsigned)n_slices);
    A.rows_per_slice = (int)((A.rows + n_slices - 1) / n_slices);
    if (storage == RELAY_BF16) RELAY_CUDA(launch_pdl(ewise2d_kernel<Body, __nv_bfloat16, true>, grid, block, 0, st, A));
    else RELAY_CUDA(launch_pdl(ewise2d_kernel<Body, float, false>, grid, block, 0, st, A));
    return check_launch(what);
}

// Column sums finished inside the kernel by clusters of kColsumCluster row slices (no partials, no second launch):
// taken when that many slices per column strip give every SM a block.  A.final / A.scale name the results.  Used for the
// cfg2 gradient body (strips of 32 lanes: two streamed inputs and one streamed result keep enough bytes in flight); the plain
// column sum, with one streamed input, needs narrower strips and more blocks (launch_colsum_cluster below).
static bool cluster_sums(int64_t rows, int64_t cols, int32_t storage)
{
    const int vec = storage == RELAY_BF16 ? 8 : 4;
    const int64_t gx = (cols + (int64_t)kTX * vec - 1) / (kTX * vec);
    return gx * kColsumCluster >= 148 && rows >= 32 * kColsumCluster;
}
template <typename Body>
relay_status_t launch_body2d_cluster(int32_t storage, const Args2D<Body::NIN, Body::NOUT> &A0, cudaStream_t st, const char *what)
{
    Args2D<Body::NIN, Body::NOUT> A = A0;
    const int vec = storage == RELAY_BF16 ? 8 : 4;
    const dim3 block(kTX, kTY), cluster(1, kColsumCluster, 1);
    const dim3 grid((unsigned)((A.cols + (int64_t)kTX * vec - 1) / (kTX * vec)), kColsumCluster);
    A.rows_per_slice = (int)((A.rows + kColsumCluster - 1) / kColsumCluster);
    if (storage == RELAY_BF16) RELAY_CUDA(launch_pdl_cluster(ewise2d_kernel<Body, __nv_bfloat16, true, kColsumCluster>, grid, block, cluster, 0, st, A));
    else RELAY_CUDA(launch_pdl_cluster(ewise2d_kernel<Body, float, false, kColsumCluster>, grid, block, cluster, 0, st, A));
    return check_launch(what);
}

// Column sum of ONE streamed input finished in clusters: narrow strips (TX lanes of 16 bytes) so that CL slices per strip
// still give every SM several blocks, and UN row passes of loads in flight per thread.  Measured on 8192 x 8192 bf16
// (two-pass form with per-slice partials and a second launch: 29.1 us): strips of 16 lanes (256 bytes of a row), clusters
// of 8 slices, 4 passes in flight 24.5 us; 8 passes in flight 36.8 us; 8 lanes 29.1 us; 32 lanes 33 us and more; clusters
// of 4 slices 33.2 us (16 lanes) / 25.2 us (8 lanes).
constexpr int kColsumStripLanes = 16;
static bool colsum_in_clusters(int64_t rows, int64_t cols, int32_t storage)
{
    const int vec = storage == RELAY_BF16 ? 8 : 4;
    const int64_t gx = (cols + (int64_t)kColsumStripLanes * vec - 1) / (kColsumStripLanes * vec);
    return gx * kColsumCluster >= 148 * 2 && rows >= 1024;
}
template <typename Body, int CL, int TX, int UN>
relay_status_t launch_colsum_cluster(int32_t storage, const Args2D<Body::NIN, Body::NOUT> &A0, cudaStream_t st, const char *what)
{
    Args2D<Body::NIN, Body::NOUT> A = A0;
    const int vec = storage == RELAY_BF16 ? 8 : 4;
    const dim3 block(TX, 256 / TX), cluster(1, CL, 1);
    const dim3 grid((unsigned)((A.cols + (int64_t)TX * vec - 1) / (TX * vec)), CL);
    A.rows_per_slice = (int)((A.rows + CL - 1) / CL);
    if (storage == RELAY_BF16) RELAY_CUDA(launch_pdl_cluster(ewise2d_kernel<Body, __nv_bfloat16, true, CL, TX, UN>, grid, block, cluster, 0, st, A));
    else RELAY_CUDA(launch_pdl_cluster(ewise2d_kernel<Body, float, false, CL, TX, UN>, grid, block, cluster, 0, st, A));
    return check_launch(what);
}

relay_status_t launch_colsum_finalize_n(const float *partial, int n_slices, int64_t cols, const float *scale, float *const *out, int n_out,
                                        cudaStream_t st)
{
    FinalizeOuts fo{};
    for (int k = 0; k < n_out; ++k) { fo.out[k] = out[k]; fo.scale[k] = scale ? scale[k] : 1.0f; }
    BoundsReg br;
    br.add(partial, (size_t)n_out * n_slices * cols * sizeof(float));
    for (int k = 0; k < n_out; ++k) br.add(out[k], (size_t)cols * sizeof(float));
    RELAY_TRY(br.commit(st));
    const dim3 grid((unsigned)((cols + 31) / 32), (unsigned)n_out);
    if (n_slices > 256) RELAY_CUDA(launch_pdl(colsum_finalize_kernel<32>, grid, dim3(32, 32), 0, st, partial, n_slices, cols, fo));
    else RELAY_CUDA(launch_pdl(colsum_finalize_kernel<8>, grid, dim3(32, 8), 0, st, partial, n_slices, cols, fo));
    return check_launch("colsum_finalize");
}

relay_status_t launch_colsum_finalize(const float *partial, int n_slices, int64_t cols, float scale, float *out,
                                      cudaStream_t st)
{
    return launch_colsum_finalize_n(partial, n_slices, cols, &scale, &out, 1, st);
}

// dZ = dy (.) act'(y) stored to dz, and (if db) db = column sums of dZ; used by the dense gradient group
relay_status_t launch_act_grad(int32_t storage, const void *dy, const void *y, void *dz, float *db, float *partials,
                               int64_t rows, int64_t cols, int act, cudaStream_t st)
{
    const size_t esz = storage == RELAY_BF16 ? 2 : 4;
    BoundsReg br;
    br.add(dy, (size_t)rows * cols * esz); br.add(y, (size_t)rows * cols * esz); br.add(dz, (size_t)rows * cols * esz);
    br.add(db, (size_t)cols * 4); br.add(partials, db ? (size_t)colsum_slices(rows, cols, storage) * cols * 4 : 0);
    RELAY_TRY(br.commit(st));
    Args2D<2, 2> A{};
    A.in[0] = dy; A.in[1] = y;
    A.out[0] = dz; A.out[1] = nullptr;
    A.partial[0] = nullptr; A.partial[1] = db ? partials : nullptr;
    A.rows = rows; A.cols = cols; A.aux = act;
    const int ns = colsum_slices(rows, cols, storage);
    RELAY_TRY(launch_body2d<BodyActGrad>(storage, A, ns, st, "act_grad"));
    if (db) RELAY_TRY(launch_colsum_finalize(partials, ns, cols, 1.0f, db, st));
    return RELAY_OK;
}

relay_status_t launch_colsum_bf16(const void *in, int64_t rows, int64_t cols, float *partials, float *out, cudaStream_t st)
{
    BoundsReg br;
    br.add(in, (size_t)rows * cols * 2); br.add(out, (size_t)cols * 4); br.add(partials, (size_t)colsum_slices(rows, cols, RELAY_BF16) * cols * 4);
    RELAY_TRY(br.commit(st));
    Args2D<1, 1> A{};
    A.in[0] = in; A.out[0] = nullptr; A.partial[0] = partials;
    A.rows = rows; A.cols = cols; A.aux = 0;
    const int ns = colsum_slices(rows, cols, RELAY_BF16);
    RELAY_TRY(launch_body2d<BodyIdentityColSum>(RELAY_BF16, A, ns, st, "ewise2d<identity_colsum>"));
    return launch_colsum_finalize(partials, ns, cols, 1.0f, out, st);
}

static relay_status_t check_output(const relay_tensor_t *o, int32_t dtype, int rank, const int64_t *shape, int k)
{
    char name[32];
    snprintf(name, sizeof name, "outputs[%d]", k);
    RELAY_TRY(check_type(o, name));
    RELAY_TRY(check_rank(o, rank, name));
    RELAY_TRY(check_dtype(o, dtype, name));
    for (int d = 0; d < rank; ++d)
        if (o->shape[d] != shape[d])
            return fail(RELAY_ERR_SHAPE, "%s: axis %d has extent %lld, the group's type gives %lld", name, d, (long long)o->shape[d],
                        (long long)shape[d]);
    return RELAY_OK;
}

static unsigned grid_for(int64_t total, int threads)
{
    int64_t g = (total + threads - 1) / threads;
    return (unsigned)std::max<int64_t>(1, std::min<int64_t>(g, 148 * 16));
}

}  // namespace relay

using namespace relay;

extern "C" relay_status_t relay_fused_ewise(const relay_ewise_prog_t *prog, const relay_tensor_t *const *inputs, int32_t n_in,
                                            const int32_t *out_values, const relay_tensor_t *const *outputs, int32_t n_out,
                                            void *ws, size_t ws_bytes, void *stream)
{
    (void)ws; (void)ws_bytes;
    clear_error();
    TypedProgram tp;
    RELAY_TRY(check_not_null(out_values, "out_values"));
    RELAY_TRY(check_not_null(outputs, "outputs"));
    if (n_out < 1 || n_out > RELAY_MAX_OUTPUTS) return fail(RELAY_ERR_ATTR, "%d outputs, 1..%d allowed", n_out, RELAY_MAX_OUTPUTS);
    for (int k = 0; k < n_out; ++k) RELAY_TRY(check_not_null(outputs[k], "outputs[k]"));
    RELAY_TRY(type_program(prog, inputs, n_in, &tp));
    if (n_in < 1) return fail(RELAY_ERR_ATTR, "an elementwise group needs at least one input");
    for (int k = 0; k < n_out; ++k) {
        if (out_values[k] < 0 || out_values[k] >= tp.n_values) return fail(RELAY_ERR_ATTR, "out_values[%d] = %d names no value", k, out_values[k]);
        RELAY_TRY(check_output(outputs[k], tp.dtype[out_values[k]], tp.rank, tp.shape, k));
    }
    for (int i = 0; i < n_in; ++i) RELAY_TRY(check_data(inputs[i], "input"));
    for (int k = 0; k < n_out; ++k) RELAY_TRY(check_data(outputs[k], "output"));
    RELAY_TRY(check_no_overlap(outputs, n_out, inputs, n_in));
    if (tp.total == 0) return RELAY_OK;
    cudaStream_t st = (cudaStream_t)stream;
    BoundsReg br;
    for (int i = 0; i < n_in; ++i) br.add(inputs[i]);
    for (int k = 0; k < n_out; ++k) br.add(outputs[k]);
    RELAY_TRY(br.commit(st));

    // pre-compiled body?
    View2D v = view2d(tp);
    if (v.ok && n_out == 1 && n_in == 3 && outputs[0]->dtype == v.storage && kinds_match<BodyTanhAffineResidualFwd>(v) &&
        canon(tp, out_values[0]) == known_tanh_affine_fwd(v.storage).out) {
        Args2D<3, 1> A{};
        for (int i = 0; i < 3; ++i) A.in[i] = inputs[i]->data;
        A.out[0] = outputs[0]->data; A.partial[0] = nullptr;
        A.rows = v.rows; A.cols = v.cols; A.aux = 0;
        const int vec = v.storage == RELAY_BF16 ? 8 : 4;
        const int64_t gx = (v.cols + (int64_t)kTX * vec - 1) / (kTX * vec);
        int ns = (int)std::max<int64_t>(1, std::min<int64_t>((148 * 16) / gx, (v.rows + kTY * 4 - 1) / (kTY * 4)));
        return launch_body2d<BodyTanhAffineResidualFwd>(v.storage, A, ns, st, "ewise2d<tanh_affine_residual_fwd>");
    }

    // any other program over the 2-D view: a body compiled for this program where a run-time compiler is present, else the
    // in-kernel interpreter (which takes fewer programs: bounded temporaries and literals)
    if (v.ok) {
        const bool no_sums[RELAY_MAX_OUTPUTS] = {false};
        int32_t odt[RELAY_MAX_OUTPUTS];
        for (int k = 0; k < n_out; ++k) odt[k] = outputs[k]->dtype;
        if (const void *jk = jit_get(tp, v, out_values, odt, no_sums, n_out))
            return jit_launch(jk, v, inputs, n_in, outputs, n_out, nullptr, jit_n_slices(v, false), st);
        VmPlan vp;
        if (vm_plan(tp, v, out_values, no_sums, n_out, &vp)) {
            const int64_t gx = (v.cols + 255) / 256;
            const int ns = (int)std::max<int64_t>(1, std::min<int64_t>((148 * 8) / gx, v.rows / 32));
            return vm_launch(vp, v, inputs, n_in, outputs, n_out, nullptr, ns, st);
        }
    }

    DevProgram P;
    fill_dev_program(tp, inputs, &P);
    DevOutputs O{};
    O.n_out = n_out;
    for (int k = 0; k < n_out; ++k) { O.value[k] = out_values[k]; O.dtype[k] = outputs[k]->dtype; O.ptr[k] = outputs[k]->data; }
    ewise_generic_kernel<<<grid_for(tp.total, 256), 256, 0, st>>>(P, O, tp.total);
    return check_launch("ewise_generic");
}

// ---- reduce ----------------------------------------------------------------------------------------
namespace relay {

// Scalar-evaluator reductions with few results over a long reduced extent (a sum over all axes, say) are cut into runs
// that separate blocks reduce; the runs' (value, position) pairs take at most this much of the workspace.
constexpr int kSplitUnitsMax = 4096;
constexpr size_t kSplitScratchBytes = (size_t)kSplitUnitsMax * (sizeof(float) + sizeof(long long));
static int generic_split(int64_t kept_elems, int64_t red_elems)
{
    if (kept_elems > 64 || red_elems < 65536) return 1;
    const int64_t n = std::min<int64_t>(kSplitUnitsMax / kept_elems, red_elems / 8192);
    return n >= 2 ? (int)n : 1;
}

struct ReducePlan {
    TypedProgram tp;
    View2D v;
    bool fast_grad = false;     // pre-compiled tanh-affine gradient group
    bool fast_colsum = false;   // identity column sum / mean over all leading axes
    bool fast_row = false;      // identity reduction over the last axis
    bool vm = false;            // vectorised evaluator: unreduced results and sums / means over all leading axes
    bool jit = false;           // in the class a body can be compiled for at run time (a superset of `vm`)
    VmPlan vmp;
    int jit_slices = 1;
    int32_t vm_values[RELAY_MAX_OUTPUTS];
    int n_slices = 1;
    size_t ws_need = 0;
    int64_t red_shape[RELAY_MAX_OUTPUTS][RELAY_MAX_RANK];
    int red_rank[RELAY_MAX_OUTPUTS];
    int32_t out_dtype[RELAY_MAX_OUTPUTS];
};

static relay_status_t plan_reduce(const relay_ewise_prog_t *prog, const relay_tensor_t *const *inputs, int32_t n_in,
                                  const relay_out_spec_t *specs, int32_t n_out, ReducePlan *pl)
{
    static const relay_ewise_prog_t empty = {0, 0, nullptr};
    if (!prog) prog = &empty;
    RELAY_TRY(check_not_null(specs, "specs"));
    if (n_out < 1 || n_out > RELAY_MAX_OUTPUTS) return fail(RELAY_ERR_ATTR, "%d outputs, 1..%d allowed", n_out, RELAY_MAX_OUTPUTS);
    RELAY_TRY(type_program(prog, inputs, n_in, &pl->tp));
    const TypedProgram &tp = pl->tp;
    if (n_in < 1) return fail(RELAY_ERR_ATTR, "a reduce group needs at least one input");
    for (int k = 0; k < n_out; ++k) {
        const relay_out_spec_t &s = specs[k];
        if (s.value < 0 || s.value >= tp.n_values) return fail(RELAY_ERR_ATTR, "specs[%d].value = %d names no value", k, s.value);
        relay_tensor_t vt{}, rt{};
        vt.dtype = tp.dtype[s.value]; vt.rank = tp.rank; vt.layout = RELAY_ROWMAJOR;
        for (int d = 0; d < tp.rank; ++d) vt.shape[d] = tp.shape[d];
        if (s.red_op != RELAY_RED_NONE && !is_float(vt.dtype))
            return fail(RELAY_ERR_DTYPE, "specs[%d]: reduction of a %s value is not defined here", k, dtype_name(vt.dtype));
        RELAY_TRY(relay_infer_reduce(&vt, s.red_op, s.axes_mask, s.keepdims, &rt));
        pl->red_rank[k] = rt.rank;
        pl->out_dtype[k] = rt.dtype;
        for (int d = 0; d < rt.rank; ++d) pl->red_shape[k][d] = rt.shape[d];
    }
    pl->v = view2d(tp);
    const View2D &v = pl->v;
    const int32_t lead_mask = tp.rank >= 2 ? ((1 << (tp.rank - 1)) - 1) : 0;
    const int32_t last_mask = tp.rank >= 1 ? (1 << (tp.rank - 1)) : 0;
    if (v.ok && tp.rank >= 2 && n_out == 3 && n_in == 4 && kinds_match<BodyTanhAffineResidualGrad>(v) && specs[0].red_op == RELAY_RED_NONE &&
        tp.dtype[specs[0].value] == v.storage && specs[1].red_op == RELAY_RED_SUM && specs[2].red_op == RELAY_RED_SUM &&
        specs[1].axes_mask == lead_mask && specs[2].axes_mask == lead_mask) {
        KnownGrad kg = known_tanh_affine_grad(v.storage);
        if (canon(tp, specs[0].value) == kg.dx && canon(tp, specs[1].value) == kg.da && canon(tp, specs[2].value) == kg.db)
            pl->fast_grad = true;
    }
    if (!pl->fast_grad && v.ok && tp.rank >= 2 && n_out == 1 && n_in == 1 && tp.n_instr == 0 && v.kind[0] == KIND_FULL &&
        (specs[0].red_op == RELAY_RED_SUM || specs[0].red_op == RELAY_RED_MEAN) && specs[0].axes_mask == lead_mask)
        pl->fast_colsum = true;
    if (v.ok && tp.rank >= 1 && n_out == 1 && n_in == 1 && tp.n_instr == 0 && v.kind[0] == KIND_FULL &&
        specs[0].red_op != RELAY_RED_NONE && specs[0].axes_mask == last_mask)
        pl->fast_row = true;
    if (pl->fast_grad || pl->fast_colsum) {
        pl->n_slices = colsum_slices(v.rows, v.cols, v.storage);
        pl->ws_need = (size_t)(pl->fast_grad ? 2 : 1) * pl->n_slices * (size_t)v.cols * sizeof(float);
    } else if (!pl->fast_row && v.ok && tp.rank >= 2) {
        bool sums[RELAY_MAX_OUTPUTS], fits = true;
        for (int k = 0; k < n_out; ++k) {
            const bool colsum = (specs[k].red_op == RELAY_RED_SUM || specs[k].red_op == RELAY_RED_MEAN) && specs[k].axes_mask == lead_mask;
            if (specs[k].red_op != RELAY_RED_NONE && !colsum) fits = false;
            sums[k] = colsum;
            pl->vm_values[k] = specs[k].value;
        }
        if (fits) {
            int n_sum = 0;
            for (int k = 0; k < n_out; ++k) n_sum += sums[k];
            pl->jit = jit_in_class(tp, v, pl->vm_values, n_out);
            pl->vm = vm_plan(tp, v, pl->vm_values, sums, n_out, &pl->vmp);
            pl->n_slices = pl->vm ? vm_grid_slices(v, colsum_slices(v.rows, v.cols, v.storage)) : 1;
            pl->jit_slices = jit_n_slices(v, true);
            // room for either route: which one runs is decided at the launch (is a run-time compiler present?)
            if (pl->jit || pl->vm) pl->ws_need = (size_t)n_sum * std::max(pl->n_slices, pl->jit_slices) * (size_t)v.cols * sizeof(float);
        }
    }
    if (!pl->fast_grad && !pl->fast_colsum && !pl->fast_row) {
        // what is neither pre-compiled, compiled at run time nor interpreted 16 elements at a time runs on the scalar
        // evaluator; whether a compiled body exists is only known at the launch, so the room for split runs is asked for
        // whenever that evaluator may run
        for (int k = 0; k < n_out; ++k) {
            if (specs[k].red_op == RELAY_RED_NONE) continue;
            int64_t kept = 1, red = 1;
            for (int d = 0; d < tp.rank; ++d) (specs[k].axes_mask >> d & 1 ? red : kept) *= tp.shape[d];
            if (generic_split(kept, red) > 1) pl->ws_need = std::max(pl->ws_need, kSplitScratchBytes);
        }
    }
    return RELAY_OK;
}

// scratch that relay_fused_reduce will really use for this group (never more than relay_workspace_bytes_reduce's bound)
relay_status_t reduce_planned_scratch(const relay_ewise_prog_t *prog, const relay_tensor_t *const *inputs, int32_t n_in,
                                      const relay_out_spec_t *specs, int32_t n_out, size_t *need)
{
    ReducePlan pl;
    RELAY_TRY(plan_reduce(prog, inputs, n_in, specs, n_out, &pl));
    *need = pl.ws_need;
    return RELAY_OK;
}

}  // namespace relay

extern "C" size_t relay_workspace_bytes_reduce(const relay_tensor_t *const *inputs, int32_t n_in, const relay_out_spec_t *specs,
                                               int32_t n_out)
{
    // The workspace depends on the shapes and on which results are column sums, not on the
    // program body: an upper bound that holds for every program over these inputs.
    clear_error();
    if (!inputs || !specs || n_in < 1 || n_in > RELAY_MAX_INPUTS || n_out < 1) return 0;
    static const relay_ewise_prog_t empty = {0, 0, nullptr};
    TypedProgram tp;
    if (type_program(&empty, inputs, n_in, &tp) != RELAY_OK) return 0;
    int n_sum = 0;
    for (int k = 0; k < n_out; ++k) n_sum += specs[k].red_op != RELAY_RED_NONE;
    // runs of a split reduction on the scalar evaluator (any shape and type), or per-slice partials of column sums
    const size_t split = n_sum ? kSplitScratchBytes : 0;
    View2D v = view2d(tp);
    if (!v.ok) return split;
    return std::max(split, (size_t)n_sum * colsum_slices(v.rows, v.cols, v.storage) * (size_t)v.cols * sizeof(float));
}

extern "C" relay_status_t relay_fused_reduce(const relay_ewise_prog_t *prog, const relay_tensor_t *const *inputs, int32_t n_in,
                                             const relay_out_spec_t *specs, const relay_tensor_t *const *outputs, int32_t n_out,
                                             void *ws, size_t ws_bytes, void *stream)
{
    clear_error();
    RELAY_TRY(check_not_null(outputs, "outputs"));
    if (n_out >= 1 && n_out <= RELAY_MAX_OUTPUTS)
        for (int k = 0; k < n_out; ++k) RELAY_TRY(check_not_null(outputs[k], "outputs[k]"));
    ReducePlan pl;
    RELAY_TRY(plan_reduce(prog, inputs, n_in, specs, n_out, &pl));
    const TypedProgram &tp = pl.tp;
    for (int k = 0; k < n_out; ++k) RELAY_TRY(check_output(outputs[k], pl.out_dtype[k], pl.red_rank[k], pl.red_shape[k], k));
    for (int i = 0; i < n_in; ++i) RELAY_TRY(check_data(inputs[i], "input"));
    for (int k = 0; k < n_out; ++k) RELAY_TRY(check_data(outputs[k], "output"));
    RELAY_TRY(check_no_overlap(outputs, n_out, inputs, n_in));
    RELAY_TRY(check_workspace(ws, ws_bytes, pl.ws_need));
    if (tp.total == 0) return RELAY_OK;
    cudaStream_t st = (cudaStream_t)stream;
    const View2D &v = pl.v;
    BoundsReg br;
    for (int i = 0; i < n_in; ++i) br.add(inputs[i]);
    for (int k = 0; k < n_out; ++k) br.add(outputs[k]);
    br.add(ws, pl.ws_need);
    RELAY_TRY(br.commit(st));

    if (pl.fast_grad) {
        Args2D<4, 3> A{};
        for (int i = 0; i < 4; ++i) A.in[i] = inputs[i]->data;
        float *part = (float *)ws;
        A.out[0] = outputs[0]->data; A.out[1] = A.out[2] = nullptr;
        A.partial[0] = nullptr; A.partial[1] = part; A.partial[2] = part + (size_t)pl.n_slices * v.cols;
        A.rows = v.rows; A.cols = v.cols; A.aux = 0;
        if (cluster_sums(v.rows, v.cols, v.storage)) {
            A.partial[1] = A.partial[2] = nullptr;
            A.final[1] = (float *)outputs[1]->data; A.final[2] = (float *)outputs[2]->data; A.scale[1] = A.scale[2] = 1.0f;
            return launch_body2d_cluster<BodyTanhAffineResidualGrad>(v.storage, A, st, "ewise2d<tanh_affine_residual_grad>");
        }
        RELAY_TRY(launch_body2d<BodyTanhAffineResidualGrad>(v.storage, A, pl.n_slices, st, "ewise2d<tanh_affine_residual_grad>"));
        float *sums[2] = {(float *)outputs[1]->data, (float *)outputs[2]->data};
        return launch_colsum_finalize_n(A.partial[1], pl.n_slices, v.cols, nullptr, sums, 2, st);
    }
    if (pl.fast_colsum) {
        Args2D<1, 1> A{};
        A.in[0] = inputs[0]->data; A.out[0] = nullptr; A.partial[0] = (float *)ws;
        A.rows = v.rows; A.cols = v.cols; A.aux = 0;
        const float scale = specs[0].red_op == RELAY_RED_MEAN ? 1.0f / (float)v.rows : 1.0f;
        if (colsum_in_clusters(v.rows, v.cols, v.storage)) {
            A.partial[0] = nullptr; A.final[0] = (float *)outputs[0]->data; A.scale[0] = scale;
            return launch_colsum_cluster<BodyIdentityColSum, kColsumCluster, kColsumStripLanes, 4>(v.storage, A, st, "ewise2d<identity_colsum>");
        }
        RELAY_TRY(launch_body2d<BodyIdentityColSum>(v.storage, A, pl.n_slices, st, "ewise2d<identity_colsum>"));
        return launch_colsum_finalize(A.partial[0], pl.n_slices, v.cols, scale, (float *)outputs[0]->data, st);
    }
    if (pl.fast_row) {
        const unsigned grid = (unsigned)((v.rows + 7) / 8);
        const float scale = specs[0].red_op == RELAY_RED_MEAN ? 1.0f / (float)v.cols : 1.0f;
        const int op = specs[0].red_op == RELAY_RED_MEAN ? RELAY_RED_SUM : specs[0].red_op;
#define ROWRED(T, OP) rowreduce_kernel<T, OP><<<grid, 256, 0, st>>>((const T *)inputs[0]->data, v.rows, v.cols, scale, outputs[0]->data)
        if (v.storage == RELAY_BF16) {
            if (op == RELAY_RED_SUM) ROWRED(__nv_bfloat16, RELAY_RED_SUM);
            else if (op == RELAY_RED_MAX) ROWRED(__nv_bfloat16, RELAY_RED_MAX);
            else ROWRED(__nv_bfloat16, RELAY_RED_ARGMAX);
        } else {
            if (op == RELAY_RED_SUM) ROWRED(float, RELAY_RED_SUM);
            else if (op == RELAY_RED_MAX) ROWRED(float, RELAY_RED_MAX);
            else ROWRED(float, RELAY_RED_ARGMAX);
        }
#undef ROWRED
        return check_launch("rowreduce");
    }

    int32_t odt[RELAY_MAX_OUTPUTS];
    bool is_sum[RELAY_MAX_OUTPUTS];
    for (int k = 0; k < n_out; ++k) { odt[k] = outputs[k]->dtype; is_sum[k] = specs[k].red_op != RELAY_RED_NONE; }
    const void *jk = pl.jit ? jit_get(tp, v, pl.vm_values, odt, is_sum, n_out) : nullptr;
    if (jk || pl.vm) {
        int slices = pl.n_slices;
        if (jk) {
            slices = pl.jit_slices;
            RELAY_TRY(jit_launch(jk, v, inputs, n_in, outputs, n_out, (float *)ws, slices, st));
        } else {
            RELAY_TRY(vm_launch(pl.vmp, v, inputs, n_in, outputs, n_out, (float *)ws, slices, st));
        }
        float *sums[RELAY_MAX_OUTPUTS];
        float scale[RELAY_MAX_OUTPUTS];
        int n_sum = 0;
        for (int k = 0; k < n_out; ++k)
            if (specs[k].red_op != RELAY_RED_NONE) {
                sums[n_sum] = (float *)outputs[k]->data;
                scale[n_sum++] = specs[k].red_op == RELAY_RED_MEAN ? 1.0f / (float)v.rows : 1.0f;
            }
        return n_sum ? launch_colsum_finalize_n((const float *)ws, slices, v.cols, scale, sums, n_sum, st) : RELAY_OK;
    }

    // generic: one evaluator pass for the unreduced results, one reduction launch per reduced result
    DevProgram P;
    fill_dev_program(tp, inputs, &P);
    DevOutputs O{};
    for (int k = 0; k < n_out; ++k)
        if (specs[k].red_op == RELAY_RED_NONE) {
            O.value[O.n_out] = specs[k].value; O.dtype[O.n_out] = outputs[k]->dtype; O.ptr[O.n_out] = outputs[k]->data;
            ++O.n_out;
        }
    if (O.n_out > 0) {
        ewise_generic_kernel<<<grid_for(tp.total, 256), 256, 0, st>>>(P, O, tp.total);
        RELAY_TRY(check_launch("ewise_generic"));
    }
    for (int k = 0; k < n_out; ++k) {
        if (specs[k].red_op == RELAY_RED_NONE) continue;
        DevReduce R{};
        R.red_op = specs[k].red_op; R.value = specs[k].value; R.out = outputs[k]->data;
        R.kept_elems = 1; R.red_elems = 1;
        for (int d = 0; d < tp.rank; ++d) {
            if (specs[k].axes_mask >> d & 1) { R.red_axis[R.n_red++] = d; R.red_elems *= tp.shape[d]; }
            else { R.kept_axis[R.n_kept++] = d; R.kept_elems *= tp.shape[d]; }
        }
        R.scale = specs[k].red_op == RELAY_RED_MEAN ? 1.0f / (float)R.red_elems : 1.0f;
        R.group = (R.kept_elems < 148 * 8 && R.red_elems >= 1024) ? 256 : 32;
        R.n_split = generic_split(R.kept_elems, R.red_elems);
        int64_t units = R.kept_elems;
        if (R.n_split > 1) {
            R.group = 256;
            R.chunk = (R.red_elems + R.n_split - 1) / R.n_split;
            R.part_val = (float *)ws;
            R.part_pos = (long long *)((char *)ws + (size_t)kSplitUnitsMax * sizeof(float));
            units *= R.n_split;
        }
        const int per_block = 256 / R.group;
        reduce_generic_kernel<<<(unsigned)((units + per_block - 1) / per_block), 256, 0, st>>>(P, R);
        RELAY_TRY(check_launch("reduce_generic"));
        if (R.n_split > 1) {
            reduce_split_finish_kernel<<<(unsigned)((R.kept_elems + 127) / 128), 128, 0, st>>>(R);
            RELAY_TRY(check_launch("reduce_split_finish"));
        }
    }
    return RELAY_OK;
}

// Which kernel tier a group would run on (host only, launches nothing): 0 a pre-compiled body, 1 the vectorised
// evaluator, 2 the scalar evaluator, 3 the row-reduction kernel; -1 if the group does not type-check.
extern "C" int32_t relay_debug_group_route(const relay_ewise_prog_t *prog, const relay_tensor_t *const *inputs, int32_t n_in,
                                           const relay_out_spec_t *specs, int32_t n_out)
{
    clear_error();
    ReducePlan pl;
    if (plan_reduce(prog, inputs, n_in, specs, n_out, &pl) != RELAY_OK) return -1;
    bool all_unreduced = true;
    for (int k = 0; k < n_out; ++k) all_unreduced = all_unreduced && specs[k].red_op == RELAY_RED_NONE;
    if (!all_unreduced) return (pl.fast_grad || pl.fast_colsum) ? 0 : pl.fast_row ? 3 : (pl.vm || (pl.jit && jit_usable())) ? 1 : 2;
    const View2D &v = pl.v;
    if (v.ok && n_out == 1 && n_in == 3 && kinds_match<BodyTanhAffineResidualFwd>(v) && pl.tp.dtype[specs[0].value] == v.storage &&
        canon(pl.tp, specs[0].value) == known_tanh_affine_fwd(v.storage).out)
        return 0;
    VmPlan vp;
    int32_t values[RELAY_MAX_OUTPUTS];
    const bool no_sums[RELAY_MAX_OUTPUTS] = {false};
    for (int k = 0; k < n_out; ++k) values[k] = specs[k].value;
    return v.ok && (vm_plan(pl.tp, v, values, no_sums, n_out, &vp) || (jit_usable() && jit_in_class(pl.tp, v, values, n_out))) ? 1 : 2;
}

// Host only: the source of the body that would be compiled at run time for this group, and whether it compiles for sm_100a.
// 1: compiled (the source, NUL-terminated and cut to `cap` bytes, is in `src` if that is not null); 0: the group does not
// run on the vectorised tier; -1: no run-time compiler on this machine; -2: it did not compile (relay_last_error has the
// compiler's messages); -3: the group does not type-check.
extern "C" int32_t relay_debug_jit_compile(const relay_ewise_prog_t *prog, const relay_tensor_t *const *inputs, int32_t n_in,
                                           const relay_out_spec_t *specs, int32_t n_out, char *src, size_t cap)
{
    clear_error();
    ReducePlan pl;
    if (plan_reduce(prog, inputs, n_in, specs, n_out, &pl) != RELAY_OK) return -3;
    bool all_unreduced = true;
    for (int k = 0; k < n_out; ++k) all_unreduced = all_unreduced && specs[k].red_op == RELAY_RED_NONE;
    int32_t values[RELAY_MAX_OUTPUTS], odt[RELAY_MAX_OUTPUTS];
    bool sums[RELAY_MAX_OUTPUTS];
    for (int k = 0; k < n_out; ++k) { values[k] = specs[k].value; sums[k] = specs[k].red_op != RELAY_RED_NONE; odt[k] = pl.tp.dtype[specs[k].value]; }
    if (all_unreduced ? !jit_in_class(pl.tp, pl.v, values, n_out) : !pl.jit) return 0;
    if (!all_unreduced && (pl.fast_grad || pl.fast_colsum || pl.fast_row)) return 0;
    std::string text, log;
    const int r = jit_compile_only(pl.tp, pl.v, values, odt, sums, n_out, &text, &log);
    if (r == -2) fail(RELAY_ERR_CUDA, "run-time compilation failed: %s", log.c_str());
    if (src && cap > 0) { snprintf(src, cap, "%s", text.c_str()); }
    return r;
}
