// Vectorised evaluator for elementwise programs that have no pre-compiled body (Fig. 1 BinOp / UnaryOp productions,
// Fig. 5 typing rules; operator fusion, Section 5.2): any straight-line program over the collapsed 2-D view
// [rows, cols] whose inputs are full-shape tensors, tensors constant down the rows, or scalars of one float storage
// type, with unreduced results and column sums.
//
// Host: the let-list is turned into code for a small ACCUMULATOR machine.  The accumulator holds 16 elements per
// thread in registers; every instruction combines it with at most one operand that is fetched from shared memory: an
// input (the TMA-filled tile ring, or the row of an input that is constant down the rows), a temporary (a
// thread-private slot that an earlier instruction stored the accumulator to) or a literal.  Expression trees are
// evaluated deeper operand first, so that the other operand is a leaf wherever possible; values used several times are
// computed once and kept in a temporary.  With one accumulator there is no register state that depends on where
// in the program the interpreter is: it branches once per instruction on the opcode, and the branch tree is shallow.
//
// Device: a block owns 256 columns x a slice of rows.  16-row tiles of every full-shape input stream into a
// shared-memory ring by TMA, issued by one lane of warp 0 ahead of use (the bytes in flight live in shared memory,
// not in registers); the 256 threads each interpret the program once per tile on 2 rows x 8 columns.  Column sums:
// per-thread accumulators -> fixed-order combine in shared memory -> one partial per row slice ->
// colsum_finalize_kernel (no float atomics: reruns are bit-identical).
#include <algorithm>
#include <cstring>
#include <new>

#include "ewise_host.h"
#include "ewise_kernels.cuh"
#include "ewise_prog.h"
#include "tc_common.cuh"

namespace relay {

relay_status_t make_tmap_2d(CUtensorMap *m, bool f32, const void *base, uint64_t inner, uint64_t outer, uint64_t row_stride,
                            uint32_t box_inner, uint32_t box_outer, bool swizzle128);

namespace {

constexpr int VM_TX = 32, VM_TY = 8, VM_V = 8, VM_R = 2;   // 256 threads; a thread owns 8 columns of rows ty and ty + 8 of a tile
constexpr int VM_E = VM_V * VM_R;                          // elements in the accumulator
constexpr int VM_COLS = VM_TX * VM_V;                      // columns per block
constexpr int VM_TILE_ROWS = VM_TY * VM_R;
constexpr int VM_THREADS = VM_TX * VM_TY;
constexpr int VM_MAXCODE = 96, VM_MAXFULL = 4, VM_MAXFIXED = 4, VM_MAXSUM = 2, VM_MAXTEMP = 4, VM_MAXCONST = 6;
constexpr int VM_RING_BYTES = 96 * 1024;                   // budget of the tile ring

// opcodes: 0 .. RELAY_OP_COUNT_-1 are the program's own operators, acc = acc (op) operand for the binary ones
enum : int {
    A_LOAD = 22,        // acc = operand
    A_RSUB, A_RDIV,     // acc = operand - acc, operand / acc (the deeper operand of a tree is evaluated first)
    A_STASH,            // temporary[operand] = acc
    A_STORE,            // output[operand] = acc
    A_COLSUM0, A_COLSUM1,
    A_ROUND_BF16, A_TO_BOOL,
    A_NOPS
};
static_assert(RELAY_OP_COUNT_ == 22, "the machine's own opcodes start after the program's operators");

// operand of an instruction: 0..7 input i; 8.. slot (temporaries first, then literals)
constexpr int OPD_SLOT = 8;

struct VmCode {
    int32_t n;
    uint8_t op[VM_MAXCODE], opd[VM_MAXCODE], opd2[VM_MAXCODE];   // opd2: SELECT's second operand
};

struct VmArgs {
    const void *fixed_ptr[VM_MAXFIXED];
    int8_t fixed_scalar[VM_MAXFIXED];
    int8_t in_kind[RELAY_MAX_INPUTS], in_slot[RELAY_MAX_INPUTS];   // kind 0: full-shape (slot = ring slot), 1: constant down the rows
    void *out[RELAY_MAX_OUTPUTS];
    int8_t out_dt[RELAY_MAX_OUTPUTS];
    float *partial[VM_MAXSUM];
    float literal[VM_MAXCONST];
    int64_t rows, cols;
    int32_t rows_per_slice, n_full, n_fixed, n_sum, n_temp, n_const, stages;
    int32_t box_cols, box_rows;        // TMA box (min(256, cols) x min(16, rows))
    int *err;
    VmCode code;
};

template <typename T> __device__ __forceinline__ int vm_col(int tx, int v)
{
    // bf16: 8 consecutive columns per thread; f32: two runs of 4 columns, 128 columns apart (16-byte shared-memory
    // reads of a warp then cover 512 consecutive bytes: no bank conflicts)
    if constexpr (sizeof(T) == 2) return tx * 8 + v;
    else return (v < 4 ? 0 : 128) + tx * 4 + (v & 3);
}

__device__ __forceinline__ uint4 lds128(uint32_t addr)
{
    uint4 r;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr));
    return r;
}
__device__ __forceinline__ void sts128(uint32_t addr, const uint4 &r)
{
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(r.x), "r"(r.y), "r"(r.z), "r"(r.w) : "memory");
}

// (register arrays are only ever indexed with constants and never passed as pointers: a pointer into one would move it
// to local memory)
template <typename T> __device__ __forceinline__ void vm_load_row(uint32_t row, bool hi_live, float (&f)[VM_V])
{
    if constexpr (sizeof(T) == 2) {
        unpack(lds128(row), f);
    } else {
        float lo[4], hi[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        unpack(lds128(row), lo);
        if (hi_live) unpack(lds128(row + 512), hi);
#pragma unroll
        for (int v = 0; v < 4; ++v) { f[v] = lo[v]; f[4 + v] = hi[v]; }
    }
}

// stores N consecutive result elements (N = 8 or 4) starting at element index `at` of an output of type `dt`
template <int N> __device__ __forceinline__ void vm_store_run(void *out, int dt, int64_t at, const float (&f)[N])
{
    if (dt == RELAY_F32) {
#pragma unroll
        for (int q = 0; q < N / 4; ++q)
            st_stream((float *)out + at + 4 * q, make_uint4(__float_as_uint(f[4 * q]), __float_as_uint(f[4 * q + 1]), __float_as_uint(f[4 * q + 2]),
                                                            __float_as_uint(f[4 * q + 3])));
    } else if (dt == RELAY_BF16) {
        if constexpr (N == 8) {
            st_stream((__nv_bfloat16 *)out + at, make_uint4(pack2(f[0], f[1]), pack2(f[2], f[3]), pack2(f[4], f[5]), pack2(f[6], f[7])));
        } else {
            if (relay_in_bounds((__nv_bfloat16 *)out + at, 8)) *reinterpret_cast<uint2 *>((__nv_bfloat16 *)out + at) = make_uint2(pack2(f[0], f[1]), pack2(f[2], f[3]));
        }
    } else {   // bool: one byte per element
        uint32_t w[N / 4];
#pragma unroll
        for (int q = 0; q < N / 4; ++q)
            w[q] = (f[4 * q] != 0.0f ? 1u : 0u) | (f[4 * q + 1] != 0.0f ? 0x100u : 0u) | (f[4 * q + 2] != 0.0f ? 0x10000u : 0u) |
                   (f[4 * q + 3] != 0.0f ? 0x1000000u : 0u);
        if (!relay_in_bounds((uint8_t *)out + at, N)) return;
        if constexpr (N == 8) *reinterpret_cast<uint2 *>((uint8_t *)out + at) = make_uint2(w[0], w[1]);
        else *reinterpret_cast<uint32_t *>((uint8_t *)out + at) = w[0];
    }
}

struct VmThread {             // shared-memory addresses are 32-bit shared-window addresses, already offset by this thread's lane
    uint32_t stage;         // ring stage of the current tile + ty * row_bytes + tx * 16
    uint32_t fixed;         // rows of the operands that are constant down the rows + tx * 16
    uint32_t temps;         // temporaries: [slot][4 pieces of 16 bytes][256 threads] + tid * 16
    uint32_t literals;      // 16 bytes each, behind the temporaries
    int tx, ty, tid;
    bool hi_live;           // f32: the thread's second run of 4 columns lies inside the tensor
    bool row_live[VM_R];
    int tile_bytes, row_bytes, n_temp;
    int64_t row0, col0;     // first row of the tile and the block's first column
};

// fetches the operand of an instruction into o[16]
template <typename T>
__device__ __forceinline__ void vm_fetch(int opd, float (&o)[VM_E], const VmArgs &A, const VmThread &th)
{
    if (opd < OPD_SLOT) {
        const int slot = A.in_slot[opd];
        if (A.in_kind[opd] == 0) {
            const uint32_t row = th.stage + slot * th.tile_bytes;
            float r0[VM_V], r1[VM_V];
            vm_load_row<T>(row, th.hi_live, r0);
            vm_load_row<T>(row + VM_TY * th.row_bytes, th.hi_live, r1);
#pragma unroll
            for (int v = 0; v < VM_V; ++v) { o[v] = r0[v]; o[VM_V + v] = r1[v]; }
        } else {
            float r0[VM_V];
            vm_load_row<T>(th.fixed + slot * (VM_COLS * (int)sizeof(T)), th.hi_live, r0);
#pragma unroll
            for (int v = 0; v < VM_V; ++v) { o[v] = r0[v]; o[VM_V + v] = r0[v]; }
        }
    } else {
        // a temporary (one 64-byte value per thread, in four pieces) or a literal (one 16-byte piece for everybody)
        const int k = opd - OPD_SLOT;
        const bool temp = k < th.n_temp;
        const uint32_t p = temp ? th.temps + k * (4 * VM_THREADS * 16) : th.literals + (k - th.n_temp) * 16;
        const uint32_t step = temp ? VM_THREADS * 16 : 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint4 w = lds128(p + q * step);
            o[4 * q] = __uint_as_float(w.x); o[4 * q + 1] = __uint_as_float(w.y); o[4 * q + 2] = __uint_as_float(w.z); o[4 * q + 3] = __uint_as_float(w.w);
        }
    }
}

template <typename T, bool FAST>
__global__ void __launch_bounds__(VM_THREADS, 3)
ewise_vm_kernel(const __grid_constant__ CUtensorMap tm0, const __grid_constant__ CUtensorMap tm1, const __grid_constant__ CUtensorMap tm2,
                const __grid_constant__ CUtensorMap tm3, const __grid_constant__ VmArgs A)
{
    extern __shared__ uint8_t vm_smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(vm_smem_raw) + 1023) & ~uintptr_t(1023));
    const int row_bytes = A.box_cols * (int)sizeof(T), tile_bytes = ((A.box_rows * row_bytes + 127) / 128) * 128;
    const int stage_bytes = A.n_full * tile_bytes, STAGES = A.stages;
    const int ring_bytes = max(STAGES * stage_bytes, VM_TY * (VM_COLS + 1) * (int)sizeof(float));   // the ring's start doubles as the combine buffer
    uint8_t *fixed = smem + ((ring_bytes + 127) / 128) * 128;
    uint8_t *slots = fixed + ((A.n_fixed * VM_COLS * (int)sizeof(T) + 127) / 128) * 128;
    uint64_t *bars = reinterpret_cast<uint64_t *>(slots + ((A.n_temp * 4 * VM_THREADS + A.n_const) * 16 + 127) / 128 * 128);
    uint64_t *full = bars, *empty = bars + 4;
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + 8);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t col0 = (int64_t)blockIdx.x * VM_COLS;
    const int64_t r0 = (int64_t)blockIdx.y * A.rows_per_slice, r1 = min(A.rows, r0 + (int64_t)A.rows_per_slice);
    const int n_tiles = r1 > r0 ? (int)((r1 - r0 + A.box_rows - 1) / A.box_rows) : 0;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&full[s], 1); tc::mbar_init(&empty[s], VM_TY); }
        *abort_flag = 0;
        tc::fence_barrier_init();
        tc::prefetch_tmap(&tm0);
    }
    pdl_wait();
    // operands that are constant down the rows: one row of this block's columns each (a scalar fills the row); literals
    for (int g = 0; g < A.n_fixed; ++g) {
        const T *p = (const T *)A.fixed_ptr[g];
        T val = T(0.0f);
        if (A.fixed_scalar[g]) { if (relay_in_bounds(p, sizeof(T))) val = p[0]; }
        else if (col0 + tid < A.cols && relay_in_bounds(p + col0 + tid, sizeof(T))) val = p[col0 + tid];
        reinterpret_cast<T *>(fixed)[g * VM_COLS + tid] = val;
    }
    if (tid < A.n_const * 4) reinterpret_cast<float *>(slots + A.n_temp * 4 * VM_THREADS * 16)[tid] = A.literal[tid >> 2];
    __syncthreads();

    float sum[VM_MAXSUM][VM_V];
#pragma unroll
    for (int k = 0; k < VM_MAXSUM; ++k)
#pragma unroll
        for (int v = 0; v < VM_V; ++v) sum[k][v] = 0.0f;

    {
        // Warp 0 is also the producer: before it interprets tile t it refills the ring with tile t + STAGES - 1, whose
        // stage the other warps released when they finished tile t - 1 (they run at most a tile or two behind).
        const CUtensorMap *tms[VM_MAXFULL] = {&tm0, &tm1, &tm2, &tm3};
        auto issue = [&](int t) -> bool {        // whole warp 0; false when a wait gave up
            const int s = t % STAGES;
            if (!__all_sync(0xffffffffu, tc::mbar_wait(&empty[s], ((t / STAGES) & 1) ^ 1, abort_flag, A.err, tc::ERR_WAIT_EMPTY))) return false;
            if (tc::elect_one()) {
                tc::mbar_expect_tx(&full[s], (uint32_t)(A.n_full * A.box_rows * row_bytes));
#pragma unroll
                for (int f = 0; f < VM_MAXFULL; ++f)
                    if (f < A.n_full) tc::tma_load_2d(smem + s * stage_bytes + f * tile_bytes, tms[f], &full[s], (int)col0, (int)(r0 + (int64_t)t * A.box_rows));
            }
            __syncwarp();
            return true;
        };
        bool ok_issue = true;
        if (warp == 0)
            for (int t = 0; t < STAGES - 1 && t < n_tiles && ok_issue; ++t) ok_issue = issue(t);
        VmThread th;
        th.fixed = tc::smem_u32(fixed) + lane * 16;
        th.temps = tc::smem_u32(slots) + tid * 16;
        th.literals = tc::smem_u32(slots) + A.n_temp * 4 * VM_THREADS * 16;
        th.tx = lane; th.ty = warp; th.tid = tid;
        th.tile_bytes = tile_bytes; th.row_bytes = row_bytes; th.n_temp = A.n_temp;
        th.col0 = col0;
        th.hi_live = sizeof(T) == 4 && col0 + 128 + lane * 4 < A.cols;
        const bool col_live = col0 + vm_col<T>(lane, 0) < A.cols;     // a thread's first column decides (its second run is checked at the store)
        float acc[VM_E];
#pragma unroll
        for (int e = 0; e < VM_E; ++e) acc[e] = 0.0f;
        for (int t = 0; t < n_tiles; ++t) {
            if (warp == 0 && t + STAGES - 1 < n_tiles && ok_issue) ok_issue = issue(t + STAGES - 1);
            const int st = t % STAGES;
            int ok = 1;
            if (lane == 0) ok = tc::mbar_wait(&full[st], (t / STAGES) & 1, abort_flag, A.err, tc::ERR_WAIT_FULL) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            th.stage = tc::smem_u32(smem + st * stage_bytes) + warp * row_bytes + lane * 16;
            th.row0 = r0 + (int64_t)t * A.box_rows;
#pragma unroll
            for (int r = 0; r < VM_R; ++r) th.row_live[r] = warp + VM_TY * r < A.box_rows && th.row0 + warp + VM_TY * r < r1;
            if (th.row_live[0] && col_live) {
#pragma unroll 1
                for (int pc = 0; pc < A.code.n; ++pc) {
                    const int op = A.code.op[pc], opd = A.code.opd[pc];
                    if (op <= A_RDIV && op != RELAY_OP_NEG && op != RELAY_OP_SQ && op != RELAY_OP_RELU && op != RELAY_OP_TANH && op != RELAY_OP_SIGMOID &&
                        op != RELAY_OP_EXP && op != RELAY_OP_LOG && op != RELAY_OP_SELECT) {
                        float o[VM_E];
                        vm_fetch<T>(opd, o, A, th);
#define VM_BIN(OP, EXPR)                                                         \
    case OP:                                                                     \
        _Pragma("unroll") for (int e = 0; e < VM_E; ++e) { const float x = acc[e], y = o[e]; acc[e] = (EXPR); } \
        break;
                        switch (op) {
                            VM_BIN(RELAY_OP_ADD, x + y)
                            VM_BIN(RELAY_OP_SUB, x - y)
                            VM_BIN(RELAY_OP_MUL, x * y)
                            VM_BIN(RELAY_OP_DIV, FAST ? __fdividef(x, y) : x / y)
                            VM_BIN(RELAY_OP_NE, x != y ? 1.0f : 0.0f)
                            VM_BIN(RELAY_OP_EQ, x == y ? 1.0f : 0.0f)
                            VM_BIN(RELAY_OP_LT, x < y ? 1.0f : 0.0f)
                            VM_BIN(RELAY_OP_LE, x <= y ? 1.0f : 0.0f)
                            VM_BIN(RELAY_OP_GT, x > y ? 1.0f : 0.0f)
                            VM_BIN(RELAY_OP_GE, x >= y ? 1.0f : 0.0f)
                            VM_BIN(RELAY_OP_MAX, fmaxf(x, y))
                            VM_BIN(RELAY_OP_MIN, fminf(x, y))
                            VM_BIN(A_RSUB, y - x)
                            VM_BIN(A_RDIV, FAST ? __fdividef(y, x) : y / x)
                        default:      // A_LOAD
#pragma unroll
                            for (int e = 0; e < VM_E; ++e) acc[e] = o[e];
                            break;
                        }
#undef VM_BIN
                    } else {
#define VM_UN(OP, EXPR)                                                          \
    case OP:                                                                     \
        _Pragma("unroll") for (int e = 0; e < VM_E; ++e) { const float x = acc[e]; acc[e] = (EXPR); } \
        break;
                        switch (op) {
                            VM_UN(RELAY_OP_NEG, -x)
                            VM_UN(RELAY_OP_SQ, x * x)
                            VM_UN(RELAY_OP_RELU, fmaxf(x, 0.0f))
                            // bf16 storage: exp2 / reciprocal approximations (absolute error about 1e-7).  The one-instruction
                            // tanh.approx of the pre-compiled bodies (relative error 2^-11) is not used here: a program may
                            // multiply the result by anything.
                            VM_UN(RELAY_OP_TANH, FAST ? 1.0f - __fdividef(2.0f, 1.0f + __expf(2.0f * x)) : tanhf(x))
                            VM_UN(RELAY_OP_SIGMOID, FAST ? __fdividef(1.0f, 1.0f + __expf(-x)) : 1.0f / (1.0f + expf(-x)))
                            VM_UN(RELAY_OP_EXP, FAST ? __expf(x) : expf(x))
                            VM_UN(RELAY_OP_LOG, FAST ? __logf(x) : logf(x))
                            VM_UN(A_ROUND_BF16, round_bf16(x))
                            VM_UN(A_TO_BOOL, x != 0.0f ? 1.0f : 0.0f)
                        case RELAY_OP_SELECT: {      // acc = acc ? operand : second operand
                            float a[VM_E], b[VM_E];
                            vm_fetch<T>(opd, a, A, th);
                            vm_fetch<T>(A.code.opd2[pc], b, A, th);
#pragma unroll
                            for (int e = 0; e < VM_E; ++e) acc[e] = acc[e] != 0.0f ? a[e] : b[e];
                            break;
                        }
                        case A_STASH: {
                            const uint32_t p = th.temps + (opd - OPD_SLOT) * (4 * VM_THREADS * 16);
#pragma unroll
                            for (int q = 0; q < 4; ++q)
                                sts128(p + q * VM_THREADS * 16, make_uint4(__float_as_uint(acc[4 * q]), __float_as_uint(acc[4 * q + 1]), __float_as_uint(acc[4 * q + 2]),
                                                                           __float_as_uint(acc[4 * q + 3])));
                            break;
                        }
                        case A_STORE: {
                            void *out = A.out[opd];
                            const int dt = A.out_dt[opd];
#pragma unroll
                            for (int r = 0; r < VM_R; ++r) {
                                if (!th.row_live[r]) continue;
                                const int64_t at = (th.row0 + warp + VM_TY * r) * A.cols + col0;
                                if constexpr (sizeof(T) == 2) {
                                    float w[8];
#pragma unroll
                                    for (int v = 0; v < 8; ++v) w[v] = acc[VM_V * r + v];
                                    vm_store_run<8>(out, dt, at + lane * 8, w);
                                } else {
                                    float lo[4], hi[4];
#pragma unroll
                                    for (int v = 0; v < 4; ++v) { lo[v] = acc[VM_V * r + v]; hi[v] = acc[VM_V * r + 4 + v]; }
                                    vm_store_run<4>(out, dt, at + lane * 4, lo);
                                    if (th.hi_live) vm_store_run<4>(out, dt, at + 128 + lane * 4, hi);
                                }
                            }
                            break;
                        }
                        case A_COLSUM0:
#pragma unroll
                            for (int v = 0; v < VM_V; ++v) sum[0][v] += acc[v] + (th.row_live[1] ? acc[VM_V + v] : 0.0f);
                            break;
                        default:      // A_COLSUM1
#pragma unroll
                            for (int v = 0; v < VM_V; ++v) sum[1][v] += acc[v] + (th.row_live[1] ? acc[VM_V + v] : 0.0f);
                            break;
                        }
#undef VM_UN
                    }
                }
            }
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(&empty[st]);      // the warp's shared-memory reads of this stage are done
        }
    }

    // column sums: combine the 8 row-threads of every column in ty order, one partial row per slice
    if (A.n_sum > 0) {
        __syncthreads();                                    // the ring is no longer read: its first bytes hold the combine buffer
        float(*sm)[VM_COLS + 1] = reinterpret_cast<float(*)[VM_COLS + 1]>(smem);
        for (int k = 0; k < A.n_sum; ++k) {
#pragma unroll
            for (int v = 0; v < VM_V; ++v) sm[warp][vm_col<T>(lane, v)] = sum[k][v];
            __syncthreads();
            if (col0 + tid < A.cols) {
                float t = 0.0f;
#pragma unroll
                for (int j = 0; j < VM_TY; ++j) t += sm[j][tid];
                if (relay_in_bounds(&A.partial[k][(int64_t)blockIdx.y * A.cols + col0 + tid], 4)) A.partial[k][(int64_t)blockIdx.y * A.cols + col0 + tid] = t;
            }
            __syncthreads();
        }
    }
}

// =================================================================================================
// host: let-list -> accumulator code
// =================================================================================================
struct Compiler {
    const TypedProgram &tp;
    VmCode &code;
    int alias[kMaxValues];       // value this one is a plain copy of (casts that change nothing), or itself
    int uses[kMaxValues];
    int home[kMaxValues];        // temporary that holds the value, -1 if none
    bool temp_used[VM_MAXTEMP] = {false};
    int n_temp = 0;              // highest temporary in use + 1
    float literal[VM_MAXCONST];
    int n_const = 0;
    int acc_holds = -1;          // value currently in the accumulator, if known
    int last_op = -1;
    bool ok = true;

    Compiler(const TypedProgram &t, VmCode &c) : tp(t), code(c) { code.n = 0; }

    void emit(int op, int opd, int opd2 = 0)
    {
        if (code.n >= VM_MAXCODE) { ok = false; return; }
        code.op[code.n] = (uint8_t)op; code.opd[code.n] = (uint8_t)opd; code.opd2[code.n] = (uint8_t)opd2;
        ++code.n;
        last_op = op;
        if (op != A_STASH && op != A_STORE && op != A_COLSUM0 && op != A_COLSUM1) acc_holds = -1;
    }
    int alloc_temp()
    {
        for (int k = 0; k < VM_MAXTEMP; ++k)
            if (!temp_used[k]) { temp_used[k] = true; n_temp = std::max(n_temp, k + 1); return k; }
        ok = false;
        return 0;
    }
    float literal_of(const relay_instr_t &in) const
    {
        float c = (float)in.imm;
        if (in.dtype == RELAY_BF16) c = __bfloat162float(__float2bfloat16_rn(c));
        else if (in.dtype == RELAY_BOOL) c = in.imm != 0.0 ? 1.0f : 0.0f;
        return c;
    }
    int const_slot(float c)
    {
        for (int i = 0; i < n_const; ++i)
            if (memcmp(&literal[i], &c, sizeof c) == 0) return i;
        if (n_const == VM_MAXCONST) { ok = false; return 0; }
        literal[n_const] = c;
        return n_const++;
    }
    bool is_const(int v) const { return v >= tp.n_in && tp.instr[v - tp.n_in].op == RELAY_OP_CONST; }
    // operands that an instruction can take straight from shared memory
    bool is_leaf(int v) const { v = alias[v]; return v < tp.n_in || home[v] >= 0 || is_const(v); }
    // operand code of a leaf; literals are numbered behind the temporaries once their count is known, so they are
    // recorded as 128 + index here and renumbered by finish()
    int operand(int v)
    {
        v = alias[v];
        if (v < tp.n_in) return v;
        if (home[v] >= 0) return OPD_SLOT + home[v];
        return 128 + const_slot(literal_of(tp.instr[v - tp.n_in]));
    }
    static int mirrored(int op)      // x op y == y mirrored(op) x
    {
        switch (op) {
        case RELAY_OP_SUB: return A_RSUB;
        case RELAY_OP_DIV: return A_RDIV;
        case RELAY_OP_LT: return RELAY_OP_GT;
        case RELAY_OP_LE: return RELAY_OP_GE;
        case RELAY_OP_GT: return RELAY_OP_LT;
        case RELAY_OP_GE: return RELAY_OP_LE;
        default: return op;          // commutative
        }
    }
    // operand code of v for SELECT: a leaf as it is, anything else through a temporary
    int as_operand(int v, int depth, int *owned_temp)
    {
        *owned_temp = -1;
        if (is_leaf(v)) return operand(v);
        gen(v, depth + 1);
        const int t = alloc_temp();
        emit(A_STASH, OPD_SLOT + t);
        *owned_temp = t;
        return OPD_SLOT + t;
    }

    // evaluates value v into the accumulator
    void gen(int v, int depth = 0)
    {
        if (!ok || depth > 40) { ok = false; return; }
        v = alias[v];
        if (acc_holds == v) return;
        if (is_leaf(v)) { emit(A_LOAD, operand(v)); acc_holds = v; return; }
        const relay_instr_t &in = tp.instr[v - tp.n_in];
        if (in.op == RELAY_OP_CAST) {       // a cast that is not a plain copy
            gen(in.a, depth + 1);
            emit(in.dtype == RELAY_BF16 ? A_ROUND_BF16 : A_TO_BOOL, 0);
        } else if (in.op == RELAY_OP_SELECT) {
            int own_b, own_c;
            const int ob = as_operand(in.b, depth, &own_b), oc = as_operand(in.c, depth, &own_c);
            gen(in.a, depth + 1);
            emit(RELAY_OP_SELECT, ob, oc);
            if (own_b >= 0) temp_used[own_b] = false;
            if (own_c >= 0) temp_used[own_c] = false;
        } else if (in.b < 0) {              // unary
            gen(in.a, depth + 1);
            emit(in.op, 0);
        } else if (is_leaf(in.b)) {
            gen(in.a, depth + 1);
            emit(in.op, operand(in.b));
        } else if (is_leaf(in.a)) {
            gen(in.b, depth + 1);
            emit(mirrored(in.op), operand(in.a));
        } else {
            gen(in.a, depth + 1);
            const int t = alloc_temp();
            emit(A_STASH, OPD_SLOT + t);
            gen(in.b, depth + 1);
            emit(mirrored(in.op), OPD_SLOT + t);
            temp_used[t] = false;
        }
        // a value of type bf16 holds a bf16 number (operators that only pick one of their operands need no rounding)
        if (in.dtype == RELAY_BF16 && in.op != RELAY_OP_CAST && in.op != RELAY_OP_SELECT && in.op != RELAY_OP_MAX && in.op != RELAY_OP_MIN &&
            in.op != RELAY_OP_NEG && in.op != RELAY_OP_RELU)
            emit(A_ROUND_BF16, 0);
        acc_holds = v;
    }
    // literals live behind the temporaries
    void finish()
    {
        for (int i = 0; i < code.n; ++i) {
            if (code.opd[i] >= 128) code.opd[i] = (uint8_t)(OPD_SLOT + n_temp + (code.opd[i] - 128));
            if (code.opd2[i] >= 128) code.opd2[i] = (uint8_t)(OPD_SLOT + n_temp + (code.opd2[i] - 128));
        }
    }
};

}  // namespace

struct VmPlanImpl {
    VmCode code;
    int in_kind[RELAY_MAX_INPUTS], in_slot[RELAY_MAX_INPUTS];
    int n_full = 0, n_fixed = 0, n_sum = 0, n_temp = 0, n_const = 0;
    float literal[VM_MAXCONST];
    int sum_of_out[RELAY_MAX_OUTPUTS];     // index of the accumulator of output k, or -1
};

// Plans the group for the vectorised evaluator.  `colsum[k]`: output k is the sum of value out_values[k] over all rows
// (else it is stored unreduced).  Returns false when the group has to run on the scalar evaluator.
bool vm_plan(const TypedProgram &tp, const View2D &v, const int32_t *out_values, const bool *colsum, int n_out, VmPlan *plan)
{
    static_assert(sizeof(VmPlan::storage) >= sizeof(VmPlanImpl), "VmPlan::storage too small");
    VmPlanImpl &P = *new (plan->storage) VmPlanImpl();
    plan->ok = false;
    if (!v.ok || v.rows < 1 || n_out < 1 || n_out > RELAY_MAX_OUTPUTS) return false;
    if (v.rows >= (1ll << 31) || v.cols >= (1ll << 31)) return false;
    for (int i = 0; i < tp.n_in; ++i) {
        if (v.kind[i] == KIND_FULL) { if (P.n_full == VM_MAXFULL) return false; P.in_kind[i] = 0; P.in_slot[i] = P.n_full++; }
        else { if (P.n_fixed == VM_MAXFIXED) return false; P.in_kind[i] = 1; P.in_slot[i] = P.n_fixed++; }
    }
    if (P.n_full < 1) return false;
    // at least two ring stages of 16-row tiles must fit
    const int64_t tile = std::min<int64_t>(VM_COLS, v.cols) * (v.storage == RELAY_F32 ? 4 : 2) * std::min<int64_t>(VM_TILE_ROWS, v.rows);
    if (2 * P.n_full * ((tile + 127) / 128 * 128) > VM_RING_BYTES) return false;
    Compiler C(tp, P.code);
    // which values are needed, and which are plain copies of another value
    bool needed[kMaxValues] = {false};
    for (int k = 0; k < n_out; ++k) needed[out_values[k]] = true;
    for (int x = tp.n_values - 1; x >= tp.n_in; --x) {
        if (!needed[x]) continue;
        const relay_instr_t &in = tp.instr[x - tp.n_in];
        if (in.a >= 0) needed[in.a] = true;
        if (in.b >= 0) needed[in.b] = true;
        if (in.c >= 0) needed[in.c] = true;
    }
    for (int x = 0; x < tp.n_values; ++x) {
        C.alias[x] = x; C.uses[x] = 0; C.home[x] = -1;
        if (needed[x] && !(tp.dtype[x] == RELAY_F32 || tp.dtype[x] == RELAY_BF16 || tp.dtype[x] == RELAY_BOOL)) return false;   // integer lanes: scalar evaluator
        if (x >= tp.n_in && needed[x]) {
            const relay_instr_t &in = tp.instr[x - tp.n_in];
            if (in.op == RELAY_OP_CAST) {
                const int32_t from = tp.dtype[in.a], to = in.dtype;
                // held as fp32 either way: widening (bf16 -> f32, bool -> float) and same-type casts copy the value
                const bool copy = from == to || to == RELAY_F32 || (from == RELAY_BOOL && to == RELAY_BF16);
                if (copy) C.alias[x] = C.alias[in.a];
            }
        }
    }
    for (int x = tp.n_in; x < tp.n_values; ++x) {
        if (!needed[x] || C.alias[x] != x) continue;
        const relay_instr_t &in = tp.instr[x - tp.n_in];
        if (in.a >= 0) ++C.uses[C.alias[in.a]];
        if (in.b >= 0) ++C.uses[C.alias[in.b]];
        if (in.c >= 0) ++C.uses[C.alias[in.c]];
    }
    for (int k = 0; k < n_out; ++k) ++C.uses[C.alias[out_values[k]]];
    // values used more than once are computed in let order and kept in a temporary
    for (int x = tp.n_in; x < tp.n_values && C.ok; ++x) {
        if (!needed[x] || C.alias[x] != x || C.uses[x] < 2 || C.is_const(x)) continue;
        C.gen(x);
        const int t = C.alloc_temp();
        C.emit(A_STASH, OPD_SLOT + t);
        C.home[x] = t;
        C.acc_holds = x;
    }
    for (int k = 0; k < n_out && C.ok; ++k) {
        C.gen(out_values[k]);
        P.sum_of_out[k] = -1;
        if (colsum[k]) {
            if (P.n_sum == VM_MAXSUM) return false;
            P.sum_of_out[k] = P.n_sum;
            C.emit(A_COLSUM0 + P.n_sum++, 0);
        } else {
            // the store of a bf16 result rounds by itself: a rounding that was emitted just for it is dropped
            if (C.last_op == A_ROUND_BF16 && tp.dtype[out_values[k]] == RELAY_BF16 && C.ok) { --P.code.n; C.acc_holds = -1; }
            C.emit(A_STORE, k);
        }
    }
    if (!C.ok) return false;
    C.finish();
    P.n_temp = C.n_temp; P.n_const = C.n_const;
    memcpy(P.literal, C.literal, sizeof P.literal);
    plan->ok = true;
    plan->n_sum = P.n_sum;
    return true;
}

relay_status_t vm_launch(const VmPlan &plan, const View2D &v, const relay_tensor_t *const *inputs, int n_in, const relay_tensor_t *const *outputs,
                         int n_out, float *partials, int n_slices, cudaStream_t st)
{
    const VmPlanImpl &P = *reinterpret_cast<const VmPlanImpl *>(plan.storage);
    const bool f32 = v.storage == RELAY_F32;
    const int esize = f32 ? 4 : 2;
    VmArgs A{};
    A.rows = v.rows; A.cols = v.cols;
    A.n_full = P.n_full; A.n_fixed = P.n_fixed; A.n_sum = P.n_sum; A.n_temp = P.n_temp; A.n_const = P.n_const;
    memcpy(A.literal, P.literal, sizeof A.literal);
    A.box_cols = (int)std::min<int64_t>(VM_COLS, v.cols);
    A.box_rows = (int)std::min<int64_t>(VM_TILE_ROWS, v.rows);
    A.rows_per_slice = (int)((v.rows + n_slices - 1) / n_slices);
    A.rows_per_slice = (A.rows_per_slice + A.box_rows - 1) / A.box_rows * A.box_rows;      // slices start on tile boundaries
    A.code = P.code;
    A.err = device_error_word();
    if (!A.err) return fail(RELAY_ERR_CUDA, "no device error word");
    BoundsReg br;
    for (int i = 0; i < n_in; ++i) br.add(inputs[i]);
    for (int k = 0; k < n_out; ++k) br.add(outputs[k]);
    br.add(partials, (size_t)P.n_sum * n_slices * v.cols * sizeof(float));
    RELAY_TRY(br.commit(st));
    CUtensorMap tm[VM_MAXFULL];
    memset(tm, 0, sizeof tm);
    for (int i = 0; i < n_in; ++i) {
        A.in_kind[i] = (int8_t)P.in_kind[i]; A.in_slot[i] = (int8_t)P.in_slot[i];
        if (P.in_kind[i] == 0) {
            RELAY_TRY(make_tmap_2d(&tm[P.in_slot[i]], f32, inputs[i]->data, (uint64_t)v.cols, (uint64_t)v.rows, (uint64_t)v.cols, (uint32_t)A.box_cols,
                                   (uint32_t)A.box_rows, false));
        } else {
            A.fixed_ptr[P.in_slot[i]] = inputs[i]->data;
            A.fixed_scalar[P.in_slot[i]] = v.kind[i] == KIND_SCALAR;
        }
    }
    for (int f = P.n_full; f < VM_MAXFULL; ++f) tm[f] = tm[0];
    for (int k = 0; k < n_out; ++k) {
        A.out[k] = outputs[k]->data; A.out_dt[k] = (int8_t)outputs[k]->dtype;
        if (P.sum_of_out[k] >= 0) A.partial[P.sum_of_out[k]] = partials + (size_t)P.sum_of_out[k] * n_slices * v.cols;
    }
    const int row_bytes = A.box_cols * esize, tile_bytes = ((A.box_rows * row_bytes + 127) / 128) * 128;
    const int stage_bytes = P.n_full * tile_bytes;
    A.stages = std::max(2, std::min(4, VM_RING_BYTES / 2 / stage_bytes));     // as many as half the budget holds (two blocks per SM), at least two
    const size_t ring = std::max((size_t)A.stages * stage_bytes, (size_t)VM_TY * (VM_COLS + 1) * sizeof(float));
    const size_t smem = 1024 + (ring + 127) / 128 * 128 + ((size_t)P.n_fixed * VM_COLS * esize + 127) / 128 * 128 +
                        ((size_t)(P.n_temp * 4 * VM_THREADS + P.n_const) * 16 + 127) / 128 * 128 + 256;
    const dim3 grid((unsigned)((v.cols + VM_COLS - 1) / VM_COLS), (unsigned)((v.rows + A.rows_per_slice - 1) / A.rows_per_slice));
    if (f32) {
        RELAY_CUDA(cudaFuncSetAttribute(ewise_vm_kernel<float, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        RELAY_CUDA(launch_pdl(ewise_vm_kernel<float, false>, grid, dim3(VM_THREADS), smem, st, tm[0], tm[1], tm[2], tm[3], A));
    } else {
        RELAY_CUDA(cudaFuncSetAttribute(ewise_vm_kernel<__nv_bfloat16, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        RELAY_CUDA(launch_pdl(ewise_vm_kernel<__nv_bfloat16, true>, grid, dim3(VM_THREADS), smem, st, tm[0], tm[1], tm[2], tm[3], A));
    }
    return check_launch("ewise_vm");
}

int vm_grid_slices(const View2D &v, int n_slices_wanted)
{
    // the slices the launch really makes (whole tiles per slice)
    const int box_rows = (int)std::min<int64_t>(VM_TILE_ROWS, v.rows);
    int rps = (int)((v.rows + n_slices_wanted - 1) / n_slices_wanted);
    rps = (rps + box_rows - 1) / box_rows * box_rows;
    return (int)((v.rows + rps - 1) / rps);
}

}  // namespace relay
