// Vectorised evaluator for elementwise programs that have no pre-compiled body (Fig. 1 BinOp / UnaryOp productions,
// Fig. 5 typing rules; operator fusion, Section 5.2): any straight-line program over the collapsed 2-D view
// [rows, cols] whose inputs are full-shape tensors, tensors constant down the rows, or scalars of one float storage
// type, with unreduced results and column sums.
//
// Host: the let-list is turned into a small STACK program.  Values used once are evaluated in place as expression
// trees; values used several times are computed once, stay on the stack, and are copied to the top where needed.
// Operands of a stack instruction are implicit (the top of the stack), so the device code can keep the stack in
// REGISTERS: the interpreter dispatches on (stack height, opcode) and every case indexes the stack with constants.
//
// Device: a block owns 256 columns x a slice of rows.  One producer thread streams 8-row tiles of every full-shape
// input into a shared-memory ring with TMA (the bytes in flight live in shared memory, not in registers); 256
// consumer threads each interpret the program once per tile on 8 elements (a 16-byte vector of bf16, two of f32),
// taking operands from shared memory; operands that are constant down the rows sit in shared memory as one row.
// Column sums: per-thread accumulators -> fixed-order combine in shared memory -> one partial per row slice ->
// colsum_finalize_kernel (no float atomics: reruns are bit-identical).
#include <algorithm>
#include <cstring>

#include "ewise_host.h"
#include "ewise_kernels.cuh"
#include "ewise_prog.h"
#include "tc_common.cuh"

namespace relay {

relay_status_t make_tmap_2d(CUtensorMap *m, bool f32, const void *base, uint64_t inner, uint64_t outer, uint64_t row_stride,
                            uint32_t box_inner, uint32_t box_outer, bool swizzle128);

namespace {

constexpr int VM_TX = 32, VM_TY = 8, VM_E = 8;           // 256 consumer threads, 8 elements each per tile
constexpr int VM_COLS = VM_TX * VM_E;                    // columns per block
constexpr int VM_STAGES = 4;
constexpr int VM_MAXSP = 8, VM_MAXCODE = 96, VM_MAXFULL = 4, VM_MAXFIXED = 4, VM_MAXSUM = 3;
constexpr int VM_THREADS = VM_TX * VM_TY + 32;           // + the producer warp

// stack opcodes: 0 .. RELAY_OP_COUNT_-1 are the program's own operators (operands on top of the stack)
enum : int { S_PUSH_IN = 32, S_PUSH_CONST, S_PICK, S_STORE, S_COLSUM, S_ROUND_BF16, S_TO_BOOL, S_POP };

struct VmCode {
    int32_t n;
    uint8_t op[VM_MAXCODE], arg[VM_MAXCODE], sp[VM_MAXCODE];   // sp: stack height BEFORE the instruction
    float imm[VM_MAXCODE];
};

struct VmArgs {
    const void *fixed_ptr[VM_MAXFIXED];
    int8_t fixed_scalar[VM_MAXFIXED];
    int8_t in_kind[RELAY_MAX_INPUTS], in_slot[RELAY_MAX_INPUTS];   // kind 0: full-shape (slot = ring slot), 1: constant down the rows
    void *out[RELAY_MAX_OUTPUTS];
    int8_t out_dt[RELAY_MAX_OUTPUTS];
    float *partial[VM_MAXSUM];
    int64_t rows, cols;
    int32_t rows_per_slice, n_full, n_fixed, n_sum;
    int32_t box_cols, box_rows;        // TMA box (min(256, cols) x min(8, rows))
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

template <typename T> __device__ __forceinline__ void vm_load(const char *row, int tx, float (&f)[VM_E])
{
    if constexpr (sizeof(T) == 2) {
        unpack(*reinterpret_cast<const uint4 *>(row + tx * 16), f);
    } else {
        float lo[4], hi[4];
        unpack(*reinterpret_cast<const uint4 *>(row + tx * 16), lo);
        unpack(*reinterpret_cast<const uint4 *>(row + 512 + tx * 16), hi);
#pragma unroll
        for (int v = 0; v < 4; ++v) { f[v] = lo[v]; f[4 + v] = hi[v]; }
    }
}

// stores `n` consecutive result elements (n = 8 or 4) starting at element index `at` of an output of type `dt`
template <int N> __device__ __forceinline__ void vm_store_run(void *out, int dt, int64_t at, const float *f)
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
            *reinterpret_cast<uint2 *>((__nv_bfloat16 *)out + at) = make_uint2(pack2(f[0], f[1]), pack2(f[2], f[3]));
        }
    } else {   // bool: one byte per element
        uint32_t w[N / 4];
#pragma unroll
        for (int q = 0; q < N / 4; ++q)
            w[q] = (f[4 * q] != 0.0f ? 1u : 0u) | (f[4 * q + 1] != 0.0f ? 0x100u : 0u) | (f[4 * q + 2] != 0.0f ? 0x10000u : 0u) |
                   (f[4 * q + 3] != 0.0f ? 0x1000000u : 0u);
        if constexpr (N == 8) *reinterpret_cast<uint2 *>((uint8_t *)out + at) = make_uint2(w[0], w[1]);
        else *reinterpret_cast<uint32_t *>((uint8_t *)out + at) = w[0];
    }
}

struct VmThread {
    const char *stage;      // ring stage of the current tile
    const char *fixed;      // rows of the operands that are constant down the rows
    int tx, ty;
    int tile_bytes, row_bytes;
    int64_t row, col0;      // this thread's row of the tile and the block's first column
};

template <typename T, bool FAST>
__device__ __forceinline__ float vm_unary(int op, float x)
{
    switch (op) {
    case RELAY_OP_NEG: return -x;
    case RELAY_OP_SQ: return x * x;
    case RELAY_OP_RELU: return fmaxf(x, 0.0f);
    case RELAY_OP_TANH: return tanh_<FAST>(x);
    case RELAY_OP_SIGMOID: return sigmoid_<FAST>(x);
    case RELAY_OP_EXP: return FAST ? __expf(x) : expf(x);
    case RELAY_OP_LOG: return FAST ? __logf(x) : logf(x);
    case S_ROUND_BF16: return round_bf16(x);
    default: return x != 0.0f ? 1.0f : 0.0f;   // S_TO_BOOL
    }
}
template <bool FAST>
__device__ __forceinline__ float vm_binary(int op, float x, float y)
{
    switch (op) {
    case RELAY_OP_ADD: return x + y;
    case RELAY_OP_SUB: return x - y;
    case RELAY_OP_MUL: return x * y;
    case RELAY_OP_DIV: return FAST ? __fdividef(x, y) : x / y;
    case RELAY_OP_NE: return x != y ? 1.0f : 0.0f;
    case RELAY_OP_EQ: return x == y ? 1.0f : 0.0f;
    case RELAY_OP_LT: return x < y ? 1.0f : 0.0f;
    case RELAY_OP_LE: return x <= y ? 1.0f : 0.0f;
    case RELAY_OP_GT: return x > y ? 1.0f : 0.0f;
    case RELAY_OP_GE: return x >= y ? 1.0f : 0.0f;
    case RELAY_OP_MAX: return fmaxf(x, y);
    default: return fminf(x, y);               // RELAY_OP_MIN
    }
}

// one stack instruction at stack height SP (every index into `s` is a compile-time constant)
template <int SP, typename T, bool FAST>
__device__ __forceinline__ void vm_exec(int op, int arg, float imm, float (&s)[VM_MAXSP][VM_E], float (&acc)[VM_MAXSUM][VM_E],
                                        const VmArgs &A, const VmThread &th)
{
    if (op == S_PUSH_IN) {
        if constexpr (SP < VM_MAXSP) {
            const int slot = A.in_slot[arg];
            const char *row = A.in_kind[arg] == 0 ? th.stage + slot * th.tile_bytes + th.ty * th.row_bytes : th.fixed + slot * th.row_bytes;
            vm_load<T>(row, th.tx, s[SP]);
        }
    } else if (op == S_PUSH_CONST) {
        if constexpr (SP < VM_MAXSP) {
#pragma unroll
            for (int v = 0; v < VM_E; ++v) s[SP][v] = imm;
        }
    } else if (op == S_PICK) {
        if constexpr (SP >= 1 && SP < VM_MAXSP) {
#pragma unroll
            for (int q = 0; q < SP; ++q)
                if (arg == q) {
#pragma unroll
                    for (int v = 0; v < VM_E; ++v) s[SP][v] = s[SP - 1 - q][v];
                }
        }
    } else if (op == S_STORE) {
        if constexpr (SP >= 1) {
            void *out = A.out[arg];
            const int dt = A.out_dt[arg];
            if constexpr (sizeof(T) == 2) {
                if (th.col0 + th.tx * 8 < A.cols) vm_store_run<8>(out, dt, th.row * A.cols + th.col0 + th.tx * 8, s[SP - 1]);
            } else {
                if (th.col0 + th.tx * 4 < A.cols) vm_store_run<4>(out, dt, th.row * A.cols + th.col0 + th.tx * 4, s[SP - 1]);
                if (th.col0 + 128 + th.tx * 4 < A.cols) vm_store_run<4>(out, dt, th.row * A.cols + th.col0 + 128 + th.tx * 4, s[SP - 1] + 4);
            }
        }
    } else if (op == S_COLSUM) {
        if constexpr (SP >= 1) {
#pragma unroll
            for (int k = 0; k < VM_MAXSUM; ++k)
                if (arg == k) {
#pragma unroll
                    for (int v = 0; v < VM_E; ++v) acc[k][v] += s[SP - 1][v];
                }
        }
    } else if (op == S_POP) {
    } else if (op == RELAY_OP_SELECT) {
        if constexpr (SP >= 3) {
#pragma unroll
            for (int v = 0; v < VM_E; ++v) s[SP - 3][v] = s[SP - 3][v] != 0.0f ? s[SP - 2][v] : s[SP - 1][v];
        }
    } else if (op == RELAY_OP_NEG || op == RELAY_OP_SQ || op == RELAY_OP_RELU || op == RELAY_OP_TANH || op == RELAY_OP_SIGMOID ||
               op == RELAY_OP_EXP || op == RELAY_OP_LOG || op == S_ROUND_BF16 || op == S_TO_BOOL) {
        if constexpr (SP >= 1) {
#pragma unroll
            for (int v = 0; v < VM_E; ++v) s[SP - 1][v] = vm_unary<T, FAST>(op, s[SP - 1][v]);
        }
    } else {
        if constexpr (SP >= 2) {
#pragma unroll
            for (int v = 0; v < VM_E; ++v) s[SP - 2][v] = vm_binary<FAST>(op, s[SP - 2][v], s[SP - 1][v]);
        }
    }
}

template <typename T, bool FAST>
__global__ void __launch_bounds__(VM_THREADS, 2)
ewise_vm_kernel(const __grid_constant__ CUtensorMap tm0, const __grid_constant__ CUtensorMap tm1, const __grid_constant__ CUtensorMap tm2,
                const __grid_constant__ CUtensorMap tm3, const __grid_constant__ VmArgs A)
{
    extern __shared__ uint8_t vm_smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(vm_smem_raw) + 1023) & ~uintptr_t(1023));
    const int row_bytes = A.box_cols * (int)sizeof(T), tile_bytes = ((A.box_rows * row_bytes + 127) / 128) * 128;
    const int stage_bytes = A.n_full * tile_bytes;
    uint8_t *fixed = smem + VM_STAGES * stage_bytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(fixed + ((A.n_fixed * VM_COLS * (int)sizeof(T) + 127) / 128) * 128);
    uint64_t *full = bars, *empty = bars + VM_STAGES;
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + 2 * VM_STAGES);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t col0 = (int64_t)blockIdx.x * VM_COLS;
    const int64_t r0 = (int64_t)blockIdx.y * A.rows_per_slice, r1 = min(A.rows, r0 + (int64_t)A.rows_per_slice);
    const int n_tiles = r1 > r0 ? (int)((r1 - r0 + A.box_rows - 1) / A.box_rows) : 0;

    if (tid == 0) {
        for (int s = 0; s < VM_STAGES; ++s) { tc::mbar_init(&full[s], 1); tc::mbar_init(&empty[s], VM_TY); }
        *abort_flag = 0;
        tc::fence_barrier_init();
        tc::prefetch_tmap(&tm0);
    }
    pdl_wait();
    // operands that are constant down the rows: one row of this block's columns each (a scalar fills the row)
    if (tid < VM_COLS) {
        for (int g = 0; g < A.n_fixed; ++g) {
            const T *p = (const T *)A.fixed_ptr[g];
            T val = T(0.0f);
            if (A.fixed_scalar[g]) val = p[0];
            else if (col0 + tid < A.cols) val = p[col0 + tid];
            reinterpret_cast<T *>(fixed)[g * VM_COLS + tid] = val;
        }
    }
    __syncthreads();

    float acc[VM_MAXSUM][VM_E];
#pragma unroll
    for (int k = 0; k < VM_MAXSUM; ++k)
#pragma unroll
        for (int v = 0; v < VM_E; ++v) acc[k][v] = 0.0f;

    if (warp == VM_TY) {
        // producer: every lane runs the loop, one elected lane issues
        const CUtensorMap *tms[VM_MAXFULL] = {&tm0, &tm1, &tm2, &tm3};
        for (int t = 0; t < n_tiles; ++t) {
            const int s = t % VM_STAGES;
            if (!__all_sync(0xffffffffu, tc::mbar_wait(&empty[s], ((t / VM_STAGES) & 1) ^ 1, abort_flag, A.err, tc::ERR_WAIT_EMPTY))) break;
            if (tc::elect_one()) {
                tc::mbar_expect_tx(&full[s], (uint32_t)(A.n_full * A.box_rows * row_bytes));
#pragma unroll
                for (int f = 0; f < VM_MAXFULL; ++f)
                    if (f < A.n_full) tc::tma_load_2d(smem + s * stage_bytes + f * tile_bytes, tms[f], &full[s], (int)col0, (int)(r0 + (int64_t)t * A.box_rows));
            }
            __syncwarp();
        }
    } else {
        VmThread th;
        th.fixed = reinterpret_cast<const char *>(fixed);
        th.tx = lane; th.ty = warp;
        th.tile_bytes = tile_bytes; th.row_bytes = row_bytes;
        th.col0 = col0;
        const bool col_live = col0 + vm_col<T>(lane, 0) < A.cols;     // a thread's first column decides (its second run is checked at the store)
        float s[VM_MAXSP][VM_E];
        for (int t = 0; t < n_tiles; ++t) {
            const int st = t % VM_STAGES;
            int ok = 1;
            if (lane == 0) ok = tc::mbar_wait(&full[st], (t / VM_STAGES) & 1, abort_flag, A.err, tc::ERR_WAIT_FULL) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            th.stage = reinterpret_cast<const char *>(smem + st * stage_bytes);
            th.row = r0 + (int64_t)t * A.box_rows + warp;
            if (warp < A.box_rows && th.row < r1 && col_live) {
#pragma unroll 1
                for (int pc = 0; pc < A.code.n; ++pc) {
                    const int op = A.code.op[pc], arg = A.code.arg[pc];
                    const float imm = A.code.imm[pc];
                    switch (A.code.sp[pc]) {
                    case 0: vm_exec<0, T, FAST>(op, arg, imm, s, acc, A, th); break;
                    case 1: vm_exec<1, T, FAST>(op, arg, imm, s, acc, A, th); break;
                    case 2: vm_exec<2, T, FAST>(op, arg, imm, s, acc, A, th); break;
                    case 3: vm_exec<3, T, FAST>(op, arg, imm, s, acc, A, th); break;
                    case 4: vm_exec<4, T, FAST>(op, arg, imm, s, acc, A, th); break;
                    case 5: vm_exec<5, T, FAST>(op, arg, imm, s, acc, A, th); break;
                    case 6: vm_exec<6, T, FAST>(op, arg, imm, s, acc, A, th); break;
                    case 7: vm_exec<7, T, FAST>(op, arg, imm, s, acc, A, th); break;
                    default: vm_exec<8, T, FAST>(op, arg, imm, s, acc, A, th); break;
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
            if (warp < VM_TY) {
#pragma unroll
                for (int v = 0; v < VM_E; ++v) sm[warp][vm_col<T>(lane, v)] = acc[k][v];
            }
            __syncthreads();
            if (tid < VM_COLS && col0 + tid < A.cols) {
                float t = 0.0f;
#pragma unroll
                for (int j = 0; j < VM_TY; ++j) t += sm[j][tid];
                A.partial[k][(int64_t)blockIdx.y * A.cols + col0 + tid] = t;
            }
            __syncthreads();
        }
    }
}

}  // namespace

// =================================================================================================
// host: let-list -> stack program
// =================================================================================================
namespace {

struct Compiler {
    const TypedProgram &tp;
    VmCode &code;
    int alias[kMaxValues];       // value this one is a plain copy of (casts that change nothing), or itself
    int uses[kMaxValues];
    int pos[kMaxValues];         // stack position of a value kept on the stack, -1 otherwise
    int sp = 0, max_sp = 0;
    bool ok = true;

    Compiler(const TypedProgram &t, VmCode &c) : tp(t), code(c) { code.n = 0; }

    void emit(int op, int arg, float imm, int delta)
    {
        if (code.n >= VM_MAXCODE) { ok = false; return; }
        code.op[code.n] = (uint8_t)op; code.arg[code.n] = (uint8_t)arg; code.sp[code.n] = (uint8_t)sp; code.imm[code.n] = imm;
        ++code.n;
        sp += delta;
        max_sp = std::max(max_sp, sp);
        if (sp > VM_MAXSP || sp < 0) ok = false;
    }
    static bool floatlike(int32_t dt) { return dt == RELAY_F32 || dt == RELAY_BF16 || dt == RELAY_BOOL; }

    // pushes value v
    void push(int v, int depth = 0)
    {
        if (!ok || depth > 40) { ok = false; return; }
        v = alias[v];
        if (v < tp.n_in) { emit(S_PUSH_IN, v, 0.0f, +1); return; }
        if (pos[v] >= 0) { emit(S_PICK, sp - 1 - pos[v], 0.0f, +1); return; }
        compute(v, depth);
    }
    // evaluates instruction value v onto the top of the stack
    void compute(int v, int depth)
    {
        const relay_instr_t &in = tp.instr[v - tp.n_in];
        if (in.op == RELAY_OP_CONST) {
            float c = (float)in.imm;
            if (in.dtype == RELAY_BF16) c = __bfloat162float(__float2bfloat16_rn(c));
            else if (in.dtype == RELAY_BOOL) c = in.imm != 0.0 ? 1.0f : 0.0f;
            emit(S_PUSH_CONST, 0, c, +1);
            return;
        }
        if (in.op == RELAY_OP_CAST) {       // a cast that is not a plain copy
            push(in.a, depth + 1);
            emit(in.dtype == RELAY_BF16 ? S_ROUND_BF16 : S_TO_BOOL, 0, 0.0f, 0);
            return;
        }
        if (in.a >= 0) push(in.a, depth + 1);
        if (in.b >= 0) push(in.b, depth + 1);
        if (in.c >= 0) push(in.c, depth + 1);
        const int ar = (in.a >= 0) + (in.b >= 0) + (in.c >= 0);
        emit(in.op, 0, 0.0f, 1 - ar);
        // a value of type bf16 holds a bf16 number (comparisons and select of already rounded values need no rounding)
        if (in.dtype == RELAY_BF16 && in.op != RELAY_OP_SELECT && in.op != RELAY_OP_MAX && in.op != RELAY_OP_MIN && in.op != RELAY_OP_NEG &&
            in.op != RELAY_OP_RELU)
            emit(S_ROUND_BF16, 0, 0.0f, 0);
    }
};

}  // namespace

struct VmPlanImpl {
    VmCode code;
    int in_kind[RELAY_MAX_INPUTS], in_slot[RELAY_MAX_INPUTS];
    int n_full = 0, n_fixed = 0, n_sum = 0;
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
        C.alias[x] = x; C.uses[x] = 0; C.pos[x] = -1;
        if (needed[x] && !Compiler::floatlike(tp.dtype[x])) return false;           // integer lanes: scalar evaluator
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
    // values used more than once are computed in let order and stay on the stack
    for (int x = tp.n_in; x < tp.n_values && C.ok; ++x) {
        if (!needed[x] || C.alias[x] != x || C.uses[x] < 2 || tp.instr[x - tp.n_in].op == RELAY_OP_CONST) continue;
        C.compute(x, 0);
        C.pos[x] = C.sp - 1;
    }
    for (int k = 0; k < n_out && C.ok; ++k) {
        C.push(out_values[k]);
        P.sum_of_out[k] = -1;
        if (colsum[k]) {
            if (P.n_sum == VM_MAXSUM) return false;
            P.sum_of_out[k] = P.n_sum;
            C.emit(S_COLSUM, P.n_sum++, 0.0f, -1);
        } else {
            C.emit(S_STORE, k, 0.0f, -1);
        }
    }
    if (!C.ok) return false;
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
    A.n_full = P.n_full; A.n_fixed = P.n_fixed; A.n_sum = P.n_sum;
    A.box_cols = (int)std::min<int64_t>(VM_COLS, v.cols);
    A.box_rows = (int)std::min<int64_t>(VM_TY, v.rows);
    A.rows_per_slice = (int)((v.rows + n_slices - 1) / n_slices);
    A.rows_per_slice = (A.rows_per_slice + A.box_rows - 1) / A.box_rows * A.box_rows;      // slices start on tile boundaries
    A.code = P.code;
    A.err = device_error_word();
    if (!A.err) return fail(RELAY_ERR_CUDA, "no device error word");
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
    const size_t ring = (size_t)VM_STAGES * P.n_full * tile_bytes;
    const size_t smem = 1024 + std::max(ring, (size_t)VM_TY * (VM_COLS + 1) * sizeof(float)) + ((size_t)P.n_fixed * VM_COLS * esize + 127) / 128 * 128 + 256;
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
    const int box_rows = (int)std::min<int64_t>(VM_TY, v.rows);
    int rps = (int)((v.rows + n_slices_wanted - 1) / n_slices_wanted);
    rps = (rps + box_rows - 1) / box_rows * box_rows;
    return (int)((v.rows + rps - 1) / rps);
}

}  // namespace relay
