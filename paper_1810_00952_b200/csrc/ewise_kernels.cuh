// Device-side building blocks of the memory-bound groups: 128-bit vector access, scalar
// operators, the pre-compiled group bodies ("type-specialised operator instances") and the
// generic in-kernel evaluator for programs that have no pre-compiled body.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "../../include/relay_b200.h"
#include "common.h"

namespace relay {

// ---- scalar operators -------------------------------------------------------------------------
// FAST = hardware approximations (one MUFU op; relative error about 2^-11), used where the
// result is stored in bf16; otherwise the accurate fp32 routines.
template <bool FAST>
__device__ __forceinline__ float tanh_(float x)
{
    if constexpr (FAST) {
        float y;
        asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
        return y;
    } else {
        return tanhf(x);
    }
}
template <bool FAST>
__device__ __forceinline__ float sigmoid_(float x)
{
    if constexpr (FAST) return fmaf(0.5f, tanh_<true>(0.5f * x), 0.5f);
    else return 1.0f / (1.0f + expf(-x));
}
__device__ __forceinline__ float round_bf16(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

template <bool FAST>
__device__ __forceinline__ float act_fwd(float z, int act)
{
    switch (act) {
    case RELAY_ACT_RELU: return fmaxf(z, 0.0f);
    case RELAY_ACT_TANH: return tanh_<FAST>(z);
    case RELAY_ACT_SIGMOID: return sigmoid_<FAST>(z);
    default: return z;
    }
}
// derivative of the activation written through the saved output y
__device__ __forceinline__ float act_grad_from_output(float y, int act)
{
    switch (act) {
    case RELAY_ACT_RELU: return y > 0.0f ? 1.0f : 0.0f;
    case RELAY_ACT_TANH: return 1.0f - y * y;
    case RELAY_ACT_SIGMOID: return y * (1.0f - y);
    default: return 1.0f;
    }
}

// ---- 16-byte vectors ----------------------------------------------------------------------------
template <typename T> struct VecN;
template <> struct VecN<__nv_bfloat16> { static constexpr int N = 8; };
template <> struct VecN<float> { static constexpr int N = 4; };

__device__ __forceinline__ void unpack(const uint4 &r, float (&f)[8])
{
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}
__device__ __forceinline__ void unpack(const uint4 &r, float (&f)[4])
{
    f[0] = __uint_as_float(r.x); f[1] = __uint_as_float(r.y); f[2] = __uint_as_float(r.z); f[3] = __uint_as_float(r.w);
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}
__device__ __forceinline__ uint4 pack(const float (&f)[8])
{
    return make_uint4(pack2(f[0], f[1]), pack2(f[2], f[3]), pack2(f[4], f[5]), pack2(f[6], f[7]));
}
__device__ __forceinline__ uint4 pack(const float (&f)[4])
{
    return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
}
// streaming 128-bit access: data is touched once, keep it out of L1
__device__ __forceinline__ uint4 ld_stream(const void *p)
{
    uint4 r;
    if (!relay_in_bounds(p, 16)) return make_uint4(0, 0, 0, 0);
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}
__device__ __forceinline__ void st_stream(void *p, const uint4 &r)
{
    if (!relay_in_bounds(p, 16)) return;
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(r.x), "r"(r.y), "r"(r.z), "r"(r.w) : "memory");
}

// ---- scalar typed access (generic evaluator) ----------------------------------------------------
// A program value is held in the lane of its base type: floats (and Bool, as 0 / 1) in `f`, IntType values in `i`
// as a 64-bit integer, so that integers are exact over their whole range whatever casts they pass through.
union Val { float f; long long i; };
__device__ __forceinline__ bool is_int_type(int dt) { return dt == RELAY_I32 || dt == RELAY_I64; }

__device__ __forceinline__ Val load_value(const void *p, int64_t i, int dt)
{
    Val v;
    v.i = 0;
    const size_t esz = dt == RELAY_BF16 ? 2 : dt == RELAY_I64 ? 8 : dt == RELAY_BOOL ? 1 : 4;
    if (!relay_in_bounds((const char *)p + i * esz, esz)) return v;
    switch (dt) {
    case RELAY_F32: v.f = ((const float *)p)[i]; break;
    case RELAY_BF16: v.f = __bfloat162float(((const __nv_bfloat16 *)p)[i]); break;
    case RELAY_I32: v.i = ((const int32_t *)p)[i]; break;
    case RELAY_I64: v.i = ((const int64_t *)p)[i]; break;
    default: v.f = ((const uint8_t *)p)[i] ? 1.0f : 0.0f; break;
    }
    return v;
}
__device__ __forceinline__ void store_value(void *p, int64_t i, int dt, Val v)
{
    const size_t esz = dt == RELAY_BF16 ? 2 : dt == RELAY_I64 ? 8 : dt == RELAY_BOOL ? 1 : 4;
    if (!relay_in_bounds((const char *)p + i * esz, esz)) return;
    switch (dt) {
    case RELAY_F32: ((float *)p)[i] = v.f; break;
    case RELAY_BF16: ((__nv_bfloat16 *)p)[i] = __float2bfloat16_rn(v.f); break;
    case RELAY_I32: ((int32_t *)p)[i] = (int32_t)v.i; break;
    case RELAY_I64: ((int64_t *)p)[i] = v.i; break;
    default: ((uint8_t *)p)[i] = v.f != 0.0f ? 1 : 0; break;
    }
}

// ---- generic evaluator --------------------------------------------------------------------------
struct DevProgram {
    int32_t n_in, n_instr, rank, pad_;
    int64_t shape[RELAY_MAX_RANK];
    int64_t in_stride[RELAY_MAX_INPUTS][RELAY_MAX_RANK];  // element stride per output axis, 0 where broadcast
    const void *in_ptr[RELAY_MAX_INPUTS];
    int8_t in_dtype[RELAY_MAX_INPUTS];
    int8_t op[RELAY_MAX_INSTR], a[RELAY_MAX_INSTR], b[RELAY_MAX_INSTR], c[RELAY_MAX_INSTR], dt[RELAY_MAX_INSTR];
    double imm[RELAY_MAX_INSTR];
};

constexpr int kDevMaxValues = RELAY_MAX_INPUTS + RELAY_MAX_INSTR;

// cast (Fig. 1): float -> int truncates toward zero (saturating at the ends of the integer type), int -> float rounds
// once to nearest even, int -> int keeps the low bits, anything -> Bool is "!= 0"
__device__ __forceinline__ Val cast_value(Val x, int from, int to)
{
    Val r;
    r.i = 0;
    if (is_int_type(from)) {
        switch (to) {
        case RELAY_I32: r.i = (int32_t)x.i; break;
        case RELAY_I64: r.i = x.i; break;
        case RELAY_F32: r.f = __ll2float_rn(x.i); break;
        case RELAY_BF16: r.f = __bfloat162float(__ll2bfloat16_rn(x.i)); break;
        default: r.f = x.i != 0 ? 1.0f : 0.0f; break;
        }
    } else {
        switch (to) {
        case RELAY_I32: r.i = __float2int_rz(x.f); break;
        case RELAY_I64: r.i = __float2ll_rz(x.f); break;
        case RELAY_BF16: r.f = round_bf16(x.f); break;
        case RELAY_BOOL: r.f = x.f != 0.0f ? 1.0f : 0.0f; break;
        default: r.f = x.f; break;
        }
    }
    return r;
}

// evaluates every value of the program at the output multi-index idx[]
__device__ __forceinline__ void eval_program(const DevProgram &P, const int64_t *idx, Val *vals)
{
    for (int i = 0; i < P.n_in; ++i) {
        int64_t off = 0;
        for (int d = 0; d < P.rank; ++d) off += idx[d] * P.in_stride[i][d];
        vals[i] = load_value(P.in_ptr[i], off, P.in_dtype[i]);
    }
    for (int j = 0; j < P.n_instr; ++j) {
        const int op = P.op[j], dt = P.dt[j];
        Val out;
        out.i = 0;
        if (op == RELAY_OP_CAST) {
            const int src = P.a[j];
            out = cast_value(vals[src], src < P.n_in ? P.in_dtype[src] : P.dt[src - P.n_in], dt);
        } else if (op == RELAY_OP_CONST) {
            if (is_int_type(dt)) out.i = (long long)P.imm[j];
            else { out.f = (float)P.imm[j]; out = cast_value(out, RELAY_F32, dt); }
        } else if (op == RELAY_OP_SELECT) {
            out = vals[P.a[j]].f != 0.0f ? vals[P.b[j]] : vals[P.c[j]];
        } else {
            const float x = P.a[j] >= 0 ? vals[P.a[j]].f : 0.0f;
            const float y = P.b[j] >= 0 ? vals[P.b[j]].f : 0.0f;
            float r;
            switch (op) {
            case RELAY_OP_ADD: r = x + y; break;
            case RELAY_OP_SUB: r = x - y; break;
            case RELAY_OP_MUL: r = x * y; break;
            case RELAY_OP_DIV: r = x / y; break;
            case RELAY_OP_NEG: r = -x; break;
            case RELAY_OP_SQ: r = x * x; break;
            case RELAY_OP_NE: r = x != y ? 1.0f : 0.0f; break;
            case RELAY_OP_EQ: r = x == y ? 1.0f : 0.0f; break;
            case RELAY_OP_LT: r = x < y ? 1.0f : 0.0f; break;
            case RELAY_OP_LE: r = x <= y ? 1.0f : 0.0f; break;
            case RELAY_OP_GT: r = x > y ? 1.0f : 0.0f; break;
            case RELAY_OP_GE: r = x >= y ? 1.0f : 0.0f; break;
            case RELAY_OP_RELU: r = fmaxf(x, 0.0f); break;
            case RELAY_OP_TANH: r = tanhf(x); break;
            case RELAY_OP_SIGMOID: r = 1.0f / (1.0f + expf(-x)); break;
            case RELAY_OP_EXP: r = expf(x); break;
            case RELAY_OP_LOG: r = logf(x); break;
            case RELAY_OP_MAX: r = fmaxf(x, y); break;
            default: r = fminf(x, y); break;
            }
            out.f = dt == RELAY_BF16 ? round_bf16(r) : r;   // a value of type bf16 holds a bf16 number
        }
        vals[P.n_in + j] = out;
    }
}

__device__ __forceinline__ void unravel(int64_t lin, int rank, const int64_t *shape, int64_t *idx)
{
    for (int d = rank - 1; d >= 0; --d) {
        idx[d] = lin % shape[d];
        lin /= shape[d];
    }
}

// operand kinds of the collapsed 2-D view [rows, cols]
enum : int { KIND_FULL = 0, KIND_ROWVEC = 1, KIND_SCALAR = 2 };

// ---- pre-compiled group bodies --------------------------------------------------------------------
// A body maps NIN loaded operands to NOUT results for one element.  kColSum[k] says whether
// result k is summed over rows (true) or stored unreduced (false); kind(i) is the operand kind
// this instance was compiled for (full-shape, constant down the rows, or scalar).

// out = tanh(a*x + b) + x                                   inputs: x, a, b
struct BodyTanhAffineResidualFwd {
    static constexpr int NIN = 3, NOUT = 1;
    __host__ __device__ static constexpr bool col_sum(int) { return false; }
    __host__ __device__ static constexpr int kind(int i) { return i == 0 ? KIND_FULL : KIND_ROWVEC; }
    template <bool FAST>
    __device__ __forceinline__ static void apply(const float (&in)[NIN], float (&out)[NOUT], int)
    {
        out[0] = tanh_<FAST>(fmaf(in[1], in[0], in[2])) + in[0];
    }
};

// gradient group of the above for upstream dout              inputs: dout, x, a, b
//   s = 1 - tanh(a*x+b)^2;  dx = dout*(a*s+1);  da = sum_rows dout*s*x;  db = sum_rows dout*s
struct BodyTanhAffineResidualGrad {
    static constexpr int NIN = 4, NOUT = 3;
    __host__ __device__ static constexpr bool col_sum(int k) { return k >= 1; }
    __host__ __device__ static constexpr int kind(int i) { return i <= 1 ? KIND_FULL : KIND_ROWVEC; }
    template <bool FAST>
    __device__ __forceinline__ static void apply(const float (&in)[NIN], float (&out)[NOUT], int)
    {
        float t = tanh_<FAST>(fmaf(in[2], in[1], in[3]));
        float s = fmaf(-t, t, 1.0f);
        float ds = in[0] * s;
        out[0] = in[0] * fmaf(in[2], s, 1.0f);
        out[1] = ds * in[1];
        out[2] = ds;
    }
};

// dZ = dy (.) act'(y), column sum of dZ (bias gradient)       inputs: dy, y; `act` at run time
struct BodyActGrad {
    static constexpr int NIN = 2, NOUT = 2;
    __host__ __device__ static constexpr bool col_sum(int k) { return k == 1; }
    __host__ __device__ static constexpr int kind(int) { return KIND_FULL; }
    template <bool FAST>
    __device__ __forceinline__ static void apply(const float (&in)[NIN], float (&out)[NOUT], int act)
    {
        float dz = in[0] * act_grad_from_output(in[1], act);
        if constexpr (FAST) dz = round_bf16(dz);   // bf16 storage: dZ is a bf16 value; db sums what is stored
        out[0] = dz;
        out[1] = dz;
    }
};

// identity body for standalone column reductions              inputs: x
struct BodyIdentityColSum {
    static constexpr int NIN = 1, NOUT = 1;
    __host__ __device__ static constexpr bool col_sum(int) { return true; }
    __host__ __device__ static constexpr int kind(int) { return KIND_FULL; }
    template <bool FAST>
    __device__ __forceinline__ static void apply(const float (&in)[NIN], float (&out)[NOUT], int)
    {
        out[0] = in[0];
    }
};

template <int NIN, int NOUT>
struct Args2D {
    const void *in[NIN];
    void *out[NOUT];        // unreduced results (storage type T); unused for summed results
    float *partial[NOUT];   // [n_slices][cols] fp32 partial column sums for summed results (launches without clusters)
    float *final[NOUT];     // cluster launches: the finished column sums, [cols] fp32 ...
    float scale[NOUT];      // ... times this factor
    int64_t rows, cols;
    int rows_per_slice;
    int aux;                // body-specific run-time attribute (e.g. activation code)
};

}  // namespace relay
