// Bodies compiled at run time for fused elementwise groups that have no pre-compiled body.
//
// The paper's compiler fuses a chain of elementwise operators into ONE kernel that is generated for that chain
// (Section 4.1: fusion of an operator group into a single type-specialised instance).  The pre-compiled bodies of
// ewise_kernels.cuh are four such instances fixed at build time; this file makes one for ANY straight-line program over
// the collapsed 2-D view (same class of groups as the vectorised interpreter of ewise_vm.cu): the let-list is written out
// as the per-element body of a CUDA kernel with the structure of ewise2d_kernel (16-byte streaming loads, operands that
// are constant down the rows kept in registers, four rows in flight per thread, column sums as per-thread accumulators ->
// shared-memory combine -> per-slice partials), compiled for sm_100a by NVRTC, loaded as a module and cached by its text.
// The compiler library is looked up at run time; where it is missing (or in the bounds-check build, whose checks the
// generated code does not carry) the group runs on the interpreter instead -- on the GPU either way.
#include <cuda.h>
#include <dlfcn.h>

#include <atomic>
#include <cmath>
#include <cstring>
#include <mutex>
#include <string>
#include <unordered_map>

#include "ewise_host.h"
#include "ewise_kernels.cuh"
#include "ewise_prog.h"

namespace relay {
namespace {

// ---- the run-time compiler and the module loader, both looked up at run time -------------------------------------------
struct Nvrtc {
    bool ok = false;
    int (*create)(void **prog, const char *src, const char *name, int n_headers, const char *const *headers, const char *const *names) = nullptr;
    int (*compile)(void *prog, int n_opts, const char *const *opts) = nullptr;
    int (*cubin_size)(void *prog, size_t *n) = nullptr;
    int (*cubin)(void *prog, char *out) = nullptr;
    int (*log_size)(void *prog, size_t *n) = nullptr;
    int (*log)(void *prog, char *out) = nullptr;
    int (*destroy)(void **prog) = nullptr;
};

const Nvrtc &nvrtc()
{
    static Nvrtc n = []() {
        Nvrtc r;
        const char *names[] = {"libnvrtc.so.12", "/usr/local/cuda/lib64/libnvrtc.so.12", "libnvrtc.so", "/usr/local/cuda/lib64/libnvrtc.so"};
        void *lib = nullptr;
        for (const char *nm : names)
            if ((lib = dlopen(nm, RTLD_NOW | RTLD_LOCAL)) != nullptr) break;
        if (!lib) return r;
        r.create = (decltype(r.create))dlsym(lib, "nvrtcCreateProgram");
        r.compile = (decltype(r.compile))dlsym(lib, "nvrtcCompileProgram");
        r.cubin_size = (decltype(r.cubin_size))dlsym(lib, "nvrtcGetCUBINSize");
        r.cubin = (decltype(r.cubin))dlsym(lib, "nvrtcGetCUBIN");
        r.log_size = (decltype(r.log_size))dlsym(lib, "nvrtcGetProgramLogSize");
        r.log = (decltype(r.log))dlsym(lib, "nvrtcGetProgramLog");
        r.destroy = (decltype(r.destroy))dlsym(lib, "nvrtcDestroyProgram");
        r.ok = r.create && r.compile && r.cubin_size && r.cubin && r.log_size && r.log && r.destroy;
        return r;
    }();
    return n;
}

struct Driver {
    bool ok = false;
    CUresult (*module_load)(CUmodule *, const void *) = nullptr;
    CUresult (*module_fn)(CUfunction *, CUmodule, const char *) = nullptr;
    CUresult (*launch)(const CUlaunchConfig *, CUfunction, void **, void **) = nullptr;
};

const Driver &driver()
{
    static Driver d = []() {
        Driver r;
        auto get = [](const char *name) -> void * {
            void *fp = nullptr;
            cudaDriverEntryPointQueryResult q;
            if (cudaGetDriverEntryPoint(name, &fp, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) { cudaGetLastError(); return nullptr; }
            return fp;
        };
        r.module_load = (decltype(r.module_load))get("cuModuleLoadData");
        r.module_fn = (decltype(r.module_fn))get("cuModuleGetFunction");
        r.launch = (decltype(r.launch))get("cuLaunchKernelEx");
        r.ok = r.module_load && r.module_fn && r.launch;
        return r;
    }();
    return d;
}

// ---- the generated source ----------------------------------------------------------------------------------------------
constexpr int kJitTX = 32, kJitTY = 8, kJitUnroll = 4;

const char *kPrologue = R"SRC(
typedef unsigned int u32;
typedef long long i64;
__device__ __forceinline__ uint4 ld16(const void *p)
{
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}
__device__ __forceinline__ void st16(void *p, u32 a, u32 b, u32 c, u32 d) { asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(a), "r"(b), "r"(c), "r"(d) : "memory"); }
__device__ __forceinline__ void st8(void *p, u32 a, u32 b) { asm volatile("st.global.cs.v2.u32 [%0], {%1,%2};" ::"l"(p), "r"(a), "r"(b) : "memory"); }
__device__ __forceinline__ void st4(void *p, u32 a) { asm volatile("st.global.cs.u32 [%0], %1;" ::"l"(p), "r"(a) : "memory"); }
// two floats -> two bf16 (round to nearest even), `lo` in the low half
__device__ __forceinline__ u32 pk(float lo, float hi) { u32 r; asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo)); return r; }
__device__ __forceinline__ float rb(float x) { return __uint_as_float(pk(0.0f, x) & 0xffff0000u); }
__device__ __forceinline__ u32 by(float a, float b, float c, float d) { return (a != 0.0f ? 1u : 0u) | (b != 0.0f ? 0x100u : 0u) | (c != 0.0f ? 0x10000u : 0u) | (d != 0.0f ? 0x1000000u : 0u); }
)SRC";

float bf16_round_host(float x)
{
    uint32_t u;
    memcpy(&u, &x, 4);
    if ((u & 0x7f800000u) == 0x7f800000u && (u & 0x007fffffu)) u |= 0x00400000u;   // NaN stays NaN
    else u += 0x7fffu + ((u >> 16) & 1u);
    u &= 0xffff0000u;
    float r;
    memcpy(&r, &u, 4);
    return r;
}
std::string lit(float x)
{
    uint32_t u;
    memcpy(&u, &x, 4);
    char buf[48];
    snprintf(buf, sizeof buf, "__uint_as_float(0x%08xu)", u);
    return buf;
}
std::string num(long long x) { return std::to_string(x); }

struct Gen {
    std::string src;
    int n_sum = 0;
    int sum_of_out[RELAY_MAX_OUTPUTS];
    bool ok = false;
};

// which values the results depend on; false if one of them is of a type the bodies do not carry (integer lanes)
bool needed_values(const TypedProgram &tp, const int32_t *out_values, int n_out, bool (&needed)[kMaxValues])
{
    for (int x = 0; x < kMaxValues; ++x) needed[x] = false;
    for (int k = 0; k < n_out; ++k) needed[out_values[k]] = true;
    for (int x = tp.n_values - 1; x >= tp.n_in; --x) {
        if (!needed[x]) continue;
        const relay_instr_t &in = tp.instr[x - tp.n_in];
        if (in.a >= 0) needed[in.a] = true;
        if (in.b >= 0) needed[in.b] = true;
        if (in.c >= 0) needed[in.c] = true;
    }
    for (int x = 0; x < tp.n_values; ++x)
        if (needed[x] && !(tp.dtype[x] == RELAY_F32 || tp.dtype[x] == RELAY_BF16 || tp.dtype[x] == RELAY_BOOL)) return false;
    return true;
}

// `out_dtype[k]`: storage type of result k (bf16, f32 or Bool as bytes); `colsum[k]`: result k is summed over the rows
Gen generate(const TypedProgram &tp, const View2D &v, const int32_t *out_values, const int32_t *out_dtype, const bool *colsum, int n_out)
{
    Gen G;
    const bool bf = v.storage == RELAY_BF16;
    const int V = bf ? 8 : 4;
    bool needed[kMaxValues];
    if (!needed_values(tp, out_values, n_out, needed)) return G;
    int n_full = 0;
    for (int i = 0; i < tp.n_in; ++i) n_full += v.kind[i] == KIND_FULL;
    for (int k = 0; k < n_out; ++k) {
        G.sum_of_out[k] = colsum[k] ? G.n_sum++ : -1;
        if (!colsum[k] && !(out_dtype[k] == RELAY_F32 || out_dtype[k] == RELAY_BF16 || out_dtype[k] == RELAY_BOOL)) return G;
    }
    const std::string Vs = num(V), esz = bf ? "2" : "4";
    std::string s = kPrologue;
    s += "struct Args { const void *in[" + num(tp.n_in) + "]; void *out[" + num(n_out) + "]; float *partial[" + num(n_out) +
         "]; i64 rows, cols; int rows_per_slice, pad_; };\n";
    s += "extern \"C\" __global__ void __launch_bounds__(256, " + num(n_full >= 4 ? 2 : 3) + ") relay_jit_kernel(const Args A)\n{\n";
    s += "    const int tx = threadIdx.x, ty = threadIdx.y;\n    const i64 col0 = ((i64)blockIdx.x * 32 + tx) * " + Vs + ";\n";
    s += "    asm volatile(\"griddepcontrol.launch_dependents;\" ::: \"memory\");\n    asm volatile(\"griddepcontrol.wait;\" ::: \"memory\");\n";
    s += "    const bool active = col0 < A.cols;\n";
    auto unpack = [&](const std::string &dst, const std::string &raw) {
        if (bf)
            return "{ const u32 w_[4] = {" + raw + ".x, " + raw + ".y, " + raw + ".z, " + raw + ".w};\n"
                   "#pragma unroll\n for (int q = 0; q < 4; ++q) { " + dst + "[2 * q] = __uint_as_float(w_[q] << 16); " + dst +
                   "[2 * q + 1] = __uint_as_float(w_[q] & 0xffff0000u); } }\n";
        return "{ " + dst + "[0] = __uint_as_float(" + raw + ".x); " + dst + "[1] = __uint_as_float(" + raw + ".y); " + dst + "[2] = __uint_as_float(" + raw +
               ".z); " + dst + "[3] = __uint_as_float(" + raw + ".w); }\n";
    };
    // operands that do not change from row to row
    for (int i = 0; i < tp.n_in; ++i) {
        if (!needed[i] || v.kind[i] == KIND_FULL) continue;
        const std::string f = "f" + num(i);
        s += "    float " + f + "[" + Vs + "];\n";
        if (v.kind[i] == KIND_ROWVEC) {
            s += "    { uint4 r_ = make_uint4(0, 0, 0, 0); if (active) r_ = ld16((const char *)A.in[" + num(i) + "] + col0 * " + esz + ");\n    " + unpack(f, "r_") + "    }\n";
        } else {
            s += bf ? "    { const float s_ = __uint_as_float((u32)(*(const unsigned short *)A.in[" + num(i) + "]) << 16);\n"
                    : "    { const float s_ = *(const float *)A.in[" + num(i) + "];\n";
            s += "#pragma unroll\n      for (int e = 0; e < " + Vs + "; ++e) " + f + "[e] = s_; }\n";
        }
    }
    for (int k = 0; k < n_out; ++k)
        if (colsum[k]) s += "    float acc" + num(k) + "[" + Vs + "];\n#pragma unroll\n    for (int e = 0; e < " + Vs + "; ++e) acc" + num(k) + "[e] = 0.0f;\n";
    s += "    const i64 r0 = (i64)blockIdx.y * A.rows_per_slice;\n    const i64 r1 = min(A.rows, r0 + (i64)A.rows_per_slice);\n";
    s += "    if (active) {\n      for (i64 r = r0 + ty; r < r1; r += " + num(kJitTY * kJitUnroll) + ") {\n";
    for (int i = 0; i < tp.n_in; ++i)
        if (needed[i] && v.kind[i] == KIND_FULL) s += "        uint4 raw" + num(i) + "[" + num(kJitUnroll) + "];\n";
    s += "#pragma unroll\n        for (int u = 0; u < " + num(kJitUnroll) + "; ++u) {\n          const i64 rr = r + u * " + num(kJitTY) + ";\n          if (rr < r1) {\n";
    for (int i = 0; i < tp.n_in; ++i)
        if (needed[i] && v.kind[i] == KIND_FULL)
            s += "            raw" + num(i) + "[u] = ld16((const char *)A.in[" + num(i) + "] + (rr * A.cols + col0) * " + esz + ");\n";
    s += "          }\n        }\n";
    s += "#pragma unroll\n        for (int u = 0; u < " + num(kJitUnroll) + "; ++u) {\n          const i64 rr = r + u * " + num(kJitTY) + ";\n          if (rr >= r1) break;\n";
    for (int i = 0; i < tp.n_in; ++i)
        if (needed[i] && v.kind[i] == KIND_FULL) s += "          float a" + num(i) + "[" + Vs + "];\n          " + unpack("a" + num(i), "raw" + num(i) + "[u]");
    for (int k = 0; k < n_out; ++k)
        if (!colsum[k]) s += "          float o" + num(k) + "[" + Vs + "];\n";
    // the let-list, once per element
    s += "#pragma unroll\n          for (int e = 0; e < " + Vs + "; ++e) {\n";
    auto val = [&](int x) { return "v" + num(x); };
    for (int i = 0; i < tp.n_in; ++i)
        if (needed[i]) s += "            const float " + val(i) + " = " + (v.kind[i] == KIND_FULL ? "a" : "f") + num(i) + "[e];\n";
    for (int x = tp.n_in; x < tp.n_values; ++x) {
        if (!needed[x]) continue;
        const relay_instr_t &in = tp.instr[x - tp.n_in];
        const int dt = tp.dtype[x];
        const std::string a = in.a >= 0 ? val(in.a) : "0.0f", b = in.b >= 0 ? val(in.b) : "0.0f", c = in.c >= 0 ? val(in.c) : "0.0f";
        std::string e;
        bool typed_round = dt == RELAY_BF16;       // a value of type bf16 holds a bf16 number
        switch (in.op) {
        case RELAY_OP_CAST: {
            const int from = tp.dtype[in.a];
            if (dt == RELAY_BOOL) e = "(" + a + " != 0.0f ? 1.0f : 0.0f)";
            else e = a;
            typed_round = dt == RELAY_BF16 && from == RELAY_F32;       // Bool and bf16 values are bf16 numbers already
            break;
        }
        case RELAY_OP_CONST: {
            float cv = (float)in.imm;
            if (dt == RELAY_BF16) cv = bf16_round_host(cv);
            else if (dt == RELAY_BOOL) cv = cv != 0.0f ? 1.0f : 0.0f;
            e = lit(cv);
            typed_round = false;
            break;
        }
        case RELAY_OP_SELECT: e = "(" + a + " != 0.0f ? " + b + " : " + c + ")"; typed_round = false; break;
        case RELAY_OP_ADD: e = a + " + " + b; break;
        case RELAY_OP_SUB: e = a + " - " + b; break;
        case RELAY_OP_MUL: e = a + " * " + b; break;
        case RELAY_OP_DIV: e = bf ? "__fdividef(" + a + ", " + b + ")" : a + " / " + b; break;
        case RELAY_OP_NEG: e = "-" + a; break;
        case RELAY_OP_SQ: e = a + " * " + a; break;
        case RELAY_OP_NE: e = "(" + a + " != " + b + " ? 1.0f : 0.0f)"; break;
        case RELAY_OP_EQ: e = "(" + a + " == " + b + " ? 1.0f : 0.0f)"; break;
        case RELAY_OP_LT: e = "(" + a + " < " + b + " ? 1.0f : 0.0f)"; break;
        case RELAY_OP_LE: e = "(" + a + " <= " + b + " ? 1.0f : 0.0f)"; break;
        case RELAY_OP_GT: e = "(" + a + " > " + b + " ? 1.0f : 0.0f)"; break;
        case RELAY_OP_GE: e = "(" + a + " >= " + b + " ? 1.0f : 0.0f)"; break;
        case RELAY_OP_RELU: e = "fmaxf(" + a + ", 0.0f)"; break;
        case RELAY_OP_TANH: e = bf ? "1.0f - __fdividef(2.0f, 1.0f + __expf(2.0f * " + a + "))" : "tanhf(" + a + ")"; break;
        case RELAY_OP_SIGMOID: e = bf ? "__fdividef(1.0f, 1.0f + __expf(-" + a + "))" : "1.0f / (1.0f + expf(-" + a + "))"; break;
        case RELAY_OP_EXP: e = bf ? "__expf(" + a + ")" : "expf(" + a + ")"; break;
        case RELAY_OP_LOG: e = bf ? "__logf(" + a + ")" : "logf(" + a + ")"; break;
        case RELAY_OP_MAX: e = "fmaxf(" + a + ", " + b + ")"; break;
        case RELAY_OP_MIN: e = "fminf(" + a + ", " + b + ")"; break;
        default: return G;
        }
        s += "            const float " + val(x) + " = " + (typed_round ? "rb(" + e + ")" : e) + ";\n";
    }
    for (int k = 0; k < n_out; ++k) {
        if (colsum[k]) s += "            acc" + num(k) + "[e] += " + val(out_values[k]) + ";\n";
        else s += "            o" + num(k) + "[e] = " + val(out_values[k]) + ";\n";
    }
    s += "          }\n";
    for (int k = 0; k < n_out; ++k) {
        if (colsum[k]) continue;
        const std::string o = "o" + num(k), at = "(rr * A.cols + col0)";
        if (out_dtype[k] == RELAY_BF16) {
            const std::string p = "(char *)A.out[" + num(k) + "] + " + at + " * 2";
            if (V == 8) s += "          st16(" + p + ", pk(" + o + "[0], " + o + "[1]), pk(" + o + "[2], " + o + "[3]), pk(" + o + "[4], " + o + "[5]), pk(" + o + "[6], " + o + "[7]));\n";
            else s += "          st8(" + p + ", pk(" + o + "[0], " + o + "[1]), pk(" + o + "[2], " + o + "[3]));\n";
        } else if (out_dtype[k] == RELAY_F32) {
            for (int q = 0; q < V / 4; ++q) {
                const std::string p = "(char *)A.out[" + num(k) + "] + (" + at + " + " + num(4 * q) + ") * 4";
                s += "          st16(" + p + ", __float_as_uint(" + o + "[" + num(4 * q) + "]), __float_as_uint(" + o + "[" + num(4 * q + 1) + "]), __float_as_uint(" + o + "[" +
                     num(4 * q + 2) + "]), __float_as_uint(" + o + "[" + num(4 * q + 3) + "]));\n";
            }
        } else {
            const std::string p = "(char *)A.out[" + num(k) + "] + " + at;
            if (V == 8) s += "          st8(" + p + ", by(" + o + "[0], " + o + "[1], " + o + "[2], " + o + "[3]), by(" + o + "[4], " + o + "[5], " + o + "[6], " + o + "[7]));\n";
            else s += "          st4(" + p + ", by(" + o + "[0], " + o + "[1], " + o + "[2], " + o + "[3]));\n";
        }
    }
    s += "        }\n      }\n    }\n";
    if (G.n_sum > 0) {
        // combine the row-threads of each column, in ty order, and publish one partial per slice
        s += "    __shared__ float sm[" + num(kJitTY) + "][" + num(kJitTX * V + 1) + "];\n";
        for (int k = 0; k < n_out; ++k) {
            if (!colsum[k]) continue;
            s += "#pragma unroll\n    for (int e = 0; e < " + Vs + "; ++e) sm[ty][tx * " + Vs + " + e] = acc" + num(k) + "[e];\n    __syncthreads();\n";
            s += "    if (ty == 0 && active) {\n#pragma unroll\n      for (int e = 0; e < " + Vs + "; ++e) {\n        float t_ = 0.0f;\n#pragma unroll\n        for (int j = 0; j < " +
                 num(kJitTY) + "; ++j) t_ += sm[j][tx * " + Vs + " + e];\n        A.partial[" + num(k) + "][(i64)blockIdx.y * A.cols + col0 + e] = t_;\n      }\n    }\n    __syncthreads();\n";
        }
    }
    s += "}\n";
    G.src = std::move(s);
    G.ok = true;
    return G;
}

// ---- cache -------------------------------------------------------------------------------------------------------------
struct Kernel {
    CUfunction fn = nullptr;
    int n_sum = 0, vec = 0;
    int sum_of_out[RELAY_MAX_OUTPUTS];
};

std::mutex g_mu;
std::unordered_map<std::string, Kernel *> g_cache;      // device ordinal + source text -> kernel (nullptr: did not compile)
std::atomic<int> g_enabled{1};
std::atomic<int> g_compiled{0};
std::string g_last_log;

// source -> machine code for sm_100a; false (with the compiler's messages in *log) if it does not compile
bool to_cubin(const std::string &src, std::string *bin, std::string *log)
{
    const Nvrtc &N = nvrtc();
    void *prog = nullptr;
    if (N.create(&prog, src.c_str(), "relay_jit.cu", 0, nullptr, nullptr) != 0) return false;
    const char *opts[] = {"--gpu-architecture=sm_100a", "--std=c++17", "-default-device"};
    const int rc = N.compile(prog, 3, opts);
    if (rc != 0) {
        size_t n = 0;
        if (log && N.log_size(prog, &n) == 0 && n > 1) { log->resize(n); N.log(prog, &(*log)[0]); }
        N.destroy(&prog);
        return false;
    }
    size_t n = 0;
    if (N.cubin_size(prog, &n) != 0 || n == 0) { N.destroy(&prog); return false; }
    bin->resize(n);
    const int got = N.cubin(prog, &(*bin)[0]);
    N.destroy(&prog);
    return got == 0;
}

Kernel *compile(const Gen &G, int vec)
{
    const Driver &D = driver();
    std::string bin;
    if (!to_cubin(G.src, &bin, &g_last_log)) return nullptr;
    cudaFree(nullptr);                                     // the runtime's context is current before the module is loaded into it
    CUmodule mod = nullptr;
    CUfunction fn = nullptr;
    if (D.module_load(&mod, bin.data()) != CUDA_SUCCESS) return nullptr;
    if (D.module_fn(&fn, mod, "relay_jit_kernel") != CUDA_SUCCESS) return nullptr;
    Kernel *k = new Kernel();
    k->fn = fn; k->n_sum = G.n_sum; k->vec = vec;
    memcpy(k->sum_of_out, G.sum_of_out, sizeof k->sum_of_out);
    g_compiled.fetch_add(1);
    return k;
}

}  // namespace

// The class of groups a body can be generated for (whether or not a compiler is present): over the collapsed 2-D view,
// float and Bool values only; the caller has checked that every result is unreduced or a sum over all leading axes.
bool jit_in_class(const TypedProgram &tp, const View2D &v, const int32_t *out_values, int n_out)
{
    bool needed[kMaxValues];
    return v.ok && n_out >= 1 && n_out <= RELAY_MAX_OUTPUTS && v.rows < (1ll << 31) && needed_values(tp, out_values, n_out, needed);
}

// Set by callers that must not allocate (compiling and loading a module allocates host and device memory): on this thread
// only bodies that are compiled already are used, any other group runs on the interpreter.
static thread_local bool t_cached_only = false;
bool jit_set_cached_only(bool on)
{
    const bool before = t_cached_only;
    t_cached_only = on;
    return before;
}

bool jit_usable()
{
#ifdef RELAY_BOUNDS_CHECK
    return false;
#else
    return g_enabled.load() != 0 && nvrtc().ok && driver().ok;
#endif
}

// The kernel for this group, compiled on first use; nullptr when the group is outside the class, when there is no run-time
// compiler on this machine, or when it is switched off (the caller then takes the interpreter).
const void *jit_get(const TypedProgram &tp, const View2D &v, const int32_t *out_values, const int32_t *out_dtype, const bool *colsum, int n_out)
{
    if (!jit_usable() || !v.ok || n_out < 1 || n_out > RELAY_MAX_OUTPUTS) return nullptr;
    Gen G = generate(tp, v, out_values, out_dtype, colsum, n_out);
    if (!G.ok) return nullptr;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    const std::string key = std::to_string(dev) + "\n" + G.src;
    std::lock_guard<std::mutex> lock(g_mu);
    auto it = g_cache.find(key);
    if (it != g_cache.end()) return it->second;
    if (t_cached_only) return nullptr;
    Kernel *k = compile(G, v.storage == RELAY_BF16 ? 8 : 4);
    g_cache.emplace(key, k);
    return k;
}

// Host only (no GPU needed): generates the source of the group's body and compiles it.  1: compiled; 0: the group is outside
// the class; -1: no run-time compiler here; -2: the source did not compile (*log has the compiler's messages).
int jit_compile_only(const TypedProgram &tp, const View2D &v, const int32_t *out_values, const int32_t *out_dtype, const bool *colsum, int n_out,
                     std::string *src, std::string *log)
{
    if (!nvrtc().ok) return -1;
    if (!v.ok || n_out < 1 || n_out > RELAY_MAX_OUTPUTS) return 0;
    Gen G = generate(tp, v, out_values, out_dtype, colsum, n_out);
    if (!G.ok) return 0;
    if (src) *src = G.src;
    std::string bin;
    return to_cubin(G.src, &bin, log) ? 1 : -2;
}

int jit_n_slices(const View2D &v, bool any_sum)
{
    const int vec = v.storage == RELAY_BF16 ? 8 : 4;
    const int64_t gx = (v.cols + (int64_t)kJitTX * vec - 1) / (kJitTX * vec);
    if (any_sum) return colsum_slices(v.rows, v.cols, v.storage);
    return (int)std::max<int64_t>(1, std::min<int64_t>((148 * 16) / gx, (v.rows + kJitTY * kJitUnroll - 1) / (kJitTY * kJitUnroll)));
}

// partials: [n_sum][n_slices][cols] floats (column sums only)
relay_status_t jit_launch(const void *kernel, const View2D &v, const relay_tensor_t *const *inputs, int n_in, const relay_tensor_t *const *outputs,
                          int n_out, float *partials, int n_slices, cudaStream_t st)
{
    const Kernel &K = *static_cast<const Kernel *>(kernel);
    uint64_t args[3 * RELAY_MAX_OUTPUTS + RELAY_MAX_INPUTS + 3];
    int w = 0;
    for (int i = 0; i < n_in; ++i) args[w++] = (uint64_t)(uintptr_t)inputs[i]->data;
    for (int k = 0; k < n_out; ++k) args[w++] = (uint64_t)(uintptr_t)outputs[k]->data;
    for (int k = 0; k < n_out; ++k)
        args[w++] = K.sum_of_out[k] >= 0 ? (uint64_t)(uintptr_t)(partials + (size_t)K.sum_of_out[k] * n_slices * v.cols) : 0;
    args[w++] = (uint64_t)v.rows;
    args[w++] = (uint64_t)v.cols;
    const uint32_t rps = (uint32_t)((v.rows + n_slices - 1) / n_slices);
    args[w++] = (uint64_t)rps;
    CUlaunchConfig cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDimX = (unsigned)((v.cols + (int64_t)kJitTX * K.vec - 1) / (kJitTX * K.vec)); cfg.gridDimY = (unsigned)n_slices; cfg.gridDimZ = 1;
    cfg.blockDimX = kJitTX; cfg.blockDimY = kJitTY; cfg.blockDimZ = 1;
    cfg.sharedMemBytes = 0;
    cfg.hStream = (CUstream)st;
    CUlaunchAttribute attr[1];
    memset(attr, 0, sizeof attr);
    attr[0].id = CU_LAUNCH_ATTRIBUTE_PROGRAMMATIC_STREAM_SERIALIZATION;
    attr[0].value.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    void *params[] = {(void *)args};
    const CUresult r = driver().launch(&cfg, K.fn, params, nullptr);
    if (r != CUDA_SUCCESS) return fail(RELAY_ERR_CUDA, "launch of a run-time compiled body failed with driver code %d", (int)r);
    count_launch();
    return RELAY_OK;
}

int jit_n_sum(const void *kernel) { return static_cast<const Kernel *>(kernel)->n_sum; }

}  // namespace relay

using namespace relay;

// Switches the run-time compiled bodies on (1) or off (0) for this process (off: such groups run on the interpreter);
// returns the previous setting.
extern "C" int32_t relay_debug_set_jit(int32_t enabled) { return g_enabled.exchange(enabled ? 1 : 0); }

// Bodies compiled so far in this process; -1 when compiled bodies cannot be used here (no run-time compiler library, or no
// driver to load them with).
extern "C" int32_t relay_debug_jit_compiled(void)
{
#ifdef RELAY_BOUNDS_CHECK
    return -1;
#else
    return nvrtc().ok && driver().ok ? g_compiled.load() : -1;
#endif
}
