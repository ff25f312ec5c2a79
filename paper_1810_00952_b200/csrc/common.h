// Internal helpers shared by the host-side entry points: status reporting, descriptor checks
// (the type relations of Fig. 4 / Fig. 5 applied to concrete tensors), launch accounting.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdarg>
#include <cstdint>
#include <cstdio>

#include "../../include/relay_b200.h"

namespace relay {

// ---- status -----------------------------------------------------------------------------------
relay_status_t fail(relay_status_t st, const char *fmt, ...);  // records text, returns st
void clear_error();
void count_launch(int n = 1);

#define RELAY_TRY(expr)                                   \
    do {                                                  \
        relay_status_t st__ = (expr);                     \
        if (st__ != RELAY_OK) return st__;                \
    } while (0)

#define RELAY_CUDA(expr)                                                                        \
    do {                                                                                        \
        cudaError_t e__ = (expr);                                                               \
        if (e__ != cudaSuccess)                                                                 \
            return ::relay::fail(RELAY_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e__)); \
    } while (0)

// checks the launch that was just issued
relay_status_t check_launch(const char *what);

// ---- descriptors --------------------------------------------------------------------------------
inline size_t dtype_size(int32_t dt)
{
    switch (dt) {
    case RELAY_F32: return 4;
    case RELAY_BF16: return 2;
    case RELAY_I32: return 4;
    case RELAY_I64: return 8;
    case RELAY_BOOL: return 1;
    default: return 0;
    }
}
inline bool is_float(int32_t dt) { return dt == RELAY_F32 || dt == RELAY_BF16; }
inline const char *dtype_name(int32_t dt)
{
    switch (dt) {
    case RELAY_F32: return "f32";
    case RELAY_BF16: return "bf16";
    case RELAY_I32: return "i32";
    case RELAY_I64: return "i64";
    case RELAY_BOOL: return "bool";
    default: return "?";
    }
}

inline int64_t numel(const relay_tensor_t *t)
{
    int64_t n = 1;
    for (int d = 0; d < t->rank; ++d) n *= t->shape[d];
    return n;
}
inline size_t nbytes(const relay_tensor_t *t) { return (size_t)numel(t) * dtype_size(t->dtype); }

// Tensor-T / Shape-T / BaseType-T on a concrete descriptor: known base type, rank in range,
// extents natural numbers.  Does not look at `data`.
relay_status_t check_type(const relay_tensor_t *t, const char *name);

// Stage-wise checks used by the entry points so that the first failing rule is reported in the
// documented order.
relay_status_t check_not_null(const void *p, const char *name);
relay_status_t check_rank(const relay_tensor_t *t, int rank, const char *name);
relay_status_t check_dtype(const relay_tensor_t *t, int32_t dt, const char *name);
relay_status_t check_layout(const relay_tensor_t *t, int32_t a, int32_t b, const char *name);
relay_status_t check_shape(const relay_tensor_t *t, std::initializer_list<int64_t> want, const char *name);
relay_status_t check_shape_n(const relay_tensor_t *t, const int64_t *want, int rank, const char *name);
relay_status_t check_data(const relay_tensor_t *t, const char *name);  // non-null (if numel>0), 16 B aligned
relay_status_t check_workspace(const void *ws, size_t have, size_t need);

struct Span { const char *lo, *hi; };
inline Span span_of(const relay_tensor_t *t)
{
    const char *p = (const char *)t->data;
    return Span{p, p + nbytes(t)};
}
// outputs must not overlap inputs or each other
relay_status_t check_no_overlap(const relay_tensor_t *const *outs, int n_out, const relay_tensor_t *const *ins,
                                int n_in);

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Launch with programmatic stream serialisation: the kernel may be scheduled while the previous kernel
// of the stream drains, runs its set-up, and blocks in pdl_wait() until that kernel has completed and
// its memory is visible.  Kernels launched this way call pdl_wait() before their first global access.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
// the same for a kernel that runs in thread-block clusters of `cluster` blocks
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, dim3 cluster, size_t smem, cudaStream_t st, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = cluster.x; attr[1].val.clusterDim.y = cluster.y; attr[1].val.clusterDim.z = cluster.z;
    cfg.attrs = attr; cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#ifdef __CUDACC__
// lets the next kernel of the stream start its set-up; then waits for the previous kernel's results
__device__ __forceinline__ void pdl_wait()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
#endif

// device-side error word (set by kernels whose bounded waits expire)
int *device_error_word();  // device address of the word on the current device (nullptr on failure)

// ---- bounds-check build (-DRELAY_BOUNDS_CHECK) -----------------------------------------------------
// A debugging variant of the library.  A launch function registers the address ranges its kernel may touch (every
// tensor of the call and the workspace); the kernels' global-memory access helpers look every address up, and an
// access outside all ranges is SKIPPED (loads return zero) and recorded in the device error word, which
// relay_poll_status reports.  Nothing traps.  The table is one __constant__ object per translation unit and is
// rewritten by every registering launch, so calls that overlap on one device confuse it: the variant is for
// single-stream test runs.  In the ordinary build all of this compiles to nothing.
constexpr int kErrBounds = 6;
#ifdef RELAY_BOUNDS_CHECK
struct BoundsTable { int n; int *err; unsigned long long lo[16], hi[16]; };
#ifdef __CUDACC__
static __constant__ BoundsTable c_bounds;
__device__ __forceinline__ bool relay_in_bounds(const void *p, size_t bytes)
{
    if (c_bounds.n == 0) return true;                    // this launch registered nothing
    const unsigned long long a = (unsigned long long)p;
    for (int i = 0; i < c_bounds.n; ++i)
        if (a >= c_bounds.lo[i] && a + bytes <= c_bounds.hi[i]) return true;
    if (c_bounds.err) atomicCAS(c_bounds.err, 0, kErrBounds);
    return false;
}
struct BoundsReg {
    BoundsTable t{};
    void add(const void *p, size_t bytes)
    {
        if (!p || !bytes || t.n >= 16) return;
        t.lo[t.n] = (unsigned long long)p; t.hi[t.n] = (unsigned long long)p + bytes; ++t.n;
    }
    void add(const relay_tensor_t *x) { if (x) add(x->data, nbytes(x)); }
    relay_status_t commit(cudaStream_t st)
    {
        t.err = device_error_word();
        RELAY_CUDA(cudaMemcpyToSymbolAsync(c_bounds, &t, sizeof t, 0, cudaMemcpyHostToDevice, st));
        return RELAY_OK;
    }
};
#endif
#else
#ifdef __CUDACC__
__device__ __forceinline__ constexpr bool relay_in_bounds(const void *, size_t) { return true; }
#endif
struct BoundsReg {
    void add(const void *, size_t) {}
    void add(const relay_tensor_t *) {}
    relay_status_t commit(cudaStream_t) { return RELAY_OK; }
};
#endif

}  // namespace relay
