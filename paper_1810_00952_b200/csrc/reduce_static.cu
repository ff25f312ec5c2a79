// relay_fused_reduce_static_scratch: the fused elementwise + reduce group for callers that cannot
// allocate device memory.  The column-sum kernels need scratch for their per-slice partial sums;
// here that scratch is a fixed array that lives in the library's device image.
#include <mutex>

#include "common.h"

namespace {

constexpr size_t kStaticScratchBytes = RELAY_STATIC_SCRATCH_BYTES;

// One copy per GPU that loads the library, held until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_mu;
void *g_scratch_addr[64] = {nullptr};

// `g_static_scratch` in host code is only a handle for the runtime, not an address a kernel can
// use: the device address is looked up once per device, with that device current.
relay_status_t static_scratch_of_current_device(void **out)
{
    int dev = -1;
    RELAY_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return relay::fail(RELAY_ERR_CUDA, "device ordinal %d not supported", dev);
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g_scratch_addr[dev]) {
        void *ptr = nullptr;
        RELAY_CUDA(cudaGetSymbolAddress((void **)&ptr, g_static_scratch));
        if (!ptr) return relay::fail(RELAY_ERR_CUDA, "static scratch has no device address");
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return RELAY_OK;
}

}  // namespace

namespace relay {
relay_status_t reduce_planned_scratch(const relay_ewise_prog_t *prog, const relay_tensor_t *const *inputs, int32_t n_in,
                                      const relay_out_spec_t *specs, int32_t n_out, size_t *need);
bool jit_set_cached_only(bool on);
}

extern "C" relay_status_t relay_fused_reduce_static_scratch(const relay_ewise_prog_t *prog, const relay_tensor_t *const *inputs,
                                                            int32_t n_in, const relay_out_spec_t *specs,
                                                            const relay_tensor_t *const *outputs, int32_t n_out, void *stream)
{
    relay::clear_error();
    // what this group's kernels will really use (a reduction over the last axis uses none), not the program-independent bound
    size_t need = 0;
    RELAY_TRY(relay::reduce_planned_scratch(prog, inputs, n_in, specs, n_out, &need));
    if (need > kStaticScratchBytes)
        return relay::fail(RELAY_ERR_WORKSPACE,
                           "this group needs %zu bytes of scratch but the built-in scratch holds %zu; use relay_fused_reduce "
                           "with a caller-provided workspace",
                           need, kStaticScratchBytes);
    void *scratch = nullptr;
    RELAY_TRY(static_scratch_of_current_device(&scratch));
    // Every partial that the second pass reads is written by the first pass of the same call, so
    // nothing in the array has to be cleared between calls.
    // Compiling a body for a new program and loading it allocates (host memory, device memory for the code), so this call
    // never does: a program whose body an earlier relay_fused_reduce / relay_fused_ewise call compiled uses it, any other
    // runs on the library's built-in kernels.
    const bool before = relay::jit_set_cached_only(true);
    const relay_status_t r = relay_fused_reduce(prog, inputs, n_in, specs, outputs, n_out, scratch, kStaticScratchBytes, stream);
    relay::jit_set_cached_only(before);
    return r;
}
