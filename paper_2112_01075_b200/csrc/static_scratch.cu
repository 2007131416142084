// redist_execute_static -- run a plan whose intermediates need scratch memory without the caller
// (or this library) allocating any: the scratch is a fixed array that is part of the loaded module.
//
// Who needs this: a caller that is handed tiles by a framework but owns no allocator of its own --
// a plug-in inside a serving process that gave all device memory to a pool at start-up and forbids
// cudaMalloc afterwards, or code on a path where an allocation could fail or stall a latency-bound
// request.  Such a caller still passes its source and destination tiles; only the ping-pong
// buffers of an unfused plan come from here.
#include <cuda_runtime.h>

#include <cstdint>
#include <mutex>

#include "kernels.h"
#include "plan.hpp"

namespace {

// The scratch itself.  Every GPU that loads this library carries these bytes until the process
// exits.  In host code the name below is only a stand-in for the symbol: it is not a device address
// and must never be passed to a kernel; the address comes from cudaGetSymbolAddress (device_scratch).
static __device__ __align__(256) unsigned char g_static_scratch[REDIST_STATIC_SCRATCH_BYTES];

constexpr int kMaxGpus = 64;
std::mutex g_setup_mutex;
unsigned char *g_scratch_addr[kMaxGpus] = {};   // device address of g_static_scratch, per GPU

// Set-up, once per device, with that device current: resolve the device address of the array.
redist_status device_scratch(unsigned char **out)
{
    int dev = -1;
    cudaError_t ce = cudaGetDevice(&dev);
    if (ce != cudaSuccess || dev < 0 || dev >= kMaxGpus) {
        redist::tl_cuda_error = int(ce);
        return ce != cudaSuccess ? REDIST_ECUDA : REDIST_EUNSUPPORTED;
    }
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[dev]) {
        void *ptr = nullptr;
        ce = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (ce != cudaSuccess || !ptr) {
            redist::tl_cuda_error = int(ce);
            return REDIST_ECUDA;
        }
        g_scratch_addr[dev] = static_cast<unsigned char *>(ptr);
    }
    *out = g_scratch_addr[dev];
    return REDIST_OK;
}

}  // namespace

extern "C" redist_status redist_execute_static(const redist_plan_t *plan, const void *const *src_shards,
                                               void *const *dst_shards, void *cuda_stream)
{
    using namespace redist;
    try {
        if (!plan || !src_shards || !dst_shards) return REDIST_EINVAL;
        const Plan &p = plan->p;
        if (p.scratch_bytes > i64(REDIST_STATIC_SCRATCH_BYTES)) return REDIST_ESCRATCH;
        unsigned char *scratch = nullptr;
        redist_status rc = device_scratch(&scratch);
        if (rc != REDIST_OK) return rc;
        // The same checks and launches as redist_execute (tables and parameter block on the stack, nothing
        // allocated).  The caller's tiles can only meet the built-in array by a wild pointer; the whole
        // array takes part in the overlap check anyway.
        return run_plan(p, src_shards, dst_shards, scratch, REDIST_STATIC_SCRATCH_BYTES, cuda_stream);
    } catch (...) {
        return REDIST_EINTERNAL;
    }
}
