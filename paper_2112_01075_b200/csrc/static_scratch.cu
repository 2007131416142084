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

bool intersects(uintptr_t a, uintptr_t an, uintptr_t b, uintptr_t bn) { return a < b + bn && b < a + an; }

}  // namespace

extern "C" redist_status redist_execute_static(const redist_plan_t *plan, const void *const *src_shards,
                                               void *const *dst_shards, void *cuda_stream)
{
    using namespace redist;
    if (!plan || !src_shards || !dst_shards) return REDIST_EINVAL;
    const Plan &p = plan->p;
    const int N = p.n_devices;
    if (p.scratch_bytes > i64(REDIST_STATIC_SCRATCH_BYTES)) return REDIST_ESCRATCH;
    unsigned char *scratch = nullptr;
    redist_status rc = device_scratch(&scratch);
    if (rc != REDIST_OK) return rc;

    const uintptr_t amask = uintptr_t(p.alignment) - 1;
    const uintptr_t sb = uintptr_t(p.local_src * p.elem_bytes), db = uintptr_t(p.local_dst * p.elem_bytes);
    for (int d = 0; d < N; ++d) {
        if (!src_shards[d] || !dst_shards[d]) return REDIST_EINVAL;
        const uintptr_t s = uintptr_t(src_shards[d]), t = uintptr_t(dst_shards[d]);
        if ((s & amask) || (t & amask)) return REDIST_EALIGN;
        // the caller's tiles can only meet the built-in array by a wild pointer; check anyway
        if (intersects(s, sb, uintptr_t(scratch), REDIST_STATIC_SCRATCH_BYTES) ||
            intersects(t, db, uintptr_t(scratch), REDIST_STATIC_SCRATCH_BYTES))
            return REDIST_EOVERLAP;
        for (int q = 0; q < N; ++q)
            if (intersects(t, db, uintptr_t(src_shards[q]), sb) ||
                (q != d && intersects(t, db, uintptr_t(dst_shards[q]), db)))
                return REDIST_EOVERLAP;
    }

    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    auto buffer = [&](BufKind kind, int32_t dev) -> char * {
        switch (kind) {
        case BUF_SRC: return static_cast<char *>(const_cast<void *>(src_shards[dev]));
        case BUF_DST: return static_cast<char *>(dst_shards[dev]);
        case BUF_SCRATCH0: return reinterpret_cast<char *>(scratch) + i64(dev) * p.slot_bytes;
        case BUF_SCRATCH1: return reinterpret_cast<char *>(scratch) + (i64(N) + dev) * p.slot_bytes;
        default: return reinterpret_cast<char *>(scratch);
        }
    };
    // pointer tables on the stack: nothing is allocated, on the host or on the device
    const char *stab[REDIST_MAX_DEVICES];
    char *dtab[REDIST_MAX_DEVICES];
    for (const Launch &L : p.launches) {
        const int ns = int(L.src_holder.size()), nd = int(L.dst_devs.size());
        if (ns > REDIST_MAX_DEVICES || nd > REDIST_MAX_DEVICES) return REDIST_EUNSUPPORTED;
        for (int t = 0; t < ns; ++t) stab[t] = buffer(L.from, L.src_holder[t] < 0 ? 0 : L.src_holder[t]);
        for (int t = 0; t < nd; ++t) dtab[t] = buffer(L.to, L.dst_devs[t] < 0 ? 0 : L.dst_devs[t]);
        if (L.geo.n_items == 0) continue;
        cudaError_t ce = launch_copy(L.kernel, L.geo, stab, ns, dtab, nd, int(L.geo.n_items), stream);
        if (ce != cudaSuccess) {
            tl_cuda_error = int(ce);
            return REDIST_ECUDA;
        }
    }
    return REDIST_OK;
}
