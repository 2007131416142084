// Launch interface between the executor (host) and the copy kernels.
#pragma once

#include <cuda_runtime.h>

#include "copy_params.h"

namespace redist {

constexpr int kSmallTable = 64;     // pointer-table capacity of the small parameter block
constexpr int kLargeTable = 1024;   // ... of the large one (REDIST_MAX_DEVICES)

// One kernel launch, ready to go: entry point, launch shape and a pointer to the complete parameter block
// (copy descriptor plus both pointer tables), which lives in storage of the caller's choosing -- the
// stack of a call, or a bound plan that is launched again and again.
struct PreparedLaunch {
    const void *fn = nullptr;
    unsigned grid = 0, block = 0;
    size_t smem = 0;
    int pdl = 1;
    void *params = nullptr;
};

// Bytes of parameter storage (16-byte aligned) a launch with this many table entries needs.
constexpr size_t param_bytes(int n_tab)
{
    return n_tab <= kSmallTable ? sizeof(CopyParams<kSmallTable>) : sizeof(CopyParams<kLargeTable>);
}

// kernel: 0 dynslice, 1 alltoall, 2 allgather, 3 allpermute, 4 copy, 5 fused, 6 naive gather,
// 7 naive slice.  src_tab / dst_tab are HOST arrays of device pointers (copied into the parameter
// block at `storage`, which must hold param_bytes(max(n_src, n_dst)) bytes).  Host only; allocates nothing.
cudaError_t prepare_copy(int kernel, const CopyGeometry &geo, const char *const *src_tab, int n_src,
                         char *const *dst_tab, int n_dst, int pdl, void *storage, size_t storage_bytes,
                         PreparedLaunch &out);

// Asynchronous on `stream`; the parameter block is read during the call.
cudaError_t launch_prepared(const PreparedLaunch &pl, cudaStream_t stream);

// Work items of the bulk-copy kernels whose bounded wait ran out on the current device (0 in a healthy
// run).  Synchronizes the device.
cudaError_t read_bulk_timeouts(unsigned int *out);

// Checked build only: {violations, source line, block, side, distance} of the accesses that failed
// their bounds test since the last call (and resets the record); cudaErrorNotSupported otherwise.
cudaError_t read_bounds_report(long long out[5]);

}  // namespace redist
