// Launch interface between the executor (host) and the copy kernels.
#pragma once

#include <cuda_runtime.h>

#include "copy_params.h"

namespace redist {

constexpr int kSmallTable = 64;     // pointer-table capacity of the small parameter block
constexpr int kLargeTable = 1024;   // ... of the large one (REDIST_MAX_DEVICES)

// kernel: 0 dynslice, 1 alltoall, 2 allgather, 3 allpermute, 4 copy, 5 fused, 6 naive gather,
// 7 naive slice.  src_tab / dst_tab are HOST arrays of device pointers (copied into the kernel
// parameters).  Asynchronous on `stream`.
cudaError_t launch_copy(int kernel, const CopyGeometry &geo, const char *const *src_tab, int n_src,
                        char *const *dst_tab, int n_dst, int grid, cudaStream_t stream);

// Work items of the bulk-copy kernel whose bounded wait ran out on the current device (0 in a healthy
// run).  Synchronizes the device.
cudaError_t read_bulk_timeouts(unsigned int *out);

}  // namespace redist
