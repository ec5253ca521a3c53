// The checked copy of the kernels (A2SGD_DEBUG_CHECKS): the same kernel source as the production
// library, compiled into its own namespace with the access checks switched on, plus the two hooks
// the host dispatch needs — the table of these kernels and the switch of the descriptor that holds
// the extents of the call in flight.
#include <cuda_runtime.h>

#include "a2sgd_kernel_table.h"
#define A2SGD_NS a2sgd_chk
#define A2SGD_CHECKED 1
#include "a2sgd_kernels.cuh"
#include "a2sgd_segments.cuh"
#include "a2sgd_select.cuh"

const a2sgd_kernel_table *a2sgd_checked_kernels()
{
    static const a2sgd_kernel_table table = a2sgd_chk::kernel_table();
    return &table;
}

// Copies a DebugChecks descriptor (see a2sgd_kernels.cuh) into the constant the checked kernels
// read, in stream order.  The source is pageable host memory: it is staged before the call returns.
cudaError_t a2sgd_checked_arm(const void *descriptor, size_t bytes, cudaStream_t stream)
{
    if (bytes != sizeof(a2sgd_chk::DebugChecks)) return cudaErrorInvalidValue;
    return cudaMemcpyToSymbolAsync(a2sgd_chk::c_debug, descriptor, bytes, 0, cudaMemcpyHostToDevice, stream);
}
