// Host-side helpers shared by the translation units that launch tensor-path kernels.
#pragma once
#include <cuda_runtime.h>

#include <atomic>

#include "dispatch.h"

namespace ekl {

// Opts the kernel into its dynamic shared memory and asks how many CTAs fit on an SM; done
// once per device and kernel (the answer is kept), so that repeated calls cost one launch.
// Racing first calls compute and store the same value.  `cached` is the caller's per-kernel
// table (kernels of different shapes can share a function-pointer type, so the table cannot
// live here).
template <typename Kernel>
cudaError_t ctas_per_sm(Kernel kernel, int threads, size_t smem, std::atomic<int> (&cached)[64],
                        int* per_sm) {
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    int n = cached[dev].load(std::memory_order_acquire);
    if (n == 0) {
        err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        n = 1;
        err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, threads, smem);
        if (err != cudaSuccess) return err;
        if (n < 1) n = 1;
        cached[dev].store(n, std::memory_order_release);
    }
    *per_sm = n;
    return cudaSuccess;
}

// Batches are handed out dynamically when a CTA would otherwise get more than one; a launch
// with at most one batch per CTA needs no counter (and keeps its launch path to one call).
inline cudaError_t tickets_for(long long batches, long long grid, cudaStream_t stream,
                               unsigned long long** tickets) {
    *tickets = nullptr;
    if (batches <= grid) return cudaSuccess;
    return next_ticket_counter(stream, tickets);
}

}  // namespace ekl
