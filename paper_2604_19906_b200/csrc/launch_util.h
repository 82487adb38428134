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

// Batches are handed out dynamically from the third batch of a CTA on (the first two are
// fixed).  A launch with up to four batches per CTA keeps the fixed round-robin deal: it is
// over in microseconds and the counter's atomics would cost more than the balance gains
// (measured at n = 8, E = 4096).
inline cudaError_t tickets_for(long long batches, long long grid, unsigned long long** tickets) {
    *tickets = nullptr;
    if (batches <= 4 * grid) return cudaSuccess;
    return next_ticket_counter(tickets);
}

}  // namespace ekl
