// Launch of one convective-flux instance on the FP64 tensor path; shared by the translation
// units that hold the instances.
#pragma once
#include "convection_dmma.cuh"
#include "dispatch.h"
#include "launch_util.h"

namespace ekl {

template <int NQ, int NV>
cudaError_t launch_conv(const double* Dvq, const double* Ivq, const double* M, const double* P,
                        double* F, long long E, cudaStream_t stream) {
    using C = dmma::ConvCfg<NQ, NV>;
    static_assert(C::kSmemBytes <= kMaxSmemBytes, "instance does not fit in shared memory");
    static std::atomic<int> prepared[64];   // racing first calls store the same value
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!prepared[dev].load(std::memory_order_acquire)) {
        err = cudaFuncSetAttribute(dmma::convection_dmma<NQ, NV>,
                                   cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::kSmemBytes);
        if (err != cudaSuccess) return err;
        prepared[dev].store(1, std::memory_order_release);
    }
    long long grid = (long long)sm_count() * C::kCtasPerSm;
    if (grid > E) grid = E;
    // no ticket counter: the elements are dealt round-robin (every element costs the same here,
    // and the fixed deal measured 0.5 % faster than the dynamic one)
    unsigned long long* tickets = nullptr;
    dmma::convection_dmma<NQ, NV><<<(unsigned)grid, C::kThreads, C::kSmemBytes, stream>>>(
        Dvq, Ivq, M, P, F, E, tickets);
    return cudaGetLastError();
}

}  // namespace ekl
