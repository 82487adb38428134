// Launch of one forward-operator instance on the FP64 tensor path; shared by the translation
// units that hold the instances.
#pragma once
#include "launch_util.h"
#include "tpo_dmma.cuh"

namespace ekl {

template <int N0, int N1, int N2, int M0, int M1, int M2, typename T>
cudaError_t launch_apply_instance(const T* A, const T* B, const T* Cm, const T* u, T* v,
                                  long long E, cudaStream_t stream) {
    using C = dmma::ApplyCfg<N0, N1, N2, M0, M1, M2>;
    auto kernel = dmma::apply_dmma<N0, N1, N2, M0, M1, M2, T>;
    static std::atomic<int> cached[64];
    int per_sm = 1;
    cudaError_t err = ctas_per_sm(kernel, C::kThreads, C::kSmemBytes, cached, &per_sm);
    if (err != cudaSuccess) return err;
    const long long batches = (E + C::kBe - 1) / C::kBe;
    long long grid = (long long)sm_count() * per_sm;
    if (grid > batches) grid = batches;
    unsigned long long* tickets = nullptr;
    err = tickets_for(batches, grid, &tickets);
    if (err != cudaSuccess) return err;
    kernel<<<(unsigned)grid, C::kThreads, C::kSmemBytes, stream>>>(A, B, Cm, u, v, E, tickets);
    return cudaGetLastError();
}

}  // namespace ekl
