// Launch of one per-direction inverse Helmholtz instance; shared by the translation units that
// hold the instances.
#pragma once
#include "dispatch.h"
#include "launch_util.h"
#include "tpo_dmma.cuh"

namespace ekl {

// One operator and one extent per direction (fp64).
template <int N0, int N1, int N2>
cudaError_t launch_ih3(const double* S0, const double* S1, const double* S2, const double* D,
                       const double* u, double* v, long long E, cudaStream_t stream) {
    using C = dmma::Ih3Cfg<N0, N1, N2>;
    auto kernel = dmma::inv_helmholtz3_dmma<N0, N1, N2>;
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
    kernel<<<(unsigned)grid, C::kThreads, C::kSmemBytes, stream>>>(S0, S1, S2, D, u, v, E, tickets);
    return cudaGetLastError();
}

}  // namespace ekl
