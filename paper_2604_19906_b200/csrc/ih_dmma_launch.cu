// Instances and launcher of the tensor-path inverse-Helmholtz kernel.
#include <cstdint>

#include "dispatch.h"
#include "ih_dmma.cuh"

namespace ekl {
namespace {

template <int N>
cudaError_t launch_n(const double* S, const double* D, const double* u, double* v, long long E,
                     cudaStream_t stream) {
    using C = dmma::Cfg<N>;
    cudaError_t err = cudaFuncSetAttribute(dmma::inv_helmholtz_dmma<N>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)C::kSmemBytes);
    if (err != cudaSuccess) return err;
    const long long batches = (E + C::kBe - 1) / C::kBe;
    int per_sm = 1;
    err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, dmma::inv_helmholtz_dmma<N>,
                                                        C::kThreads, C::kSmemBytes);
    if (err != cudaSuccess) return err;
    if (per_sm < 1) per_sm = 1;
    long long grid = (long long)sm_count() * per_sm;
    if (grid > batches) grid = batches;
    dmma::inv_helmholtz_dmma<N><<<(unsigned)grid, C::kThreads, C::kSmemBytes, stream>>>(S, D, u, v, E);
    return cudaGetLastError();
}

}  // namespace

bool try_launch_ih_dmma(const double* S, const double* D, const double* u, double* v, int n,
                        long long E, cudaStream_t stream, cudaError_t* err) {
    // the bulk copy of u needs 16-byte aligned element addresses (8 n^3 is a multiple of 16
    // for every even n)
    if (reinterpret_cast<uintptr_t>(u) % 16) return false;
    switch (n) {
        case 6: *err = launch_n<6>(S, D, u, v, E, stream); return true;
        case 10: *err = launch_n<10>(S, D, u, v, E, stream); return true;
        case 14: *err = launch_n<14>(S, D, u, v, E, stream); return true;
        default: return false;
    }
}

}  // namespace ekl
