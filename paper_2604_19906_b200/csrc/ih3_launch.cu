// Instances and launcher of the inverse Helmholtz kernel with one operator per direction.
#include <cstdint>

#include "dispatch.h"
#include "launch_util.h"
#include "tpo_dmma.cuh"

namespace ekl {
namespace {

// One operator and one extent per direction (fp64, even extents, 16-byte aligned u).
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

}  // namespace

bool try_launch_ih3_dmma(const double* S0, const double* S1, const double* S2, const double* D,
                         const double* u, double* v, int n0, int n1, int n2, long long E,
                         cudaStream_t stream, cudaError_t* err) {
    if (reinterpret_cast<uintptr_t>(u) % 16) return false;
#define EKL_IH3_CASE(A_, B_, C_)                                                  \
    if (n0 == A_ && n1 == B_ && n2 == C_) {                                       \
        *err = launch_ih3<A_, B_, C_>(S0, S1, S2, D, u, v, E, stream);            \
        return true;                                                              \
    }
    // cubic shapes with three operators
    EKL_IH3_CASE(8, 8, 8)
    EKL_IH3_CASE(10, 10, 10)
    EKL_IH3_CASE(12, 12, 12)
    EKL_IH3_CASE(14, 14, 14)
    EKL_IH3_CASE(16, 16, 16)
    // anisotropic shapes
    EKL_IH3_CASE(8, 10, 12)
    EKL_IH3_CASE(12, 10, 8)
    EKL_IH3_CASE(14, 12, 8)
    EKL_IH3_CASE(8, 8, 16)
    EKL_IH3_CASE(16, 8, 8)
#undef EKL_IH3_CASE
    return false;
}


int ih3_timeout_flag() { return dmma::take_timeout_flag(); }

}  // namespace ekl
