// Forward-operator instances for shapes that are not cubic (fp64, even extents, 16-byte aligned u):
// operators that change the resolution in some directions only, and anisotropic elements.
#include <cstdint>

#include "dispatch.h"
#include "launch_util.h"
#include "tpo_dmma.cuh"

namespace ekl {
namespace {

template <int N0, int N1, int N2, int M0, int M1, int M2>
cudaError_t launch_ap(const double* A, const double* B, const double* Cm, const double* u, double* v,
                      long long E, cudaStream_t stream) {
    using C = dmma::ApplyCfg<N0, N1, N2, M0, M1, M2>;
    auto kernel = dmma::apply_dmma<N0, N1, N2, M0, M1, M2, double>;
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

}  // namespace

bool try_launch_apply_aniso(const double* A, const double* B, const double* C, const double* u,
                            double* v, int n0, int n1, int n2, int m0, int m1, int m2, long long E,
                            cudaStream_t stream, cudaError_t* err) {
    if (reinterpret_cast<uintptr_t>(u) % 16) return false;
#define EKL_AP_CASE(a, b, c, d, e, f)                                                   \
    if (n0 == a && n1 == b && n2 == c && m0 == d && m1 == e && m2 == f) {               \
        *err = launch_ap<a, b, c, d, e, f>(A, B, C, u, v, E, stream);                   \
        return true;                                                                    \
    }
    EKL_AP_CASE(8, 8, 8, 12, 12, 8)
    EKL_AP_CASE(8, 8, 8, 8, 8, 12)
    EKL_AP_CASE(12, 12, 12, 8, 8, 12)
    EKL_AP_CASE(12, 12, 8, 8, 8, 12)
    EKL_AP_CASE(8, 10, 12, 12, 10, 8)
    EKL_AP_CASE(8, 10, 12, 8, 10, 12)
    EKL_AP_CASE(6, 8, 10, 10, 8, 6)
    EKL_AP_CASE(14, 12, 8, 8, 12, 14)
#undef EKL_AP_CASE
    return false;
}

int apply_aniso_timeout_flag() { return dmma::take_timeout_flag(); }

}  // namespace ekl
