// Instances and launcher of the inverse Helmholtz kernel with one operator per direction.
#include <cstdint>

#include "ih3_launch.h"

namespace ekl {

bool try_launch_ih3_dmma(const double* S0, const double* S1, const double* S2, const double* D,
                         const double* u, double* v, int n0, int n1, int n2, long long E,
                         cudaStream_t stream, cudaError_t* err) {
    // bulk copies of u (planes that are whole 16-byte units) need 16-byte aligned elements
    if ((n1 * n2) % 2 == 0 && reinterpret_cast<uintptr_t>(u) % 16) return false;
#define EKL_IH3_CASE(A_, B_, C_)                                                  \
    if (n0 == A_ && n1 == B_ && n2 == C_) {                                       \
        *err = launch_ih3<A_, B_, C_>(S0, S1, S2, D, u, v, E, stream);            \
        return true;                                                              \
    }
    // cubic shapes with three operators
    EKL_IH3_CASE(4, 4, 4)
    EKL_IH3_CASE(6, 6, 6)
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
    return try_launch_ih3_odd(S0, S1, S2, D, u, v, n0, n1, n2, E, stream, err);
}


int ih3_timeout_flag() { return dmma::take_timeout_flag(); }

}  // namespace ekl
