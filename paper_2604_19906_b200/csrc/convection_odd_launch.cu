// Convective-flux instances with an odd extent (fields whose planes hold an odd number of values
// come in by 8-byte asynchronous copies instead of bulk copies).
#include "convection_launch.h"

namespace ekl {

bool try_launch_convection_odd(const double* Dvq, const double* Ivq, const double* M,
                               const double* P, double* F, int nq, int nv, long long E,
                               cudaStream_t stream, cudaError_t* err) {
#define EKL_CASE(Q, V)                                                  \
    if (nq == Q && nv == V) {                                           \
        *err = launch_conv<Q, V>(Dvq, Ivq, M, P, F, E, stream);         \
        return true;                                                    \
    }
    EKL_CASE(5, 5)
    EKL_CASE(7, 5)
    EKL_CASE(7, 7)
    EKL_CASE(8, 5)
    EKL_CASE(9, 6)
    EKL_CASE(9, 7)
    EKL_CASE(9, 9)
    EKL_CASE(11, 7)
    EKL_CASE(14, 9)
    EKL_CASE(15, 10)
#undef EKL_CASE
    return false;
}

int convection_odd_timeout_flag() { return dmma::take_timeout_flag(); }

}  // namespace ekl
