// Per-direction inverse Helmholtz instances with an odd extent.
#include "ih3_launch.h"

namespace ekl {

bool try_launch_ih3_odd(const double* S0, const double* S1, const double* S2, const double* D,
                        const double* u, double* v, int n0, int n1, int n2, long long E,
                        cudaStream_t stream, cudaError_t* err) {
#define EKL_IH3_CASE(A_, B_, C_)                                                  \
    if (n0 == A_ && n1 == B_ && n2 == C_) {                                       \
        *err = launch_ih3<A_, B_, C_>(S0, S1, S2, D, u, v, E, stream);            \
        return true;                                                              \
    }
    EKL_IH3_CASE(5, 5, 5)
    EKL_IH3_CASE(7, 7, 7)
    EKL_IH3_CASE(9, 9, 9)
    EKL_IH3_CASE(11, 11, 11)
    EKL_IH3_CASE(13, 13, 13)
    EKL_IH3_CASE(15, 15, 15)
    EKL_IH3_CASE(5, 7, 9)
    EKL_IH3_CASE(9, 7, 5)
    EKL_IH3_CASE(6, 7, 8)
    EKL_IH3_CASE(7, 8, 9)
#undef EKL_IH3_CASE
    return false;
}

int ih3_odd_timeout_flag() { return dmma::take_timeout_flag(); }

}  // namespace ekl
