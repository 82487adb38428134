// Forward-operator instances for shapes that are not cubic (fp64, even extents, 16-byte aligned u):
// operators that change the resolution in some directions only, and anisotropic elements.
#include <cstdint>

#include "apply_launch.h"
#include "dispatch.h"

namespace ekl {

bool try_launch_apply_aniso(const double* A, const double* B, const double* C, const double* u,
                            double* v, int n0, int n1, int n2, int m0, int m1, int m2, long long E,
                            cudaStream_t stream, cudaError_t* err) {
    if (reinterpret_cast<uintptr_t>(u) % 16) return false;
#define EKL_AP_CASE(a, b, c, d, e, f)                                                   \
    if (n0 == a && n1 == b && n2 == c && m0 == d && m1 == e && m2 == f) {               \
        *err = launch_apply_instance<a, b, c, d, e, f, double>(A, B, C, u, v, E, stream); \
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
