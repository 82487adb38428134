// Forward-operator instances for shapes that are not cubic (even extents; fp64 fields with a
// 16-byte aligned u, or fp32 fields widened on the way in):
// operators that change the resolution in some directions only, and anisotropic elements.
#include <cstdint>

#include "apply_launch.h"
#include "dispatch.h"

namespace ekl {

template <typename T>
bool try_launch_apply_aniso(const T* A, const T* B, const T* C, const T* u, T* v, int n0, int n1,
                            int n2, int m0, int m1, int m2, long long E, cudaStream_t stream,
                            cudaError_t* err) {
    if (sizeof(T) == 8 && reinterpret_cast<uintptr_t>(u) % 16) return false;
#define EKL_AP_CASE(a, b, c, d, e, f)                                                   \
    if (n0 == a && n1 == b && n2 == c && m0 == d && m1 == e && m2 == f) {               \
        *err = launch_apply_instance<a, b, c, d, e, f, T>(A, B, C, u, v, E, stream);      \
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

template bool try_launch_apply_aniso<double>(const double*, const double*, const double*,
                                             const double*, double*, int, int, int, int, int, int,
                                             long long, cudaStream_t, cudaError_t*);
template bool try_launch_apply_aniso<float>(const float*, const float*, const float*, const float*,
                                            float*, int, int, int, int, int, int, long long,
                                            cudaStream_t, cudaError_t*);

int apply_aniso_timeout_flag() { return dmma::take_timeout_flag(); }

}  // namespace ekl
