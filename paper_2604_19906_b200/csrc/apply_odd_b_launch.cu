// Forward-operator instances on the FP64 tensor path, cubic n -> m with an odd extent: to and from the 3/2 quadrature resolution.
// Fields with an odd number of values per plane are copied in with 8-byte asynchronous copies
// instead of bulk copies (16-byte granules), so they need no alignment beyond their own.
#include "apply_launch.h"
#include "dispatch.h"

namespace ekl {

template <typename T>
bool try_launch_apply_odd_b(const T* A, const T* B, const T* C, const T* u, T* v, int n, int m,
                             long long E, cudaStream_t stream, cudaError_t* err) {
#define EKL_CASE(N_, M_)                                                                      \
    if (n == N_ && m == M_) {                                                                 \
        *err = launch_apply_instance<N_, N_, N_, M_, M_, M_, T>(A, B, C, u, v, E, stream);    \
        return true;                                                                          \
    }
    EKL_CASE(5, 8)
    EKL_CASE(8, 5)
    EKL_CASE(6, 9)
    EKL_CASE(9, 6)
    EKL_CASE(7, 11)
    EKL_CASE(11, 7)
    EKL_CASE(9, 14)
    EKL_CASE(14, 9)
    EKL_CASE(10, 15)
    EKL_CASE(15, 10)
#undef EKL_CASE
    return false;
}

template bool try_launch_apply_odd_b<double>(const double*, const double*, const double*,
                                              const double*, double*, int, int, long long,
                                              cudaStream_t, cudaError_t*);
template bool try_launch_apply_odd_b<float>(const float*, const float*, const float*, const float*,
                                             float*, int, int, long long, cudaStream_t,
                                             cudaError_t*);

int apply_odd_b_timeout_flag() { return dmma::take_timeout_flag(); }

}  // namespace ekl
