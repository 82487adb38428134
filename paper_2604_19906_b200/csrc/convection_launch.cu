// Entry point, instances and launcher of the convective-flux kernel.
#include "../../include/ekl_tpo.h"

#include <cstdint>

#include "convection_launch.h"
#include "dispatch.h"

namespace {

bool misaligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) != 0; }

bool overlaps(const void* a, size_t na, const void* b, size_t nb) {
    const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
    return na != 0 && nb != 0 && x < y + nb && y < x + na;
}

}  // namespace

namespace ekl {
int convection_timeout_flag() { return dmma::take_timeout_flag(); }
}  // namespace ekl

extern "C" ekl_tpo_status ekl_tpo_convection(const double* Dvq, const double* Ivq, const double* M,
                                             const double* P, double* F, int nq, int nv,
                                             long long E, cudaStream_t stream) {
    if (nq < 1 || nv < 1 || E < 0) return EKL_TPO_ERR_SHAPE;
    if (E == 0) return EKL_TPO_OK;
    if (!Dvq || !Ivq || !M || !P || !F) return EKL_TPO_ERR_NULL;
    if (nq > 64 || nv > 64 || ekl::generic_conv_smem(nq, nv) > ekl::kMaxSmemBytes)
        return EKL_TPO_ERR_UNSUPPORTED;
    if (misaligned(Dvq, 8) || misaligned(Ivq, 8) || misaligned(F, 8) || misaligned(M, 8) ||
        misaligned(P, 8))
        return EKL_TPO_ERR_ALIGN;
    // the tensor-path instances bulk-copy M and P where nq is even: 16-byte aligned fields
    const bool tensor_ok = ekl::tuned_kernels_allowed() &&
                           (nq % 2 != 0 || (!misaligned(M, 16) && !misaligned(P, 16)));
    const size_t q3 = (size_t)nq * nq * nq * sizeof(double), v3 = (size_t)nv * nv * nv * sizeof(double);
    const size_t fbytes = 3 * (size_t)E * v3, mat = (size_t)nv * nq * sizeof(double);
    if (overlaps(F, fbytes, M, (size_t)E * q3) || overlaps(F, fbytes, P, 9 * (size_t)E * q3) ||
        overlaps(F, fbytes, Dvq, mat) || overlaps(F, fbytes, Ivq, mat))
        return EKL_TPO_ERR_OVERLAP;
    cudaError_t err = cudaSuccess;
#define EKL_CONV_CASE(Q, V)                                                   \
    if (tensor_ok && nq == Q && nv == V) {                                    \
        err = ekl::launch_conv<Q, V>(Dvq, Ivq, M, P, F, E, stream);                \
        if (err != cudaSuccess) {                                             \
            ekl::set_last_cuda_error((int)err);                               \
            return EKL_TPO_ERR_CUDA;                                          \
        }                                                                     \
        return EKL_TPO_OK;                                                    \
    }
    EKL_CONV_CASE(4, 4)
    EKL_CONV_CASE(6, 4)
    EKL_CONV_CASE(6, 6)
    EKL_CONV_CASE(8, 4)
    EKL_CONV_CASE(8, 6)
    EKL_CONV_CASE(8, 8)
    EKL_CONV_CASE(10, 8)
    EKL_CONV_CASE(10, 10)
    EKL_CONV_CASE(12, 8)
    EKL_CONV_CASE(12, 10)
    EKL_CONV_CASE(12, 12)
    EKL_CONV_CASE(14, 12)
#undef EKL_CONV_CASE
    if (tensor_ok && ekl::try_launch_convection_odd(Dvq, Ivq, M, P, F, nq, nv, E, stream, &err)) {
        if (err != cudaSuccess) {
            ekl::set_last_cuda_error((int)err);
            return EKL_TPO_ERR_CUDA;
        }
        return EKL_TPO_OK;
    }
    err = ekl::launch_convection_generic(Dvq, Ivq, M, P, F, nq, nv, E, stream);
    if (err != cudaSuccess) {
        ekl::set_last_cuda_error((int)err);
        return EKL_TPO_ERR_CUDA;
    }
    return EKL_TPO_OK;
}
