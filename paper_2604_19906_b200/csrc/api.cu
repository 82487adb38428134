// C-ABI entry points: argument validation on the host, choice of kernel, launch.
#include "../../include/ekl_tpo.h"

#include <cstdint>
#include <cstdlib>
#include <cstring>

#include "dispatch.h"

namespace {
thread_local int g_last_cuda_error = 0;
}

namespace ekl {
void set_last_cuda_error(int err) { g_last_cuda_error = err; }
}  // namespace ekl

namespace {

ekl_tpo_status cuda_fail(cudaError_t err) {
    g_last_cuda_error = (int)err;
    return EKL_TPO_ERR_CUDA;
}

bool misaligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) != 0; }

// Do [a, a+na) and [b, b+nb) share a byte?
bool overlaps(const void* a, size_t na, const void* b, size_t nb) {
    const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
    return na != 0 && nb != 0 && x < y + nb && y < x + na;
}

template <typename T>
ekl_tpo_status inv_helmholtz_impl(const T* S, const T* D, const T* u, T* v, int n, long long E,
                                  cudaStream_t stream) {
    if (n < 1 || E < 0) return EKL_TPO_ERR_SHAPE;
    if (E == 0) return EKL_TPO_OK;
    if (!S || !D || !u || !v) return EKL_TPO_ERR_NULL;
    if (n > ekl::max_cubic_extent(sizeof(T))) return EKL_TPO_ERR_UNSUPPORTED;
    if (misaligned(S, sizeof(T)) || misaligned(D, sizeof(T)) || misaligned(u, sizeof(T)) ||
        misaligned(v, sizeof(T)))
        return EKL_TPO_ERR_ALIGN;
    const size_t field = (size_t)E * n * n * n * sizeof(T), mat = (size_t)n * n * sizeof(T);
    if (overlaps(v, field, S, mat) || overlaps(v, field, D, field)) return EKL_TPO_ERR_OVERLAP;
    if ((const void*)v != (const void*)u && overlaps(v, field, u, field))
        return EKL_TPO_ERR_OVERLAP;
    const cudaError_t err = ekl::launch_inv_helmholtz<T>(S, D, u, v, n, E, stream);
    return err == cudaSuccess ? EKL_TPO_OK : cuda_fail(err);
}

template <typename T>
ekl_tpo_status apply_impl(const T* A, const T* B, const T* C, const T* u, T* v, int n0, int n1,
                          int n2, int m0, int m1, int m2, long long E, cudaStream_t stream) {
    if (n0 < 1 || n1 < 1 || n2 < 1 || m0 < 1 || m1 < 1 || m2 < 1 || E < 0)
        return EKL_TPO_ERR_SHAPE;
    if (E == 0) return EKL_TPO_OK;
    if (!A || !B || !C || !u || !v) return EKL_TPO_ERR_NULL;
    if (!ekl::apply_fits(n0, n1, n2, m0, m1, m2, sizeof(T))) return EKL_TPO_ERR_UNSUPPORTED;
    if (misaligned(A, sizeof(T)) || misaligned(B, sizeof(T)) || misaligned(C, sizeof(T)) ||
        misaligned(u, sizeof(T)) || misaligned(v, sizeof(T)))
        return EKL_TPO_ERR_ALIGN;
    const size_t nin = (size_t)E * n0 * n1 * n2 * sizeof(T);
    const size_t nout = (size_t)E * m0 * m1 * m2 * sizeof(T);
    if (overlaps(v, nout, u, nin) || overlaps(v, nout, A, (size_t)m0 * n0 * sizeof(T)) ||
        overlaps(v, nout, B, (size_t)m1 * n1 * sizeof(T)) ||
        overlaps(v, nout, C, (size_t)m2 * n2 * sizeof(T)))
        return EKL_TPO_ERR_OVERLAP;
    const cudaError_t err =
        ekl::launch_apply<T>(A, B, C, u, v, n0, n1, n2, m0, m1, m2, E, stream);
    return err == cudaSuccess ? EKL_TPO_OK : cuda_fail(err);
}

}  // namespace

extern "C" {

ekl_tpo_status ekl_tpo_inv_helmholtz(const double* S, const double* D, const double* u,
                                     double* v, int n, long long E, cudaStream_t stream) {
    return inv_helmholtz_impl<double>(S, D, u, v, n, E, stream);
}

ekl_tpo_status ekl_tpo_inv_helmholtz_f32(const float* S, const float* D, const float* u, float* v,
                                         int n, long long E, cudaStream_t stream) {
    return inv_helmholtz_impl<float>(S, D, u, v, n, E, stream);
}

ekl_tpo_status ekl_tpo_apply(const double* A, const double* B, const double* C, const double* u,
                             double* v, int n0, int n1, int n2, int m0, int m1, int m2,
                             long long E, cudaStream_t stream) {
    return apply_impl<double>(A, B, C, u, v, n0, n1, n2, m0, m1, m2, E, stream);
}

ekl_tpo_status ekl_tpo_apply_f32(const float* A, const float* B, const float* C, const float* u,
                                 float* v, int n0, int n1, int n2, int m0, int m1, int m2,
                                 long long E, cudaStream_t stream) {
    return apply_impl<float>(A, B, C, u, v, n0, n1, n2, m0, m1, m2, E, stream);
}

ekl_tpo_status ekl_tpo_inv_helmholtz_lambda(const double* S, const double* lam, const double* c,
                                            const double* u, double* v, int n, long long E,
                                            cudaStream_t stream) {
    if (n < 1 || E < 0) return EKL_TPO_ERR_SHAPE;
    if (E == 0) return EKL_TPO_OK;
    if (!S || !lam || !c || !u || !v) return EKL_TPO_ERR_NULL;
    if (n < 4 || n > 20) return EKL_TPO_ERR_UNSUPPORTED;
    if (misaligned(S, 8) || misaligned(lam, 8) || misaligned(c, 8) || misaligned(u, 8) ||
        misaligned(v, 8) || (n % 2 == 0 && misaligned(u, 16)))
        return EKL_TPO_ERR_ALIGN;
    const size_t field = (size_t)E * n * n * n * sizeof(double);
    if (overlaps(v, field, S, (size_t)n * n * sizeof(double)) ||
        overlaps(v, field, lam, (size_t)n * sizeof(double)) ||
        overlaps(v, field, c, (size_t)E * sizeof(double)) ||
        ((const void*)v != (const void*)u && overlaps(v, field, u, field)))
        return EKL_TPO_ERR_OVERLAP;
    cudaError_t err = cudaSuccess;
    if (!ekl::try_launch_ih_lambda_dmma(S, lam, c, u, v, n, E, stream, &err))
        return EKL_TPO_ERR_UNSUPPORTED;
    return err == cudaSuccess ? EKL_TPO_OK : cuda_fail(err);
}

ekl_tpo_status ekl_tpo_inv_helmholtz3(const double* S0, const double* S1, const double* S2,
                                      const double* D, const double* u, double* v, int n0, int n1,
                                      int n2, long long E, cudaStream_t stream) {
    if (n0 < 1 || n1 < 1 || n2 < 1 || E < 0) return EKL_TPO_ERR_SHAPE;
    if (E == 0) return EKL_TPO_OK;
    if (!S0 || !S1 || !S2 || !D || !u || !v) return EKL_TPO_ERR_NULL;
    if (!ekl::ih3_fits(n0, n1, n2, sizeof(double))) return EKL_TPO_ERR_UNSUPPORTED;
    if (misaligned(S0, 8) || misaligned(S1, 8) || misaligned(S2, 8) || misaligned(D, 8) ||
        misaligned(u, 8) || misaligned(v, 8))
        return EKL_TPO_ERR_ALIGN;
    const size_t field = (size_t)E * n0 * n1 * n2 * sizeof(double);
    if (overlaps(v, field, S0, (size_t)n0 * n0 * sizeof(double)) ||
        overlaps(v, field, S1, (size_t)n1 * n1 * sizeof(double)) ||
        overlaps(v, field, S2, (size_t)n2 * n2 * sizeof(double)) || overlaps(v, field, D, field))
        return EKL_TPO_ERR_OVERLAP;
    if ((const void*)v != (const void*)u && overlaps(v, field, u, field))
        return EKL_TPO_ERR_OVERLAP;
    const cudaError_t err = ekl::launch_inv_helmholtz3(S0, S1, S2, D, u, v, n0, n1, n2, E, stream);
    return err == cudaSuccess ? EKL_TPO_OK : cuda_fail(err);
}

const char* ekl_tpo_status_string(ekl_tpo_status status) {
    switch (status) {
        case EKL_TPO_OK: return "ok";
        case EKL_TPO_ERR_NULL: return "null pointer";
        case EKL_TPO_ERR_SHAPE: return "invalid extent or element count";
        case EKL_TPO_ERR_UNSUPPORTED: return "extents too large for on-chip memory";
        case EKL_TPO_ERR_ALIGN: return "pointer not aligned to its element type";
        case EKL_TPO_ERR_OVERLAP: return "output overlaps an input";
        case EKL_TPO_ERR_CUDA: return "CUDA runtime error (see ekl_tpo_last_cuda_error)";
    }
    return "unknown status";
}

int ekl_tpo_version(void) { return 100; }

int ekl_tpo_last_cuda_error(void) { return g_last_cuda_error; }

}  // extern "C"
