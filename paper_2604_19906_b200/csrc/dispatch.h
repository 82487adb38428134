// Host-side kernel selection shared by the entry points.
#pragma once
#include <cuda_runtime.h>

#include <cstddef>

namespace ekl {

// Largest dynamic shared memory a CTA may opt into on sm_100.
constexpr size_t kMaxSmemBytes = 227 * 1024;

// Shared memory the run-time-sized inverse-Helmholtz kernel needs: S + two element buffers.
inline size_t generic_ih_smem(int n, size_t elem) {
    return ((size_t)n * n + 2 * (size_t)n * n * n) * elem;
}

// Largest cubic extent the library accepts for elements of `elem` bytes.
inline int max_cubic_extent(size_t elem) {
    int n = 1;
    while (generic_ih_smem(n + 1, elem) <= kMaxSmemBytes) ++n;
    return n;
}

// The same for one operator and one extent per direction: three matrices + two element buffers.
inline size_t generic_ih3_smem(int n0, int n1, int n2, size_t elem) {
    return ((size_t)n0 * n0 + (size_t)n1 * n1 + (size_t)n2 * n2 + 2 * (size_t)n0 * n1 * n2) * elem;
}
inline bool ih3_fits(int n0, int n1, int n2, size_t elem) {
    if ((double)n0 * n1 * n2 > 1.0e6 || n0 > 1000 || n1 > 1000 || n2 > 1000) return false;
    return generic_ih3_smem(n0, n1, n2, elem) <= kMaxSmemBytes;
}

// Elements of one ping-pong buffer of the run-time-sized forward kernel.
inline size_t generic_apply_buf(int n0, int n1, int n2, int m1, int m2) {
    size_t a = (size_t)n0 * n1 * n2, b = (size_t)n0 * n1 * m2, c = (size_t)n0 * m1 * m2;
    size_t even = a > c ? a : c;  // buffer 0 holds u then q, buffer 1 holds p
    return even > b ? even : b;
}

inline size_t generic_apply_smem(int n0, int n1, int n2, int m0, int m1, int m2, size_t elem) {
    return ((size_t)m0 * n0 + (size_t)m1 * n1 + (size_t)m2 * n2 +
            2 * generic_apply_buf(n0, n1, n2, m1, m2)) * elem;
}

inline bool apply_fits(int n0, int n1, int n2, int m0, int m1, int m2, size_t elem) {
    // guard the products against overflow before comparing
    const double est = ((double)n0 * n1 * n2 + (double)n0 * n1 * m2 + (double)n0 * m1 * m2 +
                        (double)m0 * n0 + (double)m1 * n1 + (double)m2 * n2) * (double)elem;
    if (est > 4.0 * (double)kMaxSmemBytes) return false;
    if ((double)m0 * m1 * m2 > 2.0e9) return false;
    return generic_apply_smem(n0, n1, n2, m0, m1, m2, elem) <= kMaxSmemBytes;
}

// Records the cudaError_t that ekl_tpo_last_cuda_error() reports for the calling thread.
void set_last_cuda_error(int err);

// Run-time-sized convective-flux kernel: elements of one ping-pong buffer, total shared
// memory, launcher.
inline size_t generic_conv_buf(int nq, int nv) {
    size_t a = (size_t)nq * nq * nq, b = (size_t)nq * nq * nv, c = (size_t)nq * nv * nv,
           d = (size_t)nv * nv * nv;
    size_t m = a > b ? a : b;
    m = m > c ? m : c;
    return m > d ? m : d;
}
inline size_t generic_conv_smem(int nq, int nv) {
    return (2 * (size_t)nv * nq + 2 * generic_conv_buf(nq, nv) + (size_t)nv * nv * nv) *
           sizeof(double);
}
cudaError_t launch_convection_generic(const double* Dvq, const double* Ivq, const double* M,
                                      const double* P, double* F, int nq, int nv, long long E,
                                      cudaStream_t stream);

// Convective-flux instances with an odd extent; false if there is none for (nq, nv).
bool try_launch_convection_odd(const double* Dvq, const double* Ivq, const double* M,
                               const double* P, double* F, int nq, int nv, long long E,
                               cudaStream_t stream, cudaError_t* err);

// Device error flags of the convective-flux kernels and of the per-direction inverse
// Helmholtz kernels (see ekl_tpo_device_error_flags).
int convection_timeout_flag();
int convection_odd_timeout_flag();
int ih3_timeout_flag();
int ih3_odd_timeout_flag();
int apply_aniso_timeout_flag();
int apply_odd_a_timeout_flag();
int apply_odd_b_timeout_flag();
int apply_odd_c_timeout_flag();

// False when EKL_TPO_VARIANT=generic asks for the run-time-sized kernels only.
bool tuned_kernels_allowed();

// Number of SMs of the current device (cached per device).
int sm_count();

// A ticket counter (two 64-bit words, zero) for one launch; see launch.cu.
cudaError_t next_ticket_counter(unsigned long long** out);

// Tensor-path kernels (fp64 arithmetic; T is the type of the fields in memory).  Return false
// if there is no instance for these extents or the pointers do not meet the alignment the
// instance needs; otherwise launch and set *err.
template <typename T>
bool try_launch_ih_dmma(const T* S, const T* D, const T* u, T* v, int n, long long E,
                        cudaStream_t stream, cudaError_t* err);
// Same, with the pointwise factor formed from lam[n] and c[E] instead of read from a field.
bool try_launch_ih_lambda_dmma(const double* S, const double* lam, const double* cvec,
                               const double* u, double* v, int n, long long E, cudaStream_t stream,
                               cudaError_t* err);
// One operator and one extent per direction (fp64).
bool try_launch_ih3_dmma(const double* S0, const double* S1, const double* S2, const double* D,
                         const double* u, double* v, int n0, int n1, int n2, long long E,
                         cudaStream_t stream, cudaError_t* err);
// The instances of that with an odd extent (their own translation unit).
bool try_launch_ih3_odd(const double* S0, const double* S1, const double* S2, const double* D,
                        const double* u, double* v, int n0, int n1, int n2, long long E,
                        cudaStream_t stream, cudaError_t* err);
// Forward operator, shapes that are not cubic.
template <typename T>
bool try_launch_apply_aniso(const T* A, const T* B, const T* C, const T* u, T* v, int n0, int n1,
                            int n2, int m0, int m1, int m2, long long E, cudaStream_t stream,
                            cudaError_t* err);
// Forward operator, cubic n -> m with an odd extent (three groups of instances, one translation
// unit each).
template <typename T>
bool try_launch_apply_odd_a(const T* A, const T* B, const T* C, const T* u, T* v, int n, int m,
                            long long E, cudaStream_t stream, cudaError_t* err);
template <typename T>
bool try_launch_apply_odd_b(const T* A, const T* B, const T* C, const T* u, T* v, int n, int m,
                            long long E, cudaStream_t stream, cudaError_t* err);
template <typename T>
bool try_launch_apply_odd_c(const T* A, const T* B, const T* C, const T* u, T* v, int n, int m,
                            long long E, cudaStream_t stream, cudaError_t* err);
template <typename T>
bool try_launch_apply_dmma(const T* A, const T* B, const T* C, const T* u, T* v, int n0, int n1,
                           int n2, int m0, int m1, int m2, long long E, cudaStream_t stream,
                           cudaError_t* err);

template <typename T>
cudaError_t launch_inv_helmholtz(const T* S, const T* D, const T* u, T* v, int n, long long E,
                                 cudaStream_t stream);

cudaError_t launch_inv_helmholtz3(const double* S0, const double* S1, const double* S2,
                                  const double* D, const double* u, double* v, int n0, int n1,
                                  int n2, long long E, cudaStream_t stream);

template <typename T>
cudaError_t launch_apply(const T* A, const T* B, const T* C, const T* u, T* v, int n0, int n1,
                         int n2, int m0, int m1, int m2, long long E, cudaStream_t stream);

}  // namespace ekl
