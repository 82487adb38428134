// Kernel selection and launch configuration.
#include <cstdlib>
#include <cstring>

#include "dispatch.h"
#include "generic_kernel.cuh"

namespace ekl {

int sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1)
            n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

namespace {

int round_up_warp(long long x, int cap) {
    long long t = ((x + 31) / 32) * 32;
    if (t > cap) t = cap;
    if (t < 32) t = 32;
    return (int)t;
}

template <typename T>
cudaError_t launch_ih_generic(const T* S, const T* D, const T* u, T* v, int n, long long E,
                              cudaStream_t stream) {
    const size_t smem = generic_ih_smem(n, sizeof(T));
    cudaError_t err = cudaFuncSetAttribute(inv_helmholtz_generic<T>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    const int threads = round_up_warp((long long)n * n * n, 512);
    int per_sm = 1;
    err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, inv_helmholtz_generic<T>, threads,
                                                        smem);
    if (err != cudaSuccess) return err;
    if (per_sm < 1) per_sm = 1;
    long long grid = (long long)sm_count() * per_sm;
    if (grid > E) grid = E;
    inv_helmholtz_generic<T><<<(unsigned)grid, threads, smem, stream>>>(S, D, u, v, n, E);
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_apply_generic(const T* A, const T* B, const T* C, const T* u, T* v, int n0,
                                 int n1, int n2, int m0, int m1, int m2, long long E,
                                 cudaStream_t stream) {
    const size_t smem = generic_apply_smem(n0, n1, n2, m0, m1, m2, sizeof(T));
    cudaError_t err = cudaFuncSetAttribute(apply_generic<T>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    const int threads = round_up_warp((long long)m0 * m1 * m2, 512);
    int per_sm = 1;
    err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, apply_generic<T>, threads, smem);
    if (err != cudaSuccess) return err;
    if (per_sm < 1) per_sm = 1;
    long long grid = (long long)sm_count() * per_sm;
    if (grid > E) grid = E;
    apply_generic<T><<<(unsigned)grid, threads, smem, stream>>>(
        A, B, C, u, v, n0, n1, n2, m0, m1, m2, (int)generic_apply_buf(n0, n1, n2, m1, m2), E);
    return cudaGetLastError();
}

}  // namespace

// EKL_TPO_VARIANT=generic forces the run-time-sized kernels (A/B measurements).
static bool tuned_allowed() {
    static const bool allowed = [] {
        const char* v = std::getenv("EKL_TPO_VARIANT");
        return !(v && std::strcmp(v, "generic") == 0);
    }();
    return allowed;
}

cudaError_t launch_convection_generic(const double* Dvq, const double* Ivq, const double* M,
                                      const double* P, double* F, int nq, int nv, long long E,
                                      cudaStream_t stream) {
    const size_t smem = generic_conv_smem(nq, nv);
    cudaError_t err = cudaFuncSetAttribute(convection_generic<double>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    const int threads = round_up_warp((long long)nq * nq * nv, 512);
    int per_sm = 1;
    err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, convection_generic<double>,
                                                        threads, smem);
    if (err != cudaSuccess) return err;
    if (per_sm < 1) per_sm = 1;
    long long grid = (long long)sm_count() * per_sm;
    if (grid > 3 * E) grid = 3 * E;
    convection_generic<double><<<(unsigned)grid, threads, smem, stream>>>(
        Dvq, Ivq, M, P, F, nq, nv, (int)generic_conv_buf(nq, nv), E);
    return cudaGetLastError();
}

bool tuned_kernels_allowed() { return tuned_allowed(); }

template <typename T>
cudaError_t launch_inv_helmholtz(const T* S, const T* D, const T* u, T* v, int n, long long E,
                                 cudaStream_t stream) {
    cudaError_t err = cudaSuccess;
    if (tuned_allowed() && try_launch_ih_dmma<T>(S, D, u, v, n, E, stream, &err)) return err;
    return launch_ih_generic<T>(S, D, u, v, n, E, stream);
}

template <typename T>
cudaError_t launch_apply(const T* A, const T* B, const T* C, const T* u, T* v, int n0, int n1,
                         int n2, int m0, int m1, int m2, long long E, cudaStream_t stream) {
    cudaError_t err = cudaSuccess;
    if (tuned_allowed() &&
        try_launch_apply_dmma<T>(A, B, C, u, v, n0, n1, n2, m0, m1, m2, E, stream, &err))
        return err;
    return launch_apply_generic<T>(A, B, C, u, v, n0, n1, n2, m0, m1, m2, E, stream);
}

template cudaError_t launch_inv_helmholtz<double>(const double*, const double*, const double*,
                                                  double*, int, long long, cudaStream_t);
template cudaError_t launch_inv_helmholtz<float>(const float*, const float*, const float*, float*,
                                                 int, long long, cudaStream_t);
template cudaError_t launch_apply<double>(const double*, const double*, const double*,
                                          const double*, double*, int, int, int, int, int, int,
                                          long long, cudaStream_t);
template cudaError_t launch_apply<float>(const float*, const float*, const float*, const float*,
                                         float*, int, int, int, int, int, int, long long,
                                         cudaStream_t);

}  // namespace ekl
