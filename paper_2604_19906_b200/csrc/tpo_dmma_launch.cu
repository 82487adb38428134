// Instances and launchers of the tensor-path kernels.
#include "../../include/ekl_tpo.h"

#include <cstdint>

#include "dispatch.h"
#include "launch_util.h"
#include "tpo_dmma.cuh"
#include "tpo_tf32.cuh"
#include "tpo_umma.cuh"
#include "apply_launch.h"

#include <cstdlib>
#include <cstring>

namespace ekl {
namespace {

template <int N, typename T, bool LAMBDA>
cudaError_t launch_ih(const T* S, const T* D, const double* lam, const double* cvec, const T* u, T* v,
                      long long E, cudaStream_t stream) {
    using C = dmma::IhCfg<N, T>;
    static std::atomic<int> cached[64];
    int per_sm = 1;
    cudaError_t err = ctas_per_sm(dmma::inv_helmholtz_dmma<N, T, LAMBDA>, C::kThreads,
                                  C::kSmemBytes, cached, &per_sm);
    if (err != cudaSuccess) return err;
    const long long batches = (E + C::kBe - 1) / C::kBe;
    long long grid = (long long)sm_count() * per_sm;
    if (grid > batches) grid = batches;
    unsigned long long* tickets = nullptr;
    err = tickets_for(batches, grid, &tickets);
    if (err != cudaSuccess) return err;
    dmma::inv_helmholtz_dmma<N, T, LAMBDA>
        <<<(unsigned)grid, C::kThreads, C::kSmemBytes, stream>>>(S, D, lam, cvec, u, v, E, tickets);
    return cudaGetLastError();
}

// Single precision, split-TF32 tensor path (even extents 8..16, 16-byte aligned u).
template <int N>
cudaError_t launch_ih_tf32(const float* S, const float* D, const float* u, float* v, long long E,
                           cudaStream_t stream) {
    using C = tf32::IhCfg32<N>;
    static std::atomic<int> cached[64];
    int per_sm = 1;
    cudaError_t err = ctas_per_sm(tf32::inv_helmholtz_tf32<N>, C::kThreads, C::kSmemBytes, cached,
                                  &per_sm);
    if (err != cudaSuccess) return err;
    const long long batches = (E + C::kBe - 1) / C::kBe;
    long long grid = (long long)sm_count() * per_sm;
    if (grid > batches) grid = batches;
    unsigned long long* tickets = nullptr;
    err = tickets_for(batches, grid, &tickets);
    if (err != cudaSuccess) return err;
    tf32::inv_helmholtz_tf32<N>
        <<<(unsigned)grid, C::kThreads, C::kSmemBytes, stream>>>(S, D, u, v, E, tickets);
    return cudaGetLastError();
}

// The same operator on the asynchronous tensor path (tcgen05.mma, accumulator in tensor memory).
// It is correct but slower here (the 16-column operator makes every tensor instruction re-read
// its 128-row operand from shared memory), so it only runs when EKL_TPO_F32_PATH=tcgen05 asks
// for it (A/B measurements).
template <int N>
cudaError_t launch_ih_umma(const float* S, const float* D, const float* u, float* v, long long E,
                           cudaStream_t stream) {
    using C = umma::Cfg<N>;
    static std::atomic<int> ready[64];   // racing first calls store the same value
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!ready[dev].load(std::memory_order_acquire)) {
        err = cudaFuncSetAttribute(umma::inv_helmholtz_umma<N>,
                                   cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::kSmemBytes);
        if (err != cudaSuccess) return err;
        ready[dev].store(1, std::memory_order_release);
    }
    // as many CTAs as shared memory lets an SM hold (the occupancy query answers 1 for kernels
    // that allocate tensor memory; more do run side by side, 32 columns each)
    long long grid = (long long)sm_count() * C::kCtasPerSm;
    if (grid > E) grid = E;
    umma::inv_helmholtz_umma<N><<<(unsigned)grid, C::kThreads, C::kSmemBytes, stream>>>(S, D, u, v, E);
    return cudaGetLastError();
}

static bool f32_path_is_tcgen05() {
    static const bool on = [] {
        const char* p = std::getenv("EKL_TPO_F32_PATH");
        return p && std::strcmp(p, "tcgen05") == 0;
    }();
    return on;
}

bool try_launch_ih_tf32(const float* S, const float* D, const float* u, float* v, int n, long long E,
                        cudaStream_t stream, cudaError_t* err) {
    if (reinterpret_cast<uintptr_t>(u) % 16) return false;
    if (f32_path_is_tcgen05() && reinterpret_cast<uintptr_t>(D) % 8 == 0 &&
        reinterpret_cast<uintptr_t>(v) % 8 == 0) {
        switch (n) {
            case 8: *err = launch_ih_umma<8>(S, D, u, v, E, stream); return true;
            case 10: *err = launch_ih_umma<10>(S, D, u, v, E, stream); return true;
            case 12: *err = launch_ih_umma<12>(S, D, u, v, E, stream); return true;
            case 14: *err = launch_ih_umma<14>(S, D, u, v, E, stream); return true;
            case 16: *err = launch_ih_umma<16>(S, D, u, v, E, stream); return true;
            default: break;
        }
    }
    switch (n) {
        case 8: *err = launch_ih_tf32<8>(S, D, u, v, E, stream); return true;
        case 10: *err = launch_ih_tf32<10>(S, D, u, v, E, stream); return true;
        case 12: *err = launch_ih_tf32<12>(S, D, u, v, E, stream); return true;
        case 14: *err = launch_ih_tf32<14>(S, D, u, v, E, stream); return true;
        case 16: *err = launch_ih_tf32<16>(S, D, u, v, E, stream); return true;
        default: return false;
    }
}
// the fp64 fields have no such path
bool try_launch_ih_tf32(const double*, const double*, const double*, double*, int, long long,
                        cudaStream_t, cudaError_t*) {
    return false;
}

// Forward operator, single precision, split-TF32 tensor path (cubic n -> m, even extents 8..16).
template <int N, int M>
cudaError_t launch_ap_tf32(const float* A, const float* B, const float* Cm, const float* u, float* v,
                           long long E, cudaStream_t stream) {
    using C = tf32::ApplyCfg32<N, N, N, M, M, M>;
    auto kernel = tf32::apply_tf32<N, N, N, M, M, M>;
    static std::atomic<int> cached[64];
    int per_sm = 1;
    cudaError_t err = ctas_per_sm(kernel, C::kThreads, C::kSmemBytes, cached, &per_sm);
    if (err != cudaSuccess) return err;
    const long long batches = (E + C::kBe - 1) / C::kBe;
    long long grid = (long long)sm_count() * per_sm;
    if (grid > batches) grid = batches;
    unsigned long long* tickets = nullptr;
    err = tickets_for(batches, grid, &tickets);
    if (err != cudaSuccess) return err;
    kernel<<<(unsigned)grid, C::kThreads, C::kSmemBytes, stream>>>(A, B, Cm, u, v, E, tickets);
    return cudaGetLastError();
}

template <int N>
bool apply_tf32_from(int m, const float* A, const float* B, const float* C, const float* u, float* v,
                     long long E, cudaStream_t stream, cudaError_t* err) {
    switch (m) {
        case 8: *err = launch_ap_tf32<N, 8>(A, B, C, u, v, E, stream); return true;
        case 10: *err = launch_ap_tf32<N, 10>(A, B, C, u, v, E, stream); return true;
        case 12: *err = launch_ap_tf32<N, 12>(A, B, C, u, v, E, stream); return true;
        case 14: *err = launch_ap_tf32<N, 14>(A, B, C, u, v, E, stream); return true;
        case 16: *err = launch_ap_tf32<N, 16>(A, B, C, u, v, E, stream); return true;
        default: return false;
    }
}

bool try_launch_apply_tf32(const float* A, const float* B, const float* C, const float* u, float* v,
                           int n, int m, long long E, cudaStream_t stream, cudaError_t* err) {
    switch (n) {
        case 8: return apply_tf32_from<8>(m, A, B, C, u, v, E, stream, err);
        case 10: return apply_tf32_from<10>(m, A, B, C, u, v, E, stream, err);
        case 12: return apply_tf32_from<12>(m, A, B, C, u, v, E, stream, err);
        case 14: return apply_tf32_from<14>(m, A, B, C, u, v, E, stream, err);
        case 16: return apply_tf32_from<16>(m, A, B, C, u, v, E, stream, err);
        default: return false;
    }
}
bool try_launch_apply_tf32(const double*, const double*, const double*, const double*, double*, int,
                           int, long long, cudaStream_t, cudaError_t*) {
    return false;
}

}  // namespace

template <typename T>
bool try_launch_ih_dmma(const T* S, const T* D, const T* u, T* v, int n, long long E,
                        cudaStream_t stream, cudaError_t* err) {
    // bulk copies of u (fp64, even n) need 16-byte aligned element addresses; odd n and fp32
    // fields are copied in element units, and the L2 prefetches align themselves
    if (sizeof(T) == 8 && n % 2 == 0 && reinterpret_cast<uintptr_t>(u) % 16) return false;
    if (try_launch_ih_tf32(S, D, u, v, n, E, stream, err)) return true;
    switch (n) {
        case 4: *err = launch_ih<4, T, false>(S, D, nullptr, nullptr, u, v, E, stream); return true;
        case 5: *err = launch_ih<5, T, false>(S, D, nullptr, nullptr, u, v, E, stream); return true;
        case 6: *err = launch_ih<6, T, false>(S, D, nullptr, nullptr, u, v, E, stream); return true;
        case 7: *err = launch_ih<7, T, false>(S, D, nullptr, nullptr, u, v, E, stream); return true;
        case 8: *err = launch_ih<8, T, false>(S, D, nullptr, nullptr, u, v, E, stream); return true;
        case 9: *err = launch_ih<9, T, false>(S, D, nullptr, nullptr, u, v, E, stream); return true;
        case 10: *err = launch_ih<10, T, false>(S, D, nullptr, nullptr, u, v, E, stream); return true;
        case 11: *err = launch_ih<11, T, false>(S, D, nullptr, nullptr, u, v, E, stream); return true;
        case 12: *err = launch_ih<12, T, false>(S, D, nullptr, nullptr, u, v, E, stream); return true;
        case 13: *err = launch_ih<13, T, false>(S, D, nullptr, nullptr, u, v, E, stream); return true;
        case 14: *err = launch_ih<14, T, false>(S, D, nullptr, nullptr, u, v, E, stream); return true;
        case 15: *err = launch_ih<15, T, false>(S, D, nullptr, nullptr, u, v, E, stream); return true;
        case 16: *err = launch_ih<16, T, false>(S, D, nullptr, nullptr, u, v, E, stream); return true;
        case 17: *err = launch_ih<17, T, false>(S, D, nullptr, nullptr, u, v, E, stream); return true;
        case 18: *err = launch_ih<18, T, false>(S, D, nullptr, nullptr, u, v, E, stream); return true;
        case 19: *err = launch_ih<19, T, false>(S, D, nullptr, nullptr, u, v, E, stream); return true;
        case 20: *err = launch_ih<20, T, false>(S, D, nullptr, nullptr, u, v, E, stream); return true;
        default: return false;
    }
}

namespace {

// cubic n -> m instances for even extents
template <int N, typename T>
bool apply_cubic_from(int m, const T* A, const T* B, const T* C, const T* u, T* v, long long E,
                      cudaStream_t stream, cudaError_t* err) {
    switch (m) {
        case 4: *err = launch_apply_instance<N, N, N, 4, 4, 4, T>(A, B, C, u, v, E, stream); return true;
        case 6: *err = launch_apply_instance<N, N, N, 6, 6, 6, T>(A, B, C, u, v, E, stream); return true;
        case 8: *err = launch_apply_instance<N, N, N, 8, 8, 8, T>(A, B, C, u, v, E, stream); return true;
        case 10: *err = launch_apply_instance<N, N, N, 10, 10, 10, T>(A, B, C, u, v, E, stream); return true;
        case 12: *err = launch_apply_instance<N, N, N, 12, 12, 12, T>(A, B, C, u, v, E, stream); return true;
        case 14: *err = launch_apply_instance<N, N, N, 14, 14, 14, T>(A, B, C, u, v, E, stream); return true;
        case 16: *err = launch_apply_instance<N, N, N, 16, 16, 16, T>(A, B, C, u, v, E, stream); return true;
        default: return false;
    }
}

}  // namespace

bool try_launch_ih_lambda_dmma(const double* S, const double* lam, const double* cvec,
                               const double* u, double* v, int n, long long E, cudaStream_t stream,
                               cudaError_t* err) {
    if (n % 2 == 0 && reinterpret_cast<uintptr_t>(u) % 16) return false;
    switch (n) {
#define EKL_LAMBDA_CASE(N_)                                                                 \
    case N_:                                                                                \
        *err = launch_ih<N_, double, true>(S, nullptr, lam, cvec, u, v, E, stream);         \
        return true;
        EKL_LAMBDA_CASE(4)
        EKL_LAMBDA_CASE(5)
        EKL_LAMBDA_CASE(6)
        EKL_LAMBDA_CASE(7)
        EKL_LAMBDA_CASE(8)
        EKL_LAMBDA_CASE(9)
        EKL_LAMBDA_CASE(10)
        EKL_LAMBDA_CASE(11)
        EKL_LAMBDA_CASE(12)
        EKL_LAMBDA_CASE(13)
        EKL_LAMBDA_CASE(14)
        EKL_LAMBDA_CASE(15)
        EKL_LAMBDA_CASE(16)
        EKL_LAMBDA_CASE(17)
        EKL_LAMBDA_CASE(18)
        EKL_LAMBDA_CASE(19)
        EKL_LAMBDA_CASE(20)
#undef EKL_LAMBDA_CASE
        default: return false;
    }
}

template <typename T>
bool try_launch_apply_dmma(const T* A, const T* B, const T* C, const T* u, T* v, int n0, int n1,
                           int n2, int m0, int m1, int m2, long long E, cudaStream_t stream,
                           cudaError_t* err) {
    // fp64 u is bulk-copied plane by plane where a plane is a whole number of 16-byte units:
    // 16-byte aligned element addresses
    if (sizeof(T) == 8 && (n1 * n2) % 2 == 0 && reinterpret_cast<uintptr_t>(u) % 16) return false;
    if (n0 != n1 || n1 != n2 || m0 != m1 || m1 != m2)
        return try_launch_apply_aniso(A, B, C, u, v, n0, n1, n2, m0, m1, m2, E, stream, err);
    if (try_launch_apply_tf32(A, B, C, u, v, n0, m0, E, stream, err)) return true;
    switch (n0) {
        case 4: if (apply_cubic_from<4, T>(m0, A, B, C, u, v, E, stream, err)) return true; break;
        case 6: if (apply_cubic_from<6, T>(m0, A, B, C, u, v, E, stream, err)) return true; break;
        case 8: if (apply_cubic_from<8, T>(m0, A, B, C, u, v, E, stream, err)) return true; break;
        case 10: if (apply_cubic_from<10, T>(m0, A, B, C, u, v, E, stream, err)) return true; break;
        case 12: if (apply_cubic_from<12, T>(m0, A, B, C, u, v, E, stream, err)) return true; break;
        case 14: if (apply_cubic_from<14, T>(m0, A, B, C, u, v, E, stream, err)) return true; break;
        case 16: if (apply_cubic_from<16, T>(m0, A, B, C, u, v, E, stream, err)) return true; break;
        default: break;
    }
    return try_launch_apply_odd_a(A, B, C, u, v, n0, m0, E, stream, err) ||
           try_launch_apply_odd_b(A, B, C, u, v, n0, m0, E, stream, err) ||
           try_launch_apply_odd_c(A, B, C, u, v, n0, m0, E, stream, err);
}

template bool try_launch_ih_dmma<double>(const double*, const double*, const double*, double*, int,
                                         long long, cudaStream_t, cudaError_t*);
template bool try_launch_ih_dmma<float>(const float*, const float*, const float*, float*, int,
                                        long long, cudaStream_t, cudaError_t*);
template bool try_launch_apply_dmma<double>(const double*, const double*, const double*,
                                            const double*, double*, int, int, int, int, int, int,
                                            long long, cudaStream_t, cudaError_t*);
template bool try_launch_apply_dmma<float>(const float*, const float*, const float*, const float*,
                                           float*, int, int, int, int, int, int, long long,
                                           cudaStream_t, cudaError_t*);

}  // namespace ekl

namespace {
// One warp arms a barrier for 16 bytes that nothing ever sends and waits for them: the wait
// runs out of its time budget, raises bit 0 of the error flags and the kernel returns.
__global__ void expired_wait_kernel() {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        ekl::dmma::mbar_init(&bar, 1);
        ekl::dmma::mbar_expect_tx(&bar, 16);
    }
    __syncthreads();
    ekl::dmma::wait_bulk(&bar, 0);
}
}  // namespace

extern "C" ekl_tpo_status ekl_tpo_selftest_expired_wait(cudaStream_t stream) {
    expired_wait_kernel<<<1, 32, 0, stream>>>();
    const cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) {
        ekl::set_last_cuda_error((int)err);
        return EKL_TPO_ERR_CUDA;
    }
    return EKL_TPO_OK;
}

// Reads (and clears) the flags device code raises when something that should never happen
// did: bit 0 = a bounded wait on a bulk copy gave up, bit 1 = a launch's ticket counter was
// written by something else while it ran; either way the results of that launch are not
// valid.  Synchronises the device.
extern "C" int ekl_tpo_device_error_flags(void) {
    if (cudaDeviceSynchronize() != cudaSuccess) return -1;
    const int flags[] = {ekl::dmma::take_timeout_flag(),   ekl::convection_timeout_flag(),
                         ekl::ih3_timeout_flag(),          ekl::apply_aniso_timeout_flag(),
                         ekl::apply_odd_a_timeout_flag(),  ekl::apply_odd_b_timeout_flag(),
                         ekl::apply_odd_c_timeout_flag(),    ekl::convection_odd_timeout_flag(),
                         ekl::ih3_odd_timeout_flag()};
    int all = 0;
    for (int f : flags) {
        if (f < 0) return -1;
        all |= f;
    }
    return all;
}
