// Instances and launchers of the tensor-path kernels.
#include <cstdint>

#include "dispatch.h"
#include "tpo_dmma.cuh"

namespace ekl {
namespace {

template <int N>
cudaError_t launch_ih(const double* S, const double* D, const double* u, double* v, long long E,
                      cudaStream_t stream) {
    using C = dmma::IhCfg<N>;
    cudaError_t err = cudaFuncSetAttribute(dmma::inv_helmholtz_dmma<N>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)C::kSmemBytes);
    if (err != cudaSuccess) return err;
    int per_sm = 1;
    err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, dmma::inv_helmholtz_dmma<N>,
                                                        C::kThreads, C::kSmemBytes);
    if (err != cudaSuccess) return err;
    if (per_sm < 1) per_sm = 1;
    const long long batches = (E + C::kBe - 1) / C::kBe;
    long long grid = (long long)sm_count() * per_sm;
    if (grid > batches) grid = batches;
    dmma::inv_helmholtz_dmma<N><<<(unsigned)grid, C::kThreads, C::kSmemBytes, stream>>>(S, D, u, v, E);
    return cudaGetLastError();
}

template <int N0, int N1, int N2, int M0, int M1, int M2>
cudaError_t launch_ap(const double* A, const double* B, const double* Cm, const double* u,
                      double* v, long long E, cudaStream_t stream) {
    using C = dmma::ApplyCfg<N0, N1, N2, M0, M1, M2>;
    auto kernel = dmma::apply_dmma<N0, N1, N2, M0, M1, M2>;
    cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)C::kSmemBytes);
    if (err != cudaSuccess) return err;
    int per_sm = 1;
    err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, C::kThreads, C::kSmemBytes);
    if (err != cudaSuccess) return err;
    if (per_sm < 1) per_sm = 1;
    const long long batches = (E + C::kBe - 1) / C::kBe;
    long long grid = (long long)sm_count() * per_sm;
    if (grid > batches) grid = batches;
    kernel<<<(unsigned)grid, C::kThreads, C::kSmemBytes, stream>>>(A, B, Cm, u, v, E);
    return cudaGetLastError();
}

}  // namespace

bool try_launch_ih_dmma(const double* S, const double* D, const double* u, double* v, int n,
                        long long E, cudaStream_t stream, cudaError_t* err) {
    // bulk copies of u (even n) need 16-byte aligned element addresses; odd n is copied in
    // 8-byte units, and the L2 prefetches align themselves
    if (n % 2 == 0 && reinterpret_cast<uintptr_t>(u) % 16) return false;
    switch (n) {
        case 4: *err = launch_ih<4>(S, D, u, v, E, stream); return true;
        case 5: *err = launch_ih<5>(S, D, u, v, E, stream); return true;
        case 6: *err = launch_ih<6>(S, D, u, v, E, stream); return true;
        case 7: *err = launch_ih<7>(S, D, u, v, E, stream); return true;
        case 8: *err = launch_ih<8>(S, D, u, v, E, stream); return true;
        case 9: *err = launch_ih<9>(S, D, u, v, E, stream); return true;
        case 10: *err = launch_ih<10>(S, D, u, v, E, stream); return true;
        case 11: *err = launch_ih<11>(S, D, u, v, E, stream); return true;
        case 12: *err = launch_ih<12>(S, D, u, v, E, stream); return true;
        case 13: *err = launch_ih<13>(S, D, u, v, E, stream); return true;
        case 14: *err = launch_ih<14>(S, D, u, v, E, stream); return true;
        case 15: *err = launch_ih<15>(S, D, u, v, E, stream); return true;
        case 16: *err = launch_ih<16>(S, D, u, v, E, stream); return true;
        default: return false;
    }
}

namespace {

// cubic n -> m instances for even extents
template <int N>
bool apply_cubic_from(int m, const double* A, const double* B, const double* C, const double* u,
                      double* v, long long E, cudaStream_t stream, cudaError_t* err) {
    switch (m) {
        case 4: *err = launch_ap<N, N, N, 4, 4, 4>(A, B, C, u, v, E, stream); return true;
        case 6: *err = launch_ap<N, N, N, 6, 6, 6>(A, B, C, u, v, E, stream); return true;
        case 8: *err = launch_ap<N, N, N, 8, 8, 8>(A, B, C, u, v, E, stream); return true;
        case 10: *err = launch_ap<N, N, N, 10, 10, 10>(A, B, C, u, v, E, stream); return true;
        case 12: *err = launch_ap<N, N, N, 12, 12, 12>(A, B, C, u, v, E, stream); return true;
        case 14: *err = launch_ap<N, N, N, 14, 14, 14>(A, B, C, u, v, E, stream); return true;
        case 16: *err = launch_ap<N, N, N, 16, 16, 16>(A, B, C, u, v, E, stream); return true;
        default: return false;
    }
}

}  // namespace

bool try_launch_apply_dmma(const double* A, const double* B, const double* C, const double* u,
                           double* v, int n0, int n1, int n2, int m0, int m1, int m2, long long E,
                           cudaStream_t stream, cudaError_t* err) {
    // u is bulk-copied plane by plane: 16-byte aligned element addresses
    if (reinterpret_cast<uintptr_t>(u) % 16) return false;
    if (n0 != n1 || n1 != n2 || m0 != m1 || m1 != m2) return false;
    switch (n0) {
        case 4: return apply_cubic_from<4>(m0, A, B, C, u, v, E, stream, err);
        case 6: return apply_cubic_from<6>(m0, A, B, C, u, v, E, stream, err);
        case 8: return apply_cubic_from<8>(m0, A, B, C, u, v, E, stream, err);
        case 10: return apply_cubic_from<10>(m0, A, B, C, u, v, E, stream, err);
        case 12: return apply_cubic_from<12>(m0, A, B, C, u, v, E, stream, err);
        case 14: return apply_cubic_from<14>(m0, A, B, C, u, v, E, stream, err);
        case 16: return apply_cubic_from<16>(m0, A, B, C, u, v, E, stream, err);
        default: return false;
    }
}

}  // namespace ekl

// Reads (and clears) the flags device code raises when something that should never happen
// did: bit 0 = a bounded wait on a bulk copy gave up, so the results of that launch are
// not valid.  Synchronises the device.
extern "C" int ekl_tpo_device_error_flags(void) {
    int flag = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) return -1;
    if (cudaMemcpyFromSymbol(&flag, ekl::dmma::g_bulk_wait_timeout, sizeof(int)) != cudaSuccess)
        return -1;
    if (flag) {
        const int zero = 0;
        cudaMemcpyToSymbol(ekl::dmma::g_bulk_wait_timeout, &zero, sizeof(int));
    }
    return flag ? 1 : 0;
}
