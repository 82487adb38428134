// Kernel selection and launch configuration.
#include <atomic>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <tuple>

#include "dispatch.h"
#include "generic_kernel.cuh"

namespace ekl {

int sm_count() {
    static std::atomic<int> cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    int n = cached[dev].load(std::memory_order_relaxed);
    if (n == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1)
            n = 148;
        cached[dev].store(n, std::memory_order_relaxed);
    }
    return n;
}

// ---- ticket counters for the dynamic distribution of batches (BatchQueue in tpo_dmma.cuh).
// A launch that wants one takes the next pair of 64-bit words of this ring.  The ring lives in
// the library image (nothing is allocated per call) and starts out zero; the CTA of a launch
// that leaves last puts its pair back to zero, so no call has to clear anything.  A pair comes
// round again after kTicketSlots launches, and a kernel whose pair was touched by another
// launch while it ran reports that through ekl_tpo_device_error_flags (bit 1).
namespace {
constexpr unsigned kTicketSlots = 4096;
__device__ unsigned long long g_ticket_ring[2 * kTicketSlots];
}  // namespace

cudaError_t next_ticket_counter(unsigned long long** out) {
    static std::mutex mu;
    static unsigned long long* base[64] = {nullptr};
    static std::atomic<unsigned> turn{0};
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    unsigned long long* b = nullptr;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!base[dev]) {
            void* p = nullptr;
            err = cudaGetSymbolAddress(&p, g_ticket_ring);
            if (err != cudaSuccess) return err;
            base[dev] = static_cast<unsigned long long*>(p);
        }
        b = base[dev];
    }
    *out = b + 2 * (turn.fetch_add(1, std::memory_order_relaxed) % kTicketSlots);
    return cudaSuccess;
}

namespace {

// Opts a run-time-sized kernel into the largest dynamic shared memory once per device and keeps
// the occupancy answers per (device, threads, bytes), so that a call costs one launch and
// concurrent callers with different extents cannot undo each other's setting.
template <typename Kernel>
cudaError_t generic_ctas_per_sm(Kernel kernel, int threads, size_t smem, int* per_sm) {
    static std::mutex mu;
    static std::map<std::tuple<int, const void*, int, size_t>, int> answers;
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    const void* id = reinterpret_cast<const void*>(kernel);
    std::lock_guard<std::mutex> lock(mu);
    const auto opted = std::make_tuple(dev, id, 0, (size_t)0);
    if (answers.find(opted) == answers.end()) {
        err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)kMaxSmemBytes);
        if (err != cudaSuccess) return err;
        answers.emplace(opted, 1);
    }
    const auto key = std::make_tuple(dev, id, threads, smem);
    auto it = answers.find(key);
    if (it == answers.end()) {
        int n = 1;
        err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, threads, smem);
        if (err != cudaSuccess) return err;
        it = answers.emplace(key, n < 1 ? 1 : n).first;
    }
    *per_sm = it->second;
    return cudaSuccess;
}

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
    const int threads = round_up_warp((long long)n * n * n, 512);
    int per_sm = 1;
    const cudaError_t err = generic_ctas_per_sm(inv_helmholtz_generic<T>, threads, smem, &per_sm);
    if (err != cudaSuccess) return err;
    long long grid = (long long)sm_count() * per_sm;
    if (grid > E) grid = E;
    inv_helmholtz_generic<T><<<(unsigned)grid, threads, smem, stream>>>(S, D, u, v, n, E);
    return cudaGetLastError();
}

cudaError_t launch_ih3_generic(const double* S0, const double* S1, const double* S2,
                               const double* D, const double* u, double* v, int n0, int n1, int n2,
                               long long E, cudaStream_t stream) {
    const size_t smem = generic_ih3_smem(n0, n1, n2, sizeof(double));
    const int threads = round_up_warp((long long)n0 * n1 * n2, 512);
    int per_sm = 1;
    const cudaError_t err =
        generic_ctas_per_sm(inv_helmholtz3_generic<double>, threads, smem, &per_sm);
    if (err != cudaSuccess) return err;
    long long grid = (long long)sm_count() * per_sm;
    if (grid > E) grid = E;
    inv_helmholtz3_generic<double>
        <<<(unsigned)grid, threads, smem, stream>>>(S0, S1, S2, D, u, v, n0, n1, n2, E);
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_apply_generic(const T* A, const T* B, const T* C, const T* u, T* v, int n0,
                                 int n1, int n2, int m0, int m1, int m2, long long E,
                                 cudaStream_t stream) {
    const size_t smem = generic_apply_smem(n0, n1, n2, m0, m1, m2, sizeof(T));
    const int threads = round_up_warp((long long)m0 * m1 * m2, 512);
    int per_sm = 1;
    const cudaError_t err = generic_ctas_per_sm(apply_generic<T>, threads, smem, &per_sm);
    if (err != cudaSuccess) return err;
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
    const int threads = round_up_warp((long long)nq * nq * nv, 512);
    int per_sm = 1;
    const cudaError_t err = generic_ctas_per_sm(convection_generic<double>, threads, smem, &per_sm);
    if (err != cudaSuccess) return err;
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

cudaError_t launch_inv_helmholtz3(const double* S0, const double* S1, const double* S2,
                                  const double* D, const double* u, double* v, int n0, int n1,
                                  int n2, long long E, cudaStream_t stream) {
    cudaError_t err = cudaSuccess;
    if (tuned_allowed() && try_launch_ih3_dmma(S0, S1, S2, D, u, v, n0, n1, n2, E, stream, &err))
        return err;
    return launch_ih3_generic(S0, S1, S2, D, u, v, n0, n1, n2, E, stream);
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
