// Host-buffer inverse Helmholtz for callers that must not allocate device memory.
//
// Some callers of this library cannot call cudaMalloc at the moment they need the
// operator: code running between the time steps of a solver whose memory budget was
// fixed at start-up, plug-ins loaded into a host application that owns the GPU heap,
// and anything on a latency-critical path where an allocation (which may synchronise
// the device or fail under fragmentation) is not acceptable.  The regular host-buffer
// entry point asks such a caller for a device workspace it has no way to provide.  The
// variant below stages the call in a fixed array that is part of the library image
// instead: nothing is allocated, by this code or by anything it calls.
#include "../../include/ekl_tpo.h"

#include <cstdint>
#include <mutex>

#include "dispatch.h"

namespace {

constexpr size_t kAlign = 256;
constexpr size_t kScratchBytes = EKL_TPO_STATIC_SCRATCH_BYTES;

// The staging area.  Lives in every device that loads this library until the process
// exits.  In host code this name is only a handle for cudaGetSymbolAddress -- it is not
// a device address and must never be handed to a kernel or a copy as if it were one.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

std::mutex g_setup_mutex;
unsigned char* g_scratch_addr[64] = {nullptr};

// Device address of the staging area on the current device; looked up once per device.
cudaError_t scratch_address(unsigned char** out) {
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (g_scratch_addr[dev] == nullptr) {
        void* p = nullptr;
        err = cudaGetSymbolAddress(&p, g_static_scratch);
        if (err != cudaSuccess) return err;
        if (p == nullptr || reinterpret_cast<uintptr_t>(p) % kAlign) return cudaErrorInvalidSymbol;
        g_scratch_addr[dev] = static_cast<unsigned char*>(p);
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

bool overlaps(const void* a, size_t na, const void* b, size_t nb) {
    const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
    return na != 0 && nb != 0 && x < y + nb && y < x + na;
}

#define EKL_TRY(call)                                   \
    do {                                                \
        cudaError_t e_ = (call);                        \
        if (e_ != cudaSuccess) {                        \
            ekl::set_last_cuda_error((int)e_);          \
            return EKL_TPO_ERR_CUDA;                    \
        }                                               \
    } while (0)

}  // namespace

extern "C" ekl_tpo_status ekl_tpo_inv_helmholtz_host_static(const double* S, const double* D,
                                                            const double* u, double* v, int n,
                                                            long long E, cudaStream_t stream) {
    if (n < 1 || E < 0) return EKL_TPO_ERR_SHAPE;
    if (E == 0) return EKL_TPO_OK;
    if (!S || !D || !u || !v) return EKL_TPO_ERR_NULL;
    if (n > ekl::max_cubic_extent(sizeof(double))) return EKL_TPO_ERR_UNSUPPORTED;
    const uintptr_t a = sizeof(double);
    if (reinterpret_cast<uintptr_t>(S) % a || reinterpret_cast<uintptr_t>(D) % a ||
        reinterpret_cast<uintptr_t>(u) % a || reinterpret_cast<uintptr_t>(v) % a)
        return EKL_TPO_ERR_ALIGN;
    const size_t n3 = (size_t)n * n * n;
    // The whole call must fit in the fixed staging area: S, then D, u and v for all E
    // elements.  Checked in floating point first so that a huge E cannot overflow size_t.
    const size_t mat_bytes = align_up((size_t)n * n * sizeof(double));
    if ((double)E * (double)n3 * 8.0 * 3.0 > (double)kScratchBytes) return EKL_TPO_ERR_UNSUPPORTED;
    const size_t field_bytes = (size_t)E * n3 * sizeof(double);
    const size_t field_slot = align_up(field_bytes);
    if (mat_bytes + 3 * field_slot > kScratchBytes) return EKL_TPO_ERR_UNSUPPORTED;
    if (overlaps(v, field_bytes, S, (size_t)n * n * sizeof(double)) ||
        overlaps(v, field_bytes, D, field_bytes) || (v != u && overlaps(v, field_bytes, u, field_bytes)))
        return EKL_TPO_ERR_OVERLAP;

    unsigned char* base = nullptr;
    EKL_TRY(scratch_address(&base));
    double* dS = reinterpret_cast<double*>(base);
    double* dD = reinterpret_cast<double*>(base + mat_bytes);
    double* du = reinterpret_cast<double*>(base + mat_bytes + field_slot);
    double* dv = reinterpret_cast<double*>(base + mat_bytes + 2 * field_slot);
    // Every staged byte that a kernel reads is overwritten here first, and v's region is
    // fully written by the kernel before it is copied out, so nothing left behind by an
    // earlier call can reach this one and nothing needs clearing.
    EKL_TRY(cudaMemcpyAsync(dS, S, (size_t)n * n * sizeof(double), cudaMemcpyHostToDevice, stream));
    EKL_TRY(cudaMemcpyAsync(dD, D, field_bytes, cudaMemcpyHostToDevice, stream));
    EKL_TRY(cudaMemcpyAsync(du, u, field_bytes, cudaMemcpyHostToDevice, stream));
    EKL_TRY(ekl::launch_inv_helmholtz<double>(dS, dD, du, dv, n, E, stream));
    EKL_TRY(cudaMemcpyAsync(v, dv, field_bytes, cudaMemcpyDeviceToHost, stream));
    return EKL_TPO_OK;
}
