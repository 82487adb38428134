// Entry points that take HOST buffers: the element range is cut into chunks that are
// copied to a caller-provided device workspace, processed by the same kernels as the
// device-pointer entry points, and copied back, with the three stages of successive
// chunks overlapped on separate streams (copy-in | compute | copy-out).
#include "../../include/ekl_tpo.h"

#include <cstdint>
#include <mutex>

#include "dispatch.h"

namespace {

constexpr int kSlots = 3;          // chunks in flight: one per pipeline stage
constexpr size_t kAlign = 256;

size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

// Helper streams and events of one device, created on first use and kept for the life
// of the process (streams and events only -- no device memory).
struct Pipe {
    bool ready = false;
    cudaStream_t in = nullptr, out = nullptr;
    cudaEvent_t start = nullptr, loaded[kSlots] = {}, computed[kSlots] = {}, drained[kSlots] = {};
};
Pipe g_pipes[64];
std::mutex g_mutex;

cudaError_t get_pipe(Pipe** out) {
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    Pipe& p = g_pipes[dev];
    if (!p.ready) {
        if ((err = cudaStreamCreateWithFlags(&p.in, cudaStreamNonBlocking)) != cudaSuccess) return err;
        if ((err = cudaStreamCreateWithFlags(&p.out, cudaStreamNonBlocking)) != cudaSuccess) return err;
        if ((err = cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming)) != cudaSuccess) return err;
        for (int s = 0; s < kSlots; ++s) {
            if ((err = cudaEventCreateWithFlags(&p.loaded[s], cudaEventDisableTiming)) != cudaSuccess) return err;
            if ((err = cudaEventCreateWithFlags(&p.computed[s], cudaEventDisableTiming)) != cudaSuccess) return err;
            if ((err = cudaEventCreateWithFlags(&p.drained[s], cudaEventDisableTiming)) != cudaSuccess) return err;
        }
        p.ready = true;
    }
    *out = &p;
    return cudaSuccess;
}

#define EKL_TRY(call)                                   \
    do {                                                \
        cudaError_t e_ = (call);                        \
        if (e_ != cudaSuccess) {                        \
            ekl::set_last_cuda_error((int)e_);          \
            return EKL_TPO_ERR_CUDA;                    \
        }                                               \
    } while (0)

bool overlaps(const void* a, size_t na, const void* b, size_t nb) {
    const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
    return na != 0 && nb != 0 && x < y + nb && y < x + na;
}

// One chunked pass.  mats: up to three small host matrices copied once; fields_in: one or
// two per-element host input fields; Launch(dev mats..., dev in..., dev out, count, stream).
template <typename T, typename Launch>
ekl_tpo_status pipeline(const T* const* mats, const size_t* mat_elems, int n_mats,
                        const T* const* fields_in, int n_in, size_t in_elems, T* field_out,
                        size_t out_elems, long long E, void* workspace, size_t workspace_bytes,
                        cudaStream_t stream, Launch launch) {
    if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return EKL_TPO_ERR_ALIGN;
    size_t off = 0;
    T* dmat[3] = {nullptr, nullptr, nullptr};
    for (int m = 0; m < n_mats; ++m) {
        dmat[m] = reinterpret_cast<T*>(static_cast<char*>(workspace) + off);
        off += align_up(mat_elems[m] * sizeof(T));
    }
    const size_t per_elem = align_up(in_elems * sizeof(T)) * n_in + align_up(out_elems * sizeof(T));
    if (workspace_bytes < off + kSlots * per_elem) return EKL_TPO_ERR_UNSUPPORTED;
    long long chunk = (long long)((workspace_bytes - off) / kSlots / per_elem);
    // per-slot regions are sized for `chunk` elements; alignment padding is per field
    while (chunk > 1 &&
           off + kSlots * (align_up(chunk * in_elems * sizeof(T)) * n_in +
                           align_up(chunk * out_elems * sizeof(T))) > workspace_bytes)
        --chunk;
    if (chunk > E) chunk = E;
    const size_t in_bytes = align_up(chunk * in_elems * sizeof(T));
    const size_t out_bytes = align_up(chunk * out_elems * sizeof(T));
    const size_t slot_bytes = in_bytes * n_in + out_bytes;

    std::lock_guard<std::mutex> lock(g_mutex);
    Pipe* p = nullptr;
    EKL_TRY(get_pipe(&p));
    // helper streams start after everything already enqueued on `stream`
    EKL_TRY(cudaEventRecord(p->start, stream));
    EKL_TRY(cudaStreamWaitEvent(p->in, p->start, 0));
    EKL_TRY(cudaStreamWaitEvent(p->out, p->start, 0));
    for (int m = 0; m < n_mats; ++m)
        EKL_TRY(cudaMemcpyAsync(dmat[m], mats[m], mat_elems[m] * sizeof(T), cudaMemcpyHostToDevice,
                                p->in));
    const long long n_chunks = (E + chunk - 1) / chunk;
    for (long long c = 0; c < n_chunks; ++c) {
        const int s = (int)(c % kSlots);
        const long long e0 = c * chunk;
        const long long cnt = (E - e0 < chunk) ? (E - e0) : chunk;
        char* slot = static_cast<char*>(workspace) + off + (size_t)s * slot_bytes;
        T* din[2] = {reinterpret_cast<T*>(slot), reinterpret_cast<T*>(slot + in_bytes)};
        T* dout = reinterpret_cast<T*>(slot + in_bytes * n_in);
        if (c >= kSlots) EKL_TRY(cudaStreamWaitEvent(p->in, p->drained[s], 0));
        for (int f = 0; f < n_in; ++f)
            EKL_TRY(cudaMemcpyAsync(din[f], fields_in[f] + (size_t)e0 * in_elems,
                                    (size_t)cnt * in_elems * sizeof(T), cudaMemcpyHostToDevice,
                                    p->in));
        EKL_TRY(cudaEventRecord(p->loaded[s], p->in));
        EKL_TRY(cudaStreamWaitEvent(stream, p->loaded[s], 0));
        EKL_TRY(launch(dmat, din, dout, cnt, stream));
        EKL_TRY(cudaEventRecord(p->computed[s], stream));
        EKL_TRY(cudaStreamWaitEvent(p->out, p->computed[s], 0));
        EKL_TRY(cudaMemcpyAsync(field_out + (size_t)e0 * out_elems, dout,
                                (size_t)cnt * out_elems * sizeof(T), cudaMemcpyDeviceToHost,
                                p->out));
        EKL_TRY(cudaEventRecord(p->drained[s], p->out));
    }
    // `stream` completes only after the last copies back have landed
    for (int s = 0; s < kSlots && s < n_chunks; ++s)
        EKL_TRY(cudaStreamWaitEvent(stream, p->drained[s], 0));
    return EKL_TPO_OK;
}

template <typename T>
ekl_tpo_status inv_helmholtz_host_impl(const T* S, const T* D, const T* u, T* v, int n,
                                       long long E, void* workspace, size_t workspace_bytes,
                                       cudaStream_t stream) {
    if (n < 1 || E < 0) return EKL_TPO_ERR_SHAPE;
    if (E == 0) return EKL_TPO_OK;
    if (!S || !D || !u || !v || !workspace) return EKL_TPO_ERR_NULL;
    if (n > ekl::max_cubic_extent(sizeof(T))) return EKL_TPO_ERR_UNSUPPORTED;
    const uintptr_t a = sizeof(T);
    if (reinterpret_cast<uintptr_t>(S) % a || reinterpret_cast<uintptr_t>(D) % a ||
        reinterpret_cast<uintptr_t>(u) % a || reinterpret_cast<uintptr_t>(v) % a)
        return EKL_TPO_ERR_ALIGN;
    const size_t n3 = (size_t)n * n * n;
    const size_t field = (size_t)E * n3 * sizeof(T);
    if (overlaps(v, field, S, (size_t)n * n * sizeof(T)) || overlaps(v, field, D, field) ||
        (v != u && overlaps(v, field, u, field)))
        return EKL_TPO_ERR_OVERLAP;
    const T* mats[1] = {S};
    const size_t mat_elems[1] = {(size_t)n * n};
    const T* fin[2] = {D, u};
    return pipeline<T>(
        mats, mat_elems, 1, fin, 2, n3, v, n3, E, workspace, workspace_bytes, stream,
        [n](T* const* dm, T* const* din, T* dout, long long cnt, cudaStream_t st) {
            return ekl::launch_inv_helmholtz<T>(dm[0], din[0], din[1], dout, n, cnt, st);
        });
}

template <typename T>
ekl_tpo_status apply_host_impl(const T* A, const T* B, const T* C, const T* u, T* v, int n0,
                               int n1, int n2, int m0, int m1, int m2, long long E,
                               void* workspace, size_t workspace_bytes, cudaStream_t stream) {
    if (n0 < 1 || n1 < 1 || n2 < 1 || m0 < 1 || m1 < 1 || m2 < 1 || E < 0)
        return EKL_TPO_ERR_SHAPE;
    if (E == 0) return EKL_TPO_OK;
    if (!A || !B || !C || !u || !v || !workspace) return EKL_TPO_ERR_NULL;
    if (!ekl::apply_fits(n0, n1, n2, m0, m1, m2, sizeof(T))) return EKL_TPO_ERR_UNSUPPORTED;
    const uintptr_t a = sizeof(T);
    if (reinterpret_cast<uintptr_t>(A) % a || reinterpret_cast<uintptr_t>(B) % a ||
        reinterpret_cast<uintptr_t>(C) % a || reinterpret_cast<uintptr_t>(u) % a ||
        reinterpret_cast<uintptr_t>(v) % a)
        return EKL_TPO_ERR_ALIGN;
    const size_t nout = (size_t)E * m0 * m1 * m2 * sizeof(T);
    if (overlaps(v, nout, u, (size_t)E * n0 * n1 * n2 * sizeof(T)) ||
        overlaps(v, nout, A, (size_t)m0 * n0 * sizeof(T)) ||
        overlaps(v, nout, B, (size_t)m1 * n1 * sizeof(T)) ||
        overlaps(v, nout, C, (size_t)m2 * n2 * sizeof(T)))
        return EKL_TPO_ERR_OVERLAP;
    const T* mats[3] = {A, B, C};
    const size_t mat_elems[3] = {(size_t)m0 * n0, (size_t)m1 * n1, (size_t)m2 * n2};
    const T* fin[2] = {u, nullptr};
    return pipeline<T>(
        mats, mat_elems, 3, fin, 1, (size_t)n0 * n1 * n2, v, (size_t)m0 * m1 * m2, E, workspace,
        workspace_bytes, stream,
        [=](T* const* dm, T* const* din, T* dout, long long cnt, cudaStream_t st) {
            return ekl::launch_apply<T>(dm[0], dm[1], dm[2], din[0], dout, n0, n1, n2, m0, m1,
                                             m2, cnt, st);
        });
}

}  // namespace

extern "C" {

size_t ekl_tpo_host_workspace_bytes(long long in_elems_per_element, int n_inputs,
                                    long long out_elems_per_element, long long matrix_elems,
                                    long long chunk, int elem_size) {
    if (in_elems_per_element < 1 || out_elems_per_element < 1 || chunk < 1 || n_inputs < 1 ||
        matrix_elems < 0 || elem_size < 1)
        return 0;
    const size_t w = (size_t)elem_size;
    // matrices are padded one by one; three is the most any entry point copies
    return 3 * kAlign + align_up((size_t)matrix_elems * w) +
           kSlots * (align_up((size_t)chunk * in_elems_per_element * w) * n_inputs +
                     align_up((size_t)chunk * out_elems_per_element * w));
}

ekl_tpo_status ekl_tpo_inv_helmholtz_host(const double* S, const double* D, const double* u,
                                          double* v, int n, long long E, void* workspace,
                                          size_t workspace_bytes, cudaStream_t stream) {
    return inv_helmholtz_host_impl<double>(S, D, u, v, n, E, workspace, workspace_bytes, stream);
}

ekl_tpo_status ekl_tpo_inv_helmholtz_host_f32(const float* S, const float* D, const float* u,
                                              float* v, int n, long long E, void* workspace,
                                              size_t workspace_bytes, cudaStream_t stream) {
    return inv_helmholtz_host_impl<float>(S, D, u, v, n, E, workspace, workspace_bytes, stream);
}

ekl_tpo_status ekl_tpo_apply_host(const double* A, const double* B, const double* C,
                                  const double* u, double* v, int n0, int n1, int n2, int m0,
                                  int m1, int m2, long long E, void* workspace,
                                  size_t workspace_bytes, cudaStream_t stream) {
    return apply_host_impl<double>(A, B, C, u, v, n0, n1, n2, m0, m1, m2, E, workspace,
                                   workspace_bytes, stream);
}

ekl_tpo_status ekl_tpo_apply_host_f32(const float* A, const float* B, const float* C,
                                      const float* u, float* v, int n0, int n1, int n2, int m0,
                                      int m1, int m2, long long E, void* workspace,
                                      size_t workspace_bytes, cudaStream_t stream) {
    return apply_host_impl<float>(A, B, C, u, v, n0, n1, n2, m0, m1, m2, E, workspace,
                                  workspace_bytes, stream);
}

}  // extern "C"
