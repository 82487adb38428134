/*
 * ekl_tpo -- batched, sum-factorised spectral-element tensor-product operators
 * for NVIDIA B200 (sm_100a).  C ABI; every pointer is a DEVICE pointer unless the
 * name of the function ends in "_host".
 *
 * Conventions shared by every entry point
 * ---------------------------------------
 *  - Arrays are dense, row-major (C order), last index fastest; the element
 *    index e is the slowest one.  This is the row-major C ABI the paper's
 *    kernels are linked through (Section 3, the remark on the column-major /
 *    row-major difference next to the convective-flux listing).
 *  - Kronecker ordering as in Eq. 1 of the paper: in (A (x) B (x) C) the last
 *    factor acts on the fastest (contiguous) in-element axis,
 *        ((A (x) B (x) C) x)[i,j,k] = sum_{l,m,n} A[i,l] B[j,m] C[k,n] x[l,m,n],
 *    with every matrix stored [out, in] row-major.
 *  - The result is the one the lifted ("reduction lifting", Section 5.2) sums
 *    define mathematically; floating-point association inside the library is
 *    unspecified (FMA is used), so results agree with a reference to rounding,
 *    not bit for bit.
 *  - Ownership: the caller owns every buffer.  Unless stated otherwise the
 *    library allocates nothing, frees nothing and never synchronises: a call
 *    validates its arguments on the host, enqueues work on `stream` and returns.
 *    Buffers must stay valid until the stream has passed that work.  Inputs are
 *    only read; the output is fully overwritten.
 *  - Work distribution: most kernels, in a launch that gives a CTA more than four
 *    batches of elements, hand the batches out through a counter (16 bytes) taken from a fixed
 *    ring of 4096 inside the library image.  The kernel itself puts the counter back
 *    to zero when its last CTA leaves, so a call is still one kernel launch and
 *    nothing else.  A counter comes round again after 4096 launches; a kernel whose
 *    counter was touched by another launch while it ran says so through
 *    ekl_tpo_device_error_flags (bit 1).
 *  - Errors: a status code is returned; nothing is thrown, aborted or trapped,
 *    and arguments that are accepted can never index out of bounds.  Validation
 *    happens before anything is enqueued:
 *        E > 0 and a null pointer                      -> EKL_TPO_ERR_NULL
 *        an extent < 1, or E < 0                       -> EKL_TPO_ERR_SHAPE
 *        extents too large for on-chip memory          -> EKL_TPO_ERR_UNSUPPORTED
 *        pointer not aligned to its element type       -> EKL_TPO_ERR_ALIGN
 *        output overlapping an input (see below)       -> EKL_TPO_ERR_OVERLAP
 *        a CUDA runtime call failed                    -> EKL_TPO_ERR_CUDA
 *    E == 0 is a successful no-op.  There is no CPU fallback of any kind.
 */
#ifndef EKL_TPO_H
#define EKL_TPO_H

#include <cuda_runtime_api.h>
#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    EKL_TPO_OK = 0,
    EKL_TPO_ERR_NULL = 1,
    EKL_TPO_ERR_SHAPE = 2,
    EKL_TPO_ERR_UNSUPPORTED = 3,
    EKL_TPO_ERR_ALIGN = 4,
    EKL_TPO_ERR_OVERLAP = 5,
    EKL_TPO_ERR_CUDA = 6
} ekl_tpo_status;

/*
 * Inverse Helmholtz operator (the `inv_helm` kernel of Section 2.2 / Table 2; its
 * forward stage is the lifted triple sum printed in Section 5.2):
 *
 *     v[e] = (S (x) S (x) S) . ( D[e] o ( (S^T (x) S^T (x) S^T) . u[e] ) ),   e = 0..E-1
 *
 *   S      [n,n]       one matrix shared by all elements and directions
 *   D,u,v  [E,n,n,n]   D is multiplied pointwise (it holds the reciprocals)
 *
 * fp64.  `v == u` exactly (in place) is allowed; any other overlap of v with an
 * input is rejected.  1 <= n; n is limited by shared memory (n <= 24 for fp64).
 * Every n from 4 to 20 runs on the FP64 tensor path (for even n this needs a 16-byte
 * aligned u); every other accepted case runs on a slower general kernel with the same
 * results to rounding.
 */
ekl_tpo_status ekl_tpo_inv_helmholtz(const double* S, const double* D, const double* u,
                                     double* v, int n, long long E, cudaStream_t stream);

/*
 * The same operator with the pointwise factor formed on the fly instead of read from
 * memory, for the case where it is a sum of one-dimensional eigenvalues plus a per-element
 * shift (the paper does not print this variant; it is the structure the inverse
 * Helmholtz factor has):
 *
 *     D[e,i,j,k] = 1 / (((lam[i] + lam[j]) + lam[k]) + c[e])        lam [n], c [E]
 *
 * evaluated in exactly this order with IEEE operations, so the result equals
 * ekl_tpo_inv_helmholtz on the materialised D bit for bit.  Moves 16 n^3 + 8 bytes per
 * element instead of 24 n^3 and spends n^3 divisions.  fp64, 4 <= n <= 20 (other n:
 * EKL_TPO_ERR_UNSUPPORTED); even n needs a 16-byte aligned u (EKL_TPO_ERR_ALIGN otherwise).
 * v == u is allowed.
 */
ekl_tpo_status ekl_tpo_inv_helmholtz_lambda(const double* S, const double* lam, const double* c,
                                            const double* u, double* v, int n, long long E,
                                            cudaStream_t stream);

/*
 * Inverse Helmholtz with one operator and one extent per direction.  The paper's operators
 * carry a separate small matrix for every direction (Eq. 1 and the convective-flux listing
 * of Sections 2.2 and 3 apply one matrix per axis); this is the inverse Helmholtz operator
 * in that general form:
 *
 *     v[e] = (S0 (x) S1 (x) S2) . ( D[e] o ( (S0^T (x) S1^T (x) S2^T) . u[e] ) ),   e = 0..E-1
 *
 *   S0 [n0,n0]  S1 [n1,n1]  S2 [n2,n2]     S0 acts on the slowest in-element axis, S2 on the
 *                                          contiguous one (Kronecker ordering of Eq. 1)
 *   D,u,v [E,n0,n1,n2]                     D is multiplied pointwise
 *
 * fp64.  With S0 = S1 = S2 it equals ekl_tpo_inv_helmholtz.  v == u exactly (in place) is
 * allowed; any other overlap of v with an input is rejected.  Extents are limited by shared
 * memory (three matrices and two copies of an element).  The cubic shapes with n = 4, 5, 6,
 * 7, 8, 9, 10, 11, 12, 13, 14, 15, 16 and the shapes (8,10,12), (12,10,8), (14,12,8), (8,8,16),
 * (16,8,8), (5,7,9), (9,7,5), (6,7,8), (7,8,9) run on the FP64 tensor path (u 16-byte aligned
 * where n1*n2 is even); every other accepted shape runs on a general kernel with the same
 * results to rounding.
 */
ekl_tpo_status ekl_tpo_inv_helmholtz3(const double* S0, const double* S1, const double* S2,
                                      const double* D, const double* u, double* v,
                                      int n0, int n1, int n2, long long E, cudaStream_t stream);

/*
 * Forward rectangular tensor-product operator (the operator family of Eq. 1):
 *
 *     v[e] = (A (x) B (x) C) . u[e],   e = 0..E-1
 *
 *   A [m0,n0]  B [m1,n1]  C [m2,n2]     u [E,n0,n1,n2]     v [E,m0,m1,m2]
 *
 * fp64.  v must not overlap any input.  On the FP64 tensor path run: cubic shapes n -> m
 * (n0=n1=n2, m0=m1=m2) with even n, m from 4 to 16; the cubic shapes with an odd extent
 * n -> n for odd n from 5 to 15, n <-> n+2 for odd n from 5 to 13, n <-> n+1 for n from 4 to 9,
 * and 5 <-> 8, 6 <-> 9, 7 <-> 11, 9 <-> 14, 10 <-> 15 (to and from the 3/2 quadrature
 * resolution); and the non-cubic shapes (8,8,8)->(12,12,8), (8,8,8)->(8,8,12),
 * (12,12,12)->(8,8,12), (12,12,8)->(8,8,12), (8,10,12)->(12,10,8), (8,10,12)->(8,10,12),
 * (6,8,10)->(10,8,6), (14,12,8)->(8,12,14).  Where n1*n2 is even, u must be 16-byte aligned
 * for that path.  Every other case that fits in shared memory runs on the general kernel.
 */
ekl_tpo_status ekl_tpo_apply(const double* A, const double* B, const double* C,
                             const double* u, double* v,
                             int n0, int n1, int n2, int m0, int m1, int m2,
                             long long E, cudaStream_t stream);

/*
 * Volume integral of the convective flux (Eq. 1 of the paper; the `convection` kernel,
 * the one-statement listing next to it), for the three components c = 0,1,2:
 *
 *     F[c,e] = (I (x) I (x) D) . (M[e] o P[c,0,e]) + (I (x) D (x) I) . (M[e] o P[c,1,e])
 *            + (D (x) I (x) I) . (M[e] o P[c,2,e])
 *
 *   Dvq, Ivq [nv,nq]   differentiation / interpolation from quadrature to volume points
 *   M   [E,nq,nq,nq]   pointwise factor shared by the components and directions
 *   P   [3,3,E,nq,nq,nq]   fluxes, indexed [component][direction][element]...
 *   F   [3,E,nv,nv,nv]
 *
 * In each term the last Kronecker factor acts on the contiguous in-element axis, as everywhere
 * in this header, so the differentiation matrix acts on the fastest axis for direction 0, on
 * the middle one for direction 1 and on the slowest for direction 2.  fp64.  F must not
 * overlap any input.  (nq,nv) in {(4,4),(6,4),(6,6),(8,4),(8,6),(8,8),(10,8),(10,10),(12,8),
 * (12,10),(12,12),(14,12)} and {(5,5),(7,5),(7,7),(8,5),(9,6),(9,7),(9,9),(11,7),(14,9),
 * (15,10)} run on the FP64 tensor path (M and P 16-byte aligned where nq is even); every
 * other combination that fits in shared memory (nq, nv <= 64 and about 2 max(nq,nv)^3 + nv^3
 * values) runs on a general kernel; larger extents return EKL_TPO_ERR_UNSUPPORTED.
 */
ekl_tpo_status ekl_tpo_convection(const double* Dvq, const double* Ivq, const double* M,
                                  const double* P, double* F, int nq, int nv, long long E,
                                  cudaStream_t stream);

/*
 * Single-precision twins of ekl_tpo_inv_helmholtz and ekl_tpo_apply (same layout and
 * rules; tolerance 1e-5 instead of 1e-12).  ekl_tpo_inv_helmholtz_f32 with an even n from 8
 * to 16, and ekl_tpo_apply_f32 for cubic n -> m with even n, m from 8 to 16, both with a
 * 16-byte aligned u, run on the TF32 tensor path with split operands: every
 * product is taken as a_hi*b_hi + a_lo*b_hi + a_hi*b_lo (hi = the value rounded to TF32, lo =
 * the rest) and accumulated in fp32, the fields stay fp32 on chip; measured error about 4e-7.
 * On the FP64 tensor path (the other extents from 4 to 20, the other cubic pairs listed for
 * ekl_tpo_apply) the fields
 * are widened to fp64 on chip, all arithmetic is fp64, and v is rounded to fp32 once when it
 * is stored; the general kernel computes in fp32.  With EKL_TPO_F32_PATH=tcgen05 in the
 * environment (read once, at the first call) the split-TF32 case runs on tcgen05.mma with the
 * accumulator in tensor memory instead: same results to tolerance, slower on this operator
 * (kept for comparison); it needs D and v 8-byte aligned and holds 32 columns of tensor memory
 * per CTA while it runs.
 */
ekl_tpo_status ekl_tpo_inv_helmholtz_f32(const float* S, const float* D, const float* u,
                                         float* v, int n, long long E, cudaStream_t stream);
ekl_tpo_status ekl_tpo_apply_f32(const float* A, const float* B, const float* C,
                                 const float* u, float* v,
                                 int n0, int n1, int n2, int m0, int m1, int m2,
                                 long long E, cudaStream_t stream);

/*
 * Host-buffer variants.  S (resp. A, B, C), D, u and v are HOST pointers; pinned
 * (page-locked) memory is needed for the copies to overlap with the kernels, pageable
 * memory works but serialises.  The E elements are cut into chunks; each chunk is
 * copied into `workspace`, processed by the same kernels as the device-pointer entry
 * point (Section 5.2 / Eq. 1 operators as above), and copied back, three chunks in
 * flight (copy-in, compute, copy-out).
 *
 *   workspace        DEVICE scratch owned by the caller, 256-byte aligned, of
 *   workspace_bytes  bytes.  Any size that holds the matrices plus three one-element
 *                    slots is accepted (smaller -> EKL_TPO_ERR_UNSUPPORTED); larger
 *                    workspaces give larger chunks.  ekl_tpo_host_workspace_bytes()
 *                    returns the size for a wanted chunk length.  Its contents are
 *                    scratch: undefined after the call, nothing to clear before it.
 *
 * The call enqueues everything and returns without synchronising when the host
 * buffers are pinned; `stream` completes only after the last chunk of v has landed in
 * host memory.  Two helper streams and a few events per device are created on first
 * use (no device memory is allocated).  v == u (in place) is allowed for the inverse
 * Helmholtz variant.  Calls are serialised by an internal lock while they enqueue; two
 * calls sharing one workspace must be ordered on the same stream.
 */
ekl_tpo_status ekl_tpo_inv_helmholtz_host(const double* S, const double* D, const double* u,
                                          double* v, int n, long long E, void* workspace,
                                          size_t workspace_bytes, cudaStream_t stream);
ekl_tpo_status ekl_tpo_apply_host(const double* A, const double* B, const double* C,
                                  const double* u, double* v,
                                  int n0, int n1, int n2, int m0, int m1, int m2,
                                  long long E, void* workspace, size_t workspace_bytes,
                                  cudaStream_t stream);

/* Single-precision twins of the two host-buffer variants (same rules, float buffers). */
ekl_tpo_status ekl_tpo_inv_helmholtz_host_f32(const float* S, const float* D, const float* u,
                                              float* v, int n, long long E, void* workspace,
                                              size_t workspace_bytes, cudaStream_t stream);
ekl_tpo_status ekl_tpo_apply_host_f32(const float* A, const float* B, const float* C,
                                      const float* u, float* v,
                                      int n0, int n1, int n2, int m0, int m1, int m2,
                                      long long E, void* workspace, size_t workspace_bytes,
                                      cudaStream_t stream);

/*
 * Bytes of device workspace that let the host-buffer variants run with chunks of
 * `chunk` elements: `n_inputs` per-element input fields of `in_elems_per_element`
 * values each (2 for inverse Helmholtz: D and u; 1 for the forward operator), one output
 * field of `out_elems_per_element` values, `matrix_elems` matrix entries in total,
 * `elem_size` bytes per value.  Returns 0 for nonsensical arguments.
 */
size_t ekl_tpo_host_workspace_bytes(long long in_elems_per_element, int n_inputs,
                                    long long out_elems_per_element, long long matrix_elems,
                                    long long chunk, int elem_size);

/*
 * Inverse Helmholtz with HOST buffers and no device allocation anywhere (the paper has
 * no counterpart: this entry point exists for deployment, not for the method).
 *
 * For callers that cannot obtain device memory when they need the operator -- a solver
 * step running inside a memory budget fixed at start-up, a plug-in inside an
 * application that owns the GPU heap, a latency-critical path where cudaMalloc (which
 * may synchronise the device, or fail once memory is fragmented) is off limits -- and
 * who therefore have no workspace to give ekl_tpo_inv_helmholtz_host.  Same operator,
 * layout, argument meaning and status codes as ekl_tpo_inv_helmholtz_host; S, D, u, v
 * are HOST pointers (pinned memory makes the copies asynchronous).  The staging area is
 * a fixed array of EKL_TPO_STATIC_SCRATCH_BYTES bytes inside the library image; every
 * GPU that loads the library holds that much memory until the process exits.  The call
 * and everything it calls allocate and free nothing.
 *
 *  - Limit: the whole call is staged at once, so it needs
 *        roundup256(8 n^2) + 3 * roundup256(8 E n^3)  <=  EKL_TPO_STATIC_SCRATCH_BYTES
 *    (about 509 elements at n = 14, 2730 at n = 8).  Anything larger is rejected with
 *    EKL_TPO_ERR_UNSUPPORTED before any work is enqueued; split such a batch into
 *    several calls on one stream, or use ekl_tpo_inv_helmholtz_host.
 *  - Set-up: the first call on each device looks up the staging area's device address
 *    (with that device current) and keeps it.  Make that first call outside any stream
 *    capture; `stream` must belong to the current device.
 *  - Sharing: all calls on a device use the same staging area, and it keeps whatever
 *    the previous call left there.  Nothing has to be cleared -- each call overwrites
 *    all it reads -- but two calls that can run at the same time on the GPU (different
 *    streams without an ordering between them) race on it and corrupt each other.
 *    Issue them on one stream, or order them with events.
 *  - Work is enqueued on `stream` only (copy in, kernel, copy out, in that order); the
 *    result is in v once `stream` has reached the end of the call.  v == u is allowed.
 *  - The status code is decided on the host when the work is enqueued; it cannot report
 *    that a kernel's bounded wait gave up later on the device (v is then copied back
 *    partly written).  A caller that wants to rule that out reads
 *    ekl_tpo_device_error_flags() after synchronising.
 */
#define EKL_TPO_STATIC_SCRATCH_BYTES (32u * 1024u * 1024u)
ekl_tpo_status ekl_tpo_inv_helmholtz_host_static(const double* S, const double* D,
                                                 const double* u, double* v, int n,
                                                 long long E, cudaStream_t stream);

/* Human-readable name of a status code (static storage, never NULL). */
const char* ekl_tpo_status_string(ekl_tpo_status status);

/* Library version: major*10000 + minor*100 + patch. */
int ekl_tpo_version(void);

/* cudaError_t of the most recent EKL_TPO_ERR_CUDA returned on the calling thread. */
int ekl_tpo_last_cuda_error(void);

/*
 * Device-side error flags since the last call of this function on the current device, and
 * clears them; -1 if the query itself failed.  Bit 0: a kernel's bounded wait on one of its
 * own bulk copies gave up (the kernel then stops early instead of hanging).  Bit 1: the
 * work-distribution counter of a launch was written by something else while the kernel ran
 * (see "Work distribution" above).  In both cases the output of that launch is not valid.
 * Not expected in practice; meant for health checks.
 * SYNCHRONISES the device.  (Infrastructure: the paper has no counterpart.)
 */
int ekl_tpo_device_error_flags(void);

/*
 * Self-test of that reporting path (infrastructure: the paper has no counterpart).  Enqueues
 * one warp that waits on a barrier for a copy nobody issued.  Every wait in the library's
 * kernels has a time budget of about one second; this one runs out of it twice (the wait and
 * the bounded re-wait that follows a failure), so the kernel ends by itself after about two
 * seconds and ekl_tpo_device_error_flags() then reports bit 0 once.  Nothing faults and the
 * context stays usable.
 */
ekl_tpo_status ekl_tpo_selftest_expired_wait(cudaStream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* EKL_TPO_H */
