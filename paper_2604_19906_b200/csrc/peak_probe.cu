// Measurement helper: a register-resident chain of independent double-precision FMAs,
// used to read the sustained FP64 rate of the device the operators are timed on.
#include "../../include/ekl_tpo.h"

namespace {

constexpr int kChains = 16;

__global__ void __launch_bounds__(256) fp64_fma_chain(double* __restrict__ sink, int iters,
                                                      double a, double b) {
    double acc[kChains];
#pragma unroll
    for (int c = 0; c < kChains; ++c) acc[c] = (double)(threadIdx.x + c);
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int c = 0; c < kChains; ++c) acc[c] = fma(acc[c], a, b);
    }
    double s = 0.0;
#pragma unroll
    for (int c = 0; c < kChains; ++c) s += acc[c];
    sink[(size_t)blockIdx.x * blockDim.x + threadIdx.x] = s;
}

}  // namespace

extern "C" ekl_tpo_status ekl_tpo_probe_fp64_fma(double* sink, int blocks, int iters,
                                                 double* flops, cudaStream_t stream) {
    if (!sink || !flops) return EKL_TPO_ERR_NULL;
    if (blocks < 1 || iters < 1) return EKL_TPO_ERR_SHAPE;
    fp64_fma_chain<<<blocks, 256, 0, stream>>>(sink, iters, 0.999999, 1e-9);
    *flops = 2.0 * kChains * 256.0 * (double)blocks * (double)iters;
    return cudaGetLastError() == cudaSuccess ? EKL_TPO_OK : EKL_TPO_ERR_CUDA;
}
