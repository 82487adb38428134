// Measurement helpers (libekl_probe.so, include/ekl_probe.h): the FP64 rates the roofline
// fractions refer to, and the n = 14 contraction stage in isolation on the tensor path and on
// the CUDA cores.  Nothing here is called by the operators.
#include "../../include/ekl_probe.h"

#include "tpo_dmma.cuh"

namespace {

using namespace ekl::dmma;

constexpr int kChains = 16;

__global__ void __launch_bounds__(256) fma_chain_kernel(double* __restrict__ sink, int iters,
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

// acc[o] = s[o] * x + acc[o]: 14 operator entries and the datum in registers; the datum of
// the next step is derived from the lane index so that nothing folds at compile time.
__global__ void __launch_bounds__(256) fma_contraction_kernel(double* __restrict__ sink, int iters,
                                                              double seed) {
    double s[14], acc[14];
#pragma unroll
    for (int o = 0; o < 14; ++o) {
        s[o] = seed * (double)(o + 1) + 1e-3 * (double)threadIdx.x;
        acc[o] = 0.0;
    }
    double x0 = seed, x1 = -seed;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int o = 0; o < 14; ++o) acc[o] = fma(s[o], x0, acc[o]);
#pragma unroll
        for (int o = 0; o < 14; ++o) acc[o] = fma(s[o], x1, acc[o]);
        x0 = -x0;
        x1 = -x1;
    }
    double t = 0.0;
#pragma unroll
    for (int o = 0; o < 14; ++o) t += acc[o];
    sink[(size_t)blockIdx.x * blockDim.x + threadIdx.x] = t;
}

template <int CHAINS, bool WITH_FMA>
__global__ void __launch_bounds__(256) dmma_kernel(double* __restrict__ sink, int iters, double a) {
    double c[CHAINS][2];
#pragma unroll
    for (int k = 0; k < CHAINS; ++k) c[k][0] = c[k][1] = 0.0;
    double f[4] = {0.0, 0.0, 0.0, 0.0};
    const double b = a * (double)(1 + (threadIdx.x & 3));
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int rep = 0; rep < 8 / CHAINS; ++rep) {
#pragma unroll
            for (int k = 0; k < CHAINS; ++k) mma_f64(c[k][0], c[k][1], a, b);
        }
        if (WITH_FMA) {
#pragma unroll
            for (int r = 0; r < 4; ++r) {
#pragma unroll
                for (int k = 0; k < 4; ++k) f[k] = fma(a, b, f[k]);
            }
        }
    }
    double t = f[0] + f[1] + f[2] + f[3];
#pragma unroll
    for (int k = 0; k < CHAINS; ++k) t += c[k][0] + c[k][1];
    sink[(size_t)blockIdx.x * blockDim.x + threadIdx.x] = t;
}

// ---- the n = 14 stage in isolation --------------------------------------------------------

using Cfg14 = IhCfg<14, double>;
using Mid14 = Cfg14::Mid;

__device__ __forceinline__ void fill_buffers(double* buf, int count) {
    for (int i = threadIdx.x; i < count; i += blockDim.x) buf[i] = 1.0 + 1e-3 * (double)(i % 97);
}

// The operator is the identity (so the values stay bounded however many stages run); the
// tensor pipe does the same work for any operand values.
__global__ void __launch_bounds__(Cfg14::kThreads, 2)
stage_loop_dmma_kernel(double* __restrict__ sink, int stages) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    double* bufA = reinterpret_cast<double*>(smem_raw);
    double* bufB = bufA + Cfg14::kBufElems;
    const int lane = threadIdx.x & 31;
    const int warp = ((threadIdx.x >> 5) + blockIdx.x) % Cfg14::kWarps;
    OpFrag<Mid14> op;
#pragma unroll
    for (int mt = 0; mt < Mid14::kMTiles; ++mt)
#pragma unroll
        for (int s = 0; s < Mid14::kKSteps; ++s) {
            const int o = 8 * mt + (lane >> 2), x = Mid14::k0(s) + (lane & 3);
            const bool fresh = (s == 0) || (x >= Mid14::k0(s - 1) + 4);
            op.a[mt][s] = (o == x && fresh) ? 1.0 : 0.0;
        }
    fill_buffers(bufA, 2 * Cfg14::kBufElems);
    __syncthreads();
    double dfac[1][Mid14::kMTiles][2];
    const NoFactor none;
    for (int st = 0; st < stages; st += 2) {
        run_stage<Mid14, 0, double, NoFactor, 1>(bufA, bufB, nullptr, op, dfac, none,
                                                 Mid14::kPencils, warp, lane);
        __syncthreads();
        run_stage<Mid14, 0, double, NoFactor, 1>(bufB, bufA, nullptr, op, dfac, none,
                                                 Mid14::kPencils, warp, lane);
        __syncthreads();
    }
    sink[(size_t)blockIdx.x * blockDim.x + threadIdx.x] = bufA[threadIdx.x] + bufB[threadIdx.x];
}

// CUDA-core contender: 196 threads, thread t owns pencils 2t', 2t'+1 of element t / 98.
constexpr int kFmaThreads = 196;

__global__ void __launch_bounds__(kFmaThreads, 2)
stage_loop_fma_kernel(double* __restrict__ sink, int stages) {
    constexpr int N = 14, kP = N * N, kES = Cfg14::kES, kPS = Cfg14::kPS, kRS = Cfg14::kRS;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    double* bufA = reinterpret_cast<double*>(smem_raw);
    double* bufB = bufA + Cfg14::kBufElems;
    double* sS = bufB + Cfg14::kBufElems;                  // [x][o], identity
    for (int i = threadIdx.x; i < kP; i += blockDim.x) sS[i] = (i / N == i % N) ? 1.0 : 0.0;
    fill_buffers(bufA, 2 * Cfg14::kBufElems);
    __syncthreads();
    const int e = threadIdx.x / (kP / 2);
    const int p = 2 * (threadIdx.x - e * (kP / 2));         // even: the pair shares a row
    const int p1 = p / N, p2 = p - p1 * N;
    const int in_off = e * kES + p1 * kRS + p2;
    const int out_off = e * kES + p1 * kPS + p2 * kRS;      // pencil q -> q * 14 + o
    for (int st = 0; st < stages; ++st) {
        const double* in = (st & 1) ? bufB : bufA;
        double* out = (st & 1) ? bufA : bufB;
        double acc[N][2];
#pragma unroll
        for (int o = 0; o < N; ++o) acc[o][0] = acc[o][1] = 0.0;
#pragma unroll
        for (int x = 0; x < N; ++x) {
            const double2 d = *reinterpret_cast<const double2*>(in + in_off + x * kPS);
#pragma unroll
            for (int o = 0; o < N; o += 2) {
                const double2 s = *reinterpret_cast<const double2*>(sS + x * N + o);
                acc[o][0] = fma(s.x, d.x, acc[o][0]);
                acc[o][1] = fma(s.x, d.y, acc[o][1]);
                acc[o + 1][0] = fma(s.y, d.x, acc[o + 1][0]);
                acc[o + 1][1] = fma(s.y, d.y, acc[o + 1][1]);
            }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int o = 0; o < N; o += 2)
                *reinterpret_cast<double2*>(out + out_off + h * kRS + o) =
                    make_double2(acc[o][h], acc[o + 1][h]);
        __syncthreads();
    }
    sink[(size_t)blockIdx.x * blockDim.x + threadIdx.x] = bufA[threadIdx.x] + bufB[threadIdx.x];
}

int finish(double* flops, double value) {
    *flops = value;
    return cudaGetLastError() == cudaSuccess ? 0 : 6;
}

}  // namespace

extern "C" {

int ekl_probe_fp64_fma_chain(double* sink, int blocks, int iters, double* flops,
                             cudaStream_t stream) {
    if (!sink || !flops) return 1;
    if (blocks < 1 || iters < 1) return 2;
    fma_chain_kernel<<<blocks, 256, 0, stream>>>(sink, iters, 0.999999, 1e-9);
    return finish(flops, 2.0 * kChains * 256.0 * (double)blocks * (double)iters);
}

int ekl_probe_fp64_fma_contraction(double* sink, int blocks, int iters, double* flops,
                                   cudaStream_t stream) {
    if (!sink || !flops) return 1;
    if (blocks < 1 || iters < 1) return 2;
    fma_contraction_kernel<<<blocks, 256, 0, stream>>>(sink, iters, 0.75);
    return finish(flops, 2.0 * 28.0 * 256.0 * (double)blocks * (double)iters);
}

int ekl_probe_fp64_dmma(double* sink, int blocks, int iters, int chains, double* flops,
                        cudaStream_t stream) {
    if (!sink || !flops) return 1;
    if (blocks < 1 || iters < 1 || (chains != 1 && chains != 2 && chains != 4)) return 2;
    if (chains == 1) dmma_kernel<1, false><<<blocks, 256, 0, stream>>>(sink, iters, 1.0000001);
    if (chains == 2) dmma_kernel<2, false><<<blocks, 256, 0, stream>>>(sink, iters, 1.0000001);
    if (chains == 4) dmma_kernel<4, false><<<blocks, 256, 0, stream>>>(sink, iters, 1.0000001);
    return finish(flops, 512.0 * 8.0 * 8.0 * (double)blocks * (double)iters);
}

int ekl_probe_fp64_dmma_plus_fma(double* sink, int blocks, int iters, double* flops,
                                 cudaStream_t stream) {
    if (!sink || !flops) return 1;
    if (blocks < 1 || iters < 1) return 2;
    dmma_kernel<2, true><<<blocks, 256, 0, stream>>>(sink, iters, 1.0000001);
    return finish(flops, (512.0 * 8.0 * 8.0 + 2.0 * 16.0 * 256.0) * (double)blocks * (double)iters);
}

int ekl_probe_stage_loop_n14(double* sink, int blocks, int stages, double* flops,
                             double* padded_flops, cudaStream_t stream) {
    if (!sink || !flops || !padded_flops) return 1;
    if (blocks < 1 || stages < 2 || stages % 2) return 2;
    const size_t smem = 2 * (size_t)Cfg14::kBufElems * sizeof(double);
    if (cudaFuncSetAttribute(stage_loop_dmma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)smem) != cudaSuccess)
        return 6;
    stage_loop_dmma_kernel<<<blocks, Cfg14::kThreads, smem, stream>>>(sink, stages);
    *padded_flops = 2.0 * 16 * 16 * Mid14::kTiles * 8.0 * (double)blocks * (double)stages;
    return finish(flops, 2.0 * 14 * 14 * Mid14::kPencils * (double)blocks * (double)stages);
}

int ekl_probe_stage_loop_n14_fma(double* sink, int blocks, int stages, double* flops,
                                 cudaStream_t stream) {
    if (!sink || !flops) return 1;
    if (blocks < 1 || stages < 1) return 2;
    const size_t smem = (2 * (size_t)Cfg14::kBufElems + 14 * 14) * sizeof(double);
    if (cudaFuncSetAttribute(stage_loop_fma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)smem) != cudaSuccess)
        return 6;
    stage_loop_fma_kernel<<<blocks, kFmaThreads, smem, stream>>>(sink, stages);
    return finish(flops, 2.0 * 14 * 14 * Mid14::kPencils * (double)blocks * (double)stages);
}

}  // extern "C"
