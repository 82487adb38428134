// Device-side twin of the counter-based input stream defined in inputs.py.
//
// Input generation only: nothing of the tensor-product operator is computed here.
// The stream is   h = splitmix64_finaliser(key + (index+1)*0x9E3779B97F4A7C15),
//                 r = (h >> 11) * 2^-53,   value = lo + scale*r  (multiply and add
// rounded separately), which integer arithmetic makes bit-identical to the NumPy
// implementation, so large fields can be produced directly in HBM.
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

__device__ __forceinline__ double u01(uint64_t key, uint64_t index) {
    uint64_t z = key + (index + 1ull) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    z = z ^ (z >> 31);
    return (double)(z >> 11) * 0x1.0p-53;
}

__global__ void fill_uniform_kernel(double* __restrict__ dst, long long start, long long count,
                                    uint64_t key, double lo, double scale) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long x = (long long)blockIdx.x * blockDim.x + threadIdx.x; x < count; x += stride)
        dst[x] = __dadd_rn(lo, __dmul_rn(scale, u01(key, (uint64_t)(start + x))));
}

// D[e,i,j,k] = 1 / (((lam_i + lam_j) + lam_k) + c_e),  c_e = 0.5 + 1.0*r(e)
__global__ void fill_D_kernel(double* __restrict__ D, const double* __restrict__ lam, int n,
                              long long e0, long long E, uint64_t key_c) {
    const long long n3 = (long long)n * n * n;
    const long long count = E * n3;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long x = (long long)blockIdx.x * blockDim.x + threadIdx.x; x < count; x += stride) {
        const long long e = x / n3;
        const int r = (int)(x - e * n3);
        const int i = r / (n * n), j = (r / n) % n, k = r % n;
        const double c = __dadd_rn(0.5, __dmul_rn(1.0, u01(key_c, (uint64_t)(e0 + e))));
        const double s = __dadd_rn(__dadd_rn(__dadd_rn(lam[i], lam[j]), lam[k]), c);
        D[x] = __ddiv_rn(1.0, s);
    }
}

int grid_for(long long count) {
    long long b = (count + 255) / 256;
    if (b > 148 * 16) b = 148 * 16;
    if (b < 1) b = 1;
    return (int)b;
}

}  // namespace

extern "C" int ekl_inputs_fill_uniform_f64(double* dst, long long start, long long count,
                                           uint64_t key, double lo, double scale,
                                           cudaStream_t stream) {
    if (count <= 0) return 0;
    fill_uniform_kernel<<<grid_for(count), 256, 0, stream>>>(dst, start, count, key, lo, scale);
    return (int)cudaGetLastError();
}

extern "C" int ekl_inputs_fill_D_f64(double* D, const double* lam, int n, long long e0,
                                     long long E, uint64_t key_c, cudaStream_t stream) {
    if (E <= 0) return 0;
    fill_D_kernel<<<grid_for(E * n * n * n), 256, 0, stream>>>(D, lam, n, e0, E, key_c);
    return (int)cudaGetLastError();
}
