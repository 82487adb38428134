// Single-precision inverse Helmholtz on the asynchronous tensor path (tcgen05.mma, kind::tf32,
// accumulator in tensor memory), split-TF32 arithmetic as in tpo_tf32.cuh.
//
// One CTA of 128 threads works on one element at a time.  A mode contraction is the GEMM
//     C[q][o] = sum_x A[q][x] * M[x][o],   q = pencil (N*N rows), x, o < N,
// issued by one thread as tcgen05.mma over 128-row tiles (N = 16 columns, K = 8 per instruction):
// three instructions per tile and K step for the three split products a_hi*b_hi + a_lo*b_hi +
// a_hi*b_lo, all accumulating in the same 16 columns of tensor memory.  Thread t then reads row
// t of each tile back (tcgen05.ld), i.e. one pencil (a,b) with its N outputs c, applies the
// pointwise factor after the third contraction, splits the values in hi and lo parts and
// writes them where the next contraction wants them: row (b,c), column a of the A operand.
// The A operand is K-major in the tcgen05 canonical layout without swizzle (4 consecutive K
// values in 16 bytes, the 8 rows of a group 16 bytes apart, groups kSbo bytes apart, the chunks
// of 4 K values kLbo bytes apart); kSbo = 176 bytes keeps these transposing 4-byte stores at two
// wavefronts each (a warp's rows are 14 apart; no stride does better).  An M-major A operand,
// which would let a thread store its consecutive rows as vectors, gave zeros in a probe with
// TF32 operands and is not used.  The same buffer serves every stage:
// the tensor core has finished reading it when its results are read.  The cycle
// (a,b),c -> (b,c),a returns to the natural order after three contractions, so u is gathered
// once (from a dense landing buffer filled by a bulk copy), the factor and v are addressed in
// their natural order, each thread reading/writing N consecutive values.
#pragma once
#include "tpo_dmma.cuh"
#include "tpo_tf32.cuh"

namespace ekl {
namespace umma {

using dmma::smem_addr;

__device__ __forceinline__ void tmem_alloc(uint32_t* holder, int cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_addr(holder)),
                 "r"(cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_free(uint32_t taddr, int cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols)
                 : "memory");
}
__device__ __forceinline__ void fence_before_sync() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void fence_after_sync() {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// D[tmem] (+)= A[smem] * B[smem]; `accumulate` = 0 overwrites D.
__device__ __forceinline__ void mma_tf32_ss(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc,
                                            uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The barrier gets one arrival when every tensor instruction issued so far by this thread is done.
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                     smem_addr(bar))
                 : "memory");
}
// This thread's row (tensor-memory lane) of 16 consecutive columns.
__device__ __forceinline__ void tmem_load16(float (&v)[16], uint32_t taddr) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
          "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
          "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor (no swizzle): start address, leading and stride byte offsets
// in 16-byte units, descriptor version 1.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}

template <int N>
struct Cfg {
    static_assert(N % 2 == 0 && N >= 8 && N <= 16, "even extents from 8 to 16");
    static constexpr int kRows = N * N;                       // pencils = rows of every GEMM
    static constexpr int kMT = (kRows + 127) / 128;           // 128-row tiles
    static constexpr int kThreads = 128;
    // A operand, K-major without swizzle: (m,k) at (k/4)*kLbo + (m/8)*kSbo + (m%8)*16 + (k%4)*4.
    // Only the row groups that hold pencils are laid out; the last tile's tensor instructions
    // read past them (into the next chunk or the buffers behind) for rows nobody looks at.
    static constexpr int kSbo = 176;
    static constexpr int kGroups = (kRows + 7) / 8;
    static constexpr int kLbo = kGroups * kSbo;               // one chunk of 4 K values, all rows
    static constexpr int kABytes = 4 * kLbo;                  // K = 16: four chunks
    // B operand (16 x 16), K-major without swizzle: (n,k) at (n/8)*512 + (k/4)*128 + (n%8)*16 + (k%4)*4
    static constexpr int kBBytes = 1024;
    static constexpr int kLandBytes = (N * N * N * 4 + 15) / 16 * 16;
    static constexpr int kTmemCols = (kMT * 16 < 32) ? 32 : kMT * 16;
    // layout of the dynamic shared memory
    static constexpr int kOffAhi = 0, kOffAlo = kABytes, kOffB = 2 * kABytes;      // 4 B matrices
    static constexpr int kOffLand = kOffB + 4 * kBBytes;
    static constexpr int kOffBar = kOffLand + kLandBytes;                          // 2 barriers + holder
    static constexpr size_t kSmemBytes = kOffBar + 32;
    static constexpr int kCtasPerSm = (int)((227 * 1024) / (kSmemBytes + 1024)) > 5
                                          ? 5
                                          : (int)((227 * 1024) / (kSmemBytes + 1024));
    // instruction descriptor: fp32 accumulator, TF32 operands, A and B K-major, N = 16, M = 128
    static constexpr uint32_t kIdesc = (1u << 4) | (2u << 7) | (2u << 10) | ((16u >> 3) << 17) |
                                       ((128u >> 4) << 24);
    // what a tensor instruction of the last tile may touch must still be shared memory
    static_assert(kOffAlo + 3 * kLbo + 256 + (kMT * 16) * kSbo <= (int)kSmemBytes ||
                      kMT * 16 <= kGroups,
                  "the last tile reads past the dynamic shared memory");
};

// hi/lo parts of `val[0..N)` to rows m0..m0+N-1, column k of the A operands
template <int N, class C>
__device__ __forceinline__ void scatter_row(unsigned char* smem, int m0, int k, const float (&val)[16]) {
    const int kofs = (k >> 2) * C::kLbo + (k & 3) * 4;
#pragma unroll
    for (int c = 0; c < N; ++c) {
        const int m = m0 + c;
        const int ofs = kofs + (m >> 3) * C::kSbo + (m & 7) * 16;
        uint32_t hi, lo;
        tf32::split_tf32(val[c], hi, lo);
        *reinterpret_cast<uint32_t*>(smem + C::kOffAhi + ofs) = hi;
        *reinterpret_cast<uint32_t*>(smem + C::kOffAlo + ofs) = lo;
    }
}

template <int N>
__global__ void __launch_bounds__(128, Cfg<N>::kCtasPerSm)
inv_helmholtz_umma(const float* __restrict__ S, const float* __restrict__ D, const float* u, float* v,
                   long long E) {
    using C = Cfg<N>;
    constexpr int kN3 = N * N * N;
    extern __shared__ __align__(1024) unsigned char smem[];
    float* land = reinterpret_cast<float*>(smem + C::kOffLand);
    uint64_t* bar_u = reinterpret_cast<uint64_t*>(smem + C::kOffBar);
    uint64_t* bar_mma = bar_u + 1;
    uint32_t* holder = reinterpret_cast<uint32_t*>(bar_u + 2);
    const int t = threadIdx.x, warp = t >> 5;

    // operators, split: B[n][k]; forward stages apply S^T (B_f[o][x] = S[x][o]), backward S itself
    for (int idx = t; idx < 256; idx += 128) {
        const int n = idx >> 4, k = idx & 15;
        const int ofs = (n >> 3) * 512 + (k >> 2) * 128 + (n & 7) * 16 + (k & 3) * 4;
        const bool in = n < N && k < N;
        const float f = in ? __ldg(S + k * N + n) : 0.0f, b = in ? __ldg(S + n * N + k) : 0.0f;
        uint32_t hi, lo;
        tf32::split_tf32(f, hi, lo);
        *reinterpret_cast<uint32_t*>(smem + C::kOffB + 0 * C::kBBytes + ofs) = hi;
        *reinterpret_cast<uint32_t*>(smem + C::kOffB + 1 * C::kBBytes + ofs) = lo;
        tf32::split_tf32(b, hi, lo);
        *reinterpret_cast<uint32_t*>(smem + C::kOffB + 2 * C::kBBytes + ofs) = hi;
        *reinterpret_cast<uint32_t*>(smem + C::kOffB + 3 * C::kBBytes + ofs) = lo;
    }
    // the A operands start as zeros: columns N..15 and rows beyond N*N are never written again
    for (int idx = t; idx < 2 * C::kABytes / 16; idx += 128)
        reinterpret_cast<uint4*>(smem)[idx] = make_uint4(0, 0, 0, 0);
    if (t == 0) {
        dmma::mbar_init(bar_u, 1);
        dmma::mbar_init(bar_mma, 1);
    }
    if (warp == 0) tmem_alloc(holder, C::kTmemCols);
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    const uint32_t tmem_base = *holder;
    const uint32_t tmem_row = tmem_base + ((uint32_t)(warp * 32) << 16);   // this warp's lanes

    const uint32_t a_hi = smem_addr(smem + C::kOffAhi), a_lo = smem_addr(smem + C::kOffAlo);
    const uint32_t b_base = smem_addr(smem + C::kOffB);

    long long e = blockIdx.x;
    if (e < E && t == 0) {
        dmma::mbar_expect_tx(bar_u, (unsigned)(kN3 * sizeof(float)));
        dmma::bulk_load(land, u + e * kN3, (unsigned)(kN3 * sizeof(float)), bar_u);
    }
    unsigned par_u = 0, par_mma = 0;
    bool failed = false;
    for (; e < E && !failed; e += gridDim.x) {
        const long long next = e + gridDim.x;
        // this thread's rows: pencil q = 128*mt + t = (a,b)
        // the pointwise factor of its rows, needed after the third contraction
        float dv[C::kMT][N];
#pragma unroll
        for (int mt = 0; mt < C::kMT; ++mt) {
            const int q = 128 * mt + t;
            if (q < C::kRows) {
                const float2* g = reinterpret_cast<const float2*>(D + e * kN3 + (size_t)q * N);
#pragma unroll
                for (int j = 0; j < N / 2; ++j) {
                    const float2 p = __ldg(g + j);
                    dv[mt][2 * j] = p.x;
                    dv[mt][2 * j + 1] = p.y;
                }
            }
        }
        if (t == 0 && next < E) {
            dmma::bulk_prefetch_l2(D + next * kN3, (unsigned)(kN3 * sizeof(float)));
        }
        // gather u: row (i,j) of the landing buffer goes to rows (j,k), column i
        if (__syncthreads_or(dmma::mbar_wait(bar_u, par_u) ? 0 : 1)) {
            failed = true;
            break;
        }
        par_u ^= 1u;
#pragma unroll
        for (int mt = 0; mt < C::kMT; ++mt) {
            const int q = 128 * mt + t;
            if (q < C::kRows) {
                const int a = q / N, b = q - a * N;
                float val[16];
                const float2* src = reinterpret_cast<const float2*>(land + q * N);
#pragma unroll
                for (int j = 0; j < N / 2; ++j) {
                    const float2 p = src[j];
                    val[2 * j] = p.x;
                    val[2 * j + 1] = p.y;
                }
                scatter_row<N, C>(smem, b * N, a, val);
            }
        }
        dmma::fence_async_proxy();
        fence_before_sync();
        __syncthreads();
        // the landing buffer is free: the next element's u comes in under the six contractions
        if (t == 0 && next < E) {
            dmma::mbar_expect_tx(bar_u, (unsigned)(kN3 * sizeof(float)));
            dmma::bulk_load(land, u + next * kN3, (unsigned)(kN3 * sizeof(float)), bar_u);
        }
#pragma unroll 1
        for (int stage = 0; stage < 6; ++stage) {
            if (t == 0) {
                fence_after_sync();
                const uint32_t bh = b_base + (stage < 3 ? 0 : 2) * C::kBBytes, bl = bh + C::kBBytes;
#pragma unroll
                for (int mt = 0; mt < C::kMT; ++mt) {
                    const uint32_t d = tmem_base + mt * 16;
#pragma unroll
                    for (int ks = 0; ks < 2; ++ks) {
                        const uint32_t aofs = ks * 2 * C::kLbo + mt * 16 * C::kSbo;
                        const uint64_t dah = smem_desc(a_hi + aofs, C::kLbo, C::kSbo);
                        const uint64_t dal = smem_desc(a_lo + aofs, C::kLbo, C::kSbo);
                        const uint64_t dbh = smem_desc(bh + ks * 256, 128, 512);
                        const uint64_t dbl = smem_desc(bl + ks * 256, 128, 512);
                        mma_tf32_ss(d, dal, dbh, C::kIdesc, ks);
                        mma_tf32_ss(d, dah, dbl, C::kIdesc, 1);
                        mma_tf32_ss(d, dah, dbh, C::kIdesc, 1);
                    }
                }
                mma_commit(bar_mma);
            }
            if (__syncthreads_or(dmma::mbar_wait(bar_mma, par_mma) ? 0 : 1)) {
                failed = true;
                break;
            }
            par_mma ^= 1u;
            fence_after_sync();
#pragma unroll
            for (int mt = 0; mt < C::kMT; ++mt) {
                float val[16];
                tmem_load16(val, tmem_row + mt * 16);       // every warp takes part (aligned)
                const int q = 128 * mt + t;
                if (q < C::kRows) {
                    const int a = q / N, b = q - a * N;
                    if (stage == 2) {
#pragma unroll
                        for (int c = 0; c < N; ++c) val[c] *= dv[mt][c];
                    }
                    if (stage < 5) {
                        scatter_row<N, C>(smem, b * N, a, val);
                    } else {
                        float2* dst = reinterpret_cast<float2*>(v + e * kN3 + (size_t)q * N);
#pragma unroll
                        for (int j = 0; j < N / 2; ++j) dst[j] = make_float2(val[2 * j], val[2 * j + 1]);
                    }
                }
            }
            dmma::fence_async_proxy();
            fence_before_sync();
            __syncthreads();
        }
    }
    if (failed && t == 0) {
        // not expected: flag it, then give what may still be in flight (the bulk copy into the
        // landing buffer, tensor instructions) one more bounded wait before the CTA lets go of
        // its shared and tensor memory
        atomicOr(&dmma::g_bulk_wait_timeout, 1);
        dmma::mbar_wait(bar_u, par_u);
        dmma::mbar_wait(bar_mma, par_mma);
    }
    __syncthreads();
    if (warp == 0) tmem_free(tmem_base, C::kTmemCols);
}

}  // namespace umma
}  // namespace ekl
