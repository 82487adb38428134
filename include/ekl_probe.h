/*
 * ekl_probe -- measurement helpers for the roofline figures quoted beside the operators of
 * ekl_tpo.h.  A separate library (libekl_probe.so): nothing here is on the product path and
 * the paper has no counterpart for any of it.  Every call enqueues ONE kernel on `stream`,
 * writes the number of floating-point operations that launch performs to *flops (HOST
 * pointer, written before returning) and returns 0, or a non-zero code: 1 = null pointer,
 * 2 = bad count, 6 = the launch failed.  Timing the launch with CUDA events gives the rate.
 * `sink` is a DEVICE buffer of at least blocks * threads doubles (threads is 256 unless
 * stated) that receives one value per thread, so that no work can be optimised away.
 */
#ifndef EKL_PROBE_H
#define EKL_PROBE_H

#include <cuda_runtime_api.h>

#ifdef __cplusplus
extern "C" {
#endif

/* 16 independent chains of dependent FMAs per thread, acc = acc * a + b: one register is
 * both source and destination.  Reads a little under the pipe's rate. */
int ekl_probe_fp64_fma_chain(double* sink, int blocks, int iters, double* flops,
                             cudaStream_t stream);

/* The form a mode contraction has on the CUDA cores: 14 accumulators per thread,
 * acc[o] = s[o] * x + acc[o], operator entries s[o] and the datum x all in registers. */
int ekl_probe_fp64_fma_contraction(double* sink, int blocks, int iters, double* flops,
                                   cudaStream_t stream);

/* mma.sync.m8n8k4.f64 from registers, `chains` (1, 2 or 4) independent accumulator chains
 * per warp, 16 warps per SM.  512 flops per instruction and warp. */
int ekl_probe_fp64_dmma(double* sink, int blocks, int iters, int chains, double* flops,
                        cudaStream_t stream);

/* Both at once: per iteration 8 tensor steps and 16 FMAs per thread. */
int ekl_probe_fp64_dmma_plus_fma(double* sink, int blocks, int iters, double* flops,
                                 cudaStream_t stream);

/*
 * The inner loop of the tensor-path inverse Helmholtz kernel for n = 14 without any global
 * traffic: CTAs of 8 warps, 2 per SM, each repeating `stages` times a stage of 49 tiles of 8
 * pencils (operand fragments read from shared memory, two accumulator chains of four
 * m8n8k4 steps, results written back to shared memory in the transposed layout) followed by
 * a CTA barrier.  *flops counts the USEFUL work, 2 * 14 * 14 per pencil (the tensor steps
 * compute a padded 16 x 16); *padded_flops what the tensor pipe executes.  threads = 256.
 */
int ekl_probe_stage_loop_n14(double* sink, int blocks, int stages, double* flops,
                             double* padded_flops, cudaStream_t stream);

/*
 * The same stage on the CUDA cores (the contender the tensor path has to beat): every thread
 * owns `PENCILS` = 2 pencils of a batch of 2 elements, keeps its 2 x 14 accumulators in
 * registers, reads the operator row by row with warp-uniform 128-bit shared loads and its
 * data from the same shared layout as above, and writes the transposed result back; no
 * padding of any kind.  *flops = 2 * 14 * 14 per pencil.  CTAs of 196 threads.
 */
int ekl_probe_stage_loop_n14_fma(double* sink, int blocks, int stages, double* flops,
                                 cudaStream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* EKL_PROBE_H */
