/*
 * nvfp4_measure.h -- measurement aids of the NVFP4 library. Nothing here is a step of the method (the paper has no
 * counterpart) and nothing in the product path calls it; the benchmark does.
 */
#ifndef NVFP4_MEASURE_H_
#define NVFP4_MEASURE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* In libnvfp4_b200.so: number of kernels the library has enqueued since it was loaded (all threads, all devices). */
long long nvfp4_launch_count(void);

/* In libnvfp4_measure.so: every SM of the current device issues iters x 4 block-scaled FP4 MMA instructions (M = 128,
 * N = 256, K = 64) on tiles resident in shared / tensor memory, no global traffic in the loop. *flops_out (host, optional)
 * receives the FP4 flops one launch performs; time the launch with events to get the device's tensor-core ceiling under
 * load. dev_status: optional device int, set to 8 if the kernel's single bounded wait ran out. 1 <= iters <= 2^20.
 * Returns 0, or the library's status codes 2 (iters out of range), 6 (not sm_100), 7 (CUDA error). */
int32_t nvfp4_mma_issue_probe(int32_t iters, int32_t* dev_status, double* flops_out, void* stream);
/* The same loop with more to choose:
 *   n            32, 128 or 256: instructions of M = 128, N = n, K = 64 (a 128 x 128 x 64 instruction reads 8 KB of operands
 *                from shared memory for half the arithmetic of a 128 x 256 x 64 one, which reads 12 KB; with n = 32 the
 *                arithmetic is short enough that the issuing warp's own cost per instruction shows);
 *   loop_kind    0 = only the MMAs; 1 = before each group of four MMAs the copies of its block scales from shared into
 *                tensor memory (8 for n <= 128, 12 for n = 256; four sets of scale columns in rotation), as a GEMM issues
 *                them; 2 = and a tcgen05.commit to a barrier after each group, as a GEMM releases an operand stage;
 *                3 = a ring of five stages with a second warp that declares every released stage full again at once (a
 *                GEMM's producer without its copies), walked the straightforward way (stage = iteration mod 5, a blocking
 *                wait per stage, descriptors rebuilt from the stage address); 4 = the same ring walked as the library's
 *                GEMMs walk it (running stage / phase counters, descriptors by addition to the low word, a non-blocking
 *                look at the next stage's barrier issued before this stage's instructions);
 *   side_warps   0..6 further warps per SM that keep another unit busy until the loop has drained;
 *   side_kind    what they do: 0 = 16-byte stores to a scratch region of shared memory, 1 = tcgen05.ld of their lane
 *                quarter of the accumulator columns, 2 = bulk copies (three of 8 KB per warp in flight) from a 24 KB
 *                global array, resident in L2, into shared memory, 3 = bulk stores of the same size from shared memory to
 *                one 24 KB global array (all SMs write the same lines: a test of the shared-memory side, not of the
 *                memory system);
 *   random_data  0 = every operand code and scale is 1.0; otherwise hashed codes (all sixteen values) and scales in
 *                [0.5, 1.875]: the arithmetic is the same, the switching activity, hence the power drawn and the clock the
 *                device sustains, is not.
 * dev_bytes_moved: optional device array of two 64-bit counters (zeroed by the caller): to [0] every side warp adds the
 * bytes it stored, loaded or copied; [1] receives the largest number of SM clock cycles any SM spent between its first
 * MMA and the completion of its last. With the launch's duration these give the tensor-core rate under a known rate of
 * other on-chip traffic, and the SM clock the loop ran at. All waits are bounded (dev_status 8 when one ran out). Status 2
 * for values outside the ranges above. */
int32_t nvfp4_mma_issue_probe_n(int32_t iters, int32_t n, int32_t loop_kind, int32_t side_warps, int32_t side_kind, int32_t random_data,
                                int32_t* dev_status, unsigned long long* dev_bytes_moved, double* flops_out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* NVFP4_MEASURE_H_ */
