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

#ifdef __cplusplus
}
#endif
#endif /* NVFP4_MEASURE_H_ */
