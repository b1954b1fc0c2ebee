// Measurement aid, built into its own small library (not part of the product path): the tensor-core issue loop.
// Every SM issues `iters` groups of four tcgen05.mma kind::mxf4nvf4 instructions (M = 128, N = 256, K = 64 each) on operand
// and scale tiles that stay in shared / tensor memory; no global memory is touched inside the loop. The rate it reaches is
// the tensor-core ceiling this device gives the FP4 GEMMs at the clocks it runs under load.
#include "../../include/nvfp4_measure.h"

#include "nvfp4_tc.cuh"

namespace nvfp4 {
namespace {

constexpr uint32_t PROBE_SMEM_BYTES = 16384 + 32768 + 2048 + 4096 + 1024 + 64;

__global__ void __launch_bounds__(64, 1) mma_issue_probe_kernel(int32_t iters, int32_t* dev_status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t a_tile = smem_base, b_tile = smem_base + 16384, sfa = smem_base + 49152, sfb = sfa + 2048;
  const uint32_t done_bar = sfb + 4096;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;
  const int warp = threadIdx.x >> 5;
  // operands: the E2M1 code of 1.0 everywhere (0x22), scales: the E4M3 byte of 1.0 (0x38)
  for (uint32_t i = threadIdx.x; i < (49152u >> 2); i += 64) reinterpret_cast<uint32_t*>(gen)[i] = 0x22222222u;
  for (uint32_t i = threadIdx.x; i < (6144u >> 2); i += 64) reinterpret_cast<uint32_t*>(gen + 49152)[i] = 0x38383838u;
  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    mbar_init(done_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes above, async-proxy reads below
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  pdl_prologue();
  if (warp == 1) {
    const uint32_t leader = elect_leader();
    const uint32_t idesc = instr_desc<256>();
    const uint32_t sf_tmem = tmem_base + 256;
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      tc_cp_sf(sf_tmem + kk * 4, desc_sf(sfa + kk * 512), leader);
      tc_cp_sf(sf_tmem + 16 + kk * 8, desc_sf(sfb + kk * 512), leader);
      tc_cp_sf(sf_tmem + 16 + kk * 8 + 4, desc_sf(sfb + 2048 + kk * 512), leader);
    }
    for (int32_t it = 0; it < iters; ++it) {
#pragma unroll
      for (int kk = 0; kk < 4; ++kk)
        tc_mma_nvf4(tmem_base, desc_sw128(a_tile + kk * 32), desc_sw128(b_tile + kk * 32), idesc, sf_tmem + kk * 4,
                    sf_tmem + 16 + kk * 8, (it | kk) != 0, leader);
    }
    tc_commit(done_bar, leader);
    __all_sync(0xFFFFFFFFu, mbar_wait(done_bar, 0, &abort_flag_s, dev_status, DEFAULT_WAIT_LIMIT_CYCLES));  // bounded
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}


}  // namespace
}  // namespace nvfp4

extern "C" int32_t nvfp4_mma_issue_probe(int32_t iters, int32_t* dev_status, double* flops_out, void* stream) {
  using namespace nvfp4;
  if (iters <= 0 || iters > (1 << 20)) return 2;  // NVFP4_ERR_SHAPE
  int dev = 0, major = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return 7;  // NVFP4_ERR_CUDA
  if (major != 10) return 6;  // NVFP4_ERR_ARCH
  if (cudaFuncSetAttribute(mma_issue_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PROBE_SMEM_BYTES) != cudaSuccess)
    return 7;
  if (flops_out) *flops_out = (double)sms * (double)iters * 4.0 * 2.0 * 128.0 * 256.0 * 64.0;
  mma_issue_probe_kernel<<<dim3((unsigned)sms), dim3(64), PROBE_SMEM_BYTES, static_cast<cudaStream_t>(stream)>>>(iters, dev_status);
  return cudaGetLastError() == cudaSuccess ? 0 : 7;
}
