// Measurement aid, built into its own small library (not part of the product path): the tensor-core issue loop.
// Every SM issues `iters` groups of four tcgen05.mma kind::mxf4nvf4 instructions (M = 128, N = 256 or 128, K = 64 each) on operand
// and scale tiles that stay in shared / tensor memory; the loop itself touches no global memory. The rate it reaches is
// the tensor-core ceiling this device gives the FP4 GEMMs at the clocks it runs under load. Optionally up to six more warps
// per SM keep another unit busy for as long as the loop runs and count the bytes they moved -- 16-byte stores to a scratch
// region of shared memory, tcgen05.ld of the accumulator columns, or bulk copies from an L2-resident global array into shared
// memory -- and the operand tiles can hold pseudo-random codes and scales instead of 1.0 everywhere (switching activity,
// hence power, depends on the data).
#include "../../include/nvfp4_measure.h"

#include "nvfp4_tc.cuh"

namespace nvfp4 {
namespace {

constexpr uint32_t PROBE_SCRATCH_OFFSET = 16384 + 32768 + 2048 + 4096 + 64;  // after the tiles, the scales and the barrier
constexpr uint32_t PROBE_SCRATCH_PER_WARP = 24576;
constexpr uint32_t PROBE_BULK_PIECE = 8192;  // three pieces per side warp and round
constexpr int PROBE_MAX_STORE_WARPS = 6;
constexpr uint32_t PROBE_SMEM_BYTES = PROBE_SCRATCH_OFFSET + PROBE_MAX_STORE_WARPS * PROBE_SCRATCH_PER_WARP + 1024;
__device__ __align__(128) uint8_t probe_bulk_sink[PROBE_SCRATCH_PER_WARP];    // what the bulk-store side warps write (all to the same lines)
__device__ __align__(128) uint8_t probe_bulk_source[PROBE_SCRATCH_PER_WARP];  // what the bulk-copy side warps read (stays in L2)
constexpr uint32_t PROBE_SIDE_ROUNDS_LIMIT = 1u << 24;  // bounds the side warps' loop whatever happens to the flag

template <int PN, int SIDE, int LOOP>
__global__ void __launch_bounds__(64 + 32 * PROBE_MAX_STORE_WARPS, 1)
    mma_issue_probe_kernel(int32_t iters, int32_t stage_stride, int32_t random_data, int32_t* dev_status, unsigned long long* dev_bytes_moved) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t a_tile = smem_base, b_tile = smem_base + 16384, sfa = smem_base + 49152, sfb = sfa + 2048;
  const uint32_t done_bar = sfb + 4096, group_bar = done_bar + 8;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;
  __shared__ volatile int loop_done_s;
  constexpr int RING = 5;
  __shared__ __align__(8) uint64_t ring_full_s[RING], ring_empty_s[RING];
  const int warp = threadIdx.x >> 5;
  __shared__ __align__(8) uint64_t side_bar_s[PROBE_MAX_STORE_WARPS];
  // operands: the E2M1 code of 1.0 everywhere (0x22), scales: the E4M3 byte of 1.0 (0x38); or hashed codes (all 16 values,
  // both signs) and scales in [0.5, 1.875]
  for (uint32_t i = threadIdx.x; i < (49152u >> 2); i += blockDim.x) {
    uint32_t h = (i + 1u) * 2654435761u;
    h ^= h >> 15; h *= 2246822519u; h ^= h >> 13;
    reinterpret_cast<uint32_t*>(gen)[i] = random_data ? h : 0x22222222u;
  }
  for (uint32_t i = threadIdx.x; i < (6144u >> 2); i += blockDim.x) {
    uint32_t h = (i + 77u) * 2654435761u;
    h ^= h >> 15; h *= 2246822519u; h ^= h >> 13;
    reinterpret_cast<uint32_t*>(gen + 49152)[i] = random_data ? (0x30303030u | (h & 0x0F0F0F0Fu)) : 0x38383838u;
  }
  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    loop_done_s = 0;
    mbar_init(done_bar, 1);
    mbar_init(group_bar, 1);
    for (int r = 0; r < RING; ++r) {
      mbar_init(smem_u32(&ring_full_s[r]), 1);
      mbar_init(smem_u32(&ring_empty_s[r]), 1);
    }
    for (int w = 0; w < PROBE_MAX_STORE_WARPS; ++w) mbar_init(smem_u32(&side_bar_s[w]), 1);
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
  if (warp == 0 && LOOP >= 3) {
    // stand-in for a GEMM's producer: waits for a free stage and declares it full at once (no copy)
    const uint32_t leader = elect_leader();
    bool ok = true;
    for (int32_t it = 0; it < iters && ok; ++it) {
      const int s = it % RING;
      ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&ring_empty_s[s]), ((it / RING) & 1) ^ 1, &abort_flag_s, dev_status, DEFAULT_WAIT_LIMIT_CYCLES));
      if (!ok) break;
      mbar_expect_tx(smem_u32(&ring_full_s[s]), 0, leader);
    }
  }
  if (warp == 1) {
    const uint32_t leader = elect_leader();
    const uint32_t idesc = instr_desc<PN>();
    const uint32_t sf_tmem = tmem_base + 256;
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      tc_cp_sf(sf_tmem + kk * 4, desc_sf(sfa + kk * 512), leader);
      tc_cp_sf(sf_tmem + 16 + kk * 8, desc_sf(sfb + kk * 512), leader);
      tc_cp_sf(sf_tmem + 16 + kk * 8 + 4, desc_sf(sfb + 2048 + kk * 512), leader);
    }
    const long long t_loop = clock64();
    uint32_t stage = 0, phase = 0;
    bool next_ready = false;
    const uint32_t full0 = smem_u32(&ring_full_s[0]), empty0 = smem_u32(&ring_empty_s[0]);
    // low words of the descriptors of stage 0 (the high words are constants): an address enters as (address >> 4) in the low
    // 14 bits, so the descriptor of a later stage or k step is one 32-bit addition away
    const uint32_t a_lo0 = (uint32_t)desc_sw128(a_tile), b_lo0 = (uint32_t)desc_sw128(b_tile);
    const uint32_t sfa_lo0 = (uint32_t)desc_sf(sfa), sfb_lo0 = (uint32_t)desc_sf(sfb);
    constexpr uint32_t SW_HI = (uint32_t)(((uint64_t)64 << 32 | (uint64_t)1 << 46 | (uint64_t)2 << 61) >> 32);
    constexpr uint32_t SF_HI = (uint32_t)(((uint64_t)8 << 32 | (uint64_t)1 << 46) >> 32);
    for (int32_t it = 0; it < iters; ++it) {
      // LOOP 0: only the MMAs; 1: the group's scale copies first, as a GEMM issues them (four sets of scale columns in
      // rotation); 2: and a commit to a barrier after the group; 3: a five-stage ring with a producer warp that declares a
      // released stage full at once, stage addresses and barrier waits written as in a straightforward GEMM main loop;
      // 4: the same ring as the library's GEMMs walk it: running stage / phase counters, descriptors by addition, and a
      // non-blocking look at the next stage's barrier issued before this stage's instructions
      const uint32_t sf_set = LOOP ? sf_tmem + (uint32_t)(it & 3) * 48u : sf_tmem;
      if constexpr (LOOP == 3) {
        const int sidx = it % RING;
        if (!__all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&ring_full_s[sidx]), (it / RING) & 1, &abort_flag_s, dev_status, DEFAULT_WAIT_LIMIT_CYCLES))) break;
        tc_fence_after();
        const uint32_t st = (uint32_t)(sidx * stage_stride);  // stage_stride is 0: all stages share the tiles; the compiler cannot know
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          tc_cp_sf(sf_set + kk * 4, desc_sf(sfa + st + kk * 512), leader);
          tc_cp_sf(sf_set + 16 + kk * 8, desc_sf(sfb + st + kk * 512), leader);
          if (PN == 256) tc_cp_sf(sf_set + 16 + kk * 8 + 4, desc_sf(sfb + st + 2048 + kk * 512), leader);
        }
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          tc_mma_nvf4(tmem_base, desc_sw128(a_tile + st + kk * 32), desc_sw128(b_tile + st + kk * 32), idesc, sf_set + kk * 4,
                      sf_set + 16 + kk * 8, (it | kk) != 0, leader);
        tc_commit(smem_u32(&ring_empty_s[sidx]), leader);
      } else if constexpr (LOOP == 4) {
        if (!next_ready) {
          if (!__all_sync(0xFFFFFFFFu, mbar_wait(full0 + 8u * stage, phase, &abort_flag_s, dev_status, DEFAULT_WAIT_LIMIT_CYCLES))) break;
        }
        tc_fence_after();
        const uint32_t st16 = stage * (uint32_t)stage_stride;  // in 16-byte units
        const uint32_t this_empty = empty0 + 8u * stage;
        if (++stage == (uint32_t)RING) {
          stage = 0;
          phase ^= 1;
        }
        const uint32_t next_look = mbar_test(full0 + 8u * stage, phase);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          tc_cp_sf(sf_set + kk * 4, ((uint64_t)SF_HI << 32) | (sfa_lo0 + st16 + kk * 32), leader);
          tc_cp_sf(sf_set + 16 + kk * 8, ((uint64_t)SF_HI << 32) | (sfb_lo0 + st16 + kk * 32), leader);
          if (PN == 256) tc_cp_sf(sf_set + 16 + kk * 8 + 4, ((uint64_t)SF_HI << 32) | (sfb_lo0 + st16 + 128 + kk * 32), leader);
        }
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          tc_mma_nvf4(tmem_base, ((uint64_t)SW_HI << 32) | (a_lo0 + st16 + kk * 2), ((uint64_t)SW_HI << 32) | (b_lo0 + st16 + kk * 2), idesc,
                      sf_set + kk * 4, sf_set + 16 + kk * 8, (it | kk) != 0, leader);
        tc_commit(this_empty, leader);
        next_ready = __all_sync(0xFFFFFFFFu, next_look);
      } else {
        if constexpr (LOOP >= 1) {
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            tc_cp_sf(sf_set + kk * 4, desc_sf(sfa + kk * 512), leader);
            tc_cp_sf(sf_set + 16 + kk * 8, desc_sf(sfb + kk * 512), leader);
            if (PN == 256) tc_cp_sf(sf_set + 16 + kk * 8 + 4, desc_sf(sfb + 2048 + kk * 512), leader);
          }
        }
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          tc_mma_nvf4(tmem_base, desc_sw128(a_tile + kk * 32), desc_sw128(b_tile + kk * 32), idesc, sf_set + kk * 4,
                      sf_set + 16 + kk * 8, (it | kk) != 0, leader);
        if constexpr (LOOP == 2) tc_commit(group_bar, leader);
      }
    }
    tc_commit(done_bar, leader);
    __all_sync(0xFFFFFFFFu, mbar_wait(done_bar, 0, &abort_flag_s, dev_status, DEFAULT_WAIT_LIMIT_CYCLES));  // bounded
    loop_done_s = 1;
    if (dev_bytes_moved && leader) atomicMax(dev_bytes_moved + 1, (unsigned long long)(clock64() - t_loop));
  } else if (warp >= 2) {
    // side warps: rounds of work on another unit until the MMA loop has drained (or the round limit is reached)
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t mine = smem_base + PROBE_SCRATCH_OFFSET + (uint32_t)(warp - 2) * PROBE_SCRATCH_PER_WARP;
    uint32_t rounds = 0;
    unsigned long long per_round = 0;
    if constexpr (SIDE == 0) {  // eight 16-byte stores per lane: 4 KB per warp and round
      per_round = 4096;
      while (rounds < PROBE_SIDE_ROUNDS_LIMIT && !loop_done_s) {
#pragma unroll
        for (int j = 0; j < 8; ++j)
          asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(mine + lane * 16 + j * 512), "r"(rounds) : "memory");
        ++rounds;
      }
    } else if constexpr (SIDE == 1) {  // the warp's lane quarter of the accumulator, 32 columns per load: PN / 32 loads per round
      per_round = 32ull * PN * 4;
      const uint32_t taddr = tmem_base + (((uint32_t)(warp & 3) * 32u) << 16);
      uint32_t keep = 0;
      while (rounds < PROBE_SIDE_ROUNDS_LIMIT && !loop_done_s) {
#pragma unroll 1
        for (int c = 0; c < PN; c += 32) {
          uint32_t v[32];
          tc_ld32(taddr + c, v);
          tc_wait_ld();
          keep ^= v[0] ^ v[31];
        }
        ++rounds;
      }
      if (keep == 0x12345678u && dev_status) atomicAdd(dev_status, 0);  // keeps the loaded values alive
    } else if constexpr (SIDE == 3) {  // three bulk stores of 8 KB from the warp's scratch to global (L2) per round
      per_round = 3ull * PROBE_BULK_PIECE;
      const uint32_t leader = elect_leader();
      while (rounds < PROBE_SIDE_ROUNDS_LIMIT && !loop_done_s) {
#pragma unroll
        for (int j = 0; j < 3; ++j)
          asm volatile("{\n.reg .pred q;\nsetp.ne.b32 q, %3, 0;\n@q cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;\n}" ::"l"(
                           probe_bulk_sink + j * PROBE_BULK_PIECE),
                       "r"(mine + j * PROBE_BULK_PIECE), "r"(PROBE_BULK_PIECE), "r"(leader)
                       : "memory");
        bulk_commit();
        bulk_wait_read<0>();  // the engine has read the scratch (the global writes may still be in flight)
        ++rounds;
      }
      bulk_wait_all();
    } else {  // three bulk copies of 8 KB from global (L2) into the warp's scratch per round, one barrier phase per round
      per_round = 3ull * PROBE_BULK_PIECE;
      const uint32_t bar = smem_u32(&side_bar_s[warp - 2]);
      const uint32_t leader = elect_leader();
      bool ok = true;
      while (ok && rounds < PROBE_SIDE_ROUNDS_LIMIT && !loop_done_s) {
        mbar_expect_tx(bar, 3 * PROBE_BULK_PIECE, leader);
#pragma unroll
        for (int j = 0; j < 3; ++j) bulk_load(mine + j * PROBE_BULK_PIECE, probe_bulk_source + j * PROBE_BULK_PIECE, PROBE_BULK_PIECE, bar, leader);
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar, rounds & 1, &abort_flag_s, dev_status, DEFAULT_WAIT_LIMIT_CYCLES));  // bounded
        ++rounds;
      }
    }
    if (dev_bytes_moved && lane == 0) atomicAdd(dev_bytes_moved, (unsigned long long)rounds * per_round);
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

static int32_t issue_probe(int32_t iters, int32_t n, int32_t loop_kind, int32_t side_warps, int32_t side_kind, int32_t random_data, int32_t* dev_status,
                           unsigned long long* dev_bytes_moved, double* flops_out, void* stream) {
  using namespace nvfp4;
  if (iters <= 0 || iters > (1 << 20) || (n != 128 && n != 256 && n != 32) || side_warps < 0 || side_warps > PROBE_MAX_STORE_WARPS ||
      side_kind < 0 || side_kind > 3 || loop_kind < 0 || loop_kind > 4)
    return 2;  // NVFP4_ERR_SHAPE
  int dev = 0, major = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return 7;  // NVFP4_ERR_CUDA
  if (major != 10) return 6;  // NVFP4_ERR_ARCH
  using kernel_t = void (*)(int32_t, int32_t, int32_t, int32_t*, unsigned long long*);
#define PROBE_ROW(N, S) {mma_issue_probe_kernel<N, S, 0>, mma_issue_probe_kernel<N, S, 1>, mma_issue_probe_kernel<N, S, 2>, \
                         mma_issue_probe_kernel<N, S, 3>, mma_issue_probe_kernel<N, S, 4>}
  static const kernel_t kernels[3][4][5] = {{PROBE_ROW(128, 0), PROBE_ROW(128, 1), PROBE_ROW(128, 2), PROBE_ROW(128, 3)},
                                            {PROBE_ROW(256, 0), PROBE_ROW(256, 1), PROBE_ROW(256, 2), PROBE_ROW(256, 3)},
                                            {PROBE_ROW(32, 0), PROBE_ROW(32, 1), PROBE_ROW(32, 2), PROBE_ROW(32, 3)}};
#undef PROBE_ROW
  const kernel_t kernel = kernels[n == 256 ? 1 : n == 32 ? 2 : 0][side_kind][loop_kind];
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PROBE_SMEM_BYTES) != cudaSuccess) return 7;
  if (flops_out) *flops_out = (double)sms * (double)iters * 4.0 * 2.0 * 128.0 * (double)n * 64.0;
  kernel<<<dim3((unsigned)sms), dim3(64 + 32 * (unsigned)side_warps), PROBE_SMEM_BYTES, static_cast<cudaStream_t>(stream)>>>(
      iters, /*stage_stride=*/0, random_data != 0, dev_status, dev_bytes_moved);
  return cudaGetLastError() == cudaSuccess ? 0 : 7;
}

extern "C" int32_t nvfp4_mma_issue_probe(int32_t iters, int32_t* dev_status, double* flops_out, void* stream) {
  return issue_probe(iters, 256, 0, 0, 0, 0, dev_status, nullptr, flops_out, stream);
}
extern "C" int32_t nvfp4_mma_issue_probe_n(int32_t iters, int32_t n, int32_t loop_kind, int32_t side_warps, int32_t side_kind, int32_t random_data,
                                           int32_t* dev_status, unsigned long long* dev_bytes_moved, double* flops_out,
                                           void* stream) {
  return issue_probe(iters, n, loop_kind, side_warps, side_kind, random_data, dev_status, dev_bytes_moved, flops_out, stream);
}
