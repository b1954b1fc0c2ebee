// Block-scaled FP4 GEMM for sm_100a (the "FP4 MM" of the paper's Sec. 2.3):
//     C[m, n] = sum_k (Pa Sba Sga)[m, k] (Pb Sbb Sgb)[n, k],  both operands packed along k.
//
// Design (one CTA per SM, persistent over output tiles, warp-specialised):
//   warp 0      TMA producer: per 256-wide k tile, two tiled bulk-tensor loads (A, B codes; 128-byte swizzle) and
//               two plain bulk copies (the 2 KB of E4M3 scales each operand tile needs, contiguous in the
//               TILED128x4 layout) into a ring of shared-memory stages, completion on an mbarrier.
//   warp 1      MMA issuer: copies the scales shared -> tensor memory (tcgen05.cp) and issues
//               tcgen05.mma kind::mxf4nvf4 block_scale (E2M1 data, UE4M3 scale per 16 elements, K = 64 per
//               instruction, FP32 accumulators in tensor memory, two accumulator buffers).
//   warps 2..9  epilogue (two warps per tensor-memory lane quadrant, half of the tile's columns each): tcgen05.ld the
//               accumulator, apply the FP32 global scales, convert, stage 128-byte row pieces in shared memory and
//               write them with bulk tensor stores. (The outer-block variant further down keeps four promotion
//               warps, 2..5.)
// Every wait on an mbarrier is bounded (Params::wait_limit clock cycles); when a bound is hit the kernel raises a
// status word, all roles drain and the CTA frees its tensor memory and exits.
#include <cuda.h>
#include <cuda_bf16.h>

#include "nvfp4_device.cuh"
#include "nvfp4_internal.h"
#include "nvfp4_tc.cuh"

namespace nvfp4 {

namespace {

constexpr int NUM_THREADS = 192;

// Single-CTA kernel: 128 x 128 output tiles.
constexpr int BN = 128;
struct Cfg {
  static constexpr uint32_t B_BYTES = BN * BK / 2;
  static constexpr uint32_t SFB_BYTES = 2048;
  static constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES + SFA_BYTES + SFB_BYTES;  // 36 KB, multiple of 1024
  static constexpr int STAGES = 5;
  // epilogue staging for bulk tensor stores: per epilogue warp one 32-row x 128-byte buffer
  static constexpr uint32_t STAGING_BYTES = 8 * 4096;
  static constexpr uint32_t SMEM_BYTES = STAGES * STAGE_BYTES + STAGING_BYTES + 1024 /*align slack*/ + 256 /*barriers*/;
  // tensor memory columns: two accumulators (a tile's epilogue runs under the next tile's MMAs), the optional
  // high-precision accumulator, then four scale buffers (A: 16 columns, B: 16)
  static constexpr uint32_t ACC_COLS = BN;
  static constexpr uint32_t ACC_BUFS = 2;
  // Eight epilogue warps: two per tensor-memory lane quadrant, each taking half of the tile's columns (a tile's
  // epilogue with four warps took 1.9 us and bounded every product with K <= 1024).
  static constexpr int EPI_WARPS = 8;
  static constexpr int THREADS = 64 + 32 * EPI_WARPS;
  static constexpr uint32_t SF_COLS = 32;
  static constexpr uint32_t TMEM_COLS = 512;
  static_assert(ACC_BUFS * ACC_COLS + 128 + 4 * SF_COLS <= TMEM_COLS, "tensor memory budget");
};

struct Params {
  const uint8_t* a_sf;
  const uint8_t* b_sf;
  const float* a_gscale;
  const float* b_gscale;
  void* C;
  int64_t ldc;
  int64_t M, N;
  int32_t k_tiles;        // number of 256-wide k tiles
  int32_t k_chunks;       // number of 128-wide k chunks (BLOCK128 variant)
  int64_t g_per_row;      // global scales per operand row in BLOCK128 mode
  int32_t sf_tiles_a;     // 512-byte scale tiles per 128-row tile of A (= padded k-blocks / 4)
  int32_t sf_tiles_b;
  int32_t m_tiles, n_tiles;
  int32_t c_is_f32, accumulate;
  int32_t hp_k_tiles;     // OutControl: 64-wide BF16 k tiles of the high-precision side product (0 = none)
  int32_t use_tma_store;  // C is described by a tensor map: stage the epilogue in shared memory and bulk-store it
  int32_t starve;         // test hook: the first stage's "full" barrier expects 16 bytes more than will ever arrive
  long long wait_limit;   // bound of every wait, in clock cycles
  int32_t* dev_status;
};

// When accumulating: adds the old C to W consecutive values of output row m from column n0 (a full chunk inside C).
template <int W>
__device__ __forceinline__ void add_existing(const Params& p, int64_t m, int64_t n0, float (&o)[W]) {
  if (p.accumulate) {
    if (p.c_is_f32) {
      const float* cp = reinterpret_cast<const float*>(p.C) + m * p.ldc + n0;
#pragma unroll
      for (int j = 0; j < W; j += 4) {
        const float4 q = *reinterpret_cast<const float4*>(cp + j);
        o[j] += q.x; o[j + 1] += q.y; o[j + 2] += q.z; o[j + 3] += q.w;
      }
    } else {
      const uint16_t* cp = reinterpret_cast<const uint16_t*>(p.C) + m * p.ldc + n0;
#pragma unroll
      for (int j = 0; j < W; j += 8) {
        const uint4 old = *reinterpret_cast<const uint4*>(cp + j);
        const uint32_t ow[4] = {old.x, old.y, old.z, old.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          o[j + 2 * q] += bf16_lo(ow[q]);
          o[j + 2 * q + 1] += bf16_hi(ow[q]);
        }
      }
    }
  }
}

// The columns of a chunk that sticks out past N (values final: scaled, accumulated): plain element stores, nothing beyond
// column N - 1 is touched. The bulk tensor store is kept for whole chunks only: its clipping at the edge of C was seen to
// overwrite the row's padding up to the next 16-byte boundary.
template <int W>
__device__ __forceinline__ void store_ragged(const Params& p, int64_t m, int64_t n0, const float (&o)[W]) {
  if (p.c_is_f32) {
    float* cp = reinterpret_cast<float*>(p.C) + m * p.ldc + n0;
#pragma unroll
    for (int j = 0; j < W; ++j)
      if (n0 + j < p.N) cp[j] = o[j];
  } else {
    __nv_bfloat16* cp = reinterpret_cast<__nv_bfloat16*>(p.C) + m * p.ldc + n0;
#pragma unroll
    for (int j = 0; j < W; ++j)
      if (n0 + j < p.N) cp[j] = __float2bfloat16_rn(o[j]);
  }
}

// One output row, 32 consecutive columns starting at n0 (m < M and n0 < N are the caller's business): add the old C when
// accumulating, convert, store.
__device__ __forceinline__ void store_row_chunk(const Params& p, int64_t m, int64_t n0, float (&o)[32]) {
    if (p.c_is_f32) {
      float* cp = reinterpret_cast<float*>(p.C) + m * p.ldc + n0;
      if (n0 + 32 <= p.N) {
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
          float4 q = make_float4(o[j], o[j + 1], o[j + 2], o[j + 3]);
          if (p.accumulate) {
            const float4 old = *reinterpret_cast<const float4*>(cp + j);
            q.x += old.x; q.y += old.y; q.z += old.z; q.w += old.w;
          }
          *reinterpret_cast<float4*>(cp + j) = q;
        }
      } else {
        for (int j = 0; j < 32 && n0 + j < p.N; ++j) cp[j] = p.accumulate ? cp[j] + o[j] : o[j];
      }
    } else {
      __nv_bfloat16* cp = reinterpret_cast<__nv_bfloat16*>(p.C) + m * p.ldc + n0;
      if (n0 + 32 <= p.N) {
#pragma unroll
        for (int j = 0; j < 32; j += 8) {
          if (p.accumulate) {
            const uint4 old = *reinterpret_cast<const uint4*>(cp + j);
            const uint32_t ow[4] = {old.x, old.y, old.z, old.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              o[j + 2 * q] += bf16_lo(ow[q]);
              o[j + 2 * q + 1] += bf16_hi(ow[q]);
            }
          }
          uint4 q;
          __nv_bfloat162 h;
          h = __floats2bfloat162_rn(o[j], o[j + 1]); q.x = *reinterpret_cast<uint32_t*>(&h);
          h = __floats2bfloat162_rn(o[j + 2], o[j + 3]); q.y = *reinterpret_cast<uint32_t*>(&h);
          h = __floats2bfloat162_rn(o[j + 4], o[j + 5]); q.z = *reinterpret_cast<uint32_t*>(&h);
          h = __floats2bfloat162_rn(o[j + 6], o[j + 7]); q.w = *reinterpret_cast<uint32_t*>(&h);
          *reinterpret_cast<uint4*>(cp + j) = q;
        }
      } else {
        for (int j = 0; j < 32 && n0 + j < p.N; ++j) {
          const float prev = p.accumulate ? __bfloat162float(cp[j]) : 0.0f;
          cp[j] = __float2bfloat16_rn(o[j] + prev);
        }
      }
    }
}

template <int GS>
__global__ void __launch_bounds__(Cfg::THREADS, 1)
gemm_nvfp4_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                  const __grid_constant__ CUtensorMap tmC, const __grid_constant__ CUtensorMap tmAh,
                  const __grid_constant__ CUtensorMap tmBh, const Params p) {
  using C = Cfg;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t staging_base = smem_base + C::STAGES * C::STAGE_BYTES;
  const uint32_t bar_base = staging_base + C::STAGING_BYTES;
  // barriers: full[STAGES], empty[STAGES], acc_full[2], acc_empty[2], drain
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (C::STAGES + s); };
  auto acc_full_bar = [&](int b) { return bar_base + 8u * (2 * C::STAGES + b); };
  auto acc_empty_bar = [&](int b) { return bar_base + 8u * (2 * C::STAGES + 2 + b); };
  const uint32_t drain_bar = bar_base + 8u * (2 * C::STAGES + 4);
  const uint32_t hp_empty_bar = bar_base + 8u * (2 * C::STAGES + 5);  // high-precision accumulator drained
  // tensor-memory columns of the optional high-precision accumulator and of the scale buffers
  const uint32_t hp_cols = p.hp_k_tiles > 0 ? 128u : 0u;
  const uint32_t hp_tmem_col = C::ACC_BUFS * C::ACC_COLS;
  const uint32_t sf_tmem_col = C::ACC_BUFS * C::ACC_COLS + hp_cols;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;
  volatile int* abort_flag = &abort_flag_s;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    for (int s = 0; s < C::STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(acc_full_bar(b), 1);
      mbar_init(acc_empty_bar(b), C::EPI_WARPS);
    }
    mbar_init(drain_bar, 1);
    mbar_init(hp_empty_bar, C::EPI_WARPS);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                 "r"(C::TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  pdl_prologue();  // everything above touched only shared and tensor memory

  const int64_t num_tiles = (int64_t)p.m_tiles * p.n_tiles;

  if (warp == 0) {
    // ===================================== TMA producer (warp stays converged) ===============================
    const uint32_t leader = elect_leader();
    uint32_t it = 0, s = 0, wait_parity = 1;  // running stage and the parity its "empty" barrier is waited with
    bool ok = true;
    for (int64_t t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
      const int32_t mt = (int32_t)(t / p.n_tiles), nt = (int32_t)(t % p.n_tiles);
      const uint8_t* sfa_src = p.a_sf + (size_t)mt * p.sf_tiles_a * 512;
      const uint8_t* sfb_src = p.b_sf + (size_t)nt * p.sf_tiles_b * 512;
      for (int32_t kt = 0; kt < p.k_tiles; ++kt, ++it, s = (s + 1 == (uint32_t)C::STAGES ? 0u : s + 1), wait_parity ^= (s == 0)) {
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(empty_bar(s), wait_parity, abort_flag, p.dev_status, p.wait_limit));
        if (!ok) break;
        const uint32_t st = smem_base + s * C::STAGE_BYTES;
        // (test hook of the bounded waits: with `starve` the very first stage never completes)
        mbar_expect_tx(full_bar(s), C::STAGE_BYTES + ((p.starve && it == 0) ? 16u : 0u), leader);
        tma_load_2d(st, &tmA, kt * (BK / 2), mt * BM, full_bar(s), leader);
        tma_load_2d(st + A_BYTES, &tmB, kt * (BK / 2), nt * BN, full_bar(s), leader);
        bulk_load(st + A_BYTES + C::B_BYTES, sfa_src + (size_t)kt * 2048, 2048, full_bar(s), leader);
        bulk_load(st + A_BYTES + C::B_BYTES + SFA_BYTES, sfb_src + (size_t)kt * 2048, 2048, full_bar(s), leader);
      }
      // OutControl: the BF16 outlier channels of both operands, 64 per stage, into the same stage buffers
      for (int32_t h = 0; h < p.hp_k_tiles && ok; ++h, ++it, s = (s + 1 == (uint32_t)C::STAGES ? 0u : s + 1), wait_parity ^= (s == 0)) {
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(empty_bar(s), wait_parity, abort_flag, p.dev_status, p.wait_limit));
        if (!ok) break;
        const uint32_t st = smem_base + s * C::STAGE_BYTES;
        mbar_expect_tx(full_bar(s), A_BYTES + C::B_BYTES, leader);
        tma_load_2d(st, &tmAh, h * 64, mt * BM, full_bar(s), leader);
        tma_load_2d(st + A_BYTES, &tmBh, h * 64, nt * BN, full_bar(s), leader);
      }
    }
    if (!ok) {
      // give the copies already in flight a bounded time to land before the CTA may exit
      const uint32_t n_back = it < (uint32_t)C::STAGES ? it : (uint32_t)C::STAGES;
      for (uint32_t j = 0; j < n_back; ++j) {
        const uint32_t f = it - 1 - j;
        const long long t0 = clock64();
        while (!mbar_try(full_bar(f % C::STAGES), (f / C::STAGES) & 1) && clock64() - t0 < p.wait_limit) {
        }
      }
    }
  } else if (warp == 1) {
    // ===================================== MMA issuer (warp stays converged) =================================
    const uint32_t leader = elect_leader();
    const uint32_t idesc = instr_desc<BN>();
    // The issuing warp's own instruction stream is what limits a 128 x 128 tile (13 tensor-core instructions per 256 cycles of
    // math), so the loop keeps it short: running stage / phase counters instead of divisions, descriptors formed by adding
    // to the low word of the first stage's (an address enters as address >> 4 in the low 14 bits; the high words are
    // constants), and the try on the NEXT stage's barrier issued before this stage's instructions so that its latency
    // overlaps them.
    uint32_t it = 0, tile_it = 0, stage = 0, phase = 0;
    bool ok = true;
    bool ready = false;
    constexpr uint32_t SW_HI = (uint32_t)((((uint64_t)64 << 32) | ((uint64_t)1 << 46) | ((uint64_t)2 << 61)) >> 32);
    constexpr uint32_t SF_HI = (uint32_t)((((uint64_t)8 << 32) | ((uint64_t)1 << 46)) >> 32);
    const uint32_t a_lo0 = (uint32_t)desc_sw128(smem_base), sfa_lo0 = (uint32_t)desc_sf(smem_base + A_BYTES + C::B_BYTES);
    for (int64_t t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++tile_it) {
      const uint32_t ab = tile_it % C::ACC_BUFS;
      ok = __all_sync(0xFFFFFFFFu, mbar_wait(acc_empty_bar(ab), ((tile_it / C::ACC_BUFS) & 1) ^ 1, abort_flag, p.dev_status, p.wait_limit));
      if (!ok) break;
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + ab * C::ACC_COLS;
      for (int32_t kt = 0; kt < p.k_tiles; ++kt, ++it) {
        if (!ready) {
          ok = __all_sync(0xFFFFFFFFu, mbar_wait(full_bar(stage), phase, abort_flag, p.dev_status, p.wait_limit));
          if (!ok) break;
        }
        tc_fence_after();
        const uint32_t st16 = stage * (uint32_t)(C::STAGE_BYTES >> 4);
        const uint32_t this_empty = empty_bar(stage);
        if (++stage == (uint32_t)C::STAGES) {
          stage = 0;
          phase ^= 1u;
        }
        const uint32_t next_try = mbar_test(full_bar(stage), phase);
        const uint32_t sf_tmem = tmem_base + sf_tmem_col + (it & 3) * C::SF_COLS;
        // Scales of this k tile: shared memory -> tensor memory. Per 64-wide k step: 4 columns for the 128 rows
        // of A, 4 per 128 rows of B.
#pragma unroll
        for (int kk = 0; kk < BK / 64; ++kk) {
          tc_cp_sf(sf_tmem + kk * 4, ((uint64_t)SF_HI << 32) | (sfa_lo0 + st16 + kk * 32), leader);
          tc_cp_sf(sf_tmem + 16 + kk * 4, ((uint64_t)SF_HI << 32) | (sfa_lo0 + st16 + (SFA_BYTES >> 4) + kk * 32), leader);
        }
#pragma unroll
        for (int kk = 0; kk < BK / 64; ++kk)
          tc_mma_nvf4(d_tmem, ((uint64_t)SW_HI << 32) | (a_lo0 + st16 + kk * 2), ((uint64_t)SW_HI << 32) | (a_lo0 + st16 + (A_BYTES >> 4) + kk * 2),
                      idesc, sf_tmem + kk * 4, sf_tmem + 16 + kk * 4, (kt | kk) != 0, leader);
        tc_commit(this_empty, leader);  // stage reusable once these MMAs have read it
        ready = __all_sync(0xFFFFFFFFu, next_try);
      }
      if (p.hp_k_tiles > 0 && ok) {
        // high-precision side product into its own accumulator (single buffer: wait until the previous tile's epilogue
        // has drained it, which happened a whole main loop ago)
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(hp_empty_bar, (tile_it & 1) ^ 1, abort_flag, p.dev_status, p.wait_limit));
        if (!ok) break;
        tc_fence_after();
        const uint32_t idesc_bf16 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
        for (int32_t h = 0; h < p.hp_k_tiles; ++h, ++it) {
          if (!ready) {
            ok = __all_sync(0xFFFFFFFFu, mbar_wait(full_bar(stage), phase, abort_flag, p.dev_status, p.wait_limit));
            if (!ok) break;
          }
          tc_fence_after();
          const uint32_t st = smem_base + stage * C::STAGE_BYTES;
          const uint32_t this_empty = empty_bar(stage);
          if (++stage == (uint32_t)C::STAGES) {
            stage = 0;
            phase ^= 1u;
          }
          const uint32_t next_try = mbar_test(full_bar(stage), phase);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)  // 64 BF16 = one 128-byte swizzle row = four K = 16 steps of 32 bytes
            tc_mma_bf16(tmem_base + hp_tmem_col, desc_sw128(st + kk * 32), desc_sw128(st + A_BYTES + kk * 32), idesc_bf16,
                        (h | kk) != 0, leader);
          tc_commit(this_empty, leader);
          ready = __all_sync(0xFFFFFFFFu, next_try);
        }
        if (!ok) break;
      }
      if (ok) tc_commit(acc_full_bar(ab), leader);
    }
    // make sure nothing issued is still running before tensor memory is freed
    tc_commit(drain_bar, leader);
    {
      const long long t0 = clock64();
      while (!mbar_try(drain_bar, 0) && clock64() - t0 < p.wait_limit) {
      }
    }
  } else {
    // ===================================== epilogue ========================================================
    const int quad = warp & 3;  // tensor-memory lane quadrant this warp may read
    uint32_t tile_it = 0;
    bool ok = true;
    float alpha = 1.0f;
    if (GS == kGsTensor) alpha = __fmul_rn(p.a_gscale[0], p.b_gscale[0]);
    for (int64_t t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++tile_it) {
      const int32_t mt = (int32_t)(t / p.n_tiles), nt = (int32_t)(t % p.n_tiles);
      const uint32_t ab = tile_it % C::ACC_BUFS;
      if (!(ok = mbar_wait(acc_full_bar(ab), (tile_it / C::ACC_BUFS) & 1, abort_flag, p.dev_status, p.wait_limit))) break;
      tc_fence_after();
      const int64_t m = (int64_t)mt * BM + quad * 32 + lane;
      float sa = 1.0f;
      if (GS == kGsRow && m < p.M) sa = p.a_gscale[m];
      const int half = (warp - 2) >> 2;  // which half of the tile's columns this warp owns
      {
        // Stage 128-byte row pieces (32 FP32 or 64 BF16 columns) in shared memory with the 128-byte swizzle and let the
        // bulk-tensor engine write them: full lines, clipped at the edges of C, asynchronous.
        const uint32_t my_stage = staging_base + (uint32_t)(warp - 2) * 4096u;
        const int64_t m0 = (int64_t)mt * BM + quad * 32;
        if (p.c_is_f32) {
#pragma unroll 1
          for (int c0 = half * (BN / 2); c0 < (half + 1) * (BN / 2); c0 += 32) {
            uint32_t v[32];
            tc_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + ab * C::ACC_COLS + c0, v);
            tc_wait_ld();
            const int64_t n0 = (int64_t)nt * BN + c0;
            if (n0 >= p.N) break;
            float o[32], sgb[32];
            if (GS == kGsRow) load_sgb32(p.b_gscale, n0, p.N, sgb);
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              float sc = alpha;
              if (GS == kGsRow) sc = __fmul_rn(sa, sgb[j]);
              o[j] = __uint_as_float(v[j]) * sc;
            }
            if (hp_cols) {
              tc_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + hp_tmem_col + c0, v);
              tc_wait_ld();
              if (p.k_tiles > 0) {
#pragma unroll
                for (int j = 0; j < 32; ++j) o[j] += __uint_as_float(v[j]);
              } else {  // dense BF16 product alone (no FP4 part: the main accumulator was never written): scaled like one
#pragma unroll
                for (int j = 0; j < 32; ++j) o[j] = __uint_as_float(v[j]) * alpha;
              }
            }
            if (p.accumulate && m < p.M) {
              if (n0 + 32 <= p.N) {
                add_existing<32>(p, m, n0, o);
              } else {
#pragma unroll
                for (int j = 0; j < 32; ++j)
                  if (n0 + j < p.N) o[j] += reinterpret_cast<const float*>(p.C)[m * p.ldc + n0 + j];
              }
            }
            if (n0 + 32 > p.N) {  // ragged last chunk of the row
              if (m < p.M) store_ragged<32>(p, m, n0, o);
              continue;
            }
            const uint32_t buf = my_stage;
            if (lane == 0) bulk_wait_read<0>();  // the previous store from this buffer has read it
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const uint32_t dst = buf + (uint32_t)lane * 128u + (uint32_t)((j ^ (lane & 7)) << 4);
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(__float_as_uint(o[4 * j])),
                           "r"(__float_as_uint(o[4 * j + 1])), "r"(__float_as_uint(o[4 * j + 2])),
                           "r"(__float_as_uint(o[4 * j + 3]))
                           : "memory");
            }
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
              tma_store_2d(&tmC, buf, (int32_t)n0, (int32_t)m0);
              bulk_commit();
            }
          }
        } else {
#pragma unroll 1
          for (int c0 = half * (BN / 2); c0 < (half + 1) * (BN / 2); c0 += 64) {
            uint32_t v[32], v2[32];
            tc_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + ab * C::ACC_COLS + c0, v);
            tc_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + ab * C::ACC_COLS + c0 + 32, v2);
            tc_wait_ld();
            const int64_t n0 = (int64_t)nt * BN + c0;
            if (n0 >= p.N) break;
            float o[64];
            {
              float sgb[32];
              if (GS == kGsRow) load_sgb32(p.b_gscale, n0, p.N, sgb);
#pragma unroll
              for (int j = 0; j < 32; ++j) o[j] = __uint_as_float(v[j]) * (GS == kGsRow ? __fmul_rn(sa, sgb[j]) : alpha);
              if (GS == kGsRow) load_sgb32(p.b_gscale, n0 + 32, p.N, sgb);
#pragma unroll
              for (int j = 0; j < 32; ++j) o[32 + j] = __uint_as_float(v2[j]) * (GS == kGsRow ? __fmul_rn(sa, sgb[j]) : alpha);
            }
            if (hp_cols) {
              tc_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + hp_tmem_col + c0, v);
              tc_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + hp_tmem_col + c0 + 32, v2);
              tc_wait_ld();
              if (p.k_tiles > 0) {
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                  o[j] += __uint_as_float(v[j]);
                  o[32 + j] += __uint_as_float(v2[j]);
                }
              } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                  o[j] = __uint_as_float(v[j]) * alpha;
                  o[32 + j] = __uint_as_float(v2[j]) * alpha;
                }
              }
            }
            if (p.accumulate && m < p.M) {
              if (n0 + 64 <= p.N) {
                add_existing<64>(p, m, n0, o);
              } else {
#pragma unroll
                for (int j = 0; j < 64; ++j)
                  if (n0 + j < p.N) o[j] += __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p.C)[m * p.ldc + n0 + j]);
              }
            }
            if (n0 + 64 > p.N) {  // ragged last chunk of the row
              if (m < p.M) store_ragged<64>(p, m, n0, o);
              continue;
            }
            const uint32_t buf = my_stage;
            if (lane == 0) bulk_wait_read<0>();
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              uint32_t q[4];
#pragma unroll
              for (int h = 0; h < 4; ++h) {
                const __nv_bfloat162 hh = __floats2bfloat162_rn(o[8 * j + 2 * h], o[8 * j + 2 * h + 1]);
                q[h] = *reinterpret_cast<const uint32_t*>(&hh);
              }
              const uint32_t dst = buf + (uint32_t)lane * 128u + (uint32_t)((j ^ (lane & 7)) << 4);
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(q[0]), "r"(q[1]), "r"(q[2]), "r"(q[3])
                           : "memory");
            }
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
              tma_store_2d(&tmC, buf, (int32_t)n0, (int32_t)m0);
              bulk_commit();
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(acc_empty_bar(ab));
        if (hp_cols) mbar_arrive(hp_empty_bar);
      }
    }
    if (lane == 0) bulk_wait_all();  // this lane's bulk stores are complete before the CTA may exit
  }

  // ===================================== teardown ============================================================
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(C::TMEM_COLS) : "memory");
  }
}

// =========================================================================================================
// BLOCK128 variant: the FP32 global scale changes every 128 k (the paper's 1x128 outer block, Sec. 2.2), so a
// partial product can only be accumulated over 128 k inside tensor memory. The MMA warp writes each 128-k partial
// (two K = 64 instructions) into one of three tensor-memory buffers; the epilogue warps pull it out and promote it
// into FP32 register accumulators with the rank-1 scale SgA[m, kc] * SgB[n, kc] (packed f32x2 FMAs). The SgB values
// of the tile, for all chunks, are staged in shared memory once per tile ([chunk][n] so a warp reads them as
// broadcasts). 128 x 128 tiles, K <= 16384.
// =========================================================================================================
constexpr int B128_STAGES = 4;
constexpr int B128_NBUF = 3;
constexpr int B128_MAX_CHUNKS = 128;
constexpr uint32_t B128_SGB_BYTES = (B128_MAX_CHUNKS + 1) * 128 * 4 + 512;  // + the high-precision partial; 1024-byte multiple
constexpr uint32_t B128_STAGING_BYTES = 4 * 4096;  // one 32-row x 128-byte staging buffer per epilogue warp (bulk stores)
constexpr uint32_t B128_SMEM_BYTES = B128_STAGES * Cfg::STAGE_BYTES + B128_SGB_BYTES + B128_STAGING_BYTES + 1024 + 256;

__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_nvfp4_block128_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                           const __grid_constant__ CUtensorMap tmC, const __grid_constant__ CUtensorMap tmAh,
                           const __grid_constant__ CUtensorMap tmBh, const Params p) {
  using C = Cfg;
  constexpr int BN = 128;
  constexpr int STAGES = B128_STAGES;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  float* sgb = reinterpret_cast<float*>(smem_gen + STAGES * C::STAGE_BYTES);
  const uint32_t staging_base = smem_base + STAGES * C::STAGE_BYTES + B128_SGB_BYTES;  // 1024-byte aligned
  const uint32_t bar_base = staging_base + B128_STAGING_BYTES;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto part_full_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + b); };
  auto part_empty_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + B128_NBUF + b); };
  const uint32_t drain_bar = bar_base + 8u * (2 * STAGES + 2 * B128_NBUF);
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;
  volatile int* abort_flag = &abort_flag_s;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < B128_NBUF; ++b) {
      mbar_init(part_full_bar(b), 1);
      mbar_init(part_empty_bar(b), 4);
    }
    mbar_init(drain_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  pdl_prologue();  // everything above touched only shared and tensor memory
  const int64_t num_tiles = (int64_t)p.m_tiles * p.n_tiles;
  const int32_t chunks = p.k_chunks;  // 128-wide k chunks per tile

  if (warp == 0) {
    const uint32_t leader = elect_leader();
    uint32_t it = 0;
    bool ok = true;
    for (int64_t t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
      const int32_t mt = (int32_t)(t / p.n_tiles), nt = (int32_t)(t % p.n_tiles);
      const uint8_t* sfa_src = p.a_sf + (size_t)mt * p.sf_tiles_a * 512;
      const uint8_t* sfb_src = p.b_sf + (size_t)nt * p.sf_tiles_b * 512;
      for (int32_t kt = 0; kt < p.k_tiles; ++kt, ++it) {
        const int s = it % STAGES;
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(empty_bar(s), ((it / STAGES) & 1) ^ 1, abort_flag, p.dev_status, p.wait_limit));
        if (!ok) break;
        const uint32_t st = smem_base + s * C::STAGE_BYTES;
        mbar_expect_tx(full_bar(s), C::STAGE_BYTES, leader);
        tma_load_2d(st, &tmA, kt * (BK / 2), mt * BM, full_bar(s), leader);
        tma_load_2d(st + A_BYTES, &tmB, kt * (BK / 2), nt * BN, full_bar(s), leader);
        bulk_load(st + A_BYTES + C::B_BYTES, sfa_src + (size_t)kt * 2048, 2048, full_bar(s), leader);
        bulk_load(st + A_BYTES + C::B_BYTES + SFA_BYTES, sfb_src + (size_t)kt * 2048, 2048, full_bar(s), leader);
      }
      // OutControl: the BF16 outlier channels of both operands, 64 per stage, into the same stage buffers
      for (int32_t h = 0; h < p.hp_k_tiles && ok; ++h, ++it) {
        const int s = it % STAGES;
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(empty_bar(s), ((it / STAGES) & 1) ^ 1, abort_flag, p.dev_status, p.wait_limit));
        if (!ok) break;
        const uint32_t st = smem_base + s * C::STAGE_BYTES;
        mbar_expect_tx(full_bar(s), A_BYTES + C::B_BYTES, leader);
        tma_load_2d(st, &tmAh, h * 64, mt * BM, full_bar(s), leader);
        tma_load_2d(st + A_BYTES, &tmBh, h * 64, nt * BN, full_bar(s), leader);
      }
    }
    if (!ok) {
      const uint32_t n_back = it < (uint32_t)STAGES ? it : (uint32_t)STAGES;
      for (uint32_t j = 0; j < n_back; ++j) {
        const uint32_t f = it - 1 - j;
        const long long t0 = clock64();
        while (!mbar_try(full_bar(f % STAGES), (f / STAGES) & 1) && clock64() - t0 < p.wait_limit) {
        }
      }
    }
  } else if (warp == 1) {
    const uint32_t leader = elect_leader();
    const uint32_t idesc = instr_desc<BN>();
    uint32_t it = 0, cit = 0;
    bool ok = true;
    for (int64_t t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
      for (int32_t kt = 0; kt < p.k_tiles && ok; ++kt, ++it) {
        const int s = it % STAGES;
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(full_bar(s), (it / STAGES) & 1, abort_flag, p.dev_status, p.wait_limit));
        if (!ok) break;
        tc_fence_after();
        const uint32_t st = smem_base + s * C::STAGE_BYTES;
        const uint32_t sf_tmem = tmem_base + B128_NBUF * 128 + (it & 3) * C::SF_COLS;
#pragma unroll
        for (int kk = 0; kk < BK / 64; ++kk) {
          tc_cp_sf(sf_tmem + kk * 4, desc_sf(st + A_BYTES + C::B_BYTES + kk * 512), leader);
          tc_cp_sf(sf_tmem + 16 + kk * 4, desc_sf(st + A_BYTES + C::B_BYTES + SFA_BYTES + kk * 512), leader);
        }
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          if (kt * 2 + half >= chunks) break;  // the padded half of the last k tile holds only zeros
          const uint32_t buf = cit % B128_NBUF;
          ok = __all_sync(0xFFFFFFFFu, mbar_wait(part_empty_bar(buf), ((cit / B128_NBUF) & 1) ^ 1, abort_flag, p.dev_status, p.wait_limit));
          if (!ok) break;
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + buf * 128;
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            const int kk = 2 * half + q;
            tc_mma_nvf4(d_tmem, desc_sw128(st + kk * 32), desc_sw128(st + A_BYTES + kk * 32), idesc, sf_tmem + kk * 4,
                        sf_tmem + 16 + kk * 4, q, leader);
          }
          tc_commit(part_full_bar(buf), leader);
          ++cit;
        }
        tc_commit(empty_bar(s), leader);
      }
      if (p.hp_k_tiles > 0 && ok) {
        // high-precision side product: one more partial, handed to the promotion warps like a 128-k chunk (scale 1)
        const uint32_t buf = cit % B128_NBUF;
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(part_empty_bar(buf), ((cit / B128_NBUF) & 1) ^ 1, abort_flag, p.dev_status, p.wait_limit));
        if (!ok) break;
        tc_fence_after();
        const uint32_t idesc_bf16 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
        for (int32_t h = 0; h < p.hp_k_tiles; ++h, ++it) {
          const int s = it % STAGES;
          ok = __all_sync(0xFFFFFFFFu, mbar_wait(full_bar(s), (it / STAGES) & 1, abort_flag, p.dev_status, p.wait_limit));
          if (!ok) break;
          tc_fence_after();
          const uint32_t st = smem_base + s * C::STAGE_BYTES;
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)  // 64 BF16 = one 128-byte swizzle row = four K = 16 steps of 32 bytes
            tc_mma_bf16(tmem_base + buf * 128, desc_sw128(st + kk * 32), desc_sw128(st + A_BYTES + kk * 32), idesc_bf16,
                        (h | kk) != 0, leader);
          tc_commit(empty_bar(s), leader);
        }
        if (!ok) break;
        tc_commit(part_full_bar(buf), leader);
        ++cit;
      }
    }
    tc_commit(drain_bar, leader);
    {
      const long long t0 = clock64();
      while (!mbar_try(drain_bar, 0) && clock64() - t0 < p.wait_limit) {
      }
    }
  } else {
    // ---- promotion + epilogue: thread = one output row, 128 FP32 accumulators in registers -----------------
    const int quad = warp & 3;
    const int epi_tid = (warp - 2) * 32 + lane;  // 0..127
    const int64_t G = p.g_per_row;               // global scales per operand row (= padded K / 128)
    uint32_t cit = 0;
    bool ok = true;
    for (int64_t t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
      const int32_t mt = (int32_t)(t / p.n_tiles), nt = (int32_t)(t % p.n_tiles);
      // stage SgB[n, :] of this tile as sgb[chunk][n]
      asm volatile("bar.sync 1, 128;" ::: "memory");  // everyone is done with the previous tile's values
      {
        const int64_t n = (int64_t)nt * BN + epi_tid;
        const float* src = p.b_gscale + n * G;
        if (n < p.N) {
          int32_t kc = 0;
          if ((G & 3) == 0) {  // a row's scales as 16-byte loads, sixteen values in flight per thread
#pragma unroll 4
            for (; kc + 4 <= chunks; kc += 4) {
              const float4 q = __ldg(reinterpret_cast<const float4*>(src + kc));
              sgb[kc * 128 + epi_tid] = q.x;
              sgb[(kc + 1) * 128 + epi_tid] = q.y;
              sgb[(kc + 2) * 128 + epi_tid] = q.z;
              sgb[(kc + 3) * 128 + epi_tid] = q.w;
            }
          }
          for (; kc < chunks; ++kc) sgb[kc * 128 + epi_tid] = __ldg(src + kc);
        } else {
          for (int32_t kc = 0; kc < chunks; ++kc) sgb[kc * 128 + epi_tid] = 0.0f;
        }
        if (p.hp_k_tiles > 0) sgb[chunks * 128 + epi_tid] = 1.0f;  // the high-precision partial carries no scale
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      const int64_t m = (int64_t)mt * BM + quad * 32 + lane;
      const float* sa_row = p.a_gscale + (m < p.M ? m : 0) * G;
      float2 acc[64];
#pragma unroll
      for (int j = 0; j < 64; ++j) acc[j] = make_float2(0.0f, 0.0f);
      const int32_t parts = chunks + (p.hp_k_tiles > 0 ? 1 : 0);
      // SgA[m, kc] is fetched two chunks ahead: with one promotion warp per scheduler nothing else would hide the load
      float sa_0 = chunks > 0 ? __ldg(sa_row) : 1.0f, sa_1 = chunks > 1 ? __ldg(sa_row + 1) : 1.0f;
      for (int32_t kc = 0; kc < parts && ok; ++kc, ++cit) {
        const float sa = kc < chunks ? sa_0 : 1.0f;
        sa_0 = sa_1;
        if (kc + 2 < chunks) sa_1 = __ldg(sa_row + kc + 2);
        const uint32_t buf = cit % B128_NBUF;
        if (!(ok = mbar_wait(part_full_bar(buf), (cit / B128_NBUF) & 1, abort_flag, p.dev_status, p.wait_limit))) break;
        tc_fence_after();
        const float2 sa2 = make_float2(sa, sa);
        const float4* sb4 = reinterpret_cast<const float4*>(sgb + kc * 128);
#pragma unroll
        for (int c0 = 0; c0 < 128; c0 += 32) {
          uint32_t v[32];
          tc_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + buf * 128 + c0, v);
          tc_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            const float4 sb = sb4[(c0 + j) >> 2];
            const float2 t0 = __fmul2_rn(make_float2(__uint_as_float(v[j]), __uint_as_float(v[j + 1])), sa2);
            const float2 t1 = __fmul2_rn(make_float2(__uint_as_float(v[j + 2]), __uint_as_float(v[j + 3])), sa2);
            acc[(c0 + j) >> 1] = __ffma2_rn(t0, make_float2(sb.x, sb.y), acc[(c0 + j) >> 1]);
            acc[((c0 + j) >> 1) + 1] = __ffma2_rn(t1, make_float2(sb.z, sb.w), acc[((c0 + j) >> 1) + 1]);
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(part_empty_bar(buf));
      }
      if (ok && p.use_tma_store && !p.accumulate) {
        // 128-byte row pieces staged in shared memory with the 128-byte swizzle and written by the bulk-tensor engine:
        // full lines, clipped at the edges of C (a thread-per-row store from registers took longer than the whole
        // promotion loop of a K = 1024 tile)
        const uint32_t buf = staging_base + (uint32_t)(warp - 2) * 4096u;
        const int64_t m0 = (int64_t)mt * BM + quad * 32;
        // (both loops are fully unrolled: the accumulators must be addressed with compile-time indices)
        if (p.c_is_f32) {
#pragma unroll
          for (int c0 = 0; c0 < 128; c0 += 32) {
            const int64_t n0 = (int64_t)nt * BN + c0;
            if (n0 < p.N && n0 + 32 > p.N) {  // ragged last chunk of the row
              if (m < p.M) {
                float o[32];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                  o[2 * j] = acc[(c0 >> 1) + j].x;
                  o[2 * j + 1] = acc[(c0 >> 1) + j].y;
                }
                store_ragged<32>(p, m, n0, o);
              }
            } else if (n0 < p.N) {
              if (lane == 0) bulk_wait_read<0>();  // the previous store from this buffer has read it
              __syncwarp();
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                const float2 a0 = acc[(c0 >> 1) + 2 * j], a1 = acc[(c0 >> 1) + 2 * j + 1];
                const uint32_t dst = buf + (uint32_t)lane * 128u + (uint32_t)((j ^ (lane & 7)) << 4);
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(__float_as_uint(a0.x)),
                             "r"(__float_as_uint(a0.y)), "r"(__float_as_uint(a1.x)), "r"(__float_as_uint(a1.y))
                             : "memory");
              }
              fence_async_smem();
              __syncwarp();
              if (lane == 0) {
                tma_store_2d(&tmC, buf, (int32_t)n0, (int32_t)m0);
                bulk_commit();
              }
            }
          }
        } else {
#pragma unroll
          for (int c0 = 0; c0 < 128; c0 += 64) {
            const int64_t n0 = (int64_t)nt * BN + c0;
            if (n0 < p.N && n0 + 64 > p.N) {  // ragged last chunk of the row
              if (m < p.M) {
                float o[64];
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                  o[2 * j] = acc[(c0 >> 1) + j].x;
                  o[2 * j + 1] = acc[(c0 >> 1) + j].y;
                }
                store_ragged<64>(p, m, n0, o);
              }
            } else if (n0 < p.N) {
              if (lane == 0) bulk_wait_read<0>();
              __syncwarp();
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                uint32_t q[4];
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                  const float2 a = acc[(c0 >> 1) + 4 * j + h];
                  const __nv_bfloat162 hh = __floats2bfloat162_rn(a.x, a.y);
                  q[h] = *reinterpret_cast<const uint32_t*>(&hh);
                }
                const uint32_t dst = buf + (uint32_t)lane * 128u + (uint32_t)((j ^ (lane & 7)) << 4);
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(q[0]), "r"(q[1]), "r"(q[2]), "r"(q[3])
                             : "memory");
              }
              fence_async_smem();
              __syncwarp();
              if (lane == 0) {
                tma_store_2d(&tmC, buf, (int32_t)n0, (int32_t)m0);
                bulk_commit();
              }
            }
          }
        }
      } else if (ok && m < p.M) {
#pragma unroll
        for (int c0 = 0; c0 < 128; c0 += 32) {
          const int64_t n0 = (int64_t)nt * BN + c0;
          if (n0 < p.N) {
            float o[32];
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              o[2 * j] = acc[(c0 >> 1) + j].x;
              o[2 * j + 1] = acc[(c0 >> 1) + j].y;
            }
            store_row_chunk(p, m, n0, o);
          }
        }
      }
    }
    if (lane == 0) bulk_wait_all();  // this lane's bulk stores are complete before the CTA may exit
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// =========================================================================================================
// Two-CTA variant (cta_group::2) for large products: a pair of CTAs on neighbouring SMs computes one 256 x 256 tile.
// Each CTA loads its own 128 rows of A, HALF of the B tile (128 of the 256 rows) and the scales it needs; the pair's
// tensor cores read both halves of B, so every SM pulls 38 KB per k tile instead of 54 KB (128 x 256 single-CTA
// tiles) and five stages fit. The MMAs are issued by the leader CTA (cluster rank 0) only:
//   - both CTAs' bulk-tensor loads complete on the LEADER's "full" barrier (armed for the bytes of both);
//   - tcgen05.commit multicasts the "stage free" / "accumulator ready" arrivals to the same barrier in both CTAs;
//   - both CTAs' epilogue warps arrive on the leader's "accumulator free" barrier (a remote arrive for the peer).
// No load uses cluster multicast. Accumulator: 128 lanes x 256 columns per CTA, drained into registers by eight
// epilogue warps, which hand it back at once and then scale, stage 128-byte row pieces in shared memory (one 4 KB buffer
// per warp, 128-byte swizzle) and let the bulk-tensor engine write them as full lines while the next tile's MMAs run
// (plain 16-byte stores from the registers, a lane per row, cost 16384 x 3072 x 1024 with FP32 output 112 instead of 56 us).
// =========================================================================================================
// Two tile widths. PN = 256: one accumulator of 256 columns per CTA and four sets of scale columns. PN = 192: two
// accumulators of 192 columns (a tile's epilogue runs entirely under the next tile's MMAs) and two sets of scale columns;
// each CTA loads 96 rows of B. A 192-wide tile starts at a multiple of 64 B rows, i.e. possibly in the middle of a 128-row
// scale tile: the two scale tiles it touches are copied whole and the MMA's scale address starts two columns later (one
// tensor-memory column holds the scales of 32 rows).
template <int PN>
struct Cfg2 {
  static constexpr int STAGES = 5;
  static constexpr uint32_t B_ROWS = PN / 2;                                   // this CTA's rows of the B tile
  static constexpr uint32_t B_BYTES = B_ROWS * 128;
  static constexpr uint32_t SFB_BYTES = 4096;                                  // scales of the two 128-row scale tiles touched
  static constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES + SFA_BYTES + SFB_BYTES;  // 38 KB / 34 KB
  // staging buffers of 4 KB: one per epilogue warp; with 192-wide tiles (room for it) the four warps that own 128 columns
  // alternate between two, so that a chunk does not wait for the previous chunk's bulk store to have read the buffer
  static constexpr uint32_t STAGING_BYTES = (PN == 256 ? 8 : 12) * 4096;
  static constexpr uint32_t SMEM_BYTES = STAGES * STAGE_BYTES + STAGING_BYTES + 1024 + 256;
  static constexpr int ACC_BUFS = PN == 256 ? 1 : 2;
  static constexpr uint32_t SF_COLS = 16 + 32;
  static constexpr uint32_t SF_SETS = PN == 256 ? 4 : 2;
  static constexpr uint32_t SF_TMEM_COL = ACC_BUFS * PN;                       // 256 / 384; + SF_SETS * 48 <= 512
};
constexpr int C2_THREADS = 64 + 256;

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address of the same shared-memory location in the CTA with the given cluster rank.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Arrive on a barrier of a CTA of the cluster (possibly this one). Relaxed: what it announces -- this warp's tensor-memory
// loads of the accumulator are complete -- is ordered by tcgen05.wait::ld and the tcgen05 fence before it; with release
// semantics at cluster scope the arrive took about 2500 cycles (it waits for the thread's earlier shared-memory and bulk
// traffic), and that, not the loads, was the cost of handing the accumulator over.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Bulk-tensor load of one CTA of a pair; completes on an mbarrier that may live in the peer CTA.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* tm, int32_t c0, int32_t c1,
                                                 uint32_t bar_cluster_addr, uint32_t leader) {
  asm volatile(
      "{\n.reg .pred q;\nsetp.ne.b32 q, %5, 0;\n"
      "@q cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n}" ::"r"(dst),
      "l"(tm), "r"(c0), "r"(c1), "r"(bar_cluster_addr), "r"(leader)
      : "memory");
}
__device__ __forceinline__ void tc2_commit_both(uint32_t bar, uint32_t leader) {
  asm volatile(
      "{\n.reg .pred q;\n.reg .b16 m;\nsetp.ne.b32 q, %1, 0;\nmov.b16 m, 3;\n"
      "@q tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], m;\n}" ::"r"(bar),
      "r"(leader)
      : "memory");
}
__device__ __forceinline__ void tc2_cp_sf(uint32_t taddr, uint64_t sdesc, uint32_t leader) {
  asm volatile("{\n.reg .pred q;\nsetp.ne.b32 q, %2, 0;\n@q tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;\n}" ::"r"(taddr),
               "l"(sdesc), "r"(leader)
               : "memory");
}
__device__ __forceinline__ void tc2_mma_nvf4(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                             uint32_t sfa_tmem, uint32_t sfb_tmem, uint32_t accumulate, uint32_t leader) {
  asm volatile(
      "{\n.reg .pred p, q;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "setp.ne.b32 q, %7, 0;\n"
      "@q tcgen05.mma.cta_group::2.kind::mxf4nvf4.block_scale.scale_vec::4X [%0], %1, %2, %3, [%5], [%6], p;\n}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem), "r"(leader)
      : "memory");
}

// One 128-byte-wide piece (W = 32 FP32 or 64 BF16 columns) of a warp's 32 output rows, values final except for the old C:
// accumulate, then either plain stores (a chunk that sticks out past N) or a swizzled copy into the warp's 4 KB staging
// buffer that the bulk-tensor engine writes as full lines. m0 is the first of the 32 rows, m this lane's row.
// pending: how many of this lane's earlier bulk stores may still be reading shared memory when `buf` is written again (0 with
// one staging buffer per warp, 1 when the warp alternates between two).
template <int W>
__device__ __forceinline__ void stage_and_store(const Params& p, const CUtensorMap* tmC, uint32_t buf, int lane, int64_t m, int64_t m0,
                                                int64_t n0, float (&o)[W], int pending = 0) {
  if (p.accumulate && m < p.M) {
    if (n0 + W <= p.N) {
      add_existing<W>(p, m, n0, o);
    } else if (p.c_is_f32) {
#pragma unroll
      for (int j = 0; j < W; ++j)
        if (n0 + j < p.N) o[j] += reinterpret_cast<const float*>(p.C)[m * p.ldc + n0 + j];
    } else {
#pragma unroll
      for (int j = 0; j < W; ++j)
        if (n0 + j < p.N) o[j] += __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p.C)[m * p.ldc + n0 + j]);
    }
  }
  if (n0 + W > p.N) {  // ragged last chunk of the row
    if (m < p.M) store_ragged<W>(p, m, n0, o);
    return;
  }
  if (lane == 0) {  // the previous store from this buffer has read it
    if (pending)
      bulk_wait_read<1>();
    else
      bulk_wait_read<0>();
  }
  __syncwarp();
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    uint32_t q[4];
    if (W == 32) {
#pragma unroll
      for (int h = 0; h < 4; ++h) q[h] = __float_as_uint(o[4 * j + h]);
    } else {
#pragma unroll
      for (int h = 0; h < 4; ++h) {
        const __nv_bfloat162 hh = __floats2bfloat162_rn(o[(8 * j + 2 * h) % W], o[(8 * j + 2 * h + 1) % W]);
        q[h] = *reinterpret_cast<const uint32_t*>(&hh);
      }
    }
    const uint32_t dst = buf + (uint32_t)lane * 128u + (uint32_t)((j ^ (lane & 7)) << 4);
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(q[0]), "r"(q[1]), "r"(q[2]), "r"(q[3]) : "memory");
  }
  fence_async_smem();
  __syncwarp();
  if (lane == 0) {
    tma_store_2d(tmC, buf, (int32_t)n0, (int32_t)m0);
    bulk_commit();
  }
}

template <int GS, int PN>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(C2_THREADS, 1)
gemm_nvfp4_2cta_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                       const __grid_constant__ CUtensorMap tmSFA, const __grid_constant__ CUtensorMap tmSFB,
                       const __grid_constant__ CUtensorMap tmC, const Params p) {
  using C2 = Cfg2<PN>;
  constexpr int STAGES = C2::STAGES;
  constexpr uint32_t C2_STAGE_BYTES = C2::STAGE_BYTES, C2_B_BYTES = C2::B_BYTES, C2_SF_COLS = C2::SF_COLS;
  constexpr int ACC_BUFS = C2::ACC_BUFS;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t staging_base = smem_base + STAGES * C2_STAGE_BYTES;  // eight 4 KB buffers, one per epilogue warp
  const uint32_t bar_base = staging_base + C2::STAGING_BYTES;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };             // used in the leader CTA only
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };  // one per CTA
  auto acc_full_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + b); };       // one pair per CTA
  auto acc_empty_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + 2 + b); };  // leader CTA only (16 arrivals)
  const uint32_t drain_bar = bar_base + 8u * (2 * STAGES + 4);
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;
  volatile int* abort_flag = &abort_flag_s;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();

  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(acc_full_bar(b), 1);
      mbar_init(acc_empty_bar(b), 16);
    }
    mbar_init(drain_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // the peer's barriers are initialised and its tensor memory allocated
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  pdl_prologue();

  const int64_t num_tiles = (int64_t)p.m_tiles * p.n_tiles;  // 256 x PN tiles
  const int64_t pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;

  if (warp == 0) {
    // ===================================== TMA producer (both CTAs) ========================================
    const uint32_t leader = elect_leader();
    uint32_t it = 0, s = 0, wait_parity = 1;
    bool ok = true;
    for (int64_t t = pair; t < num_tiles && ok; t += num_pairs) {
      const int32_t mt = (int32_t)(t / p.n_tiles), nt = (int32_t)(t % p.n_tiles);
      const int32_t a_row = mt * 256 + (int32_t)rank * 128, b_row = nt * PN + (int32_t)rank * (PN / 2);
      const int32_t sfa_row = ((mt * 2 + (int32_t)rank) * p.sf_tiles_a) * 4;  // in units of 128 bytes
      const int32_t sfb_tile0 = (nt * PN) >> 7;  // first 128-row scale tile the B tile touches (it touches this one and the next)
      const int32_t sfb_row0 = (sfb_tile0 * p.sf_tiles_b) * 4, sfb_row1 = ((sfb_tile0 + 1) * p.sf_tiles_b) * 4;
      for (int32_t kt = 0; kt < p.k_tiles; ++kt, ++it, s = (s + 1 == (uint32_t)STAGES ? 0u : s + 1), wait_parity ^= (s == 0)) {
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(empty_bar(s), wait_parity, abort_flag, p.dev_status, p.wait_limit));
        if (!ok) break;
        const uint32_t st = smem_base + s * C2_STAGE_BYTES;
        const uint32_t full0 = map_to_cta(full_bar(s), 0);
        if (rank == 0) mbar_expect_tx(full_bar(s), 2 * C2_STAGE_BYTES + ((p.starve && it == 0) ? 16u : 0u), leader);
        tma_load_2d_pair(st, &tmA, kt * (BK / 2), a_row, full0, leader);
        tma_load_2d_pair(st + A_BYTES, &tmB, kt * (BK / 2), b_row, full0, leader);
        tma_load_2d_pair(st + A_BYTES + C2_B_BYTES, &tmSFA, 0, sfa_row + kt * 16, full0, leader);
        tma_load_2d_pair(st + A_BYTES + C2_B_BYTES + SFA_BYTES, &tmSFB, 0, sfb_row0 + kt * 16, full0, leader);
        tma_load_2d_pair(st + A_BYTES + C2_B_BYTES + SFA_BYTES + 2048, &tmSFB, 0, sfb_row1 + kt * 16, full0, leader);
      }
    }
    if (!ok) {
      // a wait ran out: this CTA's copies in flight complete on the leader's barrier, which the peer cannot poll, so give
      // them a fixed time (far more than a copy takes) to land before the CTA may exit
      const long long t0 = clock64();
      while (clock64() - t0 < 400000) {
      }
    }
  } else if (warp == 1) {
    // ===================================== MMA issuer (leader CTA only) ====================================
    if (rank == 0) {
      const uint32_t leader = elect_leader();
      const uint32_t idesc = (1u << 7) | (1u << 10) | ((uint32_t)(PN >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
      // issue loop kept short as in the 128 x 128 kernel: running stage / phase counters, descriptors by addition to the low
      // word, the next stage's barrier tried before this stage's instructions
      uint32_t it = 0, tile_it = 0, stage = 0, phase = 0;
      bool ok = true;
      bool ready = false;
      constexpr uint32_t SW_HI = (uint32_t)((((uint64_t)64 << 32) | ((uint64_t)1 << 46) | ((uint64_t)2 << 61)) >> 32);
      constexpr uint32_t SF_HI = (uint32_t)((((uint64_t)8 << 32) | ((uint64_t)1 << 46)) >> 32);
      const uint32_t a_lo0 = (uint32_t)desc_sw128(smem_base), sfa_lo0 = (uint32_t)desc_sf(smem_base + A_BYTES + C2_B_BYTES);
      for (int64_t t = pair; t < num_tiles && ok; t += num_pairs, ++tile_it) {
        const uint32_t ab = tile_it % ACC_BUFS;
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(acc_empty_bar(ab), ((tile_it / ACC_BUFS) & 1) ^ 1, abort_flag, p.dev_status, p.wait_limit));
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + ab * PN;
        // scales of the B rows: the tile may start 64 rows into its first scale tile, i.e. two columns later
        const uint32_t sfb_col = (uint32_t)((((int32_t)(t % p.n_tiles) * PN) & 127) >> 5);
        for (int32_t kt = 0; kt < p.k_tiles; ++kt, ++it) {
          if (!ready) {
            ok = __all_sync(0xFFFFFFFFu, mbar_wait(full_bar(stage), phase, abort_flag, p.dev_status, p.wait_limit));
            if (!ok) break;
          }
          tc_fence_after();
          const uint32_t st16 = stage * (uint32_t)(C2_STAGE_BYTES >> 4);
          const uint32_t this_empty = empty_bar(stage);
          if (++stage == (uint32_t)STAGES) {
            stage = 0;
            phase ^= 1u;
          }
          const uint32_t next_try = mbar_test(full_bar(stage), phase);
          const uint32_t sf_tmem = tmem_base + C2::SF_TMEM_COL + (it % C2::SF_SETS) * C2_SF_COLS;
#pragma unroll
          for (int kk = 0; kk < BK / 64; ++kk) {
            tc2_cp_sf(sf_tmem + kk * 4, ((uint64_t)SF_HI << 32) | (sfa_lo0 + st16 + kk * 32), leader);
            tc2_cp_sf(sf_tmem + 16 + kk * 8, ((uint64_t)SF_HI << 32) | (sfa_lo0 + st16 + (SFA_BYTES >> 4) + kk * 32), leader);
            tc2_cp_sf(sf_tmem + 16 + kk * 8 + 4, ((uint64_t)SF_HI << 32) | (sfa_lo0 + st16 + ((SFA_BYTES + 2048) >> 4) + kk * 32), leader);
          }
#pragma unroll
          for (int kk = 0; kk < BK / 64; ++kk)
            tc2_mma_nvf4(d_tmem, ((uint64_t)SW_HI << 32) | (a_lo0 + st16 + kk * 2), ((uint64_t)SW_HI << 32) | (a_lo0 + st16 + (A_BYTES >> 4) + kk * 2),
                         idesc, sf_tmem + kk * 4, sf_tmem + 16 + kk * 8 + sfb_col, (kt | kk) != 0, leader);
          tc2_commit_both(this_empty, leader);
          ready = __all_sync(0xFFFFFFFFu, next_try);
        }
        if (ok) tc2_commit_both(acc_full_bar(ab), leader);
      }
      // nothing issued may still be running when tensor memory is freed; the commit covers both CTAs' work
      asm volatile(
          "{\n.reg .pred q;\nsetp.ne.b32 q, %1, 0;\n"
          "@q tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];\n}" ::"r"(drain_bar),
          "r"(leader)
          : "memory");
      {
        const long long t0 = clock64();
        while (!mbar_try(drain_bar, 0) && clock64() - t0 < p.wait_limit) {
        }
      }
    }
  } else {
    // ===================================== epilogue (both CTAs, eight warps) ================================
    const int quad = warp & 3;
    const int half = (warp - 2) >> 2;
    // columns of the tile this warp owns: [half * 128, half * 128 + 32 * nq): the first four warps 128, the others the rest
    const int nq = half == 0 ? 4 : (PN - 128) / 32;
    uint32_t tile_it = 0;
    bool ok = true;
    float alpha = 1.0f;
    if (GS == kGsTensor) alpha = __fmul_rn(p.a_gscale[0], p.b_gscale[0]);
    for (int64_t t = pair; t < num_tiles && ok; t += num_pairs, ++tile_it) {
      const int32_t mt = (int32_t)(t / p.n_tiles), nt = (int32_t)(t % p.n_tiles);
      const uint32_t ab = tile_it % ACC_BUFS;
      const uint32_t acc_empty_leader = map_to_cta(acc_empty_bar(ab), 0);
      if (!(ok = mbar_wait(acc_full_bar(ab), (tile_it / ACC_BUFS) & 1, abort_flag, p.dev_status, p.wait_limit))) break;
      tc_fence_after();
      const int64_t m = (int64_t)mt * 256 + rank * 128 + quad * 32 + lane;
      float sa = 1.0f;
      if (GS == kGsRow && m < p.M) sa = p.a_gscale[m];
      uint32_t v[4][32];
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (q < nq) tc_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + ab * PN + half * 128 + q * 32, v[q]);
      tc_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(acc_empty_leader);
      // The accumulator is free again (the pair's next tile may start); scale, stage and store from the registers.
      const bool two_bufs = PN == 192 && half == 0;
      const uint32_t my_stage = staging_base + (PN == 256 ? (uint32_t)(warp - 2) : (half == 0 ? 2u * (uint32_t)(warp - 2) : 4u + (uint32_t)(warp - 2))) * 4096u;
      const int64_t m0 = (int64_t)mt * 256 + rank * 128 + quad * 32;
      if (m0 >= p.M) continue;
      if (p.c_is_f32) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int64_t n0 = (int64_t)nt * PN + half * 128 + q * 32;
          if (q >= nq || n0 >= p.N) break;
          float o[32], sgb[32];
          if (GS == kGsRow) load_sgb32(p.b_gscale, n0, p.N, sgb);
#pragma unroll
          for (int j = 0; j < 32; ++j) o[j] = __uint_as_float(v[q][j]) * (GS == kGsRow ? __fmul_rn(sa, sgb[j]) : alpha);
          stage_and_store<32>(p, &tmC, my_stage + (two_bufs ? (uint32_t)(q & 1) * 4096u : 0u), lane, m, m0, n0, o, two_bufs ? 1 : 0);
        }
      } else {
#pragma unroll
        for (int qq = 0; qq < 2; ++qq) {
          const int64_t n0 = (int64_t)nt * PN + half * 128 + qq * 64;
          if (2 * qq >= nq || n0 >= p.N) break;
          float o[64], sgb[32];
          if (GS == kGsRow) load_sgb32(p.b_gscale, n0, p.N, sgb);
#pragma unroll
          for (int j = 0; j < 32; ++j) o[j] = __uint_as_float(v[2 * qq][j]) * (GS == kGsRow ? __fmul_rn(sa, sgb[j]) : alpha);
          if (GS == kGsRow) load_sgb32(p.b_gscale, n0 + 32, p.N, sgb);
#pragma unroll
          for (int j = 0; j < 32; ++j) o[32 + j] = __uint_as_float(v[2 * qq + 1][j]) * (GS == kGsRow ? __fmul_rn(sa, sgb[j]) : alpha);
          stage_and_store<64>(p, &tmC, my_stage + (two_bufs ? (uint32_t)(qq & 1) * 4096u : 0u), lane, m, m0, n0, o, two_bufs ? 1 : 0);
        }
      }
    }
    if (lane == 0) bulk_wait_all();  // this lane's bulk stores are complete before the CTA may exit
  }

  // ===================================== teardown ============================================================
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // the peer may still be reading this CTA's shared memory through the pair's MMAs until here
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// =========================================================================================================
// OutControl's high-precision weight-gradient columns (paper Sec. 4.2):  dW[:, A] = dY^T X[:, A], BF16 inputs, FP32
// accumulation, on the tensor cores (tcgen05 kind::f16).  G[c, j] = sum_t dY[t, c] * X_out[t, j]  with
// M = C, N = Kh (a slab of at most 256 columns of the compact outlier matrix), K = tokens. Both operands are stored with the
// contraction index t as the SLOW index, i.e. "MN-major": a bulk-tensor box of 64 columns x 64 tokens lands in
// shared memory as 64 rows of 128 bytes (8 swizzle atoms of 8 tokens), which is the MN-major 128-byte-swizzle
// operand layout (leading byte offset = distance between 64-column boxes, stride byte offset = 1024).
// Only C / 128 output tiles exist, so the token range is split over blockIdx.y; FP32 partial tiles go to a workspace
// that dw_assemble_kernel sums in a fixed order. One tile per CTA: no accumulator double buffering needed.
// =========================================================================================================
constexpr int HPDW_STAGES = 4;
constexpr int HPDW_THREADS = 192;

__global__ void __launch_bounds__(HPDW_THREADS, 1)
hp_dw_mma_kernel(const __grid_constant__ CUtensorMap tmDY, const __grid_constant__ CUtensorMap tmXO, float* __restrict__ partial,
                 int64_t C, int32_t Kh, int64_t ld_partial, int64_t T, int32_t t_per_split, int32_t* dev_status, long long wait_limit) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t b_bytes = (uint32_t)(Kh / 64) * 8192u;
  const uint32_t stage_bytes = A_BYTES + b_bytes;  // A: two boxes of 64 channels x 64 tokens; B: Kh / 64 boxes
  const uint32_t bar_base = smem_base + HPDW_STAGES * stage_bytes;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (HPDW_STAGES + s); };
  const uint32_t acc_full_bar = bar_base + 8u * (2 * HPDW_STAGES);
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;
  volatile int* abort_flag = &abort_flag_s;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t tmem_cols = Kh <= 64 ? 64u : (Kh <= 128 ? 128u : 256u);

  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    for (int s = 0; s < HPDW_STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    mbar_init(acc_full_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  pdl_prologue();

  const int32_t c0 = (int32_t)blockIdx.x * 128;
  const int64_t t_begin = (int64_t)blockIdx.y * t_per_split;
  const int64_t t_end = min(T, t_begin + t_per_split);
  const int32_t k_tiles = (int32_t)((t_end - t_begin + 63) / 64);  // tokens beyond T read as zero

  if (warp == 0) {
    const uint32_t leader = elect_leader();
    for (int32_t kt = 0; kt < k_tiles; ++kt) {
      const int s = kt % HPDW_STAGES;
      if (!__all_sync(0xFFFFFFFFu, mbar_wait(empty_bar(s), ((kt / HPDW_STAGES) & 1) ^ 1, abort_flag, dev_status, wait_limit))) break;
      const uint32_t st = smem_base + s * stage_bytes;
      const int32_t t0 = (int32_t)(t_begin + (int64_t)kt * 64);
      mbar_expect_tx(full_bar(s), stage_bytes, leader);
      tma_load_2d(st, &tmDY, c0, t0, full_bar(s), leader);
      tma_load_2d(st + 8192, &tmDY, c0 + 64, t0, full_bar(s), leader);
      for (int32_t h = 0; h < Kh / 64; ++h) tma_load_2d(st + A_BYTES + h * 8192, &tmXO, h * 64, t0, full_bar(s), leader);
    }
  } else if (warp == 1) {
    const uint32_t leader = elect_leader();
    // BF16 x BF16 -> FP32, M = 128, N = Kh, both operands MN-major
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((uint32_t)(Kh >> 3) << 17) |
                           ((uint32_t)(128 >> 4) << 24);
    bool ok = true;
    for (int32_t kt = 0; kt < k_tiles && ok; ++kt) {
      const int s = kt % HPDW_STAGES;
      ok = __all_sync(0xFFFFFFFFu, mbar_wait(full_bar(s), (kt / HPDW_STAGES) & 1, abort_flag, dev_status, wait_limit));
      if (!ok) break;
      tc_fence_after();
      const uint32_t st = smem_base + s * stage_bytes;
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {  // 16 tokens = two 8-token swizzle atoms = 2048 bytes per step
        const uint64_t adesc = (uint64_t)(((st + kk * 2048) >> 4) & 0x3FFFu) | ((uint64_t)(8192 >> 4) << 16) |
                               ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
        const uint64_t bdesc = (uint64_t)(((st + A_BYTES + kk * 2048) >> 4) & 0x3FFFu) | ((uint64_t)(8192 >> 4) << 16) |
                               ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
        tc_mma_bf16(tmem_base, adesc, bdesc, idesc, (kt | kk) != 0, leader);
      }
      tc_commit(empty_bar(s), leader);
    }
    tc_commit(acc_full_bar, leader);  // also covers the k_tiles == 0 case (arrives at once)
  } else {
    const int quad = warp & 3;
    if (mbar_wait(acc_full_bar, 0, abort_flag, dev_status, wait_limit)) {
      tc_fence_after();
      const int64_t c = (int64_t)c0 + quad * 32 + lane;
      float* dst = partial + ((int64_t)blockIdx.y * C + (c < C ? c : 0)) * ld_partial;
      for (int j0 = 0; j0 < Kh; j0 += 32) {
        uint32_t v[32];
        tc_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + j0, v);
        tc_wait_ld();
        if (c < C) {
#pragma unroll
          for (int j = 0; j < 32; j += 4)
            *reinterpret_cast<float4*>(dst + j0 + j) = k_tiles > 0 ? make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]),
                                                                                 __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]))
                                                                   : make_float4(0.f, 0.f, 0.f, 0.f);
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// Codes of an operand [R, Kp/2 bytes] as a 2-D byte tensor; box = 128 bytes x box_rows; out-of-range reads give 0.
bool make_codes_map(CUtensorMap* tm, const uint8_t* codes, int64_t R, int64_t Kp, uint32_t box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)(Kp / 2), (cuuint64_t)R};
  const cuuint64_t strides[1] = {(cuuint64_t)(Kp / 2)};
  const cuuint32_t box[2] = {128, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(codes), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// C [M, N] (BF16 or FP32, leading dimension ldc) as a 2-D tensor; box = 128 bytes of a row x 32 rows, 128-byte swizzle.
bool make_c_map(CUtensorMap* tm, void* Cp, int64_t M, int64_t N, int64_t ldc, bool is_f32) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  const cuuint64_t esz = is_f32 ? 4 : 2;
  const cuuint64_t dims[2] = {(cuuint64_t)N, (cuuint64_t)M};
  const cuuint64_t strides[1] = {(cuuint64_t)ldc * esz};
  const cuuint32_t box[2] = {(cuuint32_t)(128 / esz), 32};
  const cuuint32_t estr[2] = {1, 1};
  return fn(tm, is_f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Cp, dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// A compact BF16 side matrix [R, Kh] (Kh a multiple of 64) as a 2-D tensor; box = 64 columns (128 bytes) x 128 rows.
bool make_hp_map(CUtensorMap* tm, const void* base, int64_t R, int64_t Kh) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)Kh, (cuuint64_t)R};
  const cuuint64_t strides[1] = {(cuuint64_t)Kh * 2};
  const cuuint32_t box[2] = {64, 128};
  const cuuint32_t estr[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline int sm_count() { return device_sm_count(); }
inline long long wait_limit_of(const GemmArgs& a) { return a.wait_limit > 0 ? a.wait_limit : DEFAULT_WAIT_LIMIT_CYCLES; }

template <int GS>
cudaError_t launch_tile128(const GemmArgs& a, cudaStream_t st) {
  using C = Cfg;
  const int64_t Kp = (a.K + 127) & ~(int64_t)127;
  CUtensorMap tmA, tmB, tmC;
  if (!make_codes_map(&tmA, a.a_codes, a.M, Kp, BM) || !make_codes_map(&tmB, a.b_codes, a.N, Kp, BN))
    return cudaErrorInvalidValue;
  if (!make_c_map(&tmC, a.C, a.M, a.N, a.ldc, a.c_is_f32 != 0)) return cudaErrorInvalidValue;
  CUtensorMap tmAh = tmA, tmBh = tmB;  // placeholders unless the high-precision side product is requested
  Params p{};
  p.use_tma_store = 1;
  p.starve = a.starve_first_stage;
  p.wait_limit = wait_limit_of(a);
  if (a.hp_Kh > 0) {
    if (!make_hp_map(&tmAh, a.hp_a, a.M, a.hp_Kh) || !make_hp_map(&tmBh, a.hp_b, a.N, a.hp_Kh)) return cudaErrorInvalidValue;
    p.hp_k_tiles = (int32_t)(a.hp_Kh / 64);
  }
  p.a_sf = a.a_sf;
  p.b_sf = a.b_sf;
  p.a_gscale = a.a_gscale;
  p.b_gscale = a.b_gscale;
  p.C = a.C;
  p.ldc = a.ldc;
  p.M = a.M;
  p.N = a.N;
  p.k_tiles = (int32_t)((Kp + BK - 1) / BK);
  p.k_chunks = (int32_t)(Kp / 128);
  p.g_per_row = Kp / 128;
  const int64_t kb_padded = ((Kp >> 4) + 15) & ~(int64_t)15;
  p.sf_tiles_a = p.sf_tiles_b = (int32_t)(kb_padded >> 2);
  p.m_tiles = (int32_t)((a.M + BM - 1) / BM);
  p.n_tiles = (int32_t)((a.N + BN - 1) / BN);
  p.c_is_f32 = a.c_is_f32;
  p.accumulate = a.accumulate;
  p.dev_status = a.dev_status;
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(gemm_nvfp4_kernel<GS>), C::SMEM_BYTES);
  if (e != cudaSuccess) return e;
  const int64_t tiles = (int64_t)p.m_tiles * p.n_tiles;
  const unsigned grid = (unsigned)std::min<int64_t>(tiles, sm_count());
  launch_kernel(gemm_nvfp4_kernel<GS>, dim3(grid), dim3(C::THREADS), C::SMEM_BYTES, st, tmA, tmB, tmC, tmAh, tmBh, p);
  return cudaGetLastError();
}

// Scale bytes of an operand as a 2-D byte tensor of 128-byte rows; box = 16 rows = the 2 KB of one (row tile, k tile).
bool make_sf_map(CUtensorMap* tm, const uint8_t* sf, int64_t total_bytes) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {128, (cuuint64_t)(total_bytes / 128)};
  const cuuint64_t strides[1] = {128};
  const cuuint32_t box[2] = {128, 16};
  const cuuint32_t estr[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(sf), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int GS, int PN>
cudaError_t launch_2cta(const GemmArgs& a, cudaStream_t st) {
  using C2 = Cfg2<PN>;
  const int64_t Kp = (a.K + 127) & ~(int64_t)127;
  const int64_t kb_padded = ((Kp >> 4) + 15) & ~(int64_t)15;
  const int64_t sfa_bytes = ((a.M + 127) / 128) * 128 * kb_padded, sfb_bytes = ((a.N + 127) / 128) * 128 * kb_padded;
  CUtensorMap tmA, tmB, tmSFA, tmSFB, tmC;
  if (!make_codes_map(&tmA, a.a_codes, a.M, Kp, 128) || !make_codes_map(&tmB, a.b_codes, a.N, Kp, PN / 2) ||
      !make_sf_map(&tmSFA, a.a_sf, sfa_bytes) || !make_sf_map(&tmSFB, a.b_sf, sfb_bytes) ||
      !make_c_map(&tmC, a.C, a.M, a.N, a.ldc, a.c_is_f32 != 0))
    return cudaErrorInvalidValue;
  Params p{};
  p.a_sf = a.a_sf;
  p.b_sf = a.b_sf;
  p.a_gscale = a.a_gscale;
  p.b_gscale = a.b_gscale;
  p.C = a.C;
  p.ldc = a.ldc;
  p.M = a.M;
  p.N = a.N;
  p.k_tiles = (int32_t)((Kp + BK - 1) / BK);
  p.sf_tiles_a = p.sf_tiles_b = (int32_t)(kb_padded >> 2);
  p.m_tiles = (int32_t)((a.M + 255) / 256);
  p.n_tiles = (int32_t)((a.N + PN - 1) / PN);
  p.c_is_f32 = a.c_is_f32;
  p.accumulate = a.accumulate;
  p.dev_status = a.dev_status;
  p.starve = a.starve_first_stage;
  p.wait_limit = wait_limit_of(a);
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(gemm_nvfp4_2cta_kernel<GS, PN>), C2::SMEM_BYTES);
  if (e != cudaSuccess) return e;
  const int64_t tiles = (int64_t)p.m_tiles * p.n_tiles;
  const unsigned pairs = (unsigned)std::min<int64_t>(tiles, sm_count() / 2);
  launch_kernel(gemm_nvfp4_2cta_kernel<GS, PN>, dim3(2 * pairs), dim3(C2_THREADS), C2::SMEM_BYTES, st, tmA, tmB, tmSFA, tmSFB, tmC, p);
  return cudaGetLastError();
}

cudaError_t launch_block128(const GemmArgs& a, cudaStream_t st) {
  const int64_t Kp = (a.K + 127) & ~(int64_t)127;
  if (Kp / 128 > B128_MAX_CHUNKS) return cudaErrorInvalidValue;
  CUtensorMap tmA, tmB, tmC;
  if (!make_codes_map(&tmA, a.a_codes, a.M, Kp, BM) || !make_codes_map(&tmB, a.b_codes, a.N, Kp, 128)) return cudaErrorInvalidValue;
  Params p{};
  CUtensorMap tmAh = tmA, tmBh = tmB;  // placeholders unless the high-precision side product is requested
  if (a.hp_Kh > 0) {
    if (!make_hp_map(&tmAh, a.hp_a, a.M, a.hp_Kh) || !make_hp_map(&tmBh, a.hp_b, a.N, a.hp_Kh)) return cudaErrorInvalidValue;
    p.hp_k_tiles = (int32_t)(a.hp_Kh / 64);
  }
  p.use_tma_store = make_c_map(&tmC, a.C, a.M, a.N, a.ldc, a.c_is_f32 != 0) ? 1 : 0;
  if (!p.use_tma_store) tmC = tmA;  // unused by the kernel then
  p.a_sf = a.a_sf;
  p.b_sf = a.b_sf;
  p.a_gscale = a.a_gscale;
  p.b_gscale = a.b_gscale;
  p.C = a.C;
  p.ldc = a.ldc;
  p.M = a.M;
  p.N = a.N;
  p.k_tiles = (int32_t)((Kp + BK - 1) / BK);
  p.k_chunks = (int32_t)(Kp / 128);
  p.g_per_row = Kp / 128;
  const int64_t kb_padded = ((Kp >> 4) + 15) & ~(int64_t)15;
  p.sf_tiles_a = p.sf_tiles_b = (int32_t)(kb_padded >> 2);
  p.m_tiles = (int32_t)((a.M + BM - 1) / BM);
  p.n_tiles = (int32_t)((a.N + 127) / 128);
  p.c_is_f32 = a.c_is_f32;
  p.accumulate = a.accumulate;
  p.dev_status = a.dev_status;
  p.wait_limit = wait_limit_of(a);
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(gemm_nvfp4_block128_kernel), B128_SMEM_BYTES);
  if (e != cudaSuccess) return e;
  const int64_t tiles = (int64_t)p.m_tiles * p.n_tiles;
  const unsigned grid = (unsigned)std::min<int64_t>(tiles, sm_count());
  launch_kernel(gemm_nvfp4_block128_kernel, dim3(grid), dim3(NUM_THREADS), B128_SMEM_BYTES, st, tmA, tmB, tmC, tmAh, tmBh, p);
  return cudaGetLastError();
}

// BF16 matrix [T, W] (leading dimension ld elements) as a 2-D tensor; box = 64 columns x 64 rows, 128-byte swizzle.
bool make_tokens_map(CUtensorMap* tm, const void* base, int64_t T, int64_t W, int64_t ld) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)W, (cuuint64_t)T};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  const cuuint32_t box[2] = {64, 64};
  const cuuint32_t estr[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// partial[(split * C + c) * Kh + j] = sum over the split's tokens of dY[t, c] * X_out[t, j]. Kh is any multiple of 64:
// the outlier channels are taken in slabs of at most 256 (the widest MMA), one launch per slab.
cudaError_t launch_hp_dw_mma(const uint16_t* dY, int64_t lddy, const uint16_t* X_out, int64_t Kh, int64_t T, int64_t C,
                             float* partial, int n_split, int64_t t_per_split, int32_t* dev_status, cudaStream_t st) {
  if (Kh <= 0 || Kh % 64 != 0) return cudaErrorInvalidValue;
  CUtensorMap tmDY, tmXO;
  if (!make_tokens_map(&tmDY, dY, T, C, lddy)) return cudaErrorInvalidValue;
  for (int64_t j0 = 0; j0 < Kh; j0 += 256) {
    const int64_t w = std::min<int64_t>(256, Kh - j0);
    if (!make_tokens_map(&tmXO, X_out + j0, T, w, Kh)) return cudaErrorInvalidValue;
    const uint32_t stage_bytes = A_BYTES + (uint32_t)(w / 64) * 8192u;
    const size_t smem = (size_t)HPDW_STAGES * stage_bytes + 1024 + 256;
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(hp_dw_mma_kernel), smem);
    if (e != cudaSuccess) return e;
    const dim3 grid((unsigned)((C + 127) / 128), (unsigned)n_split);
    launch_kernel(hp_dw_mma_kernel, dim3(grid), dim3(HPDW_THREADS), smem, st, tmDY, tmXO, partial + j0, C, (int32_t)w, Kh, T,
                  (int32_t)t_per_split, dev_status, DEFAULT_WAIT_LIMIT_CYCLES);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  return cudaSuccess;
}

// Dense BF16 product (the simulated FP6 x FP4 layer): C = (SgA SgB) * A B^T with A [M, ld], B [N, ld] BF16 row-major, ld a
// multiple of 64 and the same for both. It is the 128 x 128 kernel with no FP4 k tiles at all: only its BF16 side-product path
// runs (64-wide k tiles, kind::f16, FP32 accumulation in the side accumulator) and the epilogue scales that accumulator.
cudaError_t launch_dense_gemm(const void* A, const void* B, int64_t M, int64_t N, int64_t ld, const float* a_gscale,
                              const float* b_gscale, void* Cp, int c_is_f32, int64_t ldc, int32_t* dev_status, cudaStream_t st) {
  using C = Cfg;
  if (M == 0 || N == 0) return cudaSuccess;
  CUtensorMap tmAh, tmBh, tmC;
  if (!make_hp_map(&tmAh, A, M, ld) || !make_hp_map(&tmBh, B, N, ld) || !make_c_map(&tmC, Cp, M, N, ldc, c_is_f32 != 0))
    return cudaErrorInvalidValue;
  Params p{};
  p.use_tma_store = 1;
  p.wait_limit = DEFAULT_WAIT_LIMIT_CYCLES;
  p.hp_k_tiles = (int32_t)(ld / 64);
  p.a_gscale = a_gscale;
  p.b_gscale = b_gscale;
  p.C = Cp;
  p.ldc = ldc;
  p.M = M;
  p.N = N;
  p.k_tiles = 0;
  p.m_tiles = (int32_t)((M + BM - 1) / BM);
  p.n_tiles = (int32_t)((N + BN - 1) / BN);
  p.c_is_f32 = c_is_f32;
  p.dev_status = dev_status;
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(gemm_nvfp4_kernel<kGsTensor>), C::SMEM_BYTES);
  if (e != cudaSuccess) return e;
  const int64_t tiles = (int64_t)p.m_tiles * p.n_tiles;
  const unsigned grid = (unsigned)std::min<int64_t>(tiles, sm_count());
  launch_kernel(gemm_nvfp4_kernel<kGsTensor>, dim3(grid), dim3(C::THREADS), C::SMEM_BYTES, st, tmAh, tmBh, tmC, tmAh, tmBh, p);
  return cudaGetLastError();
}

size_t gemm_workspace_bytes(int64_t, int64_t, int64_t) { return 0; }
int64_t gemm_block128_max_k() { return (int64_t)B128_MAX_CHUNKS * 128; }

// Variant choice. All kernels are bound by what the L2 delivers to the SMs (about 13 - 16 TB/s over all SMs): the 128 x 128
// kernel pulls 36 KB per k tile and SM, a pair on a 256 x 256 tile 38 KB per SM for twice the math. The 128 x 128 kernel has
// two accumulators (a tile's epilogue overlaps the next tile's MMAs entirely); the 256-wide pair kernel has one and hands it
// over once its sixteen epilogue warps hold the tile in registers (a few hundred cycles per tile), and 256-wide tiles fill
// the last wave worse. Pairs therefore run when there are enough tiles: from K = 1024 with five tiles per pair, from
// K = 2048 with two, and from K = 8192 already when half of the pairs get a tile (the weight gradients of a model: few
// tiles, K = tokens). Measured, BF16 output, 128 x 128 / 256 x 256 / 256 x 192, us: 16384 x 3072 x 1024 38.9 / 34.8 / 36.9;
// 16384 x 1024 x 1024 (256 pair tiles) 18.5 / 19.2 / 22.4; 8192 x 3072 x 1024 (384) 24.5 / 22.7 / 22.5; 4096 x 4096 x 1024
// (256) 18.4 / 18.5 / 20.4; 16384 x 1024 x 2816 31.6 / 28.8 / 32.8; 16384 x 3072 x 2048 61.4 / 51.2 / 55.8; 8192 x 8192 x 3072
// 100.4 / 77.8 / 87.9; 4096^3 38.9 / 34.8 / 34.8; 16384 x 14336 x 4096 426 / 342 / 387; 4096 x 8192 x 8192 114.8 / 88.1 /
// 104.4; 16384 x 8192 x 8192 455 / 352 / 408; 3072 x 1024 x 16384 (48 / 72 pair tiles) 38.9 / 30.8 / 30.7, FP32 output 40.9 /
// 32.7 / 30.7; 1024 x 1024 x 16384 (16 / 24) 22.6 / 30.8 / 28.7; 2048 x 2048 x 16384 (64 / 88) 38.9 / 32.8 / 46.9.
// A 256-row tile of an operand spans two 128-row scale tiles, and rows are padded to 128 in the scale layout, so any M, N
// work. The fused high-precision side product and the outer-block scales live in the single-CTA kernels only.
cudaError_t launch_gemm(const GemmArgs& a, cudaStream_t st) {
  if (a.M == 0 || a.N == 0) return cudaSuccess;
  if (a.gs_mode == kGsBlock128) return a.variant >= 2 ? cudaErrorInvalidValue : launch_block128(a, st);
  const int64_t tiles256 = ((a.M + 255) / 256) * ((a.N + 255) / 256), n_pairs = sm_count() / 2;
  // (ROW scales: the pair kernels' epilogue holds a quarter tile in registers and has two more multiplies per element to do,
  // it spills and becomes the bound at short K -- 16384 x 3072 x 1024, BF16 output: 40.9 / 53.4 / 74.7 us -- so pairs start at
  // K = 2048 there and the 192-wide kernel, which has the least time per tile to hide it in, is not used.)
  const bool row_scales = a.gs_mode == kGsRow;
  bool pairs = (!row_scales && a.K >= 1024 && tiles256 >= 5 * n_pairs) || (a.K >= 2048 && tiles256 >= 2 * n_pairs) ||
               (a.K >= 8192 && 2 * tiles256 >= n_pairs);
  // Between the two pair kernels, by a cost model in units of one 256-wide k tile: rounds of the pair grid x (k tiles x the
  // relative cost of a k tile + 1 per tile). A 192-wide k tile costs 0.85 (three quarters of the math, but more operand
  // traffic per flop); what the 192-wide tiles have is the finer last wave, which decides when tiles are few.
  bool pairs192 = false;
  if (pairs) {
    const int64_t tiles192 = ((a.M + 255) / 256) * ((a.N + 191) / 192);
    const double k_tiles = (double)((a.K + BK - 1) / BK);
    const double cost256 = (double)((tiles256 + n_pairs - 1) / n_pairs) * (k_tiles + 1.0);
    const double cost192 = (double)((tiles192 + n_pairs - 1) / n_pairs) * (0.85 * k_tiles + 1.0);
    pairs192 = !row_scales && cost192 < cost256;
  }
  if (pairs192) pairs = false;
  if (a.variant == 1) pairs = pairs192 = false;
  if (a.variant == 2) { pairs = true; pairs192 = false; }
  if (a.variant == 3) { pairs192 = true; pairs = false; }
  if (a.hp_Kh > 0) {
    if (a.variant == 2 || a.variant == 3) return cudaErrorInvalidValue;
    pairs = pairs192 = false;
  }
  if (pairs192) return a.gs_mode == kGsTensor ? launch_2cta<kGsTensor, 192>(a, st) : launch_2cta<kGsRow, 192>(a, st);
  if (pairs) return a.gs_mode == kGsTensor ? launch_2cta<kGsTensor, 256>(a, st) : launch_2cta<kGsRow, 256>(a, st);
  return a.gs_mode == kGsTensor ? launch_tile128<kGsTensor>(a, st) : launch_tile128<kGsRow>(a, st);
}

}  // namespace nvfp4
