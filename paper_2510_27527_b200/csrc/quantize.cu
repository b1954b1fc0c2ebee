// Quantize kernels of the NVFP4 linear layer (paper Sec. 2.2 double-block quantization, Sec. 2.1 rounding):
//   - amax pre-passes (whole tensor, per source row, per source column) for the TENSOR and ROW scale modes;
//   - row-axis quantize from BF16 (Q1, Q2, Q3 of Sec. 2.3): one thread per 16-element inner block;
//   - transposing quantize (Q5 from BF16; Q4, Q6 from the forward operand's codes, i.e. from X-hat / W-hat):
//     a 128(k) x 64(operand rows) tile is staged in shared memory as FP32 and read back column-wise.
// With a non-zero sign stream the backward quantizers first apply the random Hadamard transformation of Sec. 4.1 to each
// 16-element block along K (the block a thread already holds in registers), and the amax pre-passes see transformed data.
// All of them are HBM streaming kernels; the launch wrappers at the bottom are called by the C-ABI layer.
#include <type_traits>

#include "nvfp4_device.cuh"
#include "nvfp4_internal.h"

namespace nvfp4 {

// =========================================================================================================
// amax pre-passes. Results are bit patterns of non-negative floats combined with atomicMax (order-free, hence
// deterministic). The cells must be zero before the launch.
// =========================================================================================================
__device__ __forceinline__ void amax_tensor_bf16_body(const uint16_t* __restrict__ src, int64_t rows, int64_t cols, int64_t ld,
                                                      uint32_t* amax_bits, unsigned block, unsigned n_blocks) {
  // One 16-byte chunk (8 BF16) per thread per step; rows are walked through a flattened chunk index.
  const int64_t chunks_per_row = (cols + 7) >> 3;
  const int64_t total = rows * chunks_per_row;
  uint32_t m = 0;
  if (ld == cols && (cols & 7) == 0) {  // one contiguous run of 16-byte chunks: no row arithmetic, four loads in flight
    const uint4* p4 = reinterpret_cast<const uint4*>(src);
    const int64_t stride = (int64_t)n_blocks * blockDim.x;
    int64_t i = (int64_t)block * blockDim.x + threadIdx.x;
    for (; i + 3 * stride < total; i += 4 * stride) {
      const uint4 v0 = p4[i], v1 = p4[i + stride], v2 = p4[i + 2 * stride], v3 = p4[i + 3 * stride];
      const uint32_t a0 = amax16x2(amax16x2(v0.x, v0.y), amax16x2(v0.z, v0.w));
      const uint32_t a1 = amax16x2(amax16x2(v1.x, v1.y), amax16x2(v1.z, v1.w));
      const uint32_t a2 = amax16x2(amax16x2(v2.x, v2.y), amax16x2(v2.z, v2.w));
      const uint32_t a3 = amax16x2(amax16x2(v3.x, v3.y), amax16x2(v3.z, v3.w));
      m = amax16x2(m, amax16x2(amax16x2(a0, a1), amax16x2(a2, a3)));
    }
    for (; i < total; i += stride) {
      const uint4 v = p4[i];
      m = amax16x2(m, amax16x2(amax16x2(v.x, v.y), amax16x2(v.z, v.w)));
    }
  } else
  for (int64_t i = (int64_t)block * blockDim.x + threadIdx.x; i < total; i += (int64_t)n_blocks * blockDim.x) {
    const int64_t r = i / chunks_per_row, c = (i - r * chunks_per_row) << 3;
    const uint16_t* p = src + r * ld + c;
    if (c + 8 <= cols) {
      const uint4 v = *reinterpret_cast<const uint4*>(p);
      m = amax16x2(m, amax16x2(amax16x2(v.x, v.y), amax16x2(v.z, v.w)));
    } else {
      for (int64_t j = c; j < cols; ++j) m = amax16x2(m, (uint32_t)p[j - c]);
    }
  }
  uint32_t a = hmax_of_pair(bf16x2_abs_bits(m));
#pragma unroll
  for (int o = 16; o; o >>= 1) a = max(a, __shfl_xor_sync(0xFFFFFFFFu, a, o));
  __shared__ uint32_t warp_max[8];
  if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = a;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w) a = max(a, warp_max[w]);
    if (a) atomicMax(amax_bits, a << 16);  // BF16 pattern -> FP32 pattern
  }
}

__global__ void __launch_bounds__(256) amax_tensor_bf16_kernel(const uint16_t* __restrict__ src, int64_t rows,
                                                              int64_t cols, int64_t ld, uint32_t* amax_bits) {
  pdl_prologue();
  amax_tensor_bf16_body(src, rows, cols, ld, amax_bits, blockIdx.x, gridDim.x);
}

// Two tensors in one launch (the forward pass's X and W): the first grid_a CTAs take A, the rest take B.
__global__ void __launch_bounds__(256) amax_tensor_pair_kernel(const uint16_t* __restrict__ a, int64_t rows_a, int64_t cols_a, int64_t ld_a,
                                                              uint32_t* cell_a, unsigned grid_a, const uint16_t* __restrict__ b,
                                                              int64_t rows_b, int64_t cols_b, int64_t ld_b, uint32_t* cell_b) {
  pdl_prologue();
  if (blockIdx.x < grid_a)
    amax_tensor_bf16_body(a, rows_a, cols_a, ld_a, cell_a, blockIdx.x, grid_a);
  else
    amax_tensor_bf16_body(b, rows_b, cols_b, ld_b, cell_b, blockIdx.x - grid_a, gridDim.x - grid_a);
}

// amax of a BF16 matrix over all columns EXCEPT a sorted list of excluded ones (OutControl: the outlier channels do not
// take part in the FP4 operand's tensor scale). Each CTA builds, in shared memory, one 16-byte AND mask per 8-column
// chunk (0x7FFF for a column that takes part: the sign goes with it; 0 for an excluded one or one past the end), then
// streams a contiguous slab of rows with 16-byte loads: per chunk one mask load, four ANDs and four packed maxima.
// The (row, chunk) position of a thread advances by additions only. Folded into cells[0] by atomic max.
// With `out` the excluded columns of the slab are then copied, in list order, to out[r, 0 .. n_excl) (zero up to ld_out):
// the high-precision side operand, picked from rows this CTA has just pulled through L1 / L2.
__global__ void __launch_bounds__(256) amax_tensor_masked_kernel(const uint16_t* __restrict__ src, int64_t rows, int64_t cols,
                                                                int64_t ld, const int32_t* __restrict__ excluded, int64_t n_excl,
                                                                uint32_t* amax_bits, uint16_t* __restrict__ out, int64_t ld_out,
                                                                int64_t rows_per_cta, uint64_t inv_o) {
  pdl_prologue();
  extern __shared__ __align__(16) uint16_t lane_mask[];  // [chunks * 8]
  const uint32_t chunks = (uint32_t)((cols + 7) >> 3);
  for (uint32_t i = threadIdx.x; i < chunks * 8; i += 256) lane_mask[i] = (int64_t)i < cols ? (uint16_t)0x7FFFu : (uint16_t)0;
  __syncthreads();
  for (int64_t i = threadIdx.x; i < n_excl; i += 256) lane_mask[excluded[i]] = 0;
  __syncthreads();
  const int64_t r0 = (int64_t)blockIdx.x * rows_per_cta;
  const int64_t r1 = min(rows, r0 + rows_per_cta);
  const uint32_t n_rows = r1 > r0 ? (uint32_t)(r1 - r0) : 0u;
  // thread t starts at item t of the slab (row-major (row, chunk) pairs) and advances by 256 items
  const uint32_t step_r = 256u / chunks, step_c = 256u % chunks;
  uint32_t rr = threadIdx.x / chunks, c = threadIdx.x % chunks;
  const bool row_tail = (cols & 7) != 0;  // the last chunk of a row is ragged: read element by element
  uint32_t m = 0;
  while (rr < n_rows) {
    // four items per pass: positions first, then all loads, then the masks and maxima
    uint4 v[4];
    uint32_t cc[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      cc[u] = 0xFFFFFFFFu;
      v[u] = make_uint4(0, 0, 0, 0);
      if (rr < n_rows) {
        cc[u] = c;
        const uint16_t* p = src + (r0 + rr) * ld + ((int64_t)c << 3);
        if (!row_tail || c + 1 < chunks) {
          v[u] = *reinterpret_cast<const uint4*>(p);
        } else {
          uint32_t t[4] = {0, 0, 0, 0};
          for (int q = 0; q < 8; ++q)
            if (((int64_t)c << 3) + q < cols) t[q >> 1] |= (uint32_t)p[q] << (16 * (q & 1));
          v[u] = make_uint4(t[0], t[1], t[2], t[3]);
        }
        c += step_c;
        rr += step_r;
        if (c >= chunks) {
          c -= chunks;
          rr += 1;
        }
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (cc[u] != 0xFFFFFFFFu) {
        const uint4 k = *reinterpret_cast<const uint4*>(lane_mask + (cc[u] << 3));
        m = amax16x2(m, amax16x2(amax16x2(v[u].x & k.x, v[u].y & k.y), amax16x2(v[u].z & k.z, v[u].w & k.w)));  // (sign bits: see amax16x2)
      }
    }
  }
  if (out && n_rows) {
    const uint32_t ldo = (uint32_t)ld_out, n_out_items = n_rows * ldo;  // inv_o = 2^32 / ldo + 1, prepared by the launcher
    for (uint32_t e = threadIdx.x; e < n_out_items; e += 256) {
      const uint32_t ro = (uint32_t)(((uint64_t)e * inv_o) >> 32), j = e - ro * ldo;
      out[(r0 + ro) * ld_out + j] = j < n_excl ? src[(r0 + ro) * ld + excluded[j]] : (uint16_t)0;
    }
  }
  uint32_t a = hmax_of_pair(bf16x2_abs_bits(m));
#pragma unroll
  for (int o = 16; o; o >>= 1) a = max(a, __shfl_xor_sync(0xFFFFFFFFu, a, o));
  __shared__ uint32_t warp_max[8];
  if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = a;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w) a = max(a, warp_max[w]);
    if (a) atomicMax(amax_bits, a << 16);
  }
}

// amax of each source row over the kept columns -> cells[row] (ROW scale mode of the row-axis quantizer).
__global__ void __launch_bounds__(256) amax_rows_bf16_kernel(const uint16_t* __restrict__ src, int64_t rows,
                                                            int64_t cols, int64_t ld,
                                                            const int32_t* __restrict__ keep, int64_t n_keep,
                                                            uint32_t* cells, int single_cell) {
  pdl_prologue();
  const int64_t r = blockIdx.x;
  const uint16_t* p = src + r * ld;
  uint32_t m = 0;
  if (keep) {
    for (int64_t j = threadIdx.x; j < n_keep; j += blockDim.x) m = max(m, (uint32_t)(p[keep[j]] & 0x7FFFu));
  } else {
    const int64_t nchunk = cols >> 3;
    for (int64_t c = threadIdx.x; c < nchunk; c += blockDim.x) {
      const uint4 v = *reinterpret_cast<const uint4*>(p + (c << 3));
      m = amax16x2(m, amax16x2(amax16x2(v.x, v.y), amax16x2(v.z, v.w)));
    }
    for (int64_t j = (nchunk << 3) + threadIdx.x; j < cols; j += blockDim.x) m = amax16x2(m, (uint32_t)p[j]);
    m = hmax_of_pair(bf16x2_abs_bits(m));
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  __shared__ uint32_t warp_max[8];
  if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w) m = max(m, warp_max[w]);
    if (single_cell) {
      if (m) atomicMax(cells, m << 16);
    } else {
      cells[r] = m << 16;
    }
  }
}

// amax of each source row, one warp per row (ROW scale mode of the row-axis quantizer without a column list): 16-byte
// loads, four in flight per lane, packed maxima, one shuffle reduction; no shared memory, no barrier. cells[row] is
// written, not accumulated. Needs ld % 8 == 0 and a 16-byte aligned base.
__global__ void __launch_bounds__(256) amax_rows_warp_kernel(const uint16_t* __restrict__ src, int64_t rows, int64_t cols, int64_t ld,
                                                            uint32_t* __restrict__ cells) {
  pdl_prologue();
  const int lane = threadIdx.x & 31;
  const int64_t r = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (r >= rows) return;
  const uint16_t* p = src + r * ld;
  const int64_t nchunk = cols >> 3;
  uint32_t m = 0;
  int64_t c = lane;
  for (; c + 96 < nchunk; c += 128) {
    const uint4 v0 = *reinterpret_cast<const uint4*>(p + (c << 3)), v1 = *reinterpret_cast<const uint4*>(p + ((c + 32) << 3));
    const uint4 v2 = *reinterpret_cast<const uint4*>(p + ((c + 64) << 3)), v3 = *reinterpret_cast<const uint4*>(p + ((c + 96) << 3));
    const uint32_t a0 = amax16x2(amax16x2(v0.x, v0.y), amax16x2(v0.z, v0.w)), a1 = amax16x2(amax16x2(v1.x, v1.y), amax16x2(v1.z, v1.w));
    const uint32_t a2 = amax16x2(amax16x2(v2.x, v2.y), amax16x2(v2.z, v2.w)), a3 = amax16x2(amax16x2(v3.x, v3.y), amax16x2(v3.z, v3.w));
    m = amax16x2(m, amax16x2(amax16x2(a0, a1), amax16x2(a2, a3)));
  }
  for (; c < nchunk; c += 32) {
    const uint4 v = *reinterpret_cast<const uint4*>(p + (c << 3));
    m = amax16x2(m, amax16x2(amax16x2(v.x, v.y), amax16x2(v.z, v.w)));
  }
  for (int64_t j = (nchunk << 3) + lane; j < cols; j += 32) m = amax16x2(m, (uint32_t)p[j]);
  uint32_t a = hmax_of_pair(bf16x2_abs_bits(m));
#pragma unroll
  for (int o = 16; o; o >>= 1) a = max(a, __shfl_xor_sync(0xFFFFFFFFu, a, o));
  if (lane == 0) cells[r] = a << 16;
}

// amax of each COLUMN of a BF16 matrix [rowsK, D] (the per-row scales of the transposed operand in ROW mode). CTA = 32 lanes
// x 8 row lanes over a strip of 256 columns and a slab of rows: a lane owns eight neighbouring columns (one 16-byte load
// per row, a warp reads 512 contiguous bytes), keeps eight running maxima in four packed registers, the eight row lanes
// are combined through shared memory and the slab's result is folded into cells[column] (zero before the launch) by one
// atomic max per column. ld % 8 == 0, 16-byte aligned base.
__global__ void __launch_bounds__(256) amax_cols_bf16_kernel(const uint16_t* __restrict__ src, int64_t rowsK, int64_t D, int64_t ld,
                                                            int64_t rows_per_slab, uint32_t* cells) {
  pdl_prologue();
  const int lane = threadIdx.x & 31, ry = threadIdx.x >> 5;
  const int64_t d0 = (int64_t)blockIdx.x * 256 + lane * 8;
  const int64_t k0 = (int64_t)blockIdx.y * rows_per_slab, k1 = min(rowsK, k0 + rows_per_slab);
  uint32_t m[4] = {0, 0, 0, 0};
  if (d0 + 8 <= D) {
    int64_t k = k0 + ry;
    for (; k + 24 < k1; k += 32) {  // four rows in flight
      const uint4 v0 = *reinterpret_cast<const uint4*>(src + k * ld + d0), v1 = *reinterpret_cast<const uint4*>(src + (k + 8) * ld + d0);
      const uint4 v2 = *reinterpret_cast<const uint4*>(src + (k + 16) * ld + d0), v3 = *reinterpret_cast<const uint4*>(src + (k + 24) * ld + d0);
      m[0] = amax16x2(amax16x2(m[0], v0.x), amax16x2(amax16x2(v1.x, v2.x), v3.x));
      m[1] = amax16x2(amax16x2(m[1], v0.y), amax16x2(amax16x2(v1.y, v2.y), v3.y));
      m[2] = amax16x2(amax16x2(m[2], v0.z), amax16x2(amax16x2(v1.z, v2.z), v3.z));
      m[3] = amax16x2(amax16x2(m[3], v0.w), amax16x2(amax16x2(v1.w, v2.w), v3.w));
    }
    for (; k < k1; k += 8) {
      const uint4 v = *reinterpret_cast<const uint4*>(src + k * ld + d0);
      m[0] = amax16x2(m[0], v.x);
      m[1] = amax16x2(m[1], v.y);
      m[2] = amax16x2(m[2], v.z);
      m[3] = amax16x2(m[3], v.w);
    }
  } else if (d0 < D) {  // ragged last chunk of the rows
    for (int64_t k = k0 + ry; k < k1; k += 8)
      for (int i = 0; d0 + i < D; ++i) m[i >> 1] = amax16x2(m[i >> 1], (uint32_t)src[k * ld + d0 + i] << (16 * (i & 1)));
  }
  __shared__ uint32_t red[8][4][32];
#pragma unroll
  for (int i = 0; i < 4; ++i) red[ry][i][lane] = bf16x2_abs_bits(m[i]);
  __syncthreads();
  {
    // thread t combines the eight row lanes of packed pair (t >> 5 & 3) of lane (t & 31); two threads share... keep it simple:
    // 128 threads, one packed pair each
    if (threadIdx.x < 128) {
      const int i = threadIdx.x >> 5, ln = threadIdx.x & 31;
      uint32_t a = red[0][i][ln];
#pragma unroll
      for (int y = 1; y < 8; ++y) a = umax16x2(a, red[y][i][ln]);
      const int64_t d = (int64_t)blockIdx.x * 256 + ln * 8 + 2 * i;
      const uint32_t lo = a & 0xFFFFu, hi = a >> 16;
      if (d < D && lo) atomicMax(cells + d, lo << 16);
      if (d + 1 < D && hi) atomicMax(cells + d + 1, hi << 16);
    }
  }
}

// amax of the transformed matrix (x S) H along the rows' K axis: per row (ROW mode) or folded into cells[0]. One thread
// per 16-element block; atomic max on cells that are zero before the launch.
__global__ void __launch_bounds__(256) amax_rows_rht_kernel(const uint16_t* __restrict__ src, int64_t rows, int64_t K, int64_t ld,
                                                           uint64_t seed, uint32_t rht_stream, uint32_t* cells, int per_row) {
  pdl_prologue();
  const int64_t nb16 = (K + 15) >> 4;
  const int64_t total = rows * nb16;
  float acc = 0.0f;
  for (int64_t base = (int64_t)blockIdx.x * 256; base < total; base += (int64_t)gridDim.x * 256) {
    const int64_t gid = base + threadIdx.x;
    const bool active = gid < total;
    const int64_t r = active ? gid / nb16 : -1;
    const int64_t k0 = active ? (gid - r * nb16) << 4 : 0;
    float x[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) x[i] = 0.0f;
    if (active) {
      const uint16_t* p = src + r * ld + k0;
      if (k0 + 16 <= K && (ld & 7) == 0) {
        const uint4 v0 = *reinterpret_cast<const uint4*>(p), v1 = *reinterpret_cast<const uint4*>(p + 8);
        const uint32_t w[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          x[2 * i] = bf16_lo(w[i]);
          x[2 * i + 1] = bf16_hi(w[i]);
        }
      } else {
        for (int i = 0; i < 16; ++i)
          if (k0 + i < K) x[i] = bf16_bits_to_float(p[i]);
      }
    }
    rht_scale16(x, rht_sign16(seed, rht_stream, k0));
    hadamard16_butterflies(x);
    float m = 0.0f;
#pragma unroll
    for (int i = 0; i < 16; ++i) m = fmaxf(m, fabsf(x[i]));
    if (per_row) {
      // a warp usually sits inside one row: one atomic per warp then, else one per block
      const int64_t r0 = __shfl_sync(0xFFFFFFFFu, r, 0);
      if (__all_sync(0xFFFFFFFFu, r == r0)) {
#pragma unroll
        for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
        if ((threadIdx.x & 31) == 0 && r0 >= 0 && m > 0.0f) atomicMax(cells + r0, __float_as_uint(m));
      } else if (active && m > 0.0f) {
        atomicMax(cells + r, __float_as_uint(m));
      }
    } else {
      acc = fmaxf(acc, m);
    }
  }
  if (!per_row) {
#pragma unroll
    for (int o = 16; o; o >>= 1) acc = fmaxf(acc, __shfl_xor_sync(0xFFFFFFFFu, acc, o));
    __shared__ float warp_max[8];
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
      for (int w = 1; w < 8; ++w) acc = fmaxf(acc, warp_max[w]);
      if (acc > 0.0f) atomicMax(cells, __float_as_uint(acc));
    }
  }
}

// =========================================================================================================
// Shared epilogue of one 16-element inner block: scale, round, pack.
// =========================================================================================================
// =========================================================================================================
// Row-axis quantize from BF16: one thread per inner block, eight neighbouring threads per 128-wide outer block.
//   GS      scale mode. TENSOR reads the amax cell gs_cells[0]; ROW reads gs_cells[row]; BLOCK128 reduces the
//           group amax over the 8 threads of the group with shuffles (single pass over the data).
//   GATHER  columns come from the list `keep` (OutControl compaction) instead of 0..cols-1.
//   RHT     each block is replaced by (x S) H_16 before anything else looks at it (never together with GATHER).
// =========================================================================================================
template <int GS, bool SR, bool TILED, bool GATHER, bool RHT>
__global__ void __launch_bounds__(256, 4)
quantize_rows_kernel(const uint16_t* __restrict__ src, int64_t rows, int64_t K, int64_t ld,
                     const int32_t* __restrict__ keep, uint64_t seed, uint32_t stream_id,
                     const uint32_t* __restrict__ gs_cells, uint8_t* __restrict__ codes, uint8_t* __restrict__ sf,
                     float* __restrict__ gscale, uint32_t div_mul, uint32_t div_shift, int wide_loads, int64_t cols_src,
                     int64_t stage_cols8, uint32_t rht_stream, int sb_up, const __grid_constant__ PhiloxKeys pk) {
  pdl_prologue();
  constexpr int NB = 4;  // inner blocks per thread; all loads are issued before any arithmetic
  extern __shared__ uint16_t row_stage[];  // GATHER only: the source rows this CTA touches, [n_rows][cols_src8]
  const int64_t Kp = (K + 127) & ~(int64_t)127;
  const int64_t K16 = (K + 15) & ~(int64_t)15;
  const int64_t nb = Kp >> 4;  // inner blocks per operand row (multiple of 8)
  const int64_t total = rows * nb;
  const int64_t cta_base = (int64_t)blockIdx.x * (256 * NB) + threadIdx.x;
  // GATHER (OutControl compaction): the CTA's blocks cover a few whole or partial source rows; copy those rows to
  // shared memory with coalesced 16-byte loads, then pick the kept columns from there.
  int64_t stage_row0 = 0;
  if (GATHER && stage_cols8 > 0) {
    const int64_t first = (int64_t)blockIdx.x * (256 * NB);
    const int64_t last = min(first + 256 * NB, total) - 1;
    stage_row0 = first / nb;
    const int64_t n_rows = last / nb - stage_row0 + 1;
    const uint32_t chunks_per_row = (uint32_t)(stage_cols8 >> 3);
    const uint32_t n_chunks = (uint32_t)n_rows * chunks_per_row;
    // e / chunks_per_row by multiplication (exact while e * chunks_per_row < 2^32, and a CTA stages a few thousand chunks)
    const uint64_t inv = (1ull << 32) / chunks_per_row + 1ull;
    // eight chunks per thread and pass, every load issued before the first store: one exposed memory latency per pass
    for (uint32_t e0 = threadIdx.x; e0 < n_chunks; e0 += 256 * 8) {
      uint4 v[8];
      uint32_t off[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const uint32_t e = e0 + q * 256;
        v[q] = make_uint4(0, 0, 0, 0);
        off[q] = 0xFFFFFFFFu;
        if (e < n_chunks) {
          const uint32_t rr = (uint32_t)(((uint64_t)e * inv) >> 32), ch = (e - rr * chunks_per_row) << 3;
          off[q] = rr * (uint32_t)stage_cols8 + ch;
          const uint16_t* p = src + (stage_row0 + rr) * ld + ch;
          if ((int64_t)ch + 8 <= cols_src) {
            v[q] = *reinterpret_cast<const uint4*>(p);
          } else {
            uint32_t t[4] = {0, 0, 0, 0};
            for (int i = 0; i < 8; ++i)
              if ((int64_t)ch + i < cols_src) t[i >> 1] |= (uint32_t)p[i] << (16 * (i & 1));
            v[q] = make_uint4(t[0], t[1], t[2], t[3]);
          }
        }
      }
#pragma unroll
      for (int q = 0; q < 8; ++q)
        if (off[q] != 0xFFFFFFFFu) *reinterpret_cast<uint4*>(row_stage + off[q]) = v[q];
    }
    __syncthreads();
  }

  // Rows, K and the leading dimension are below 2^31 (checked by the launcher): row / block / column indices are 32-bit,
  // only the final byte offsets are formed in 64 bits (one widening multiply each).
  const uint32_t K32 = (uint32_t)K, ld32 = (uint32_t)ld, nb32 = (uint32_t)nb;
  // Interior CTAs (all of their 1024 blocks exist and are full 16-element blocks) run a copy of the body in which every
  // bounds check is compiled out; only the last CTA and ragged shapes take the checked copy.
  auto body = [&](auto full_tag) {
    constexpr bool FULL = decltype(full_tag)::value;
    uint32_t w[NB][8];
    int32_t row[NB];
    uint32_t blk[NB];
  #pragma unroll
    for (int j = 0; j < NB; ++j) {
      const int64_t gid = cta_base + j * 256;
      const bool active = FULL || gid < total;
      uint32_t r = 0, b = 0;
      if (active) {
        // gid / nb: by multiply-high when the launcher could prepare the constants (gid < 2^31), else plain division
        if (div_mul) {
          const uint32_t n = (uint32_t)gid, t = __umulhi(div_mul, n);
          r = (t + ((n - t) >> 1)) >> div_shift;
          b = n - r * nb32;
        } else if (div_shift != 0xFFFFFFFFu) {
          r = (uint32_t)gid >> div_shift;
          b = (uint32_t)gid & (nb32 - 1u);
        } else {
          r = (uint32_t)(gid / nb);
          b = (uint32_t)(gid - (int64_t)r * nb);
        }
      }
      row[j] = active ? (int32_t)r : -1;
      blk[j] = b;
      const uint32_t k0 = b << 4;
  #pragma unroll
      for (int i = 0; i < 8; ++i) w[j][i] = 0;
      if (FULL || (active && k0 < K32)) {
        const uint16_t* p = src + (size_t)r * ld32;
        if (!GATHER && (FULL || k0 + 16 <= K32)) {
          if (wide_loads) {  // rows start on 32-byte boundaries: one 256-bit load, a warp reads 1 KB contiguously
            asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                         : "=r"(w[j][0]), "=r"(w[j][1]), "=r"(w[j][2]), "=r"(w[j][3]), "=r"(w[j][4]), "=r"(w[j][5]),
                           "=r"(w[j][6]), "=r"(w[j][7])
                         : "l"(p + k0));
          } else {
            const uint4 v0 = *reinterpret_cast<const uint4*>(p + k0);
            const uint4 v1 = *reinterpret_cast<const uint4*>(p + k0 + 8);
            w[j][0] = v0.x; w[j][1] = v0.y; w[j][2] = v0.z; w[j][3] = v0.w;
            w[j][4] = v1.x; w[j][5] = v1.y; w[j][6] = v1.z; w[j][7] = v1.w;
          }
        } else if (GATHER && stage_cols8 > 0 && k0 + 16 <= K32) {
          const uint16_t* sp = row_stage + ((int64_t)r - stage_row0) * stage_cols8;
          const int4* kp = reinterpret_cast<const int4*>(keep + k0);  // keep is 16-byte aligned, k0 a multiple of 16
  #pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int4 id = kp[q];
            w[j][2 * q] = (uint32_t)sp[id.x] | ((uint32_t)sp[id.y] << 16);
            w[j][2 * q + 1] = (uint32_t)sp[id.z] | ((uint32_t)sp[id.w] << 16);
          }
        } else {
          for (int i = 0; i < 16; ++i) {
            if (k0 + i < K32) {
              const uint32_t e = GATHER ? p[keep[k0 + i]] : p[k0 + i];
              w[j][i >> 1] |= e << (16 * (i & 1));
            }
          }
        }
      }
    }

    float Sg_t = 1.0f;
    if (GS == kGsTensor) {
      Sg_t = global_scale_from_amax(__uint_as_float(gs_cells[0]));
      if (blockIdx.x == 0 && threadIdx.x == 0) gscale[0] = Sg_t;
    }

  #pragma unroll
    for (int j = 0; j < NB; ++j) {
      const bool active = FULL || row[j] >= 0;
      const uint32_t r = active ? (uint32_t)row[j] : 0u;
      const uint32_t b = blk[j];
      const uint32_t k0 = b << 4;
      float x[16];
      uint32_t amax_b_bits;  // binary32 pattern of the block's amax (non-negative, so integer order = float order)
      if (RHT) {
  #pragma unroll
        for (int i = 0; i < 8; ++i) {
          x[2 * i] = bf16_lo(w[j][i]);
          x[2 * i + 1] = bf16_hi(w[j][i]);
        }
        // blocks past K (layout padding up to 128) take no signs, so that they stay +0 and encode as zero bytes
        rht_scale16(x, (FULL || k0 < K32) ? rht_sign16(seed, rht_stream, (int64_t)k0) : 0u);
        hadamard16_butterflies(x);
        float m = 0.0f;
  #pragma unroll
        for (int i = 0; i < 16; ++i) m = fmaxf(m, fabsf(x[i]));
        amax_b_bits = __float_as_uint(m);
      } else {
        uint32_t m2 = 0;
  #pragma unroll
        for (int i = 0; i < 8; ++i) m2 = amax16x2(m2, w[j][i]);
        amax_b_bits = hmax_of_pair(bf16x2_abs_bits(m2)) << 16;
      }

      // ---- global scale -------------------------------------------------------------------------------------
      float Sg;
      if (GS == kGsBlock128) {
        uint32_t g = amax_b_bits;
        g = max(g, __shfl_xor_sync(0xFFFFFFFFu, g, 1));
        g = max(g, __shfl_xor_sync(0xFFFFFFFFu, g, 2));
        g = max(g, __shfl_xor_sync(0xFFFFFFFFu, g, 4));
        Sg = global_scale_from_amax(__uint_as_float(g));
        if (active && (b & 7) == 0) gscale[(size_t)r * (uint32_t)(Kp >> 7) + (b >> 3)] = Sg;
      } else if (GS == kGsRow) {
        Sg = global_scale_from_amax(__uint_as_float(gs_cells[r]));
        if (active && b == 0) gscale[r] = Sg;
      } else {
        Sg = Sg_t;
      }

      // ---- block scale, rounding, packing -------------------------------------------------------------------
      float rcp;
      const uint32_t sb = block_scale(__uint_as_float(amax_b_bits), Sg, rcp, SR && sb_up);
      if (!RHT) {
  #pragma unroll
        for (int i = 0; i < 8; ++i) {
          x[2 * i] = bf16_lo(w[j][i]);
          x[2 * i + 1] = bf16_hi(w[j][i]);
        }
      }
      const uint2 packed = quantize_block16<SR>(x, rcp, pk, stream_id, ((uint64_t)r * (uint32_t)K16 + k0) >> 3);

      // four neighbouring threads own the four scale bytes of one 32-bit word in either layout
      uint32_t sf4 = sb << (8 * (b & 3));
      sf4 |= __shfl_xor_sync(0xFFFFFFFFu, sf4, 1);
      sf4 |= __shfl_xor_sync(0xFFFFFFFFu, sf4, 2);
      if (active) {
        *reinterpret_cast<uint2*>(codes + (size_t)r * (uint32_t)(Kp >> 1) + (k0 >> 1)) = packed;
        if ((b & 3) == 0) {
          size_t off;
          if (TILED) {
            const uint32_t tile = (r >> 7) * (((nb32 + 15u) & ~15u) >> 2) + (b >> 2);  // 512-byte tiles, k fastest
            off = (size_t)tile * 512u + ((r & 31u) * 16u + ((r >> 5) & 3u) * 4u);       // b & 3 == 0 here
          } else {
            off = (size_t)r * nb32 + b;
          }
          *reinterpret_cast<uint32_t*>(sf + off) = sf4;
        }
      }
    }
  };
  const bool full = !GATHER && K32 == (uint32_t)Kp && (int64_t)blockIdx.x * (256 * NB) + 256 * NB <= total;  // CTA-uniform
  if (full)
    body(std::true_type{});
  else
    body(std::false_type{});
}

// =========================================================================================================
// Row-axis quantize from BF16, four ADJACENT inner blocks per thread (64 consecutive k of one operand row).
// What a thread does once per inner block in the kernel above (row / block index from the flat index, address
// arithmetic, the shuffles that assemble a word of scale bytes and reduce the 128-wide group maximum) it does here once per
// four blocks: the four scale bytes of a thread are one aligned 32-bit word of either scale layout, its codes are 32
// contiguous bytes, a 128-wide outer group is two neighbouring lanes, and the sign bits of the random Hadamard
// transformation for all four blocks come from one generator call. That bookkeeping was about 40 % of the instructions of
// the stochastic-rounding quantizers. Loads are 32 bytes per lane at a 128-byte stride (every sector is used in full; the
// four loads of a warp cover a contiguous 4 KB).
//   RMODE  0 round to nearest, 1 stochastic rounding, 2 stochastic rounding with the block scale rounded up.
// No column list (OutControl's compaction keeps the kernel above).
// =========================================================================================================
template <int GS, int RMODE, bool TILED, bool RHT>
__global__ void __launch_bounds__(256, 3)
quantize_rows4_kernel(const uint16_t* __restrict__ src, int64_t rows, int64_t K, int64_t ld, uint64_t seed, uint32_t stream_id,
                      const uint32_t* __restrict__ gs_cells, uint8_t* __restrict__ codes, uint8_t* __restrict__ sf,
                      float* __restrict__ gscale, uint32_t div_mul, uint32_t div_shift, int wide_loads, uint32_t rht_stream,
                      const __grid_constant__ PhiloxKeys pk) {
  pdl_prologue();
  constexpr bool SR = RMODE != 0;
  const uint32_t K32 = (uint32_t)K;
  const uint32_t Kp = (K32 + 127u) & ~127u;
  const uint32_t K16 = (K32 + 15u) & ~15u;
  const uint32_t nu = Kp >> 6;  // units (four inner blocks) per operand row: even, as rows are padded to 128
  const int64_t total = rows * (int64_t)nu;
  const int64_t unit = (int64_t)blockIdx.x * 256 + threadIdx.x;
  const bool full = K32 == Kp && (int64_t)blockIdx.x * 256 + 256 <= total;  // CTA-uniform: every block exists and is whole

  auto body = [&](auto full_tag) {
    constexpr bool FULL = decltype(full_tag)::value;
    const bool active = FULL || unit < total;
    uint32_t r = 0, q = 0;
    if (active) {
      if (div_mul) {
        const uint32_t n = (uint32_t)unit, t = __umulhi(div_mul, n);
        r = (t + ((n - t) >> 1)) >> div_shift;
        q = n - r * nu;
      } else if (div_shift != 0xFFFFFFFFu) {
        r = (uint32_t)unit >> div_shift;
        q = (uint32_t)unit & (nu - 1u);
      } else {
        r = (uint32_t)(unit / nu);
        q = (uint32_t)(unit - (int64_t)r * nu);
      }
    }
    const uint32_t k0 = q << 6;
    uint32_t w[4][8];
    {
      const uint16_t* p = src + (size_t)r * (uint32_t)ld + k0;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint32_t k = k0 + 16u * j;
#pragma unroll
        for (int i = 0; i < 8; ++i) w[j][i] = 0;
        if (FULL || (active && k + 16u <= K32)) {
          if (wide_loads) {
            asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                         : "=r"(w[j][0]), "=r"(w[j][1]), "=r"(w[j][2]), "=r"(w[j][3]), "=r"(w[j][4]), "=r"(w[j][5]),
                           "=r"(w[j][6]), "=r"(w[j][7])
                         : "l"(p + 16 * j));
          } else {
            const uint4 v0 = *reinterpret_cast<const uint4*>(p + 16 * j);
            const uint4 v1 = *reinterpret_cast<const uint4*>(p + 16 * j + 8);
            w[j][0] = v0.x; w[j][1] = v0.y; w[j][2] = v0.z; w[j][3] = v0.w;
            w[j][4] = v1.x; w[j][5] = v1.y; w[j][6] = v1.z; w[j][7] = v1.w;
          }
        } else if (active && k < K32) {
          for (int i = 0; i < 16; ++i)
            if (k + i < K32) w[j][i >> 1] |= (uint32_t)p[16 * j + i] << (16 * (i & 1));
        }
      }
    }
    // the 64 sign bits of this thread's k range (one half of a 128-group's generator block); none past K rounded up to 16
    uint32_t sgn_lo = 0, sgn_hi = 0;
    if (RHT) {
      const uint4 sw = rht_sign_words(seed, rht_stream, (uint64_t)(k0 >> 7));
      sgn_lo = (k0 & 64u) ? sw.z : sw.x;
      sgn_hi = (k0 & 64u) ? sw.w : sw.y;
    }

    // block maxima (binary32 patterns of non-negative values: integer order = float order)
    uint32_t amax_bits[4];
    float xr[RHT ? 4 : 1][16];  // transformed values (RHT only)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (RHT) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          xr[RHT ? j : 0][2 * i] = bf16_lo(w[j][i]);
          xr[RHT ? j : 0][2 * i + 1] = bf16_hi(w[j][i]);
        }
        const uint32_t s16 = ((j & 2) ? sgn_hi : sgn_lo) >> (16 * (j & 1));
        rht_scale16(xr[RHT ? j : 0], (FULL || k0 + 16u * j < K16) ? (s16 & 0xFFFFu) : 0u);
        hadamard16_butterflies(xr[RHT ? j : 0]);
        float m = 0.0f;
#pragma unroll
        for (int i = 0; i < 16; ++i) m = fmaxf(m, fabsf(xr[RHT ? j : 0][i]));
        amax_bits[j] = __float_as_uint(m);
      } else {
        uint32_t m2 = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) m2 = amax16x2(m2, w[j][i]);
        amax_bits[j] = hmax_of_pair(bf16x2_abs_bits(m2)) << 16;
      }
    }

    float Sg;
    if (GS == kGsBlock128) {
      uint32_t g = max(max(amax_bits[0], amax_bits[1]), max(amax_bits[2], amax_bits[3]));
      g = max(g, __shfl_xor_sync(0xFFFFFFFFu, g, 1));  // the other half of the 128-wide group is the neighbouring lane
      Sg = global_scale_from_amax(__uint_as_float(g));
      if (active && (q & 1u) == 0) gscale[(size_t)r * (Kp >> 7) + (q >> 1)] = Sg;
    } else if (GS == kGsRow) {
      Sg = global_scale_from_amax(__uint_as_float(gs_cells[r]));
      if (active && q == 0) gscale[r] = Sg;
    } else {
      Sg = global_scale_from_amax(__uint_as_float(gs_cells[0]));
      if (unit == 0) gscale[0] = Sg;
    }

    const uint64_t idx8 = ((uint64_t)r * K16 + k0) >> 3;
    uint32_t sf4 = 0;
    uint32_t packed[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float rcp;
      const uint32_t sb = block_scale(__uint_as_float(amax_bits[j]), Sg, rcp, RMODE == 2);
      sf4 |= sb << (8 * j);
      float x[16];
      if (RHT) {
#pragma unroll
        for (int i = 0; i < 16; ++i) x[i] = xr[RHT ? j : 0][i];
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          x[2 * i] = bf16_lo(w[j][i]);
          x[2 * i + 1] = bf16_hi(w[j][i]);
        }
      }
      const uint2 c = quantize_block16<SR>(x, rcp, pk, stream_id, idx8 + 2 * j);
      packed[2 * j] = c.x;
      packed[2 * j + 1] = c.y;
    }
    if (active) {
      uint4* cp = reinterpret_cast<uint4*>(codes + (size_t)r * (Kp >> 1) + (k0 >> 1));
      cp[0] = make_uint4(packed[0], packed[1], packed[2], packed[3]);
      cp[1] = make_uint4(packed[4], packed[5], packed[6], packed[7]);
      const uint32_t nb = Kp >> 4;
      size_t off;
      if (TILED) {
        const uint32_t tile = (r >> 7) * (((nb + 15u) & ~15u) >> 2) + q;  // 512-byte tiles, k fastest; this unit is one of them
        off = (size_t)tile * 512u + ((r & 31u) * 16u + ((r >> 5) & 3u) * 4u);
      } else {
        off = (size_t)r * nb + (q << 2);
      }
      *reinterpret_cast<uint32_t*>(sf + off) = sf4;
    }
  };
  if (full)
    body(std::true_type{});
  else
    body(std::false_type{});
}

// =========================================================================================================
// Transposing quantizers. Operand element (d, k) = source element (row k, column d).
// Tile = 128 k x 64 d. Phase 1 stages the tile as FP32 in shared memory; phase 2 gives each thread one
// (d, 16-k block); phase 3 writes the packed rows back in 16-byte pieces.
//   SRC = 0: BF16 source matrix [rowsK, colsD] (Q5).
//   SRC = 1: forward operand [rowsK, Kin] as codes + scales + global scales, optionally remapped per d and
//            mixed with a BF16 matrix for the rows whose map entry is negative (Q4, Q6 of Sec. 2.3 / 4.2).
// =========================================================================================================
__device__ __forceinline__ float load_aligned_value(const TransposeSrc& s, int64_t k, int64_t j) {
  // x_hat = (P * S_block) * S_global of input operand element (row k, column j): one binary32 rounding.
  const int64_t Kp = (s.in_K + 127) & ~(int64_t)127;
  const uint32_t byte = s.in_codes[k * (Kp >> 1) + (j >> 1)];
  const uint32_t code = (byte >> (4 * (j & 1))) & 15u;
  const int64_t nb = Kp >> 4;
  const size_t sfo = s.in_sf_tiled ? sf_tiled_offset(k, j >> 4, (nb + 15) & ~(int64_t)15) : (size_t)(k * nb + (j >> 4));
  const float sbf = e4m3_decode(s.in_sf[sfo]);
  const float sg = s.in_gs_mode == kGsTensor ? s.in_gscale[0]
                   : s.in_gs_mode == kGsRow  ? s.in_gscale[k]
                                             : s.in_gscale[k * (Kp >> 7) + (j >> 7)];
  return __fmul_rn(__fmul_rn(e2m1_decode(code), sbf), sg);
}

template <int SRC>
__device__ __forceinline__ float load_transpose_elem(const TransposeSrc& s, int64_t k, int64_t d) {
  if (SRC == 0) return bf16_bits_to_float(s.bf16[k * s.ld + d]);
  int64_t j = d;
  if (s.row_map) {
    const int32_t mj = s.row_map[d];
    if (mj < 0) return bf16_bits_to_float(s.hp[k * s.hp_ld + d]);
    j = mj;
  }
  return load_aligned_value(s, k, j);
}

// Column amax of a transposing quantizer's source: per source column (ROW scale mode: operand row = column) or
// folded into one cell. `only_hp` restricts the pass to the columns whose row-map entry is negative (the BF16 rows
// that OutControl mixes into W-hat). 64 columns x 256 rows per CTA, reduced in the CTA before any atomic.
template <int SRC>
__global__ void __launch_bounds__(256) amax_cols_generic_kernel(TransposeSrc s, int64_t rowsK, int64_t D,
                                                               uint32_t* cells, int per_column, int only_hp) {
  pdl_prologue();
  __shared__ float red[4][64];
  __shared__ float fin[2];
  const int dl = threadIdx.x & 63, g = threadIdx.x >> 6;
  const int64_t d = (int64_t)blockIdx.x * 64 + dl;
  const int64_t r0 = (int64_t)blockIdx.y * 256;
  float m = 0.0f;
  if (d < D && !(only_hp && s.row_map[d] >= 0))
    for (int64_t k = r0 + g; k < min(r0 + 256, rowsK); k += 4) m = fmaxf(m, fabsf(load_transpose_elem<SRC>(s, k, d)));
  red[g][dl] = m;
  __syncthreads();
  if (g == 0) {
    m = fmaxf(fmaxf(red[0][dl], red[1][dl]), fmaxf(red[2][dl], red[3][dl]));
    if (per_column) {
      if (d < D && m > 0.0f) atomicMax(cells + (s.out_rows ? (int64_t)s.out_rows[d] : d), __float_as_uint(m));
    } else {
#pragma unroll
      for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
      if ((threadIdx.x & 31) == 0) fin[threadIdx.x >> 5] = m;
    }
  }
  if (!per_column) {
    __syncthreads();
    if (threadIdx.x == 0) {
      m = fmaxf(fin[0], fin[1]);
      if (m > 0.0f) atomicMax(cells, __float_as_uint(m));
    }
  }
}

//   RHT        the 16-blocks along k are replaced by (x S) H_16: the sign and the 1/4 are applied while staging (one
//              factor per source row), the butterflies on the 16 values a thread reads back.
//   AMAX_ONLY  stop after the block maxima and fold them into the amax cells (pre-pass for TENSOR / ROW under RHT;
//              gs_cells is then written, and codes / sf / gscale are not touched).
template <int SRC, int GS, bool SR, bool TILED, bool RHT, bool AMAX_ONLY>
__global__ void __launch_bounds__(256)
quantize_transpose_generic_kernel(TransposeSrc s, int64_t rowsK, int64_t D, uint64_t seed, uint32_t stream_id,
                          uint32_t* __restrict__ gs_cells, int tensor_closed_form, uint8_t* __restrict__ codes,
                          uint8_t* __restrict__ sf, float* __restrict__ gscale, uint32_t rht_stream, int sb_up,
                          const __grid_constant__ PhiloxKeys pk) {
  pdl_prologue();
  __shared__ float tile[128][65];
  __shared__ float blk_amax[8][64];
  __shared__ __align__(16) uint8_t out_codes[64][64];
  const int64_t K = rowsK;  // operand K
  const int64_t Kp = (K + 127) & ~(int64_t)127;
  const int64_t nb = Kp >> 4;
  const int64_t k_base = (int64_t)blockIdx.x * 128;
  const int64_t d_base = (int64_t)blockIdx.y * 64;
  const int tid = threadIdx.x;
  uint4 sw = make_uint4(0, 0, 0, 0);  // the tile's 128 sign bits (k_base is a multiple of 128)
  if (RHT) {
    sw = rht_sign_words(seed, rht_stream, (uint64_t)blockIdx.x);
    // rows past K rounded up to 16 are layout padding: no signs there, so that they stay +0 and encode as zero bytes
    const int64_t live = ((rowsK + 15) & ~(int64_t)15) - k_base;
    if (live < 128) {
      const uint32_t n = live > 0 ? (uint32_t)live : 0u;
      sw.x &= n >= 32 ? 0xFFFFFFFFu : (1u << n) - 1u;
      sw.y &= n >= 64 ? 0xFFFFFFFFu : n > 32 ? (1u << (n - 32)) - 1u : 0u;
      sw.z &= n >= 96 ? 0xFFFFFFFFu : n > 64 ? (1u << (n - 64)) - 1u : 0u;
      sw.w &= n > 96 ? (1u << (n - 96)) - 1u : 0u;
    }
  }

  // ---- phase 1: stage (zero outside the matrix) ------------------------------------------------------------
  if (SRC == 0 && (s.ld & 7) == 0) {
    // 128 rows x 8 chunks of 8 BF16; the one chunk that straddles D (ragged last column tile) is read element by element
    for (int c = tid; c < 1024; c += 256) {
      const int kr = c >> 3, dc = (c & 7) << 3;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (k_base + kr < rowsK) {
        const uint16_t* src = s.bf16 + (k_base + kr) * s.ld + d_base + dc;
        if (d_base + dc + 8 <= D) {
          v = *reinterpret_cast<const uint4*>(src);
        } else if (d_base + dc < D) {
          uint32_t w[4] = {0, 0, 0, 0};
          const int n = (int)(D - d_base - dc);
          for (int i = 0; i < n; ++i) w[i >> 1] |= (uint32_t)src[i] << (16 * (i & 1));
          v = make_uint4(w[0], w[1], w[2], w[3]);
        }
      }
      float f8[8] = {bf16_lo(v.x), bf16_hi(v.x), bf16_lo(v.y), bf16_hi(v.y), bf16_lo(v.z), bf16_hi(v.z), bf16_lo(v.w), bf16_hi(v.w)};
      if (RHT) {
        const float f = rht_factor(sw, (uint32_t)kr);
#pragma unroll
        for (int i = 0; i < 8; ++i) f8[i] = __fmul_rn(f8[i], f);
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) tile[kr][dc + i] = f8[i];
    }
  } else if (SRC == 1 && !s.row_map) {
    // forward operand without a row map: 32 codes (16 bytes) and their two scale bytes per thread. A tile that sticks out
    // past D still lies inside the operand's row (K is padded to 128 there, with zero codes and zero scales), so the last
    // column tile is staged the same way and the columns past D simply hold zeros that nobody stores.
    const int kr = tid >> 1, half = tid & 1;
    const int64_t k = k_base + kr;
    float v[32];
    if (k < rowsK) {
      const int64_t in_Kp = (s.in_K + 127) & ~(int64_t)127;
      const int64_t in_nb = in_Kp >> 4;
      const uint4 c4 = *reinterpret_cast<const uint4*>(s.in_codes + k * (in_Kp >> 1) + (d_base >> 1) + half * 16);
      const int64_t kb = (d_base >> 4) + half * 2;
      const size_t sfo = s.in_sf_tiled ? sf_tiled_offset(k, kb, (in_nb + 15) & ~(int64_t)15) : (size_t)(k * in_nb + kb);
      const uint32_t sf2 = *reinterpret_cast<const uint16_t*>(s.in_sf + sfo);
      const float sg = s.in_gs_mode == kGsTensor ? s.in_gscale[0]
                       : s.in_gs_mode == kGsRow  ? s.in_gscale[k]
                                                 : s.in_gscale[k * (in_Kp >> 7) + (d_base >> 7)];
      decode8(c4.x, sf2 & 0xFFu, sg, v);
      decode8(c4.y, sf2 & 0xFFu, sg, v + 8);
      decode8(c4.z, sf2 >> 8, sg, v + 16);
      decode8(c4.w, sf2 >> 8, sg, v + 24);
    } else {
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] = 0.0f;
    }
    if (RHT) {
      const float f = rht_factor(sw, (uint32_t)kr);
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] = __fmul_rn(v[i], f);
    }
#pragma unroll
    for (int i = 0; i < 32; ++i) tile[kr][half * 32 + i] = v[i];
  } else {
    for (int e = tid; e < 128 * 64; e += 256) {
      const int kr = e >> 6, dl = e & 63;
      const int64_t k = k_base + kr, d = d_base + dl;
      float v = (k < rowsK && d < D) ? load_transpose_elem<SRC>(s, k, d) : 0.0f;
      if (RHT) v = __fmul_rn(v, rht_factor(sw, (uint32_t)kr));
      tile[kr][dl] = v;
    }
  }
  __syncthreads();

  // ---- phase 2: two (d, k-block) items per thread -----------------------------------------------------------
  const int dl = tid & 63;
  const int64_t d = d_base + dl;
  // operand row produced by source column d (identity unless the caller scatters rows, as OutControl's W-hat does)
  const int64_t o = (d < D && s.out_rows) ? (int64_t)s.out_rows[d] : d;
  float xs[2][16];
  float am[2];
#pragma unroll
  for (int it = 0; it < 2; ++it) {
    const int kb = (tid >> 6) + 4 * it;  // 0..7
#pragma unroll
    for (int i = 0; i < 16; ++i) xs[it][i] = tile[kb * 16 + i][dl];
    if (RHT) hadamard16_butterflies(xs[it]);
    float m = 0.0f;
#pragma unroll
    for (int i = 0; i < 16; ++i) m = fmaxf(m, fabsf(xs[it][i]));
    am[it] = m;
    if (GS == kGsBlock128) blk_amax[kb][dl] = m;
  }
  if (AMAX_ONLY) {
    float m = fmaxf(am[0], am[1]);
    if (GS == kGsRow) {  // one cell per operand row
      blk_amax[tid >> 6][dl] = m;
      __syncthreads();
      if (tid < 64 && d < D) {
        m = fmaxf(fmaxf(blk_amax[0][dl], blk_amax[1][dl]), fmaxf(blk_amax[2][dl], blk_amax[3][dl]));
        if (m > 0.0f) atomicMax(gs_cells + o, __float_as_uint(m));
      }
    } else {
#pragma unroll
      for (int q = 16; q; q >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, q));
      if ((tid & 31) == 0) blk_amax[0][tid >> 5] = m;
      __syncthreads();
      if (tid == 0) {
        for (int q = 1; q < 8; ++q) m = fmaxf(m, blk_amax[0][q]);
        if (m > 0.0f) atomicMax(gs_cells, __float_as_uint(m));
      }
    }
    return;
  }
  float Sg;
  if (GS == kGsBlock128) {
    __syncthreads();
    float g = 0.0f;
#pragma unroll
    for (int j = 0; j < 8; ++j) g = fmaxf(g, blk_amax[j][dl]);
    Sg = global_scale_from_amax(g);
    if (d < D && tid < 64 && k_base < K) gscale[o * (Kp >> 7) + blockIdx.x] = Sg;
  } else if (GS == kGsRow) {
    Sg = global_scale_from_amax(d < D ? __uint_as_float(gs_cells[o]) : 0.0f);
    if (d < D && tid < 64 && blockIdx.x == 0) gscale[o] = Sg;
  } else {
    // (tensor_closed_form == 2: the cell carries nothing and may be uninitialised)
    float amax = tensor_closed_form == 2 ? 0.0f : __uint_as_float(gs_cells[0]);
    // TENSOR -> TENSOR re-quantization: the aligned tensor's maximum is float32(2688 * S_global) of the forward
    // operand (its largest block has scale 448 and a magnitude-6 element); gs_cells[0] then only covers BF16 rows.
    if (SRC == 1 && tensor_closed_form) amax = fmaxf(amax, __fmul_rn(2688.0f, s.in_gscale[0]));
    if (s.closed_form_sg) amax = fmaxf(amax, __fmul_rn(2688.0f, s.closed_form_sg[0]));
    Sg = global_scale_from_amax(amax);
    if (blockIdx.x == 0 && blockIdx.y == 0 && tid == 0) gscale[0] = Sg;
  }
  const int64_t K16 = (K + 15) & ~(int64_t)15;
#pragma unroll
  for (int it = 0; it < 2; ++it) {
    const int kb = (tid >> 6) + 4 * it;
    float rcp;
    const uint32_t sb = block_scale(am[it], Sg, rcp, SR && sb_up);
    const int64_t k0 = k_base + kb * 16;
    const uint2 packed = quantize_block16<SR>(xs[it], rcp, pk, stream_id, (uint64_t)((o * K16 + k0) >> 3));
    *reinterpret_cast<uint2*>(&out_codes[dl][kb * 8]) = packed;
    if (d < D && k0 < Kp) {
      const int64_t b = k0 >> 4;
      const size_t off = TILED ? sf_tiled_offset(o, b, (nb + 15) & ~(int64_t)15) : (size_t)(o * nb + b);
      sf[off] = (uint8_t)sb;
    }
  }
  __syncthreads();

  // ---- phase 3: 64 rows x 64 bytes, 16 bytes per thread ------------------------------------------------------
  {
    const int row = tid >> 2, piece = tid & 3;
    const int64_t dd = d_base + row;
    const int64_t oo = (dd < D && s.out_rows) ? (int64_t)s.out_rows[dd] : dd;
    if (dd < D && k_base + piece * 32 < Kp)
      *reinterpret_cast<uint4*>(codes + oo * (Kp >> 1) + (k_base >> 1) + piece * 16) =
          *reinterpret_cast<const uint4*>(&out_codes[row][piece * 16]);
  }
}

// =========================================================================================================
// Transposing quantizers, fast path (no per-column remapping of the source). The 128 k x 64 d tile is staged as 16-bit
// values: the BF16 source as it is (SRC = 0), or P * S_block of the forward operand as FP16 (SRC = 1, exact; the FP32
// global scale of the source row is applied after the transposition, which is the same single rounding
// x_hat = (P * S_block) * S_global). A tile row is 128 bytes; its 16-byte chunks are XOR-swizzled with the row number so that
// both the row-wise 16-byte stores of the staging phase and the column-wise 4-byte reads of the quantizing phase are free of
// bank conflicts. Each thread then owns TWO neighbouring operand rows (one 32-bit word per k holds both values) and one
// 16-k block of each: half the shared-memory loads, packed maxima for BF16 sources, and all bookkeeping once per two blocks.
// Codes and scale bytes are collected in shared memory and written as 16-byte / 4-byte pieces.
//   RMODE  0 round to nearest, 1 stochastic rounding, 2 stochastic rounding with the block scale rounded up.
// =========================================================================================================
template <int SRC, int GS, int RMODE, bool TILED, bool RHT, bool AMAX_ONLY>
__global__ void __launch_bounds__(256, 3)
quantize_transpose_kernel(TransposeSrc s, int64_t rowsK, int64_t D, uint64_t seed, uint32_t stream_id,
                          uint32_t* __restrict__ gs_cells, int tensor_closed_form, uint8_t* __restrict__ codes,
                          uint8_t* __restrict__ sf, float* __restrict__ gscale, uint32_t rht_stream,
                          const __grid_constant__ PhiloxKeys pk) {
  pdl_prologue();
  constexpr bool SR = RMODE != 0;
  __shared__ __align__(16) uint32_t tile[128 * 32];
  __shared__ float sg_row[128];
  __shared__ float blk_amax[8][64];
  __shared__ __align__(16) uint8_t out_codes[64][80];  // 64 code bytes per operand row (+16: spreads the rows over the banks)
  __shared__ __align__(4) uint8_t out_sf[64][8];
  // Sizes and indices are below 2^31 (checked by the launcher): 32-bit arithmetic throughout, 64 bits only where a byte
  // offset is formed (one widening multiply each).
  const uint32_t K = (uint32_t)rowsK;  // operand K
  const uint32_t D32 = (uint32_t)D;
  const uint32_t Kp = (K + 127u) & ~127u;
  const uint32_t nb = Kp >> 4;
  const uint32_t nbp4 = ((nb + 15u) & ~15u) >> 2;  // 512-byte scale tiles per 128-row tile of the output operand
  const uint32_t k_base = blockIdx.x * 128u;
  const uint32_t d_base = blockIdx.y * 64u;
  const int tid = threadIdx.x;
  uint4 sw = make_uint4(0, 0, 0, 0);  // the tile's 128 sign bits (k_base is a multiple of 128)
  if (RHT) {
    sw = rht_sign_words(seed, rht_stream, (uint64_t)blockIdx.x);
    // rows past K rounded up to 16 are layout padding: no signs there, so that they stay +0 and encode as zero bytes
    const int32_t live = (int32_t)((K + 15u) & ~15u) - (int32_t)k_base;
    if (live < 128) {
      const uint32_t n = live > 0 ? (uint32_t)live : 0u;
      sw.x &= n >= 32 ? 0xFFFFFFFFu : (1u << n) - 1u;
      sw.y &= n >= 64 ? 0xFFFFFFFFu : n > 32 ? (1u << (n - 32)) - 1u : 0u;
      sw.z &= n >= 96 ? 0xFFFFFFFFu : n > 64 ? (1u << (n - 64)) - 1u : 0u;
      sw.w &= n > 96 ? (1u << (n - 96)) - 1u : 0u;
    }
  }

  // ---- phase 1: stage (zero outside the matrix) ------------------------------------------------------------
  if (SRC == 0) {
    // 128 rows x 8 chunks of 8 BF16, four chunks per thread, all loads first; the chunk that straddles D is read by element
    uint4 v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t c = tid + 256 * i, kr = c >> 3, dc = (c & 7) << 3;
      v[i] = make_uint4(0, 0, 0, 0);
      if (k_base + kr < K) {
        const uint16_t* src = s.bf16 + (size_t)(k_base + kr) * (uint32_t)s.ld + (d_base + dc);
        if (d_base + dc + 8 <= D32) {
          v[i] = *reinterpret_cast<const uint4*>(src);
        } else if (d_base + dc < D32) {
          uint32_t t[4] = {0, 0, 0, 0};
          const int n = (int)(D32 - d_base - dc);
          for (int e = 0; e < n; ++e) t[e >> 1] |= (uint32_t)src[e] << (16 * (e & 1));
          v[i] = make_uint4(t[0], t[1], t[2], t[3]);
        }
      }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int c = tid + 256 * i, kr = c >> 3, ch = c & 7;
      *reinterpret_cast<uint4*>(&tile[kr * 32 + ((ch ^ (kr & 7)) << 2)]) = v[i];
    }
  } else {
    // forward operand: 32 codes (16 bytes) and their two scale bytes per thread. A tile that sticks out past D still lies
    // inside the operand's row (K is padded to 128 there, with zero codes and zero scales): the columns past D hold zeros
    // that nobody stores.
    const int kr = tid >> 1, half = tid & 1;
    const uint32_t k = k_base + kr;
    uint32_t h[4][4];
    float sg = 0.0f;
    if (k < K) {
      const uint32_t in_Kp = ((uint32_t)s.in_K + 127u) & ~127u;
      const uint32_t in_nb = in_Kp >> 4;
      const uint4 c4 = *reinterpret_cast<const uint4*>(s.in_codes + (size_t)k * (in_Kp >> 1) + ((d_base >> 1) + half * 16));
      const uint32_t kb = (d_base >> 4) + half * 2;
      const size_t sfo = s.in_sf_tiled ? (size_t)((k >> 7) * (((in_nb + 15u) & ~15u) >> 2) + (kb >> 2)) * 512u +
                                             ((k & 31u) * 16u + ((k >> 5) & 3u) * 4u + (kb & 3u))
                                       : (size_t)k * in_nb + kb;
      const uint32_t sf2 = *reinterpret_cast<const uint16_t*>(s.in_sf + sfo);
      sg = s.in_gs_mode == kGsTensor ? s.in_gscale[0]
           : s.in_gs_mode == kGsRow  ? s.in_gscale[k]
                                     : s.in_gscale[(size_t)k * (in_Kp >> 7) + (d_base >> 7)];
      decode8_h2(c4.x, sf2 & 0xFFu, h[0]);
      decode8_h2(c4.y, sf2 & 0xFFu, h[1]);
      decode8_h2(c4.z, sf2 >> 8, h[2]);
      decode8_h2(c4.w, sf2 >> 8, h[3]);
    } else {
#pragma unroll
      for (int w = 0; w < 4; ++w)
#pragma unroll
        for (int i = 0; i < 4; ++i) h[w][i] = 0u;
    }
    if (half == 0) sg_row[kr] = sg;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const int ch = half * 4 + w;
      *reinterpret_cast<uint4*>(&tile[kr * 32 + ((ch ^ (kr & 7)) << 2)]) = make_uint4(h[w][0], h[w][1], h[w][2], h[w][3]);
    }
  }
  __syncthreads();

  // ---- phase 2: per thread two neighbouring operand rows (d, d + 1), one 16-k block of each ------------------
  const int dp = tid & 31, kb = tid >> 5;
  uint32_t hw[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) hw[i] = tile[(kb * 16 + i) * 32 + ((((dp >> 2) ^ (i & 7)) << 2) | (dp & 3))];  // row & 7 = i & 7
  const uint32_t s16 = RHT ? ((rht_pick_word(sw, (uint32_t)kb >> 1) >> (16 * (kb & 1))) & 0xFFFFu) : 0u;
  float xs[2][16];
  float am[2];
  if (SRC == 0 && !RHT) {
    // block maxima of both rows at once on the packed pairs; the values are expanded further down, one row at a time
    uint32_t m2 = 0;
#pragma unroll
    for (int i = 0; i < 16; ++i) m2 = amax16x2(m2, hw[i]);
    m2 = bf16x2_abs_bits(m2);
    am[0] = __uint_as_float(m2 << 16);
    am[1] = __uint_as_float(m2 & 0xFFFF0000u);
  } else {
    const bool uniform_sg = SRC == 1 && s.in_gs_mode == kGsTensor;
    const float sg_t = uniform_sg ? s.in_gscale[0] : 1.0f;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      if (SRC == 0) {
        xs[0][i] = bf16_lo(hw[i]);
        xs[1][i] = bf16_hi(hw[i]);
      } else {
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&hw[i]));
        const float sgk = uniform_sg ? sg_t : sg_row[kb * 16 + i];
        xs[0][i] = __fmul_rn(f.x, sgk);
        xs[1][i] = __fmul_rn(f.y, sgk);
      }
    }
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      if (RHT) {
        rht_scale16(xs[c], s16);
        hadamard16_butterflies(xs[c]);
      }
      float m = 0.0f;
#pragma unroll
      for (int i = 0; i < 16; ++i) m = fmaxf(m, fabsf(xs[c][i]));
      am[c] = m;
    }
  }
  const uint32_t d0 = d_base + 2 * dp;
  // operand rows produced by source columns d0, d0 + 1 (identity unless the caller scatters rows, as OutControl's W-hat does)
  uint32_t o[2];
#pragma unroll
  for (int c = 0; c < 2; ++c) o[c] = (d0 + c < D32 && s.out_rows) ? (uint32_t)s.out_rows[d0 + c] : d0 + c;
  if (GS == kGsBlock128 || (AMAX_ONLY && GS == kGsRow)) {
    blk_amax[kb][2 * dp] = am[0];
    blk_amax[kb][2 * dp + 1] = am[1];
  }
  if (AMAX_ONLY) {
    if (GS == kGsRow) {  // one cell per operand row
      __syncthreads();
      if (tid < 64 && d_base + tid < D32) {
        float m = 0.0f;
#pragma unroll
        for (int j = 0; j < 8; ++j) m = fmaxf(m, blk_amax[j][tid]);
        const uint32_t oo = s.out_rows ? (uint32_t)s.out_rows[d_base + tid] : d_base + tid;
        if (m > 0.0f) atomicMax(gs_cells + oo, __float_as_uint(m));
      }
    } else {
      float m = fmaxf(am[0], am[1]);
#pragma unroll
      for (int q = 16; q; q >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, q));
      if ((tid & 31) == 0) blk_amax[0][tid >> 5] = m;
      __syncthreads();
      if (tid == 0) {
        for (int q = 1; q < 8; ++q) m = fmaxf(m, blk_amax[0][q]);
        if (m > 0.0f) atomicMax(gs_cells, __float_as_uint(m));
      }
    }
    return;
  }
  float Sg[2];
  if (GS == kGsBlock128) {
    __syncthreads();
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      float g = 0.0f;
#pragma unroll
      for (int j = 0; j < 8; ++j) g = fmaxf(g, blk_amax[j][2 * dp + c]);
      Sg[c] = global_scale_from_amax(g);
      if (d0 + c < D32 && kb == 0 && k_base < K) gscale[(size_t)o[c] * (Kp >> 7) + blockIdx.x] = Sg[c];
    }
  } else if (GS == kGsRow) {
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      Sg[c] = global_scale_from_amax(d0 + c < D32 ? __uint_as_float(gs_cells[o[c]]) : 0.0f);
      if (d0 + c < D32 && kb == 0 && blockIdx.x == 0) gscale[o[c]] = Sg[c];
    }
  } else {
    // (tensor_closed_form == 2: the cell carries nothing and may be uninitialised)
    float amax = tensor_closed_form == 2 ? 0.0f : __uint_as_float(gs_cells[0]);
    // TENSOR -> TENSOR re-quantization: the aligned tensor's maximum is float32(2688 * S_global) of the forward
    // operand (its largest block has scale 448 and a magnitude-6 element); gs_cells[0] then only covers BF16 rows.
    if (SRC == 1 && tensor_closed_form) amax = fmaxf(amax, __fmul_rn(2688.0f, s.in_gscale[0]));
    if (s.closed_form_sg) amax = fmaxf(amax, __fmul_rn(2688.0f, s.closed_form_sg[0]));
    Sg[0] = Sg[1] = global_scale_from_amax(amax);
    if (blockIdx.x == 0 && blockIdx.y == 0 && tid == 0) gscale[0] = Sg[0];
  }
  const uint32_t K16 = (K + 15u) & ~15u;
  const uint32_t k0 = k_base + kb * 16u;
#pragma unroll
  for (int c = 0; c < 2; ++c) {
    float rcp;
    const uint32_t sb = block_scale(am[c], Sg[c], rcp, RMODE == 2);
    if (SRC == 0 && !RHT) {
#pragma unroll
      for (int i = 0; i < 16; ++i) xs[c][i] = c ? bf16_hi(hw[i]) : bf16_lo(hw[i]);
    }
    const uint2 packed = quantize_block16<SR>(xs[c], rcp, pk, stream_id, ((uint64_t)o[c] * K16 + k0) >> 3);
    *reinterpret_cast<uint2*>(&out_codes[2 * dp + c][kb * 8]) = packed;
    out_sf[2 * dp + c][kb] = (uint8_t)sb;
  }
  __syncthreads();

  // ---- phase 3: 64 rows x 64 code bytes, 16 bytes per thread; 64 rows x 8 scale bytes, 4 bytes per thread -----
  {
    const int row = tid >> 2, piece = tid & 3;
    const uint32_t dd = d_base + row;
    if (dd < D32) {
      const uint32_t oo = s.out_rows ? (uint32_t)s.out_rows[dd] : dd;
      *reinterpret_cast<uint4*>(codes + (size_t)oo * (Kp >> 1) + ((k_base >> 1) + piece * 16)) =
          *reinterpret_cast<const uint4*>(&out_codes[row][piece * 16]);
      if (piece < 2) {  // scale bytes of k blocks 4 * piece .. 4 * piece + 3 of this tile: one aligned word in either layout
        const uint32_t b = (k_base >> 4) + 4 * piece;
        const size_t off = TILED ? (size_t)((oo >> 7) * nbp4 + (b >> 2)) * 512u + ((oo & 31u) * 16u + ((oo >> 5) & 3u) * 4u)
                                 : (size_t)oo * nb + b;
        *reinterpret_cast<uint32_t*>(sf + off) = *reinterpret_cast<const uint32_t*>(&out_sf[row][4 * piece]);
      }
    }
  }
}

// =========================================================================================================
// Column-axis quantize from BF16 without a shared-memory transposition (Q5 of Sec. 2.3: the operand is dY^T, its blocks
// run along the tokens), for the TENSOR and ROW scale modes. A lane owns FOUR neighbouring source columns (= operand rows)
// and 64 consecutive source rows (= operand k). It reads 8 bytes per source row, so one warp instruction covers two source
// rows of 128 contiguous bytes (lanes 0..15: rows k .. , lanes 16..31: rows k + 64 ..), and the 16 values of an inner block
// are the same half of 16 loaded words: the transposition is the choice of that half. Per 16 source rows the lane quantizes
// four blocks (one per column) and stores 8 code bytes to each of its four operand rows; the four scale bytes of an operand
// row (64 k) are one aligned word of either scale layout. No barrier, no shared memory, and the index arithmetic is paid
// once per 256 elements.
//   RMODE      0 round to nearest, 1 stochastic rounding, 2 stochastic rounding with the block scale rounded up.
//   RHT        every block is replaced by (x S) H_16 first (Sec. 4.1): the lane's 64 sign bits are half of one generator
//              block, the butterflies run on the 16 values it holds anyway.
//   AMAX_ONLY  the pre-pass of RHT: only the maximum of the transformed values, folded into gs_cells (one cell, or one per
//              operand row in ROW mode); nothing else is written.
// Preconditions (the launcher falls back to the staged kernel otherwise): D and ld multiples of 4, src 8-byte aligned,
// identity row order.
// =========================================================================================================
__device__ __forceinline__ uint2 ld_nc_8(const uint16_t* p) {
  uint2 v;
  asm volatile("ld.global.nc.v2.b32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
  return v;
}

template <int GS, int RMODE, bool TILED, bool RHT, bool AMAX_ONLY>
__global__ void __launch_bounds__(128, 4)
quantize_cols4_kernel(const uint16_t* __restrict__ src, uint32_t K, uint32_t D, uint32_t ld, uint64_t seed, uint32_t stream_id,
                      uint32_t rht_stream, uint32_t* __restrict__ gs_cells, uint8_t* __restrict__ codes, uint8_t* __restrict__ sf,
                      float* __restrict__ gscale, const __grid_constant__ PhiloxKeys pk) {
  static_assert(GS != kGsBlock128, "the outer-block mode has a kernel of its own");
  pdl_prologue();
  constexpr bool SR = RMODE != 0;
  const uint32_t Kp = (K + 127u) & ~127u;
  const uint32_t K16 = (K + 15u) & ~15u;
  const uint32_t nb = Kp >> 4;
  const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
  const uint32_t d0 = blockIdx.y * 64u + (lane & 15u) * 4u;                          // first of this lane's operand rows
  const uint32_t k_start = blockIdx.x * 512u + warp * 128u + (lane >> 4) * 64u;      // first of its 64 k
  const bool live = d0 < D && k_start < Kp;  // (all four rows exist or none: D is a multiple of 4)
  const uint16_t* p = src + (size_t)k_start * ld + d0;

  float Sg[4] = {1.0f, 1.0f, 1.0f, 1.0f};
  if (!AMAX_ONLY) {
    if (GS == kGsRow) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        Sg[c] = global_scale_from_amax(live ? __uint_as_float(gs_cells[d0 + c]) : 0.0f);
        if (live && k_start == 0) gscale[d0 + c] = Sg[c];
      }
    } else {
      Sg[0] = Sg[1] = Sg[2] = Sg[3] = global_scale_from_amax(__uint_as_float(gs_cells[0]));
      if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) gscale[0] = Sg[0];
    }
  }
  // the 64 sign bits of this lane's k range (one half of a 128-group's generator block)
  uint32_t sgn_lo = 0, sgn_hi = 0;
  if (RHT && live) {
    const uint4 sw = rht_sign_words(seed, rht_stream, (uint64_t)(k_start >> 7));
    sgn_lo = (k_start & 64u) ? sw.z : sw.x;
    sgn_hi = (k_start & 64u) ? sw.w : sw.y;
  }
  float am_run[4] = {0.0f, 0.0f, 0.0f, 0.0f};  // AMAX_ONLY: running maxima of the four operand rows

  uint32_t sfw[4] = {0u, 0u, 0u, 0u};
  if (live) {
#pragma unroll 1
    for (uint32_t tb = 0; tb < 4; ++tb) {
      const uint32_t k0 = k_start + 16u * tb;
      if (AMAX_ONLY && k0 >= K16) break;  // layout padding: zeros
      uint2 w[16];
      if (k0 + 16u <= K) {
#pragma unroll
        for (int t = 0; t < 16; ++t) w[t] = ld_nc_8(p + (size_t)(16u * tb + t) * ld);
      } else {
#pragma unroll
        for (int t = 0; t < 16; ++t) w[t] = k0 + t < K ? ld_nc_8(p + (size_t)(16u * tb + t) * ld) : make_uint2(0u, 0u);
      }
      float am[4];
      if (!RHT) {
        uint32_t mx = 0, my = 0;
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          mx = amax16x2(mx, w[t].x);
          my = amax16x2(my, w[t].y);
        }
        mx = bf16x2_abs_bits(mx);
        my = bf16x2_abs_bits(my);
        am[0] = __uint_as_float(mx << 16);
        am[1] = __uint_as_float(mx & 0xFFFF0000u);
        am[2] = __uint_as_float(my << 16);
        am[3] = __uint_as_float(my & 0xFFFF0000u);
      }
      // signs of rows k0 .. k0 + 15; rows past K rounded up to 16 are layout padding and take none (they stay +0)
      const uint32_t s16 = RHT && k0 < K16 ? ((((tb & 2u) ? sgn_hi : sgn_lo) >> (16u * (tb & 1u))) & 0xFFFFu) : 0u;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        float x[16];
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          const uint32_t word = c < 2 ? w[t].x : w[t].y;
          x[t] = (c & 1) ? bf16_hi(word) : bf16_lo(word);
        }
        if (RHT) {
          rht_scale16(x, s16);
          hadamard16_butterflies(x);
          float m = 0.0f;
#pragma unroll
          for (int t = 0; t < 16; ++t) m = fmaxf(m, fabsf(x[t]));
          am[c] = m;
        }
        if (AMAX_ONLY) {
          am_run[c] = fmaxf(am_run[c], am[c]);
        } else {
          float rcp;
          const uint32_t sb = block_scale(am[c], Sg[c], rcp, RMODE == 2);
          sfw[c] |= sb << (8u * tb);
          const uint2 packed = quantize_block16<SR>(x, rcp, pk, stream_id, ((uint64_t)(d0 + c) * K16 + k0) >> 3);
          *reinterpret_cast<uint2*>(codes + (size_t)(d0 + c) * (Kp >> 1) + (k0 >> 1)) = packed;
        }
      }
    }
  }
  if (AMAX_ONLY) {
    if (GS == kGsRow) {  // one cell per operand row; the two lanes that share the rows first combine
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const float m = fmaxf(am_run[c], __shfl_xor_sync(0xFFFFFFFFu, am_run[c], 16));
        if (live && lane < 16 && m > 0.0f) atomicMax(gs_cells + d0 + c, __float_as_uint(m));
      }
    } else {
      float m = fmaxf(fmaxf(am_run[0], am_run[1]), fmaxf(am_run[2], am_run[3]));
#pragma unroll
      for (int q = 16; q; q >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, q));
      if (lane == 0 && m > 0.0f) atomicMax(gs_cells, __float_as_uint(m));
    }
    return;
  }
  if (!live) return;
  const uint32_t b = k_start >> 4;  // first of this lane's four k blocks: a multiple of 4
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const uint32_t o = d0 + c;
    const size_t off = TILED ? (size_t)((o >> 7) * (((nb + 15u) & ~15u) >> 2) + (b >> 2)) * 512u + ((o & 31u) * 16u + ((o >> 5) & 3u) * 4u)
                             : (size_t)o * nb + b;
    *reinterpret_cast<uint32_t*>(sf + off) = sfw[c];
  }
}

// The same for the 1 x 128 outer block (BLOCK128), where the scale of a block depends on all 128 k of its group: a lane owns
// TWO neighbouring source columns and keeps its 64 source rows in registers (one 32-bit word per row), so the data is read
// once; the two lanes of a group exchange the group maximum with one shuffle. A warp instruction covers two source rows of
// 64 contiguous bytes. With RHT the group maximum is that of the transformed values: the eight blocks are transformed once
// for their maxima and once more when they are quantized (80 floating-point operations per block and pass; holding the 128
// transformed values beside the 64 raw words does not fit the register file at a useful occupancy).
template <int RMODE, bool TILED, bool RHT>
__global__ void __launch_bounds__(128, 3)
quantize_cols2_block128_kernel(const uint16_t* __restrict__ src, uint32_t K, uint32_t D, uint32_t ld, uint64_t seed, uint32_t stream_id,
                               uint32_t rht_stream, uint8_t* __restrict__ codes, uint8_t* __restrict__ sf, float* __restrict__ gscale,
                               const __grid_constant__ PhiloxKeys pk) {
  pdl_prologue();
  constexpr bool SR = RMODE != 0;
  const uint32_t Kp = (K + 127u) & ~127u;
  const uint32_t K16 = (K + 15u) & ~15u;
  const uint32_t nb = Kp >> 4;
  const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
  const uint32_t d0 = blockIdx.y * 32u + (lane & 15u) * 2u;
  const uint32_t k_start = blockIdx.x * 512u + warp * 128u + (lane >> 4) * 64u;
  const bool live = d0 < D && k_start < Kp;  // (both rows exist or none: D is even)
  const uint16_t* p = src + (size_t)k_start * ld + d0;

  uint32_t w[64];
  if (live && k_start + 64u <= K) {
#pragma unroll
    for (int t = 0; t < 64; ++t) asm volatile("ld.global.nc.L1::no_allocate.b32 %0, [%1];" : "=r"(w[t]) : "l"(p + (size_t)t * ld));
  } else {
#pragma unroll
    for (int t = 0; t < 64; ++t) {
      w[t] = 0u;
      if (live && k_start + t < K) asm volatile("ld.global.nc.L1::no_allocate.b32 %0, [%1];" : "=r"(w[t]) : "l"(p + (size_t)t * ld));
    }
  }
  // the 64 sign bits of this lane's k range; rows past K rounded up to 16 are layout padding and take none (they stay +0)
  uint32_t sgn[2] = {0u, 0u};
  if (RHT && live) {
    const uint4 sw = rht_sign_words(seed, rht_stream, (uint64_t)(k_start >> 7));
    sgn[0] = (k_start & 64u) ? sw.z : sw.x;
    sgn[1] = (k_start & 64u) ? sw.w : sw.y;
  }
  auto sign16 = [&](int tb) -> uint32_t { return k_start + 16u * tb < K16 ? ((sgn[tb >> 1] >> (16 * (tb & 1))) & 0xFFFFu) : 0u; };

  float Sg[2];
  float bam[RHT ? 4 : 1][2];  // RHT: block maxima of the transformed values
  uint32_t bm[4];             // otherwise: packed block maxima (sign bits meaningless until masked)
  if (RHT) {
    float g0 = 0.0f, g1 = 0.0f;
#pragma unroll
    for (int tb = 0; tb < 4; ++tb) {
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        float x[16];
#pragma unroll
        for (int t = 0; t < 16; ++t) x[t] = c ? bf16_hi(w[16 * tb + t]) : bf16_lo(w[16 * tb + t]);
        rht_scale16(x, sign16(tb));
        hadamard16_butterflies(x);
        float m = 0.0f;
#pragma unroll
        for (int t = 0; t < 16; ++t) m = fmaxf(m, fabsf(x[t]));
        bam[RHT ? tb : 0][c] = m;
        if (c) g1 = fmaxf(g1, m); else g0 = fmaxf(g0, m);
      }
    }
    g0 = fmaxf(g0, __shfl_xor_sync(0xFFFFFFFFu, g0, 16));  // the other half of the 128-wide group
    g1 = fmaxf(g1, __shfl_xor_sync(0xFFFFFFFFu, g1, 16));
    Sg[0] = global_scale_from_amax(g0);
    Sg[1] = global_scale_from_amax(g1);
  } else {
#pragma unroll
    for (int tb = 0; tb < 4; ++tb) {
      uint32_t m = 0;
#pragma unroll
      for (int t = 0; t < 16; ++t) m = amax16x2(m, w[16 * tb + t]);
      bm[tb] = m;
    }
    uint32_t g = amax16x2(amax16x2(bm[0], bm[1]), amax16x2(bm[2], bm[3]));
    g = bf16x2_abs_bits(amax16x2(g, __shfl_xor_sync(0xFFFFFFFFu, g, 16)));
    Sg[0] = global_scale_from_amax(__uint_as_float(g << 16));
    Sg[1] = global_scale_from_amax(__uint_as_float(g & 0xFFFF0000u));
  }
  if (!live) return;
  if ((lane >> 4) == 0) {
    gscale[(size_t)d0 * (Kp >> 7) + (k_start >> 7)] = Sg[0];
    gscale[(size_t)(d0 + 1) * (Kp >> 7) + (k_start >> 7)] = Sg[1];
  }
  uint32_t sfw[2] = {0u, 0u};
#pragma unroll
  for (int tb = 0; tb < 4; ++tb) {
    const uint32_t k0 = k_start + 16u * tb;
    const uint32_t m = RHT ? 0u : bf16x2_abs_bits(bm[tb]);
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      const float am = RHT ? bam[RHT ? tb : 0][c] : __uint_as_float(c ? (m & 0xFFFF0000u) : (m << 16));
      float rcp;
      const uint32_t sb = block_scale(am, Sg[c], rcp, RMODE == 2);
      sfw[c] |= sb << (8 * tb);
      float x[16];
#pragma unroll
      for (int t = 0; t < 16; ++t) x[t] = c ? bf16_hi(w[16 * tb + t]) : bf16_lo(w[16 * tb + t]);
      if (RHT) {
        rht_scale16(x, sign16(tb));
        hadamard16_butterflies(x);
      }
      const uint2 packed = quantize_block16<SR>(x, rcp, pk, stream_id, ((uint64_t)(d0 + c) * K16 + k0) >> 3);
      *reinterpret_cast<uint2*>(codes + (size_t)(d0 + c) * (Kp >> 1) + (k0 >> 1)) = packed;
    }
  }
  const uint32_t b = k_start >> 4;
#pragma unroll
  for (int c = 0; c < 2; ++c) {
    const uint32_t o = d0 + c;
    const size_t off = TILED ? (size_t)((o >> 7) * (((nb + 15u) & ~15u) >> 2) + (b >> 2)) * 512u + ((o & 31u) * 16u + ((o >> 5) & 3u) * 4u)
                             : (size_t)o * nb + b;
    *reinterpret_cast<uint32_t*>(sf + off) = sfw[c];
  }
}

// Transposing re-quantize of a forward operand (Q4, Q6 of Sec. 2.3) without a shared-memory transposition, for the TENSOR
// and ROW scale modes of the output. A lane owns EIGHT neighbouring source columns (one 32-bit word of codes per source row,
// all under one source scale byte) and 64 consecutive source rows; a warp instruction covers two source rows of 64
// contiguous code bytes. Per 16 source rows the lane keeps the 16 code words and walks its four column pairs in a ROLLED loop
// (the loop body -- decode one byte per row into P * S_block as an FP16 pair, exact, then two blocks of 16 values down the
// rows -- stays small enough for the instruction cache, which a fully unrolled version did not). x_hat = (P * S_block) *
// S_global of the source row is the same single binary32 rounding as everywhere else. The scale bytes of a lane (8 rows x 4
// blocks) are collected in a private strip of shared memory and written as one aligned word per operand row.
//   UNIFORM  the source has one global scale (TENSOR mode); otherwise it is fetched per source row (ROW) or per source row and
//            128-column group (BLOCK128; a lane's eight columns lie in one group).
//   TBT      16-row blocks per lane: 4 (64 source rows, CTA tile 512 x 128) for operands large enough to fill the chip with such
//            tiles, 1 (CTA tile 128 x 128; scale bytes stored one by one) for the model's 16384 x 1024 activations.
// Preconditions (else the staged kernel runs): identity row order, no row map, no Hadamard transformation.
template <int GS, int RMODE, bool TILED, bool UNIFORM, int TBT>
__global__ void __launch_bounds__(128, 4)
requantize_cols8_kernel(const TransposeSrc s, uint32_t K, uint32_t D, uint32_t stream_id, const uint32_t* __restrict__ gs_cells,
                        int tensor_closed_form, uint8_t* __restrict__ codes, uint8_t* __restrict__ sf, float* __restrict__ gscale,
                        const __grid_constant__ PhiloxKeys pk) {
  static_assert(GS != kGsBlock128, "the outer-block mode keeps the staged kernel");
  pdl_prologue();
  constexpr bool SR = RMODE != 0;
  __shared__ __align__(4) uint8_t sf_strip[128][36];  // per thread: 8 operand rows x 4 k blocks (+4: spreads the banks)
  const uint32_t Kp = (K + 127u) & ~127u;
  const uint32_t K16 = (K + 15u) & ~15u;
  const uint32_t nb = Kp >> 4;
  const uint32_t in_Kp = ((uint32_t)s.in_K + 127u) & ~127u;
  const uint32_t in_nb = in_Kp >> 4;
  const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
  const uint32_t d0 = blockIdx.y * 128u + (lane & 15u) * 8u;                       // first of this lane's operand rows
  const uint32_t k_start = (blockIdx.x * 8u + warp * 2u + (lane >> 4)) * (16u * TBT);  // first of its 16 * TBT k
  if (d0 >= D || k_start >= Kp) return;
  // (d0 + 7 < in_Kp always: the source rows are padded to 128 columns with zero codes and zero scales)
  const uint8_t* cp = s.in_codes + (size_t)k_start * (in_Kp >> 1) + (d0 >> 1);
  const uint32_t kb_in = d0 >> 4;
  const uint32_t in_tile_stride = ((in_nb + 15u) & ~15u) >> 2;

  float Sg_t = 1.0f;
  if (GS == kGsTensor) {
    // (tensor_closed_form == 2: the cell carries nothing and may be uninitialised; otherwise it covers what the closed form
    // does not. The closed form: the source's maximum is float32(2688 * S_global), its largest block has scale 448 and a
    // magnitude-6 element.)
    float amax = tensor_closed_form == 2 ? 0.0f : __uint_as_float(gs_cells[0]);
    if (tensor_closed_form) amax = fmaxf(amax, __fmul_rn(2688.0f, s.in_gscale[0]));
    Sg_t = global_scale_from_amax(amax);
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) gscale[0] = Sg_t;
  }
  const float sg_uniform = UNIFORM ? s.in_gscale[0] : 1.0f;
  uint8_t* my_sf = &sf_strip[threadIdx.x][0];

#pragma unroll 1
  for (uint32_t tb = 0; tb < (uint32_t)TBT; ++tb) {
    const uint32_t k0 = k_start + 16u * tb;
    // the 16 scale bytes of rows k0 .. k0 + 15 (k0 a multiple of 16) lie at a constant stride in either layout
    const size_t sf0 = s.in_sf_tiled ? (size_t)((k0 >> 7) * in_tile_stride + (kb_in >> 2)) * 512u +
                                           ((k0 & 31u) * 16u + ((k0 >> 5) & 3u) * 4u + (kb_in & 3u))
                                     : (size_t)k0 * in_nb + kb_in;
    const uint32_t sf_step = s.in_sf_tiled ? 16u : in_nb;
    const uint8_t* crow = cp + (size_t)(16u * tb) * (in_Kp >> 1);
    uint32_t cw[16], s2[16];
    float sgk[UNIFORM ? 1 : 16];
    {
      uint32_t sbv[16];
      if (k0 + 16u <= K) {
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          cw[t] = *reinterpret_cast<const uint32_t*>(crow + (size_t)t * (in_Kp >> 1));
          sbv[t] = s.in_sf[sf0 + (size_t)t * sf_step];
        }
      } else {
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          cw[t] = sbv[t] = 0u;
          if (k0 + t < K) {
            cw[t] = *reinterpret_cast<const uint32_t*>(crow + (size_t)t * (in_Kp >> 1));
            sbv[t] = s.in_sf[sf0 + (size_t)t * sf_step];
          }
        }
      }
#pragma unroll
      for (int t = 0; t < 16; ++t)  // the row's block scale as an FP16 pair (both halves equal)
        asm("{.reg .b16 q; cvt.u16.u32 q, %1; cvt.rn.f16x2.e4m3x2 %0, q;}" : "=r"(s2[t]) : "r"(sbv[t] | (sbv[t] << 8)));
    }
    if (!UNIFORM) {
#pragma unroll
      for (int t = 0; t < 16; ++t) {
        const uint32_t k = k0 + t;
        sgk[UNIFORM ? 0 : t] = k >= K ? 0.0f : s.in_gs_mode == kGsRow ? s.in_gscale[k] : s.in_gscale[(size_t)k * (in_Kp >> 7) + (d0 >> 7)];
      }
    }
#pragma unroll 1
    for (uint32_t j = 0; j < 4; ++j) {  // column pair (d0 + 2j, d0 + 2j + 1) = byte j of every code word
      float xs[2][16];
#pragma unroll
      for (int t = 0; t < 16; ++t) {
        uint32_t h2;
        asm("{\n.reg .b8 b0, b1, b2, b3;\nmov.b32 {b0, b1, b2, b3}, %1;\ncvt.rn.f16x2.e2m1x2 %0, b0;\n}" : "=r"(h2) : "r"(__byte_perm(cw[t], 0u, j)));
        const __half2 pv = __hmul2(*reinterpret_cast<const __half2*>(&h2), *reinterpret_cast<const __half2*>(&s2[t]));  // exact
        const float2 f = __half22float2(pv);
        const float g = UNIFORM ? sg_uniform : sgk[UNIFORM ? 0 : t];
        xs[0][t] = __fmul_rn(f.x, g);
        xs[1][t] = __fmul_rn(f.y, g);
      }
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        const uint32_t o = d0 + 2u * j + c;
        float m = 0.0f;
#pragma unroll
        for (int t = 0; t < 16; ++t) m = fmaxf(m, fabsf(xs[c][t]));
        float Sg = Sg_t;
        if (GS == kGsRow) {
          Sg = global_scale_from_amax(o < D ? __uint_as_float(gs_cells[o]) : 0.0f);
          if (o < D && k0 == 0) gscale[o] = Sg;
        }
        float rcp;
        const uint32_t sb = block_scale(m, Sg, rcp, RMODE == 2);
        if (TBT == 4) {
          my_sf[(2u * j + c) * 4u + tb] = (uint8_t)sb;
        } else if (o < D) {
          const uint32_t bk = k0 >> 4;
          const size_t off1 = TILED ? (size_t)((o >> 7) * (((nb + 15u) & ~15u) >> 2) + (bk >> 2)) * 512u +
                                          ((o & 31u) * 16u + ((o >> 5) & 3u) * 4u + (bk & 3u))
                                    : (size_t)o * nb + bk;
          sf[off1] = (uint8_t)sb;
        }
        const uint2 packed = quantize_block16<SR>(xs[c], rcp, pk, stream_id, ((uint64_t)o * K16 + k0) >> 3);
        if (o < D) *reinterpret_cast<uint2*>(codes + (size_t)o * (Kp >> 1) + (k0 >> 1)) = packed;
      }
    }
  }
  if (TBT != 4) return;
  // (the strip is private to the thread: its own byte stores are ordered before its word loads)
  const uint32_t b = k_start >> 4;
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    const uint32_t o = d0 + c;
    if (o < D) {
      const size_t off = TILED ? (size_t)((o >> 7) * (((nb + 15u) & ~15u) >> 2) + (b >> 2)) * 512u + ((o & 31u) * 16u + ((o >> 5) & 3u) * 4u)
                               : (size_t)o * nb + b;
      *reinterpret_cast<uint32_t*>(sf + off) = *reinterpret_cast<const uint32_t*>(my_sf + 4 * c);
    }
  }
}

// =========================================================================================================
// Host-side launchers
// =========================================================================================================
static inline unsigned blocks_for(int64_t n, int per) { return (unsigned)((n + per - 1) / per); }

template <int GS, bool SR, bool TILED>
static cudaError_t launch_rows_g(const QuantRowsArgs& a, cudaStream_t st) {
  const int64_t Kp = (a.K + 127) & ~(int64_t)127;
  const int64_t total = a.rows * (Kp >> 4);
  const unsigned grid = blocks_for(total, 256 * 4);
  // constants for gid / nb without a hardware division (n / d = (t + ((n - t) >> 1)) >> (s - 1), t = mulhi(m, n))
  uint32_t div_mul = 0, div_shift = 0xFFFFFFFFu;
  const uint64_t d = (uint64_t)(Kp >> 4);
  if (total + 1024 < (int64_t)1 << 31) {
    if ((d & (d - 1)) == 0) {
      div_shift = 0;
      while (((uint64_t)1 << div_shift) < d) ++div_shift;
    } else {
      uint32_t sft = 0;
      while (((uint64_t)1 << sft) < d) ++sft;
      div_mul = (uint32_t)((((uint64_t)1 << 32) * (((uint64_t)1 << sft) - d)) / d + 1);
      div_shift = sft - 1;
    }
  }
  const int wide_loads = ((reinterpret_cast<uintptr_t>(a.src) & 31u) == 0 && (a.ld & 15) == 0) ? 1 : 0;
  if (a.keep) {
    // rows a CTA can touch: its 1024 blocks span at most 1024 / nb + 2 rows; stage them if they fit in shared memory
    const int64_t cols8 = (a.cols_src + 7) & ~(int64_t)7;
    const int64_t max_rows = 1024 / (int64_t)d + 2;
    size_t smem = (size_t)(max_rows * cols8 * 2);
    int64_t stage_cols8 = cols8;
    if (smem > 160 * 1024 || (reinterpret_cast<uintptr_t>(a.keep) & 15u) != 0 || (a.ld & 7) != 0) {
      smem = 0;
      stage_cols8 = 0;  // fall back to per-element global loads
    } else {
      cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(quantize_rows_kernel<GS, SR, TILED, true, false>), smem);
      if (e != cudaSuccess) return e;
    }
    launch_kernel(quantize_rows_kernel<GS, SR, TILED, true, false>, dim3(grid), dim3(256), smem, st, a.src, a.rows, a.K, a.ld, a.keep, a.seed,
                  a.stream_id, a.gs_cells, a.codes, a.sf, a.gscale, div_mul, div_shift, wide_loads, a.cols_src, stage_cols8, 0u, a.sr == 2, make_philox_keys(a.seed));
  } else if (a.rht_stream) {
    launch_kernel(quantize_rows_kernel<GS, SR, TILED, false, true>, dim3(grid), dim3(256), 0, st, a.src, a.rows, a.K, a.ld, nullptr, a.seed,
                  a.stream_id, a.gs_cells, a.codes, a.sf, a.gscale, div_mul, div_shift, wide_loads, a.cols_src, (int64_t)0, a.rht_stream, a.sr == 2, make_philox_keys(a.seed));
  } else {
    launch_kernel(quantize_rows_kernel<GS, SR, TILED, false, false>, dim3(grid), dim3(256), 0, st, a.src, a.rows, a.K, a.ld, nullptr, a.seed,
                  a.stream_id, a.gs_cells, a.codes, a.sf, a.gscale, div_mul, div_shift, wide_loads, a.cols_src, (int64_t)0, 0u, a.sr == 2, make_philox_keys(a.seed));
  }
  return cudaGetLastError();
}

// The four-adjacent-blocks kernel (stochastic rounding without a column list).
template <int GS, int RMODE, bool TILED>
static cudaError_t launch_rows4(const QuantRowsArgs& a, cudaStream_t st) {
  const int64_t Kp = (a.K + 127) & ~(int64_t)127;
  const uint64_t d = (uint64_t)(Kp >> 6);  // units per row
  const int64_t total = a.rows * (int64_t)d;
  const unsigned grid = blocks_for(total, 256);
  uint32_t div_mul = 0, div_shift = 0xFFFFFFFFu;
  if (total + 256 < (int64_t)1 << 31) {
    if ((d & (d - 1)) == 0) {
      div_shift = 0;
      while (((uint64_t)1 << div_shift) < d) ++div_shift;
    } else {
      uint32_t sft = 0;
      while (((uint64_t)1 << sft) < d) ++sft;
      div_mul = (uint32_t)((((uint64_t)1 << 32) * (((uint64_t)1 << sft) - d)) / d + 1);
      div_shift = sft - 1;
    }
  }
  const int wide_loads = ((reinterpret_cast<uintptr_t>(a.src) & 31u) == 0 && (a.ld & 15) == 0) ? 1 : 0;
  if (a.rht_stream)
    launch_kernel(quantize_rows4_kernel<GS, RMODE, TILED, true>, dim3(grid), dim3(256), 0, st, a.src, a.rows, a.K, a.ld, a.seed, a.stream_id,
                  a.gs_cells, a.codes, a.sf, a.gscale, div_mul, div_shift, wide_loads, a.rht_stream, make_philox_keys(a.seed));
  else
    launch_kernel(quantize_rows4_kernel<GS, RMODE, TILED, false>, dim3(grid), dim3(256), 0, st, a.src, a.rows, a.K, a.ld, a.seed, a.stream_id,
                  a.gs_cells, a.codes, a.sf, a.gscale, div_mul, div_shift, wide_loads, 0u, make_philox_keys(a.seed));
  return cudaGetLastError();
}

template <int GS, bool SR>
static cudaError_t launch_rows_t(const QuantRowsArgs& a, cudaStream_t st) {
  return a.sf_tiled ? launch_rows_g<GS, SR, true>(a, st) : launch_rows_g<GS, SR, false>(a, st);
}

template <int GS>
static cudaError_t launch_rows_r(const QuantRowsArgs& a, cudaStream_t st) {
  // stochastic rounding is bound by instruction issue: the kernel with the least bookkeeping per block wins there; round to
  // nearest is a streaming kernel and keeps the strided one (fully coalesced loads, four loads in flight per thread)
  if (a.sr && !a.keep && (a.ld & 7) == 0 && (reinterpret_cast<uintptr_t>(a.src) & 15u) == 0 && a.K < ((int64_t)1 << 31)) {
    if (a.sr == 2) return a.sf_tiled ? launch_rows4<GS, 2, true>(a, st) : launch_rows4<GS, 2, false>(a, st);
    return a.sf_tiled ? launch_rows4<GS, 1, true>(a, st) : launch_rows4<GS, 1, false>(a, st);
  }
  return a.sr ? launch_rows_t<GS, true>(a, st) : launch_rows_t<GS, false>(a, st);
}

static cudaError_t launch_quantize_rows_impl(const QuantRowsArgs& a, cudaStream_t st, bool& side_copy_done) {
  if (a.rows == 0 || a.K == 0) return cudaSuccess;
  if (a.rows >= ((int64_t)1 << 31) || a.cols_src >= ((int64_t)1 << 31) || a.ld >= ((int64_t)1 << 31)) return cudaErrorInvalidValue;
  cudaError_t e;
  if (a.rht_stream) {  // the scales come from the transformed data; column lists are not combined with the transformation
    if (a.keep) return cudaErrorInvalidValue;
    if (a.gs_mode != kGsBlock128 && (a.gs_mode == kGsRow || a.compute_amax)) {
      const int per_row = a.gs_mode == kGsRow;
      if (!a.cells_zeroed && (e = launch_zero_words(a.gs_cells, per_row ? a.rows : 1, st)) != cudaSuccess) return e;
      const int64_t blocks16 = a.rows * ((a.K + 15) >> 4);
      const unsigned grid = (unsigned)std::min<int64_t>((blocks16 + 255) / 256, device_sm_count() * 16);
      launch_kernel(amax_rows_rht_kernel, dim3(grid), dim3(256), 0, st, a.src, a.rows, a.K, a.ld, a.seed, a.rht_stream, a.gs_cells, per_row);
      if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    return a.gs_mode == kGsTensor ? launch_rows_r<kGsTensor>(a, st)
           : a.gs_mode == kGsRow  ? launch_rows_r<kGsRow>(a, st)
                                  : launch_rows_r<kGsBlock128>(a, st);
  }
  if (a.gs_mode == kGsTensor) {
    if (a.compute_amax) {
      if (!a.cells_zeroed && (e = launch_zero_words(a.gs_cells, 1, st)) != cudaSuccess) return e;
      if (a.keep && a.excluded && (a.ld & 7) == 0 && a.cols_src <= 20 * 1024) {
        // amax over the kept columns only: full-width vector loads with the excluded (outlier) columns masked out
        const size_t smem = (size_t)((a.cols_src + 7) >> 3) * 16;  // one 16-byte mask per chunk (at most 40 KB)
        // a contiguous slab of rows per CTA. The side copy divides item numbers by the side operand's width through a
        // 32-bit reciprocal, exact while items * width < 2^32: slabs stay below 2^32 / d^2 rows (d also covers the chunk count)
        int64_t rows_per_cta = (a.rows + device_sm_count() * 4 - 1) / (device_sm_count() * 4);  // few, fat CTAs: the per-thread setup is paid once
        const int64_t dmax = std::max<int64_t>((a.cols_src + 7) >> 3, a.excl_out ? a.ld_excl_out : 1);
        rows_per_cta = std::max<int64_t>(1, std::min<int64_t>(rows_per_cta, (((int64_t)1 << 32) - 1) / (dmax * dmax)));
        const unsigned grid = (unsigned)((a.rows + rows_per_cta - 1) / rows_per_cta);
        launch_kernel(amax_tensor_masked_kernel, dim3(grid), dim3(256), smem, st, a.src, a.rows, a.cols_src, a.ld, a.excluded,
                      a.cols_src - a.K, a.gs_cells, a.excl_out, a.ld_excl_out, rows_per_cta,
                      (uint64_t)((1ull << 32) / (uint64_t)std::max<int64_t>(1, a.ld_excl_out) + 1ull));
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        side_copy_done = a.excl_out != nullptr;
        return launch_rows_r<kGsTensor>(a, st);
      }
      if (a.keep) {  // amax over the kept columns only: one row per CTA, one atomic per row
        launch_kernel(amax_rows_bf16_kernel, dim3((unsigned)a.rows), dim3(256), 0, st, a.src, a.rows, a.cols_src, a.ld, a.keep, a.K, a.gs_cells, 1);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        return launch_rows_r<kGsTensor>(a, st);
      }
      const int64_t chunks = a.rows * ((a.cols_src + 7) >> 3);
      const unsigned grid = (unsigned)std::min<int64_t>((chunks + 255) / 256, device_sm_count() * 8);
      launch_kernel(amax_tensor_bf16_kernel, dim3(grid), dim3(256), 0, st, a.src, a.rows, a.cols_src, a.ld, a.gs_cells);
      if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    return launch_rows_r<kGsTensor>(a, st);
  }
  if (a.gs_mode == kGsRow) {
    if (!a.keep && (a.ld & 7) == 0 && (reinterpret_cast<uintptr_t>(a.src) & 15u) == 0)  // a warp per row
      launch_kernel(amax_rows_warp_kernel, dim3((unsigned)((a.rows + 7) / 8)), dim3(256), 0, st, a.src, a.rows, a.cols_src, a.ld, a.gs_cells);
    else
      launch_kernel(amax_rows_bf16_kernel, dim3((unsigned)a.rows), dim3(256), 0, st, a.src, a.rows, a.cols_src, a.ld, a.keep, a.K, a.gs_cells, 0);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    return launch_rows_r<kGsRow>(a, st);
  }
  return launch_rows_r<kGsBlock128>(a, st);
}

cudaError_t launch_quantize_rows(const QuantRowsArgs& a, cudaStream_t st) {
  bool side_copy_done = false;
  cudaError_t e = launch_quantize_rows_impl(a, st, side_copy_done);
  if (e != cudaSuccess) return e;
  if (a.excl_out && a.excluded && !side_copy_done)
    e = launch_gather_cols(a.src, a.ld, a.rows, a.excluded, a.cols_src - a.K, a.excl_out, a.ld_excl_out, st);
  return e;
}

// The fast kernel takes every source that needs no per-column choice between the forward operand and a BF16 matrix
// (nvfp4_requantize_t with a row map is the one caller that does) and whose BF16 rows can be read in 16-byte pieces.
static bool transpose_fast_path(const TransposeSrc& s, int from_codes) {
  if (s.ld >= ((int64_t)1 << 31) || s.in_K >= ((int64_t)1 << 31)) return false;
  if (from_codes) return s.row_map == nullptr;
  return (s.ld & 7) == 0 && (reinterpret_cast<uintptr_t>(s.bf16) & 15u) == 0;
}

// The register-transposing kernels take a plain BF16 source whose rows can be read in 8-byte pieces: identity row order, no
// closed-form maximum handed in by OutControl's two-pass W-hat.
static bool cols4_path(const QuantTransposeArgs& a) {
  const TransposeSrc& s = a.src;
  return !s.out_rows && !s.closed_form_sg && !a.tensor_closed_form && (a.D & 3) == 0 && (s.ld & 3) == 0 &&
         (reinterpret_cast<uintptr_t>(s.bf16) & 7u) == 0 && s.ld < ((int64_t)1 << 31) && a.rowsK < ((int64_t)1 << 31) - 1024 &&
         a.D < ((int64_t)1 << 31) - 64;
}

// ... and its counterpart for a forward operand as the source, from 8 M elements on (smaller operands, such as a layer's
// weights, do not fill the chip with its 128 x 128 tiles of 128 threads and stay with the staged kernel).
static bool cols8_path(const QuantTransposeArgs& a) {
  const TransposeSrc& s = a.src;
  return a.rowsK * a.D >= ((int64_t)8 << 20) && !a.rht_stream && !s.out_rows && !s.closed_form_sg && !s.row_map && s.in_K < ((int64_t)1 << 31) - 128 &&
         a.rowsK < ((int64_t)1 << 31) - 1024 && a.D < ((int64_t)1 << 31) - 128;
}

template <int SRC, int GS, int RMODE>
static cudaError_t launch_tr_t(const QuantTransposeArgs& a, cudaStream_t st) {
  const dim3 grid(blocks_for(a.rowsK, 128), blocks_for(a.D, 64));
  const bool fast = transpose_fast_path(a.src, SRC);
  if constexpr (SRC == 1 && GS != kGsBlock128) {
    if (cols8_path(a)) {
      // 512 x 128 tiles when they fill the chip about twice over, else 128 x 128 tiles
      const bool big = (int64_t)blocks_for(a.rowsK, 512) * blocks_for(a.D, 128) >= 8 * (int64_t)device_sm_count();
      const dim3 g8(blocks_for(a.rowsK, big ? 512 : 128), blocks_for(a.D, 128));
      const bool uniform = a.src.in_gs_mode == kGsTensor;
      const PhiloxKeys keys = make_philox_keys(a.seed);
#define NVFP4_LAUNCH_C8(TILED_, UNI_, TBT_)                                                                                          \
  launch_kernel(requantize_cols8_kernel<GS, RMODE, TILED_, UNI_, TBT_>, g8, dim3(128), 0, st, a.src, (uint32_t)a.rowsK,                \
                (uint32_t)a.D, a.stream_id, (const uint32_t*)a.gs_cells, a.tensor_closed_form, a.codes, a.sf, a.gscale, keys)
#define NVFP4_LAUNCH_C8B(TILED_, UNI_)                                                                                               \
  if (big) NVFP4_LAUNCH_C8(TILED_, UNI_, 4); else NVFP4_LAUNCH_C8(TILED_, UNI_, 1)
      if (a.sf_tiled) {
        if (uniform) { NVFP4_LAUNCH_C8B(true, true); } else { NVFP4_LAUNCH_C8B(true, false); }
      } else {
        if (uniform) { NVFP4_LAUNCH_C8B(false, true); } else { NVFP4_LAUNCH_C8B(false, false); }
      }
#undef NVFP4_LAUNCH_C8B
#undef NVFP4_LAUNCH_C8
      return cudaGetLastError();
    }
  }
  if constexpr (SRC == 0) {
    if (cols4_path(a)) {
      const PhiloxKeys keys = make_philox_keys(a.seed);
      const uint32_t K32 = (uint32_t)a.rowsK, D32 = (uint32_t)a.D, ld32 = (uint32_t)a.src.ld;
#define NVFP4_LAUNCH_COLS(TILED_, RHT_)                                                                                             \
  if constexpr (GS == kGsBlock128)                                                                                                  \
    launch_kernel(quantize_cols2_block128_kernel<RMODE, TILED_, RHT_>, dim3(blocks_for(a.rowsK, 512), blocks_for(a.D, 32)),         \
                  dim3(128), 0, st, a.src.bf16, K32, D32, ld32, a.seed, a.stream_id, a.rht_stream, a.codes, a.sf, a.gscale, keys);  \
  else                                                                                                                              \
    launch_kernel(quantize_cols4_kernel<GS, RMODE, TILED_, RHT_, false>, dim3(blocks_for(a.rowsK, 512), blocks_for(a.D, 64)),       \
                  dim3(128), 0, st, a.src.bf16, K32, D32, ld32, a.seed, a.stream_id, a.rht_stream, a.gs_cells, a.codes, a.sf,       \
                  a.gscale, keys)
      if (a.sf_tiled) {
        if (a.rht_stream) { NVFP4_LAUNCH_COLS(true, true); } else { NVFP4_LAUNCH_COLS(true, false); }
      } else {
        if (a.rht_stream) { NVFP4_LAUNCH_COLS(false, true); } else { NVFP4_LAUNCH_COLS(false, false); }
      }
#undef NVFP4_LAUNCH_COLS
      return cudaGetLastError();
    }
  }
#define NVFP4_LAUNCH_TR(TILED_, RHT_)                                                                                                  \
  if (fast)                                                                                                                            \
    launch_kernel(quantize_transpose_kernel<SRC, GS, RMODE, TILED_, RHT_, false>, dim3(grid), dim3(256), 0, st, a.src, a.rowsK, a.D,    \
                  a.seed, a.stream_id, a.gs_cells, a.tensor_closed_form, a.codes, a.sf, a.gscale, a.rht_stream,                        \
                  make_philox_keys(a.seed));                                                                                           \
  else                                                                                                                                 \
    launch_kernel(quantize_transpose_generic_kernel<SRC, GS, RMODE != 0, TILED_, RHT_, false>, dim3(grid), dim3(256), 0, st, a.src,     \
                  a.rowsK, a.D, a.seed, a.stream_id, a.gs_cells, a.tensor_closed_form, a.codes, a.sf, a.gscale, a.rht_stream,          \
                  RMODE == 2, make_philox_keys(a.seed))
  if (a.sf_tiled) {
    if (a.rht_stream) { NVFP4_LAUNCH_TR(true, true); } else { NVFP4_LAUNCH_TR(true, false); }
  } else {
    if (a.rht_stream) { NVFP4_LAUNCH_TR(false, true); } else { NVFP4_LAUNCH_TR(false, false); }
  }
#undef NVFP4_LAUNCH_TR
  return cudaGetLastError();
}

// amax pre-pass with the quantizer's own tile walk, stopped after the block maxima (its vectorised staging decodes a
// forward operand several times faster than the element-wise column kernel; under the Hadamard transformation it is the
// only pass that sees the transformed values)
template <int SRC, int GS>
static cudaError_t launch_tr_amax_rht(const TransposeSrc& src, int64_t rowsK, int64_t D, uint64_t seed, uint32_t rht_stream,
                                      uint32_t* cells, cudaStream_t st) {
  const dim3 grid(blocks_for(rowsK, 128), blocks_for(D, 64));
  uint8_t* const no_bytes = nullptr;
  float* const no_floats = nullptr;
  if constexpr (SRC == 0 && GS != kGsBlock128) {
    // the register-transposing kernel's own pre-pass (same conditions as cols4_path)
    if (rht_stream && !src.out_rows && (D & 3) == 0 && (src.ld & 3) == 0 && (reinterpret_cast<uintptr_t>(src.bf16) & 7u) == 0 &&
        src.ld < ((int64_t)1 << 31) && rowsK < ((int64_t)1 << 31) - 1024 && D < ((int64_t)1 << 31) - 64) {
      launch_kernel(quantize_cols4_kernel<GS, 0, false, true, true>, dim3(blocks_for(rowsK, 512), blocks_for(D, 64)), dim3(128), 0, st,
                    src.bf16, (uint32_t)rowsK, (uint32_t)D, (uint32_t)src.ld, seed, 0u, rht_stream, cells, no_bytes, no_bytes, no_floats,
                    make_philox_keys(seed));
      return cudaGetLastError();
    }
  }
  if (transpose_fast_path(src, SRC)) {
    if (rht_stream)
      launch_kernel(quantize_transpose_kernel<SRC, GS, 0, false, true, true>, dim3(grid), dim3(256), 0, st, src, rowsK, D, seed, 0u, cells, 0,
                    no_bytes, no_bytes, no_floats, rht_stream, make_philox_keys(seed));
    else
      launch_kernel(quantize_transpose_kernel<SRC, GS, 0, false, false, true>, dim3(grid), dim3(256), 0, st, src, rowsK, D, seed, 0u, cells, 0,
                    no_bytes, no_bytes, no_floats, 0u, make_philox_keys(seed));
  } else if (rht_stream) {
    launch_kernel(quantize_transpose_generic_kernel<SRC, GS, false, false, true, true>, dim3(grid), dim3(256), 0, st, src, rowsK, D, seed, 0u, cells,
                  0, no_bytes, no_bytes, no_floats, rht_stream, 0, make_philox_keys(seed));
  } else {
    launch_kernel(quantize_transpose_generic_kernel<SRC, GS, false, false, false, true>, dim3(grid), dim3(256), 0, st, src, rowsK, D, seed, 0u, cells,
                  0, no_bytes, no_bytes, no_floats, 0u, 0, make_philox_keys(seed));
  }
  return cudaGetLastError();
}

template <int SRC, int GS>
static cudaError_t launch_tr_r(const QuantTransposeArgs& a, cudaStream_t st) {
  return a.sr == 2 ? launch_tr_t<SRC, GS, 2>(a, st) : a.sr ? launch_tr_t<SRC, GS, 1>(a, st) : launch_tr_t<SRC, GS, 0>(a, st);
}

template <int SRC>
static cudaError_t launch_tr_s(const QuantTransposeArgs& a0, cudaStream_t st) {
  QuantTransposeArgs a = a0;
  a.tensor_closed_form = 0;
  cudaError_t e;
  const dim3 agrid(blocks_for(a.D, 64), blocks_for(a.rowsK, 256));
  if (a.rht_stream && a.gs_mode != kGsBlock128) {
    const bool per_row = a.gs_mode == kGsRow;
    if (per_row || a.compute_amax) {
      if (!a.cells_zeroed && (e = launch_zero_words(a.gs_cells, per_row ? a.D : 1, st)) != cudaSuccess) return e;
      e = per_row ? launch_tr_amax_rht<SRC, kGsRow>(a.src, a.rowsK, a.D, a.seed, a.rht_stream, a.gs_cells, st)
                  : launch_tr_amax_rht<SRC, kGsTensor>(a.src, a.rowsK, a.D, a.seed, a.rht_stream, a.gs_cells, st);
      if (e != cudaSuccess) return e;
    }
    return per_row ? launch_tr_r<SRC, kGsRow>(a, st) : launch_tr_r<SRC, kGsTensor>(a, st);
  }
  if (a.gs_mode == kGsTensor) {
    if (a.compute_amax) {
      const bool cell_unused = SRC == 1 && a.src.in_gs_mode == kGsTensor && !a.src.row_map;
      if (!cell_unused && !a.cells_zeroed && (e = launch_zero_words(a.gs_cells, 1, st)) != cudaSuccess) return e;
      if (SRC == 0) {
        const int64_t chunks = a.rowsK * ((a.D + 7) >> 3);
        const unsigned grid = (unsigned)std::min<int64_t>((chunks + 255) / 256, device_sm_count() * 8);
        launch_kernel(amax_tensor_bf16_kernel, dim3(grid), dim3(256), 0, st, a.src.bf16, a.rowsK, a.D, a.src.ld, a.gs_cells);
      } else if (a.src.in_gs_mode == kGsTensor) {
        a.tensor_closed_form = a.src.row_map ? 1 : 2;  // only the BF16 rows (if any) need a pass
        if (a.src.row_map) {
          launch_kernel(amax_cols_generic_kernel<SRC>, dim3(agrid), dim3(256), 0, st, a.src, a.rowsK, a.D, a.gs_cells, 0, 1);
        }
      } else {
        if ((e = launch_tr_amax_rht<SRC, kGsTensor>(a.src, a.rowsK, a.D, a.seed, 0u, a.gs_cells, st)) != cudaSuccess) return e;
      }
      if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    return launch_tr_r<SRC, kGsTensor>(a, st);
  }
  if (a.gs_mode == kGsRow) {
    if (!a.cells_zeroed && (e = launch_zero_words(a.gs_cells, a.D, st)) != cudaSuccess) return e;
    if (SRC == 0 && !a.src.out_rows && (a.src.ld & 7) == 0 && (reinterpret_cast<uintptr_t>(a.src.bf16) & 15u) == 0) {
      // per-column maxima of the BF16 source by a streaming kernel (about 2 CTAs per SM worth of row slabs per column strip)
      const int64_t strips = (a.D + 255) / 256;
      int64_t slabs = std::max<int64_t>(1, (device_sm_count() * 4 + strips - 1) / strips);
      slabs = std::min<int64_t>(slabs, (a.rowsK + 63) / 64);
      const int64_t rows_per_slab = ((a.rowsK + slabs - 1) / slabs + 7) / 8 * 8;
      launch_kernel(amax_cols_bf16_kernel, dim3((unsigned)strips, (unsigned)((a.rowsK + rows_per_slab - 1) / rows_per_slab)), dim3(256), 0, st,
                    a.src.bf16, a.rowsK, a.D, a.src.ld, rows_per_slab, a.gs_cells);
      if ((e = cudaGetLastError()) != cudaSuccess) return e;
    } else if ((e = launch_tr_amax_rht<SRC, kGsRow>(a.src, a.rowsK, a.D, a.seed, 0u, a.gs_cells, st)) != cudaSuccess) {
      return e;
    }
    return launch_tr_r<SRC, kGsRow>(a, st);
  }
  return launch_tr_r<SRC, kGsBlock128>(a, st);
}

cudaError_t launch_amax_tensor(const uint16_t* src, int64_t rows, int64_t cols, int64_t ld, uint32_t* cell, cudaStream_t st) {
  if (rows == 0 || cols == 0) return cudaSuccess;
  const int64_t chunks = rows * ((cols + 7) >> 3);
  const unsigned grid = (unsigned)std::min<int64_t>((chunks + 255) / 256, device_sm_count() * 8);
  launch_kernel(amax_tensor_bf16_kernel, dim3(grid), dim3(256), 0, st, src, rows, cols, ld, cell);
  return cudaGetLastError();
}

// Clears amax cells with a kernel instead of a memset node, so that the programmatic launch chain is not interrupted.
__global__ void __launch_bounds__(256) zero_words_kernel(uint32_t* p, int64_t n) {
  pdl_prologue();
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < n; i += (int64_t)gridDim.x * 256) p[i] = 0u;
}
cudaError_t launch_zero_words(uint32_t* p, int64_t n, cudaStream_t st) {
  if (n <= 0) return cudaSuccess;
  launch_kernel(zero_words_kernel, dim3((unsigned)std::min<int64_t>((n + 255) / 256, (int64_t)device_sm_count())), dim3(256), 0, st, p, n);
  return cudaGetLastError();
}

cudaError_t launch_amax_tensor_pair(const uint16_t* a, int64_t rows_a, int64_t cols_a, int64_t ld_a, uint32_t* cell_a, const uint16_t* b,
                                    int64_t rows_b, int64_t cols_b, int64_t ld_b, uint32_t* cell_b, cudaStream_t st) {
  auto grid_of = [](int64_t rows, int64_t cols) {
    const int64_t chunks = rows * ((cols + 7) >> 3);
    return (unsigned)std::max<int64_t>(1, std::min<int64_t>((chunks + 255) / 256, device_sm_count() * 8));
  };
  const unsigned ga = grid_of(rows_a, cols_a), gb = grid_of(rows_b, cols_b);
  launch_kernel(amax_tensor_pair_kernel, dim3(ga + gb), dim3(256), 0, st, a, rows_a, cols_a, ld_a, cell_a, ga, b, rows_b, cols_b, ld_b, cell_b);
  return cudaGetLastError();
}

cudaError_t launch_amax_transpose_src(const TransposeSrc& s, int from_codes, int64_t rowsK, int64_t D, uint32_t* cell,
                                      cudaStream_t st, uint64_t seed, uint32_t rht_stream) {
  if (rowsK == 0 || D == 0) return cudaSuccess;
  if (rht_stream)
    return from_codes ? launch_tr_amax_rht<1, kGsTensor>(s, rowsK, D, seed, rht_stream, cell, st)
                      : launch_tr_amax_rht<0, kGsTensor>(s, rowsK, D, seed, rht_stream, cell, st);
  const dim3 agrid(blocks_for(D, 64), blocks_for(rowsK, 256));
  if (from_codes)
    launch_kernel(amax_cols_generic_kernel<1>, dim3(agrid), dim3(256), 0, st, s, rowsK, D, cell, 0, 0);
  else
    launch_kernel(amax_cols_generic_kernel<0>, dim3(agrid), dim3(256), 0, st, s, rowsK, D, cell, 0, 0);
  return cudaGetLastError();
}

cudaError_t launch_quantize_transpose(const QuantTransposeArgs& a, cudaStream_t st) {
  if (a.rowsK == 0 || a.D == 0) return cudaSuccess;
  if (a.rowsK >= ((int64_t)1 << 31) - 128 || a.D >= ((int64_t)1 << 31) - 128) return cudaErrorInvalidValue;
  return a.from_codes ? launch_tr_s<1>(a, st) : launch_tr_s<0>(a, st);
}

}  // namespace nvfp4
