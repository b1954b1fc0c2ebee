// OutControl calibration (paper Sec. 4.2, the paragraph that defines the outlier index set): per-channel l2-norms of
// the activations are accumulated over a calibration window, and the channels with the largest accumulated value form
// the outlier set. Two entry points:
//   nvfp4_outlier_accumulate   acc[d] += sqrt(sum_t X[t, d]^2) for one step's activations (HBM streaming, 2 B/element)
//   nvfp4_outlier_select       top-n_out channels of acc -> sorted outlier list, sorted kept list, channel map
// Both are deterministic: partial sums are combined in a fixed order, ties go to the lower channel index.
#include "../../include/nvfp4.h"

#include "nvfp4_device.cuh"
#include "nvfp4_internal.h"

namespace nvfp4 {

// Sum of squares of a slab of rows, per channel. Block = 32 lanes x 8 row lanes; a lane owns 8 neighbouring channels (one
// 16-byte load per row), so a warp reads 512 contiguous bytes of a row. partial[slab][channel], channel padded to 256.
__global__ void __launch_bounds__(256) colsq_partial_kernel(const uint16_t* __restrict__ X, int64_t ld, int64_t N, int64_t D,
                                                           int64_t rows_per_slab, float* __restrict__ partial, int64_t Dp) {
  pdl_prologue();
  const int lane = threadIdx.x & 31, ry = threadIdx.x >> 5;
  const int64_t c0 = (int64_t)blockIdx.x * 256 + lane * 8;
  const int64_t r_begin = (int64_t)blockIdx.y * rows_per_slab;
  const int64_t r_end = min(N, r_begin + rows_per_slab);
  float s[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) s[i] = 0.0f;
  auto add8 = [&](const uint4& v) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float lo = bf16_lo(w[i]), hi = bf16_hi(w[i]);
      s[2 * i] = fmaf(lo, lo, s[2 * i]);
      s[2 * i + 1] = fmaf(hi, hi, s[2 * i + 1]);
    }
  };
  if (c0 + 8 <= D) {
    int64_t r = r_begin + ry;
    for (; r + 56 < r_end; r += 64) {  // eight rows in flight
      uint4 v[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) v[q] = *reinterpret_cast<const uint4*>(X + (r + 8 * q) * ld + c0);
#pragma unroll
      for (int q = 0; q < 8; ++q) add8(v[q]);
    }
    for (; r < r_end; r += 8) add8(*reinterpret_cast<const uint4*>(X + r * ld + c0));
  } else if (c0 < D) {  // ragged last chunk of a row
    for (int64_t r = r_begin + ry; r < r_end; r += 8)
      for (int i = 0; i < 8; ++i)
        if (c0 + i < D) {
          const float v = bf16_bits_to_float(X[r * ld + c0 + i]);
          s[i] = fmaf(v, v, s[i]);
        }
  }
  __shared__ float red[8][8][32];  // [row lane][i][lane]: conflict-free both ways
#pragma unroll
  for (int i = 0; i < 8; ++i) red[ry][i][lane] = s[i];
  __syncthreads();
  {
    const int i = threadIdx.x >> 5, ln = threadIdx.x & 31;
    float t = 0.0f;
#pragma unroll
    for (int y = 0; y < 8; ++y) t += red[y][i][ln];  // fixed order
    partial[(int64_t)blockIdx.y * Dp + (int64_t)blockIdx.x * 256 + ln * 8 + i] = t;
  }
}

__global__ void __launch_bounds__(256) colsq_finalize_kernel(const float* __restrict__ partial, int64_t n_slabs, int64_t Dp, int64_t D,
                                                            float* __restrict__ acc) {
  pdl_prologue();
  const int64_t d = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (d >= D) return;
  float s = 0.0f;
  for (int64_t k = 0; k < n_slabs; ++k) s += partial[k * Dp + d];  // fixed order
  acc[d] = acc[d] + __fsqrt_rn(s);
}

// rank of channel d in the order (value descending, index ascending); col_map[d] = -1 if rank < n_out, else 0
__global__ void __launch_bounds__(256) outlier_rank_kernel(const float* __restrict__ acc, int64_t D, int64_t n_out,
                                                          int32_t* __restrict__ col_map) {
  pdl_prologue();
  __shared__ float tile[1024];
  const int64_t d = (int64_t)blockIdx.x * 256 + threadIdx.x;
  const float a_d = d < D ? acc[d] : 0.0f;
  int64_t rank = 0;
  for (int64_t j0 = 0; j0 < D; j0 += 1024) {
    for (int q = threadIdx.x; q < 1024; q += 256) tile[q] = (j0 + q < D) ? acc[j0 + q] : 0.0f;
    __syncthreads();
    const int n = (int)min((int64_t)1024, D - j0);
    int r = 0;
    for (int jj = 0; jj < n; ++jj) {
      const float a_j = tile[jj];
      r += (a_j > a_d || (a_j == a_d && j0 + jj < d)) ? 1 : 0;
    }
    rank += r;
    __syncthreads();
  }
  if (d < D) col_map[d] = rank < n_out ? -1 : 0;
}

// One CTA: stable compaction of the flagged (outlier) and unflagged (kept) channels; fills col_map for the kept ones.
__global__ void __launch_bounds__(1024) outlier_compact_kernel(int64_t D, int32_t* __restrict__ col_map, int32_t* __restrict__ outl,
                                                              int32_t* __restrict__ keep) {
  pdl_prologue();
  __shared__ int warp_cnt[32];
  __shared__ int chunk_total;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  int64_t out_base = 0, keep_base = 0;
  for (int64_t c0 = 0; c0 < D; c0 += 1024) {
    const int64_t d = c0 + tid;
    const bool valid = d < D;
    const bool flag = valid && col_map[d] < 0;
    const uint32_t bal = __ballot_sync(0xFFFFFFFFu, flag);
    if (lane == 0) warp_cnt[wid] = __popc(bal);
    __syncthreads();
    if (wid == 0) {
      int v = warp_cnt[lane], incl = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += t;
      }
      warp_cnt[lane] = incl - v;  // exclusive
      if (lane == 31) chunk_total = incl;
    }
    __syncthreads();
    const int excl = warp_cnt[wid] + __popc(bal & ((1u << lane) - 1u));
    if (valid) {
      if (flag) {
        outl[out_base + excl] = (int32_t)d;
      } else {
        const int64_t pos = keep_base + (tid - excl);
        keep[pos] = (int32_t)d;
        col_map[d] = (int32_t)pos;
      }
    }
    const int n_valid = (int)min((int64_t)1024, D - c0);
    out_base += chunk_total;
    keep_base += n_valid - chunk_total;
    __syncthreads();
  }
}

// Row slabs of the partial-sum pass. A tuning constant, not a hardware query: the workspace size derived from it must not
// depend on the device (about six CTAs per SM on a 148-SM part).
constexpr int64_t kCalibTargetCtas = 888;
static int64_t calib_slabs(int64_t N, int64_t D) {
  const int64_t col_ctas = (D + 255) / 256;
  int64_t slabs = (kCalibTargetCtas + col_ctas - 1) / col_ctas;
  slabs = std::max<int64_t>(1, std::min<int64_t>(slabs, (N + 31) / 32));
  return slabs;
}

}  // namespace nvfp4

using namespace nvfp4;

extern "C" {

size_t nvfp4_outlier_accumulate_workspace_bytes(int64_t N_tok, int64_t D) {
  if (N_tok <= 0 || D <= 0) return 256;
  const int64_t Dp = (D + 255) / 256 * 256;
  return (size_t)(calib_slabs(N_tok, D) * Dp * 4 + 256);
}

nvfp4_status nvfp4_outlier_accumulate(const void* X_bf16, int64_t ldx, int64_t N_tok, int64_t D, float* acc, void* workspace,
                                      size_t ws_bytes, void* stream) {
  if (!X_bf16 || !acc) return NVFP4_ERR_NULL;
  if (N_tok < 0 || D < 0) return NVFP4_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(X_bf16) & 15u) || ldx < D || (ldx * 2) % 16 != 0 || (reinterpret_cast<uintptr_t>(acc) & 3u))
    return NVFP4_ERR_ALIGN;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 15u) || ws_bytes < nvfp4_outlier_accumulate_workspace_bytes(N_tok, D))
    return NVFP4_ERR_WORKSPACE;
  if (!device_is_sm100()) return NVFP4_ERR_ARCH;
  if (N_tok == 0 || D == 0) return NVFP4_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t Dp = (D + 255) / 256 * 256;
  const int64_t slabs = calib_slabs(N_tok, D);
  const int64_t rows_per_slab = ((N_tok + slabs - 1) / slabs + 7) / 8 * 8;
  const int64_t used_slabs = (N_tok + rows_per_slab - 1) / rows_per_slab;
  float* partial = static_cast<float*>(workspace);
  launch_kernel(colsq_partial_kernel, dim3((unsigned)(Dp / 256), (unsigned)used_slabs), dim3(256), 0, st, static_cast<const uint16_t*>(X_bf16),
                ldx, N_tok, D, rows_per_slab, partial, Dp);
  if (cudaGetLastError() != cudaSuccess) return NVFP4_ERR_CUDA;
  launch_kernel(colsq_finalize_kernel, dim3((unsigned)((D + 255) / 256)), dim3(256), 0, st, static_cast<const float*>(partial), used_slabs, Dp, D,
                acc);
  return cudaGetLastError() == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

nvfp4_status nvfp4_outlier_select(const float* acc, int64_t D, int64_t n_out, int32_t* outlier_cols, int32_t* keep_cols,
                                  int32_t* col_map, void* stream) {
  if (D < 0 || n_out < 0 || n_out > D || D > 0x7FFFFFFF) return NVFP4_ERR_SHAPE;
  if (D == 0) return NVFP4_OK;
  if (!acc || !col_map || (n_out > 0 && !outlier_cols) || (n_out < D && !keep_cols)) return NVFP4_ERR_NULL;
  if (!device_is_sm100()) return NVFP4_ERR_ARCH;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  launch_kernel(outlier_rank_kernel, dim3((unsigned)((D + 255) / 256)), dim3(256), 0, st, acc, D, n_out, col_map);
  if (cudaGetLastError() != cudaSuccess) return NVFP4_ERR_CUDA;
  launch_kernel(outlier_compact_kernel, dim3(1), dim3(1024), 0, st, D, col_map, outlier_cols, keep_cols);
  return cudaGetLastError() == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

}  // extern "C"
