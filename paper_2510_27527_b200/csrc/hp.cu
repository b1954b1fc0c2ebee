// High-precision side of OutControl (paper Sec. 4.2): the few outlier channels of X / W stay in BF16 and their
// products are accumulated in FP32 on the CUDA cores. With the paper-scale channel counts used here (about 1 % of
// the hidden size) these products are a tiny fraction of the layer's flops; the kernels are bound by reading dY and
// by writing the FP32 addend.
#include "nvfp4_device.cuh"
#include "nvfp4_internal.h"

namespace nvfp4 {

// Y[m, n] = sum_j X[m, outl[j]] * W[n, outl[j]].  CTA tile 64 x 64, outlier channels in chunks of 32.
__global__ void __launch_bounds__(256) hp_fwd_kernel(HpFwdArgs a) {
  pdl_prologue();
  __shared__ float xs[32][65];
  __shared__ float ws[32][65];
  const int64_t m0 = (int64_t)blockIdx.y * 64, n0 = (int64_t)blockIdx.x * 64;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;  // 16 x 16 threads, 4 x 4 outputs each
  float acc[4][4] = {};
  for (int64_t j0 = 0; j0 < a.n_out; j0 += 32) {
    for (int e = threadIdx.x; e < 32 * 64; e += 256) {
      const int jj = e & 31, rr = e >> 5;
      const int64_t j = j0 + jj;
      float xv = 0.0f, wv = 0.0f;
      if (j < a.n_out) {
        const int64_t col = a.outl[j];
        if (m0 + rr < a.M) xv = bf16_bits_to_float(a.X[(m0 + rr) * a.ldx + col]);
        if (n0 + rr < a.N) wv = bf16_bits_to_float(a.W[(n0 + rr) * a.ldw + col]);
      }
      xs[jj][rr] = xv;
      ws[jj][rr] = wv;
    }
    __syncthreads();
#pragma unroll 4
    for (int jj = 0; jj < 32; ++jj) {
      float xv[4], wv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        xv[i] = xs[jj][ty * 4 + i];
        wv[i] = ws[jj][tx * 4 + i];
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int k = 0; k < 4; ++k) acc[i][k] = fmaf(xv[i], wv[k], acc[i][k]);
    }
    __syncthreads();
  }
  for (int i = 0; i < 4; ++i) {
    const int64_t m = m0 + ty * 4 + i;
    if (m >= a.M) continue;
    for (int k = 0; k < 4; ++k) {
      const int64_t n = n0 + tx * 4 + k;
      if (n < a.N) a.Y[m * a.ldy + n] = acc[i][k];
    }
  }
}

// dW[c, outl[j]] = sum_t dY[t, c] * X[t, outl[j]].  One CTA per (64 output channels c, 8 outlier channels j);
// four token groups per CTA reduced through shared memory in a fixed order.
__global__ void __launch_bounds__(256) hp_dw_kernel(HpDwArgs a) {
  pdl_prologue();
  __shared__ float red[4][8][64];
  const int cl = threadIdx.x & 63, tg = threadIdx.x >> 6;
  const int64_t c = (int64_t)blockIdx.x * 64 + cl;
  const int64_t j0 = (int64_t)blockIdx.y * 8;
  int64_t cols[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) cols[j] = (j0 + j < a.n_out) ? a.outl[j0 + j] : -1;
  float acc[8] = {};
  if (c < a.C) {
    for (int64_t t = tg; t < a.T; t += 4) {
      const float g = bf16_bits_to_float(a.dY[t * a.lddy + c]);
      const uint16_t* xr = a.X + t * a.ldx;
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (cols[j] >= 0) acc[j] = fmaf(g, bf16_bits_to_float(xr[cols[j]]), acc[j]);
    }
  }
#pragma unroll
  for (int j = 0; j < 8; ++j) red[tg][j][cl] = acc[j];
  __syncthreads();
  if (tg == 0 && c < a.C) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (cols[j] < 0) continue;
      const float v = ((red[0][j][cl] + red[1][j][cl]) + red[2][j][cl]) + red[3][j][cl];
      if (a.dw_is_f32)
        reinterpret_cast<float*>(a.dW)[c * a.lddw + cols[j]] = v;
      else
        reinterpret_cast<uint16_t*>(a.dW)[c * a.lddw + cols[j]] = f32_to_bf16_bits(v);
    }
  }
}

// dst[r, keep[j]] = src[r, j]
__global__ void __launch_bounds__(256) scatter_cols_kernel(const void* src, int64_t ld_src, int src_is_f32, void* dst,
                                                          int64_t ld_dst, int dst_is_f32, int64_t rows, int64_t n_keep,
                                                          const int32_t* __restrict__ keep) {
  pdl_prologue();
  const int64_t total = rows * n_keep;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = i / n_keep, j = i - r * n_keep;
    const int64_t o = r * ld_dst + keep[j];
    if (src_is_f32) {
      const float v = reinterpret_cast<const float*>(src)[r * ld_src + j];
      if (dst_is_f32) {
        reinterpret_cast<float*>(dst)[o] = v;
      } else {
        reinterpret_cast<uint16_t*>(dst)[o] = f32_to_bf16_bits(v);
      }
    } else {
      const uint16_t v = reinterpret_cast<const uint16_t*>(src)[r * ld_src + j];
      if (dst_is_f32)
        reinterpret_cast<float*>(dst)[o] = bf16_bits_to_float(v);
      else
        reinterpret_cast<uint16_t*>(dst)[o] = v;
    }
  }
}

cudaError_t launch_hp_fwd(const HpFwdArgs& a, cudaStream_t st) {
  if (a.M == 0 || a.N == 0) return cudaSuccess;
  const dim3 grid((unsigned)((a.N + 63) / 64), (unsigned)((a.M + 63) / 64));
  launch_kernel(hp_fwd_kernel, dim3(grid), dim3(256), 0, st, a);
  return cudaGetLastError();
}

cudaError_t launch_hp_dw(const HpDwArgs& a, cudaStream_t st) {
  if (a.C == 0 || a.n_out == 0) return cudaSuccess;
  const dim3 grid((unsigned)((a.C + 63) / 64), (unsigned)((a.n_out + 7) / 8));
  launch_kernel(hp_dw_kernel, dim3(grid), dim3(256), 0, st, a);
  return cudaGetLastError();
}

cudaError_t launch_scatter_cols(const void* src, int64_t ld_src, int src_is_f32, void* dst, int64_t ld_dst,
                                int dst_is_f32, int64_t rows, int64_t n_keep, const int32_t* keep, cudaStream_t st) {
  const int64_t total = rows * n_keep;
  if (total == 0) return cudaSuccess;
  const unsigned grid = (unsigned)std::min<int64_t>((total + 255) / 256, 148 * 32);
  launch_kernel(scatter_cols_kernel, dim3(grid), dim3(256), 0, st, src, ld_src, src_is_f32, dst, ld_dst, dst_is_f32, rows, n_keep, keep);
  return cudaGetLastError();
}

}  // namespace nvfp4
