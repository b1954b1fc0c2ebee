// The 16x16 weight-block recipe that the paper compares its 1x16 weight blocks with (Sec. 2.3, third difference to
// NVIDIA's recipe; appendix on the overhead of the 1x16 weight scaling): the E4M3 scale of a weight is shared by a 16x16
// square, so W and W^T carry the same quantized values and the backward product dX = Q3(dY) x W-hat reads the forward
// codes as they are. Two kernels:
//   quantize_w16_kernel        BF16 W [C, D] -> operand [C, D] whose 16 rows of a square repeat the square's scale
//                              (per-tensor global scale from an amax cell; round to nearest)
//   transpose_operand_kernel   operand [C, D] -> operand [D, C]: nibbles transposed, scales re-indexed; no arithmetic
#include "../../include/nvfp4.h"

#include "nvfp4_device.cuh"
#include "nvfp4_internal.h"

namespace nvfp4 {

// CTA = 16 rows x 16 column blocks (256 columns). A warp holds two squares: lane = row in the square + 16 * (which square),
// so the square's maximum is four xor-shuffles over 16 lanes.
__global__ void __launch_bounds__(256) quantize_w16_kernel(const uint16_t* __restrict__ src, int64_t C, int64_t D, int64_t ld,
                                                          const uint32_t* __restrict__ amax_cell, uint8_t* __restrict__ codes,
                                                          uint8_t* __restrict__ sf, float* __restrict__ gscale, int tiled) {
  pdl_prologue();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t Kp = (D + 127) & ~(int64_t)127;
  const int64_t nb = Kp >> 4;
  const int64_t r = (int64_t)blockIdx.y * 16 + (lane & 15);
  const int64_t b = (int64_t)blockIdx.x * 16 + warp * 2 + (lane >> 4);
  const int64_t k0 = b << 4;
  float x[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) x[i] = 0.0f;
  if (r < C && b < nb && k0 < D) {
    const uint16_t* p = src + r * ld + k0;
    if (k0 + 16 <= D && (ld & 7) == 0) {
      const uint4 v0 = *reinterpret_cast<const uint4*>(p), v1 = *reinterpret_cast<const uint4*>(p + 8);
      const uint32_t w[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        x[2 * i] = bf16_lo(w[i]);
        x[2 * i + 1] = bf16_hi(w[i]);
      }
    } else {
      for (int i = 0; i < 16; ++i)
        if (k0 + i < D) x[i] = bf16_bits_to_float(p[i]);
    }
  }
  float m = 0.0f;
#pragma unroll
  for (int i = 0; i < 16; ++i) m = fmaxf(m, fabsf(x[i]));
#pragma unroll
  for (int o = 1; o < 16; o <<= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));  // over the square's 16 rows
  const float Sg = global_scale_from_amax(__uint_as_float(amax_cell[0]));
  if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) gscale[0] = Sg;
  float rcp;
  const uint32_t sb = block_scale(m, Sg, rcp);
  if (r < C && b < nb) {
    PhiloxKeys unused{};
    const uint2 packed = quantize_block16<false>(x, rcp, unused, 0u, 0ull);
    *reinterpret_cast<uint2*>(codes + r * (Kp >> 1) + (k0 >> 1)) = packed;
    const size_t off = tiled ? sf_tiled_offset(r, b, (nb + 15) & ~(int64_t)15) : (size_t)(r * nb + b);
    sf[off] = k0 < D ? (uint8_t)sb : (uint8_t)0;
  }
}

// Tile = 64 source rows (c) x 64 source columns (d). in: codes [C, Dp / 2], scales per (c, d / 16); out: codes [D, Cp / 2],
// scales per (d, c / 16). Only defined for operands made by quantize_w16_kernel (the 16 rows of a square share a scale).
__global__ void __launch_bounds__(256) transpose_operand_kernel(const uint8_t* __restrict__ in_codes, const uint8_t* __restrict__ in_sf,
                                                               int in_tiled, const float* __restrict__ in_gscale, int64_t C, int64_t D,
                                                               uint8_t* __restrict__ out_codes, uint8_t* __restrict__ out_sf, int out_tiled,
                                                               float* __restrict__ out_gscale) {
  pdl_prologue();
  __shared__ uint8_t nib[64][65];  // [c][d], one code per byte
  const int64_t Dp = (D + 127) & ~(int64_t)127, Cp = (C + 127) & ~(int64_t)127;
  const int64_t c_base = (int64_t)blockIdx.x * 64, d_base = (int64_t)blockIdx.y * 64;
  const int tid = threadIdx.x;
  {
    const int row = tid >> 2, piece = tid & 3;  // 16 codes (8 bytes) per thread
    const int64_t c = c_base + row;
    uint2 v = make_uint2(0, 0);
    if (c < C && d_base + piece * 16 < Dp) v = *reinterpret_cast<const uint2*>(in_codes + c * (Dp >> 1) + (d_base >> 1) + piece * 8);
    const uint32_t w[2] = {v.x, v.y};
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const int64_t d = d_base + piece * 16 + i;
      nib[row][piece * 16 + i] = d < D ? (uint8_t)((w[i >> 3] >> (4 * (i & 7))) & 15u) : (uint8_t)0;
    }
  }
  __syncthreads();
  {
    const int row = tid >> 2, piece = tid & 3;
    const int64_t d = d_base + row;
    if (d < D && c_base + piece * 16 < Cp) {
      uint32_t w[2] = {0, 0};
#pragma unroll
      for (int i = 0; i < 16; ++i) w[i >> 3] |= (uint32_t)nib[piece * 16 + i][row] << (4 * (i & 7));
      *reinterpret_cast<uint2*>(out_codes + d * (Cp >> 1) + (c_base >> 1) + piece * 8) = make_uint2(w[0], w[1]);
      // the scale of (d, block c / 16) is the square's: read it at the square's first row
      const int64_t cb = (c_base >> 4) + piece, c0 = cb << 4;
      const int64_t in_nb = Dp >> 4, out_nb = Cp >> 4;
      uint8_t sv = 0;
      if (c0 < C) sv = in_sf[in_tiled ? sf_tiled_offset(c0, d >> 4, (in_nb + 15) & ~(int64_t)15) : (size_t)(c0 * in_nb + (d >> 4))];
      out_sf[out_tiled ? sf_tiled_offset(d, cb, (out_nb + 15) & ~(int64_t)15) : (size_t)(d * out_nb + cb)] = sv;
    }
  }
  if (blockIdx.x == 0 && blockIdx.y == 0 && tid == 0) out_gscale[0] = in_gscale[0];
}

cudaError_t launch_quantize_w16(const uint16_t* src, int64_t C, int64_t D, int64_t ld, const uint32_t* amax_cell, uint8_t* codes,
                                uint8_t* sf, float* gscale, int tiled, cudaStream_t st) {
  if (C == 0 || D == 0) return cudaSuccess;
  const int64_t nb = ((D + 127) & ~(int64_t)127) >> 4;
  const dim3 grid((unsigned)((nb + 15) / 16), (unsigned)((C + 15) / 16));
  launch_kernel(quantize_w16_kernel, grid, dim3(256), 0, st, src, C, D, ld, amax_cell, codes, sf, gscale, tiled);
  return cudaGetLastError();
}

cudaError_t launch_transpose_operand(const uint8_t* in_codes, const uint8_t* in_sf, int in_tiled, const float* in_gscale, int64_t C, int64_t D,
                                     uint8_t* out_codes, uint8_t* out_sf, int out_tiled, float* out_gscale, cudaStream_t st) {
  if (C == 0 || D == 0) return cudaSuccess;
  const int64_t Cp = (C + 127) & ~(int64_t)127;
  const dim3 grid((unsigned)(Cp / 64), (unsigned)((D + 63) / 64));
  launch_kernel(transpose_operand_kernel, grid, dim3(256), 0, st, in_codes, in_sf, in_tiled, in_gscale, C, D, out_codes, out_sf, out_tiled,
                out_gscale);
  return cudaGetLastError();
}

}  // namespace nvfp4
