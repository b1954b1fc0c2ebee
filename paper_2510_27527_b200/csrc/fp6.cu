// Simulated FP6 x FP4 linear layer of the paper's precision-switching study (Sec. 5.4, "Precision Switching in Final Stage"):
//     Y = Q6_D(X) x Q4_D(W^T),   dX = Q6_S(dY) x Q4_S(W-hat),   dW = Q4_S(dY^T) x Q6_S(X-hat).
// The paper names FP6 without a recipe; this library's: element format E2M3 (32 magnitudes up to 7.5), the scale sequence of
// the FP4 quantizer (Sec. 2.2) with Q_max = 7.5 -- Sg = amax / 3360, t = amax_b / Sg, s = t / 7.5, Sb = e4m3(s), d = Sg Sb,
// r = 1 / d, y = x r, one binary32 operation each, |y| clamped to 7.5 -- per-tensor global scale, round to nearest (ties to
// the even code) or the 16-bit stochastic rounding of the FP4 quantizer with the same Philox addressing.
// No tensor-core instruction multiplies E2M3 by E2M1 under E4M3 block scales, and the paper itself simulates: the operands
// of the simulated products are "dense": P * S_block as BF16, which is exact for both formats (at most 4 + 4 significant
// bits), plus the FP32 global scale; the product runs on the BF16 tensor-core path of the 128 x 128 GEMM kernel with FP32
// accumulation and the two global scales in the epilogue.
#include <algorithm>

#include "nvfp4_device.cuh"
#include "nvfp4_internal.h"

namespace nvfp4 {

namespace {

// Round 16 scaled values to E2M3 and return them times the block scale as packed BF16 pairs (8 words).
// Stochastic rounding, exactly as for E2M1 with three mantissa bits instead of one: for a >= 1 the cell index and the
// position inside the cell are the exponent / top three mantissa bits and the low 20 mantissa bits of a itself; the cells
// below 1 (width 1/8) are mapped onto [0.5, 1) by z = 0.5 + a / 2 computed with round-up (an integer n is < x iff
// n < ceil(x)); adding 2^20 - 1 - ((2u + 1) << 3) to the bits carries into the cell index iff position > (2u + 1) << 3,
// i.e. iff (u + 0.5) / 65536 < position / 2^20; clearing the low 20 bits then leaves the rounded magnitude as a float (the
// carry moves through the exponent like the value does), mapped back by 2 z - 1 below 1.
template <bool SR>
__device__ __forceinline__ void fp6_block16(const float (&x)[16], float rcp, float Sbf, const PhiloxKeys& pk, uint32_t stream_id,
                                            uint64_t idx8, uint32_t (&out)[8]) {
  uint4 w[2];
  if (SR) {
    w[0] = sr_words(pk, stream_id, idx8);
    w[1] = sr_words(pk, stream_id, idx8 + 1);
  }
  float v[16];
#pragma unroll
  for (int i = 0; i < 16; i += 2) {
    const float y0 = __fmul_rn(x[i], rcp), y1 = __fmul_rn(x[i + 1], rcp);
    float p0, p1;
    if (SR) {
      const uint4& ww = w[i >> 3];
      const uint32_t word = ((i >> 1) & 3) == 0 ? ww.x : ((i >> 1) & 3) == 1 ? ww.y : ((i >> 1) & 3) == 2 ? ww.z : ww.w;
      const uint32_t u[2] = {word & 0xFFFFu, word >> 16};
      const float ys[2] = {y0, y1};
      float ps[2];
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const float a = fminf(fabsf(ys[e]), 7.5f);
        const float z = fmaxf(a, __fmaf_ru(a, 0.5f, 0.5f));
        const uint32_t bits = __float_as_uint(z) + (((~u[e] & 0xFFFFu) << 4) | 0x7u);
        const float zq = __uint_as_float(bits & 0xFFF00000u);
        const float mag = a >= 1.0f ? zq : __fmaf_rn(zq, 2.0f, -1.0f);
        ps[e] = __uint_as_float(__float_as_uint(mag) | (__float_as_uint(ys[e]) & 0x80000000u));
      }
      p0 = ps[0];
      p1 = ps[1];
    } else {
      // hardware conversion: round to nearest even, saturating at 7.5; then back to FP16 (exact)
      uint16_t packed;
      asm("cvt.rn.satfinite.e2m3x2.f32 %0, %1, %2;" : "=h"(packed) : "f"(y1), "f"(y0));
      uint32_t h2;
      asm("cvt.rn.f16x2.e2m3x2 %0, %1;" : "=r"(h2) : "h"(packed));
      const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&h2));
      p0 = f.x;
      p1 = f.y;
    }
    v[i] = __fmul_rn(p0, Sbf);  // exact: at most 4 + 4 significant bits
    v[i + 1] = __fmul_rn(p1, Sbf);
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) out[i] = (uint32_t)f32_to_bf16_bits(v[2 * i]) | ((uint32_t)f32_to_bf16_bits(v[2 * i + 1]) << 16);
}

// The scale pair of a block: E4M3 block scale as a float and the reciprocal that maps x onto the E2M3 grid.
__device__ __forceinline__ float fp6_block_scale(float amax_b, float Sg, float& rcp) {
  const float t = __fdiv_rn(amax_b, Sg);
  const float s = __fdiv_rn(t, 7.5f);
  const float Sbf = e4m3_decode(e4m3_encode(s));
  const float d = __fmul_rn(Sg, Sbf);
  rcp = Sbf == 0.0f ? 0.0f : __frcp_rn(d);
  return Sbf;
}
__device__ __forceinline__ float fp6_global_scale(float amax) { return amax == 0.0f ? 1.0f : __fdiv_rn(amax, 3360.0f); }

// Row-axis FP6 quantize from BF16 [rows, cols] (leading dimension ld): one thread per 16-element block of the padded output
// row (ld_out / 16 blocks: those past K are written as zeros). cell[0] = bits of max |x| over the tensor.
template <bool SR>
__global__ void __launch_bounds__(256)
fp6_quantize_rows_kernel(const uint16_t* __restrict__ src, int64_t rows, int64_t K, int64_t ld, uint32_t stream_id,
                         const uint32_t* __restrict__ cell, uint16_t* __restrict__ out, int64_t ld_out, float* __restrict__ gscale,
                         const __grid_constant__ PhiloxKeys pk) {
  pdl_prologue();
  const int64_t nb = ld_out >> 4;
  const int64_t gid = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (gid >= rows * nb) return;
  const int64_t r = gid / nb, b = gid - r * nb;
  const int64_t k0 = b << 4;
  const int64_t K16 = (K + 15) & ~(int64_t)15;
  const float Sg = fp6_global_scale(__uint_as_float(cell[0]));
  if (gid == 0) gscale[0] = Sg;
  uint4* dst = reinterpret_cast<uint4*>(out + r * ld_out + k0);
  if (k0 >= K) {
    dst[0] = dst[1] = make_uint4(0, 0, 0, 0);
    return;
  }
  float x[16];
  const uint16_t* p = src + r * ld + k0;
  if (k0 + 16 <= K && (ld & 7) == 0 && (reinterpret_cast<uintptr_t>(src) & 15u) == 0) {
    const uint4 a = *reinterpret_cast<const uint4*>(p), c = *reinterpret_cast<const uint4*>(p + 8);
    const uint32_t w[8] = {a.x, a.y, a.z, a.w, c.x, c.y, c.z, c.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      x[2 * i] = bf16_lo(w[i]);
      x[2 * i + 1] = bf16_hi(w[i]);
    }
  } else {
#pragma unroll
    for (int i = 0; i < 16; ++i) x[i] = k0 + i < K ? bf16_bits_to_float(p[i]) : 0.0f;
  }
  float m = 0.0f;
#pragma unroll
  for (int i = 0; i < 16; ++i) m = fmaxf(m, fabsf(x[i]));
  float rcp;
  const float Sbf = fp6_block_scale(m, Sg, rcp);
  uint32_t o[8];
  fp6_block16<SR>(x, rcp, Sbf, pk, stream_id, (uint64_t)(r * K16 + k0) >> 3, o);
  dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
  dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
}

// Transposing FP6 re-quantize of a dense operand: in [rowsK, D] (values v, global scale Sg_in) -> out [D, rowsK] with blocks
// along the source rows. x_hat = float32(v * Sg_in) is the aligned tensor (one rounding). A lane owns four neighbouring
// source columns and one 16-row block (8 bytes per source row: a warp reads 256 contiguous bytes per row). cell[0] = bits of
// max |v|; the maximum of x_hat is float32(max |v| * Sg_in) because the multiplication is monotonic.
template <bool SR>
__global__ void __launch_bounds__(128)
fp6_requantize_t_kernel(const uint16_t* __restrict__ in, int64_t rowsK, int64_t D, int64_t ld_in, const float* __restrict__ in_gscale,
                        uint32_t stream_id, const uint32_t* __restrict__ cell, uint16_t* __restrict__ out, int64_t ld_out,
                        float* __restrict__ gscale, const __grid_constant__ PhiloxKeys pk) {
  pdl_prologue();
  const int64_t d0 = ((int64_t)blockIdx.y * 32 + (threadIdx.x & 31)) * 4;
  const int64_t k0 = ((int64_t)blockIdx.x * 4 + (threadIdx.x >> 5)) * 16;
  const float sg_in = in_gscale[0];
  const float Sg = fp6_global_scale(__fmul_rn(__uint_as_float(cell[0]), sg_in));
  if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) gscale[0] = Sg;
  if (d0 >= D || k0 >= ld_out) return;
  const int64_t K16 = (rowsK + 15) & ~(int64_t)15;
  uint2 w[16];
#pragma unroll
  for (int t = 0; t < 16; ++t)
    w[t] = k0 + t < rowsK ? *reinterpret_cast<const uint2*>(in + (k0 + t) * ld_in + d0) : make_uint2(0u, 0u);  // ld_in, d0: multiples of 4
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    if (d0 + c >= D) break;
    uint4* dst = reinterpret_cast<uint4*>(out + (d0 + c) * ld_out + k0);
    if (k0 >= rowsK) {
      dst[0] = dst[1] = make_uint4(0, 0, 0, 0);
      continue;
    }
    float x[16], m = 0.0f;
#pragma unroll
    for (int t = 0; t < 16; ++t) {
      const uint32_t word = c < 2 ? w[t].x : w[t].y;
      x[t] = __fmul_rn((c & 1) ? bf16_hi(word) : bf16_lo(word), sg_in);
      m = fmaxf(m, fabsf(x[t]));
    }
    float rcp;
    const float Sbf = fp6_block_scale(m, Sg, rcp);
    uint32_t o[8];
    fp6_block16<SR>(x, rcp, Sbf, pk, stream_id, (uint64_t)((d0 + c) * K16 + k0) >> 3, o);
    dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
    dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
  }
}

// FP4 operand (codes + E4M3 scales in either layout) -> dense BF16 values P * S_block [R, ld_out]; one thread per 8 codes.
__global__ void __launch_bounds__(256)
expand_operand_kernel(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ sf, int sf_tiled, int64_t R, int64_t K,
                      const float* __restrict__ in_gscale, uint16_t* __restrict__ out, int64_t ld_out, float* __restrict__ gscale) {
  pdl_prologue();
  const int64_t n8 = ld_out >> 3;
  const int64_t gid = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (gid == 0) gscale[0] = in_gscale[0];
  if (gid >= R * n8) return;
  const int64_t r = gid / n8, k0 = (gid - r * n8) << 3;
  const int64_t Kp = (K + 127) & ~(int64_t)127;
  uint4 o = make_uint4(0, 0, 0, 0);
  if (k0 < Kp) {
    const uint32_t word = *reinterpret_cast<const uint32_t*>(codes + r * (Kp >> 1) + (k0 >> 1));
    const int64_t nb = Kp >> 4;
    const size_t sfo = sf_tiled ? sf_tiled_offset(r, k0 >> 4, (nb + 15) & ~(int64_t)15) : (size_t)(r * nb + (k0 >> 4));
    uint32_t h[4];
    decode8_h2(word, sf[sfo], h);
    uint32_t q[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&h[i]));
      q[i] = (uint32_t)f32_to_bf16_bits(f.x) | ((uint32_t)f32_to_bf16_bits(f.y) << 16);  // exact: 2 + 4 significant bits
    }
    o = make_uint4(q[0], q[1], q[2], q[3]);
  }
  *reinterpret_cast<uint4*>(out + r * ld_out + k0) = o;
}

}  // namespace

cudaError_t launch_fp6_quantize_rows(const uint16_t* src, int64_t rows, int64_t K, int64_t ld, int sr, uint64_t seed, uint32_t stream_id,
                                     uint32_t* cell, uint16_t* out, int64_t ld_out, float* gscale, cudaStream_t st) {
  if (rows == 0) return cudaSuccess;
  cudaError_t e;
  if ((e = launch_zero_words(cell, 1, st)) != cudaSuccess) return e;
  if ((e = launch_amax_tensor(src, rows, K, ld, cell, st)) != cudaSuccess) return e;
  const unsigned grid = (unsigned)((rows * (ld_out >> 4) + 255) / 256);
  const uint32_t* ccell = cell;
  if (sr)
    launch_kernel(fp6_quantize_rows_kernel<true>, dim3(grid), dim3(256), 0, st, src, rows, K, ld, stream_id, ccell, out, ld_out, gscale,
                  make_philox_keys(seed));
  else
    launch_kernel(fp6_quantize_rows_kernel<false>, dim3(grid), dim3(256), 0, st, src, rows, K, ld, stream_id, ccell, out, ld_out, gscale,
                  make_philox_keys(seed));
  return cudaGetLastError();
}

cudaError_t launch_fp6_requantize_t(const uint16_t* in, int64_t rowsK, int64_t D, int64_t ld_in, const float* in_gscale, int sr,
                                    uint64_t seed, uint32_t stream_id, uint32_t* cell, uint16_t* out, int64_t ld_out, float* gscale,
                                    cudaStream_t st) {
  if (rowsK == 0 || D == 0) return cudaSuccess;
  cudaError_t e;
  if ((e = launch_zero_words(cell, 1, st)) != cudaSuccess) return e;
  if ((e = launch_amax_tensor(in, rowsK, D, ld_in, cell, st)) != cudaSuccess) return e;
  const dim3 grid((unsigned)((ld_out / 16 + 3) / 4), (unsigned)((D + 127) / 128));
  const uint32_t* ccell = cell;
  if (sr)
    launch_kernel(fp6_requantize_t_kernel<true>, grid, dim3(128), 0, st, in, rowsK, D, ld_in, in_gscale, stream_id, ccell, out, ld_out,
                  gscale, make_philox_keys(seed));
  else
    launch_kernel(fp6_requantize_t_kernel<false>, grid, dim3(128), 0, st, in, rowsK, D, ld_in, in_gscale, stream_id, ccell, out, ld_out,
                  gscale, make_philox_keys(seed));
  return cudaGetLastError();
}

cudaError_t launch_expand_operand(const uint8_t* codes, const uint8_t* sf, int sf_tiled, int64_t R, int64_t K, const float* in_gscale,
                                  uint16_t* out, int64_t ld_out, float* gscale, cudaStream_t st) {
  if (R == 0) return cudaSuccess;
  const unsigned grid = (unsigned)((R * (ld_out >> 3) + 255) / 256);
  launch_kernel(expand_operand_kernel, dim3(grid), dim3(256), 0, st, codes, sf, sf_tiled, R, K, in_gscale, out, ld_out, gscale);
  return cudaGetLastError();
}

}  // namespace nvfp4
