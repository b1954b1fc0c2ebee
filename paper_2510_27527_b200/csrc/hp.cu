// High-precision side of OutControl (paper Sec. 4.2): the outlier channels of X / W stay in BF16. The forward side
// product runs on the tensor cores inside the FP4 GEMM kernels and dW[:, outliers] = dY^T X_out in a BF16 tensor-core
// kernel of its own (gemm.cu); here are the copy that builds a compact side operand, the FP8 snap of the side operands,
// and the pass that assembles dW from the compact FP4 product and the side product's token splits.
#include "nvfp4_device.cuh"
#include "nvfp4_internal.h"

namespace nvfp4 {

// Token splits of the side product dW[c, outl[j]] = sum_t dY[t, c] * X_out[t, j]: at most kHpDwSplit partial sums per output
// element go to a workspace and are added in a fixed order (bit-reproducible results).
constexpr int kHpDwSplit = 16;

// dW[c, d] for whole output rows (OutControl's weight gradient): a kept channel takes its value from the compact FP4
// product, an outlier channel the sum of the high-precision side product's token splits. One coalesced pass over dW
// instead of a column scatter plus a scattered reduce. Each CTA first builds, in shared memory, where every channel comes
// from: src_of[d] = position in the compact product (>= 0) or -(1 + rank among the outliers). Rows are then taken four at a
// time: all threads first reduce the splits of the group's outlier channels into shared memory (fixed order), then all
// threads assemble and store the four rows.
constexpr int kAsmRows = 4;
template <bool F32>
__global__ void __launch_bounds__(256) dw_assemble_kernel(HpDwArgs a, int n_split, const float* __restrict__ compact, int64_t ld_compact,
                                                         const int32_t* __restrict__ col_map, int64_t D, int vec) {
  pdl_prologue();
  extern __shared__ int32_t src_of[];                                       // [D]
  float* osum = reinterpret_cast<float*>(src_of + ((D + 3) & ~(int64_t)3));  // [kAsmRows][n_out]
  for (int64_t d = threadIdx.x; d < D; d += 256) src_of[d] = col_map[d];
  __syncthreads();
  for (int64_t j = threadIdx.x; j < a.n_out; j += 256) src_of[a.outl[j]] = -(int32_t)(1 + j);
  __syncthreads();
  const uint32_t n_out = (uint32_t)a.n_out, D32 = (uint32_t)D;
  const uint32_t chunks = (D32 + 3) >> 2;
  for (int64_t c0 = (int64_t)blockIdx.x * kAsmRows; c0 < a.C; c0 += (int64_t)gridDim.x * kAsmRows) {
    const uint32_t nr = (uint32_t)min((int64_t)kAsmRows, a.C - c0);
    for (uint32_t e = threadIdx.x; e < nr * n_out; e += 256) {
      const uint32_t rr = e / n_out, j = e - rr * n_out;
      const float* p = a.partial + (c0 + rr) * a.Kh + j;
      float v = 0.0f;
      for (int sp = 0; sp < n_split; ++sp) v += p[(int64_t)sp * a.C * a.Kh];  // fixed order
      osum[rr * n_out + j] = v;
    }
    __syncthreads();
    if (vec) {  // four channels per item, one 16-byte (FP32) or 8-byte (BF16) store
      for (uint32_t e = threadIdx.x; e < nr * chunks; e += 256) {
        const uint32_t rr = e / chunks, d = (e - rr * chunks) << 2;
        const int64_t c = c0 + rr;
        float v[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          v[i] = 0.0f;
          if (d + i < D32) {
            const int32_t m = src_of[d + i];
            v[i] = m >= 0 ? compact[c * ld_compact + m] : osum[rr * n_out + (uint32_t)(-m - 1)];
          }
        }
        if (d + 4 <= D32) {
          if (F32)
            *reinterpret_cast<float4*>(reinterpret_cast<float*>(a.dW) + c * a.lddw + d) = make_float4(v[0], v[1], v[2], v[3]);
          else
            *reinterpret_cast<uint2*>(reinterpret_cast<uint16_t*>(a.dW) + c * a.lddw + d) =
                make_uint2((uint32_t)f32_to_bf16_bits(v[0]) | ((uint32_t)f32_to_bf16_bits(v[1]) << 16),
                           (uint32_t)f32_to_bf16_bits(v[2]) | ((uint32_t)f32_to_bf16_bits(v[3]) << 16));
        } else {
          for (int i = 0; d + i < D32; ++i) {
            if (F32)
              reinterpret_cast<float*>(a.dW)[c * a.lddw + d + i] = v[i];
            else
              reinterpret_cast<uint16_t*>(a.dW)[c * a.lddw + d + i] = f32_to_bf16_bits(v[i]);
          }
        }
      }
    } else {
      for (uint32_t e = threadIdx.x; e < nr * D32; e += 256) {
        const uint32_t rr = e / D32, d = e - rr * D32;
        const int64_t c = c0 + rr;
        const int32_t m = src_of[d];
        const float v = m >= 0 ? compact[c * ld_compact + m] : osum[rr * n_out + (uint32_t)(-m - 1)];
        if (F32)
          reinterpret_cast<float*>(a.dW)[c * a.lddw + d] = v;
        else
          reinterpret_cast<uint16_t*>(a.dW)[c * a.lddw + d] = f32_to_bf16_bits(v);
      }
    }
    __syncthreads();  // osum is rewritten by the next group
  }
}

// FP8 option for the outlier channels (paper Sec. 4.2 names FP8 as a possible precision of the outlier part; the recipe
// is this library's): a compact side operand T (BF16, contiguous) is replaced in place by the values an E4M3 tensor
// with a per-tensor power-of-two scale represents:  e = smallest integer with amax / 2^e <= 448,  T8 = E4M3(T / 2^e) 2^e.
// Both scalings are exact and T8 is exactly representable in BF16, so the BF16 tensor-core products that consume the
// side operands give what an FP8 product times the two scales would give. cell holds the float bits of amax(|T|).
__device__ __forceinline__ void fp8_snap_body(uint16_t* __restrict__ t, int64_t n, const uint32_t* __restrict__ cell, unsigned block,
                                              unsigned n_blocks) {
  const uint32_t ab = cell[0];
  int e = 0;
  if (ab) {
    const int k = (int)((ab >> 23) & 0xFFu) - 127;
    e = (ab & 0x7FFFFFu) <= 0x600000u ? k - 8 : k - 7;  // mantissa <= 1.75: amax / 2^(k - 8) = m 2^8 <= 448
  }
  const float r = __uint_as_float((uint32_t)(127 - e) << 23), s = __uint_as_float((uint32_t)(127 + e) << 23);
  const int64_t pairs = n >> 1;  // n is even (the padded width is a multiple of 64)
  uint32_t* t2 = reinterpret_cast<uint32_t*>(t);
  for (int64_t i = (int64_t)block * blockDim.x + threadIdx.x; i < pairs; i += (int64_t)n_blocks * blockDim.x) {
    const uint32_t w = t2[i];
    const float lo = __fmul_rn(bf16_lo(w), r), hi = __fmul_rn(bf16_hi(w), r);
    uint32_t h2;
    asm("{\n.reg .b16 q;\ncvt.rn.satfinite.e4m3x2.f32 q, %1, %2;\ncvt.rn.f16x2.e4m3x2 %0, q;\n}" : "=r"(h2) : "f"(hi), "f"(lo));
    const float qlo = __half2float(__ushort_as_half((unsigned short)(h2 & 0xFFFFu)));
    const float qhi = __half2float(__ushort_as_half((unsigned short)(h2 >> 16)));
    t2[i] = (uint32_t)f32_to_bf16_bits(__fmul_rn(qlo, s)) | ((uint32_t)f32_to_bf16_bits(__fmul_rn(qhi, s)) << 16);
  }
}
__global__ void __launch_bounds__(256) fp8_snap_pair_kernel(uint16_t* a, int64_t n_a, const uint32_t* cell_a, unsigned grid_a, uint16_t* b,
                                                           int64_t n_b, const uint32_t* cell_b) {
  pdl_prologue();
  if (blockIdx.x < grid_a)
    fp8_snap_body(a, n_a, cell_a, blockIdx.x, grid_a);
  else
    fp8_snap_body(b, n_b, cell_b, blockIdx.x - grid_a, gridDim.x - grid_a);
}

cudaError_t launch_fp8_snap_pair(uint16_t* a, int64_t rows_a, uint16_t* b, int64_t rows_b, int64_t Kh, uint32_t* cells2, cudaStream_t st) {
  if (Kh == 0 || (rows_a == 0 && rows_b == 0)) return cudaSuccess;
  cudaError_t e;
  if ((e = launch_zero_words(cells2, 2, st)) != cudaSuccess) return e;
  if ((e = launch_amax_tensor_pair(a, rows_a, Kh, Kh, cells2, b, rows_b, Kh, Kh, cells2 + 1, st)) != cudaSuccess) return e;
  const int64_t cap = (int64_t)device_sm_count() * 4;
  auto grid_of = [cap](int64_t n) { return (unsigned)std::max<int64_t>(1, std::min<int64_t>((n / 2 + 255) / 256, cap)); };
  const unsigned ga = grid_of(rows_a * Kh), gb = grid_of(rows_b * Kh);
  launch_kernel(fp8_snap_pair_kernel, dim3(ga + gb), dim3(256), 0, st, a, rows_a * Kh, static_cast<const uint32_t*>(cells2), ga, b,
                rows_b * Kh, static_cast<const uint32_t*>(cells2 + 1));
  return cudaGetLastError();
}

// dst[r, j] = src[r, cols[j]] (j < n), 0 for n <= j < ld_dst. One warp per row.
__global__ void __launch_bounds__(256) gather_cols_kernel(const uint16_t* __restrict__ src, int64_t ld_src, int64_t rows,
                                                         const int32_t* __restrict__ cols, int64_t n, uint16_t* __restrict__ dst,
                                                         int64_t ld_dst) {
  pdl_prologue();
  const int64_t r = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (r >= rows) return;
  for (int64_t j = threadIdx.x & 31; j < ld_dst; j += 32) dst[r * ld_dst + j] = j < n ? src[r * ld_src + cols[j]] : (uint16_t)0;
}

size_t hp_dw_partial_floats(int64_t T, int64_t C, int64_t Kh) { return (size_t)kHpDwSplit * (size_t)C * (size_t)Kh; }

// token splits of the side product: as many as fill the SMs once with (C / 128) x splits CTAs, at most kHpDwSplit (the
// workspace's size)
static void hp_dw_splits(const HpDwArgs& a, int64_t& t_per_split, int& n_split) {
  const int64_t want = std::max<int64_t>(1, std::min<int64_t>(kHpDwSplit, device_sm_count() / std::max<int64_t>(1, (a.C + 127) / 128)));
  t_per_split = ((a.T + want - 1) / want + 63) / 64 * 64;
  n_split = (int)((a.T + t_per_split - 1) / t_per_split);
}

// First half of dW under OutControl: the split partial sums of dY^T X_out (needs nothing of the FP4 product).
cudaError_t launch_hp_dw_product(const HpDwArgs& a, cudaStream_t st) {
  if (a.C == 0 || a.n_out == 0) return cudaSuccess;
  int64_t t_per_split;
  int n_split;
  hp_dw_splits(a, t_per_split, n_split);
  return launch_hp_dw_mma(a.dY, a.lddy, a.X_out, a.Kh, a.T, a.C, a.partial, n_split, t_per_split, a.dev_status, st);
}

// Second half: dW from the compact FP4 product and the split partial sums.
cudaError_t launch_hp_dw_finish(const HpDwArgs& a, cudaStream_t st) {
  if (a.C == 0 || a.n_out == 0) return cudaSuccess;
  int64_t t_per_split;
  int n_split;
  hp_dw_splits(a, t_per_split, n_split);
  if (!a.compact || !a.col_map || !hp_dw_assemble_fits(a.D, a.n_out)) return cudaErrorInvalidValue;
  // kept and outlier channels written together, row by row
  const size_t smem = (size_t)(((a.D + 3) & ~(int64_t)3) + kAsmRows * a.n_out) * 4;
  const int f32 = a.dw_is_f32;
  const int elt = f32 ? 4 : 2;
  const int vec = (a.lddw & 3) == 0 && (reinterpret_cast<uintptr_t>(a.dW) & (size_t)(4 * elt - 1)) == 0;
  const cudaError_t e = ensure_dynamic_smem(f32 ? reinterpret_cast<const void*>(dw_assemble_kernel<true>)
                                                : reinterpret_cast<const void*>(dw_assemble_kernel<false>), smem);
  if (e != cudaSuccess) return e;
  const dim3 grid((unsigned)std::min<int64_t>((a.C + kAsmRows - 1) / kAsmRows, (int64_t)device_sm_count() * 8));
  if (f32)
    launch_kernel(dw_assemble_kernel<true>, grid, dim3(256), smem, st, a, n_split, a.compact, a.ld_compact, a.col_map, a.D, vec);
  else
    launch_kernel(dw_assemble_kernel<false>, grid, dim3(256), smem, st, a, n_split, a.compact, a.ld_compact, a.col_map, a.D, vec);
  return cudaGetLastError();
}

// The assembling pass keeps one source index per channel and kAsmRows sums per outlier channel in shared memory.
bool hp_dw_assemble_fits(int64_t D, int64_t n_out) { return (D + 4 + kAsmRows * n_out) * 4 <= 200 * 1024; }

cudaError_t launch_hp_dw(const HpDwArgs& a, cudaStream_t st) {
  const cudaError_t e = launch_hp_dw_product(a, st);
  return e != cudaSuccess ? e : launch_hp_dw_finish(a, st);
}

cudaError_t launch_gather_cols(const uint16_t* src, int64_t ld_src, int64_t rows, const int32_t* cols, int64_t n, uint16_t* dst,
                               int64_t ld_dst, cudaStream_t st) {
  if (rows == 0 || ld_dst == 0) return cudaSuccess;
  launch_kernel(gather_cols_kernel, dim3((unsigned)((rows + 7) / 8)), dim3(256), 0, st, src, ld_src, rows, cols, n, dst, ld_dst);
  return cudaGetLastError();
}

}  // namespace nvfp4
