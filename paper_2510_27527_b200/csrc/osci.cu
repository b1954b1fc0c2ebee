// OsciReset kernels (paper Sec. 3.2-3.3): per-element oscillation statistics (Algorithm 2 of the appendix) and the reset
// of high-risk master weights to the centre of their quantization bin (Algorithm 1).
//   Q(W) = FP4 quant-dequant of the master weights as the layer's forward weight quantizer sees them: cast to BF16
//   (round to nearest even), double-block quantize along the input-feature axis with round-to-nearest, dequantize as
//   float32((P * S_block) * S_global).
// One thread owns one 16-element block of a row for W (and, in the statistics kernel, for the snapshot W'): everything
// else is elementwise FP32 on those 16 values. HBM streaming kernels: 28 B/element (statistics), 16 B/element (reset),
// plus 4 B/element per amax pre-pass in the TENSOR and ROW scale modes.
#include "../../include/nvfp4.h"

#include "nvfp4_device.cuh"
#include "nvfp4_internal.h"

namespace nvfp4 {

namespace {

// 16 floats of row r starting at column k0 (zero beyond K); vector loads when the row is 16-byte aligned
__device__ __forceinline__ void load16f(const float* __restrict__ row, int64_t k0, int64_t K, bool vec, float (&v)[16]) {
  if (vec && k0 + 16 <= K) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float4 t = *reinterpret_cast<const float4*>(row + k0 + 4 * q);
      v[4 * q] = t.x; v[4 * q + 1] = t.y; v[4 * q + 2] = t.z; v[4 * q + 3] = t.w;
    }
  } else {
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = (k0 + i < K) ? row[k0 + i] : 0.0f;
  }
}
__device__ __forceinline__ void store16f(float* __restrict__ row, int64_t k0, int64_t K, bool vec, const float (&v)[16]) {
  if (vec && k0 + 16 <= K) {
#pragma unroll
    for (int q = 0; q < 4; ++q)
      *reinterpret_cast<float4*>(row + k0 + 4 * q) = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
  } else {
#pragma unroll
    for (int i = 0; i < 16; ++i)
      if (k0 + i < K) row[k0 + i] = v[i];
  }
}

// In place: w (master values) -> Q(w) for one 16-block. amax_cell: binary32 pattern of the group's amax over the master
// values (TENSOR / ROW), unused for BLOCK128 where the 8 threads of a 128-group reduce their block maxima by shuffles.
template <int GS>
__device__ __forceinline__ void quant_dequant16(float (&w)[16], uint32_t amax_cell) {
  float m = 0.0f;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    w[i] = bf16_bits_to_float(f32_to_bf16_bits(w[i]));
    m = fmaxf(m, fabsf(w[i]));
  }
  float Sg;
  if (GS == kGsBlock128) {
    uint32_t g = __float_as_uint(m);
    g = max(g, __shfl_xor_sync(0xFFFFFFFFu, g, 1));
    g = max(g, __shfl_xor_sync(0xFFFFFFFFu, g, 2));
    g = max(g, __shfl_xor_sync(0xFFFFFFFFu, g, 4));
    Sg = global_scale_from_amax(__uint_as_float(g));
  } else {
    // the cell holds max |w| over the master values; BF16 rounding is monotonic, so rounding it gives max |bf16(w)|
    Sg = global_scale_from_amax(bf16_bits_to_float(f32_to_bf16_bits(__uint_as_float(amax_cell))));
  }
  float rcp;
  const uint32_t sb = block_scale(m, Sg, rcp);
  // x_hat = (P * S_block) * S_global with P = the E2M1 value nearest to y (ties to the even code, saturating): the
  // hardware conversion to a packed pair of codes followed by the conversion of that byte back to FP16, inside one asm
  // block. (Packing the codes into a 32-bit word and unpacking that word through byte registers again in the same thread
  // came back as zeros on the device; this form never leaves the byte register.) P * S_block is exact in binary32.
  const float Sbf = e4m3_decode(sb);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float ylo = __fmul_rn(w[2 * i], rcp), yhi = __fmul_rn(w[2 * i + 1], rcp);
    uint32_t h2;
    asm("{\n"
        ".reg .b8 t;\n"
        "cvt.rn.satfinite.e2m1x2.f32 t, %2, %1;\n"
        "cvt.rn.f16x2.e2m1x2 %0, t;\n"
        "}"
        : "=r"(h2)
        : "f"(ylo), "f"(yhi));
    const float2 pv = __half22float2(*reinterpret_cast<__half2*>(&h2));
    w[2 * i] = __fmul_rn(__fmul_rn(pv.x, Sbf), Sg);
    w[2 * i + 1] = __fmul_rn(__fmul_rn(pv.y, Sbf), Sg);
  }
}

// max |w| per row (cells[r]) or over the matrix (cells[0]); cells are zero before the launch
__global__ void __launch_bounds__(256) amax_f32_kernel(const float* __restrict__ W, int64_t ld, int64_t C, int64_t D, uint32_t* cells,
                                                      int per_row) {
  pdl_prologue();
  const int64_t chunks = (D + 3) >> 2;
  const bool vec = (ld & 3) == 0;
  float m = 0.0f;
  for (int64_t r = blockIdx.x; r < C; r += gridDim.x) {
    const float* p = W + r * ld;
    float mr = 0.0f;
    int64_t c = threadIdx.x;
    if (vec) {
      for (; ((c + 768) << 2) + 4 <= D; c += 1024) {  // four 16-byte loads in flight
        const float4 v0 = *reinterpret_cast<const float4*>(p + (c << 2));
        const float4 v1 = *reinterpret_cast<const float4*>(p + ((c + 256) << 2));
        const float4 v2 = *reinterpret_cast<const float4*>(p + ((c + 512) << 2));
        const float4 v3 = *reinterpret_cast<const float4*>(p + ((c + 768) << 2));
        mr = fmaxf(mr, fmaxf(fmaxf(fabsf(v0.x), fabsf(v0.y)), fmaxf(fabsf(v0.z), fabsf(v0.w))));
        mr = fmaxf(mr, fmaxf(fmaxf(fabsf(v1.x), fabsf(v1.y)), fmaxf(fabsf(v1.z), fabsf(v1.w))));
        mr = fmaxf(mr, fmaxf(fmaxf(fabsf(v2.x), fabsf(v2.y)), fmaxf(fabsf(v2.z), fabsf(v2.w))));
        mr = fmaxf(mr, fmaxf(fmaxf(fabsf(v3.x), fabsf(v3.y)), fmaxf(fabsf(v3.z), fabsf(v3.w))));
      }
    }
    for (; c < chunks; c += 256) {
      if (vec && (c << 2) + 4 <= D) {
        const float4 v = *reinterpret_cast<const float4*>(p + (c << 2));
        mr = fmaxf(mr, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
      } else {
        for (int64_t j = c << 2; j < min(D, (c << 2) + 4); ++j) mr = fmaxf(mr, fabsf(p[j]));
      }
    }
    if (per_row) {
#pragma unroll
      for (int o = 16; o; o >>= 1) mr = fmaxf(mr, __shfl_xor_sync(0xFFFFFFFFu, mr, o));
      if ((threadIdx.x & 31) == 0 && mr > 0.0f) atomicMax(cells + r, __float_as_uint(mr));
    } else {
      m = fmaxf(m, mr);
    }
  }
  if (!per_row) {
#pragma unroll
    for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    __shared__ float wm[8];
    if ((threadIdx.x & 31) == 0) wm[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
      for (int w = 1; w < 8; ++w) m = fmaxf(m, wm[w]);
      if (m > 0.0f) atomicMax(cells, __float_as_uint(m));
    }
  }
}

// Algorithm 2, t0 = 0: clear the statistics, take the snapshot
__global__ void __launch_bounds__(256) osci_init_kernel(const float* __restrict__ W, int64_t ldw, int64_t C, int64_t D,
                                                       float* __restrict__ Wp, float* __restrict__ DM, float* __restrict__ DQ) {
  pdl_prologue();
  const int64_t nb = (D + 15) >> 4;
  const int64_t gid = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (gid >= C * nb) return;
  const int64_t r = gid / nb, k0 = (gid - r * nb) << 4;
  const bool vw = (ldw & 3) == 0, vs = (D & 3) == 0;
  float v[16], z[16];
  load16f(W + r * ldw, k0, D, vw, v);
#pragma unroll
  for (int i = 0; i < 16; ++i) z[i] = 0.0f;
  store16f(Wp + r * D, k0, D, vs, v);
  store16f(DM + r * D, k0, D, vs, z);
  store16f(DQ + r * D, k0, D, vs, z);
}

// Algorithm 2, t0 > 0: D_M += |W - W'|, D_Q += |Q(W) - Q(W')|, W' <- W
template <int GS>
__global__ void __launch_bounds__(256) osci_update_kernel(const float* __restrict__ W, int64_t ldw, int64_t C, int64_t D,
                                                         float* __restrict__ Wp, float* __restrict__ DM, float* __restrict__ DQ,
                                                         const uint32_t* __restrict__ cells) {
  pdl_prologue();
  const int64_t nb = ((D + 127) & ~(int64_t)127) >> 4;  // blocks per row, padded so that 8 lanes share a 128-group
  const int64_t gid = (int64_t)blockIdx.x * 256 + threadIdx.x;
  const bool active = gid < C * nb;
  const int64_t r = active ? gid / nb : 0;
  const int64_t k0 = active ? (gid - r * nb) << 4 : D;  // inactive lanes read nothing and still take part in shuffles
  const bool vw = (ldw & 3) == 0, vs = (D & 3) == 0;
  float w[16], p[16];
  load16f(W + r * ldw, k0, D, vw, w);
  load16f(Wp + r * D, k0, D, vs, p);
  float a[16], aq[16];
  load16f(DM + r * D, k0, D, vs, a);  // requested before the arithmetic
  load16f(DQ + r * D, k0, D, vs, aq);
  float dm[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) dm[i] = fabsf(__fsub_rn(w[i], p[i]));
  if (active && k0 < D) store16f(Wp + r * D, k0, D, vs, w);
  const uint32_t cw = GS == kGsTensor ? cells[0] : GS == kGsRow ? cells[r] : 0u;
  const uint32_t cp = GS == kGsTensor ? cells[1] : GS == kGsRow ? cells[C + r] : 0u;
  quant_dequant16<GS>(w, cw);
  quant_dequant16<GS>(p, cp);
  if (!(active && k0 < D)) return;
#pragma unroll
  for (int i = 0; i < 16; ++i) a[i] = __fadd_rn(a[i], dm[i]);
  store16f(DM + r * D, k0, D, vs, a);
#pragma unroll
  for (int i = 0; i < 16; ++i) aq[i] = __fadd_rn(aq[i], fabsf(__fsub_rn(w[i], p[i])));
  store16f(DQ + r * D, k0, D, vs, aq);
}

// Algorithm 1: w <- Q(w) where D_Q / D_M >= tau
template <int GS>
__global__ void __launch_bounds__(256, 3) osci_suppress_kernel(float* __restrict__ W, int64_t ldw, int64_t C, int64_t D,
                                                           const float* __restrict__ DM, const float* __restrict__ DQ, float tau,
                                                           const uint32_t* __restrict__ cells, unsigned long long* n_reset) {
  pdl_prologue();
  const int64_t nb = ((D + 127) & ~(int64_t)127) >> 4;
  const int64_t gid = (int64_t)blockIdx.x * 256 + threadIdx.x;
  const bool active = gid < C * nb;
  const int64_t r = active ? gid / nb : 0;
  const int64_t k0 = active ? (gid - r * nb) << 4 : D;
  const bool vw = (ldw & 3) == 0, vs = (D & 3) == 0;
  float w[16], q[16];
  uint32_t hits = 0;
  {
    float dm[16], dq[16];
    load16f(W + r * ldw, k0, D, vw, w);  // all three streams are requested before any arithmetic
    load16f(DM + r * D, k0, D, vs, dm);
    load16f(DQ + r * D, k0, D, vs, dq);
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      // NaN (0 / 0) compares false; an element whose quantized value never moved has risk 0 (or 0 / 0): no division
      const bool hit = (k0 + i < D) && ((dq[i] == 0.0f && tau > 0.0f) ? false : (__fdiv_rn(dq[i], dm[i]) >= tau));
      hits |= (hit ? 1u : 0u) << i;
    }
  }
#pragma unroll
  for (int i = 0; i < 16; ++i) q[i] = w[i];
  quant_dequant16<GS>(q, GS == kGsTensor ? cells[0] : GS == kGsRow ? cells[r] : 0u);
  const int n = __popc(hits);
  if (active && n) {
#pragma unroll
    for (int i = 0; i < 16; ++i)
      if ((hits >> i) & 1u) w[i] = q[i];
    store16f(W + r * ldw, k0, D, vw, w);
  }
  if (n_reset) {
    int total = n;
#pragma unroll
    for (int o = 16; o; o >>= 1) total += __shfl_xor_sync(0xFFFFFFFFu, total, o);
    if ((threadIdx.x & 31) == 0 && total) atomicAdd(n_reset, (unsigned long long)total);
  }
}

size_t osci_cells(int64_t C, int32_t gs_mode) { return gs_mode == kGsRow ? (size_t)(2 * std::max<int64_t>(C, 1)) : 2; }

bool bad_f32(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

cudaError_t run_amax(const float* W, int64_t ld, int64_t C, int64_t D, uint32_t* cells, int per_row, cudaStream_t st) {
  const unsigned grid = (unsigned)std::min<int64_t>(C, 148 * 8);
  launch_kernel(amax_f32_kernel, dim3(grid), dim3(256), 0, st, W, ld, C, D, cells, per_row);
  return cudaGetLastError();
}

}  // namespace
}  // namespace nvfp4

using namespace nvfp4;

extern "C" {

size_t nvfp4_osci_workspace_bytes(int64_t C, int32_t gs_mode) { return (osci_cells(C, gs_mode) * 4 + 255) / 256 * 256; }

nvfp4_status nvfp4_osci_update(const float* W, int64_t ldw, int64_t C, int64_t D, int32_t gs_mode, int32_t t0, float* W_prev,
                               float* D_M, float* D_Q, void* workspace, size_t ws_bytes, void* stream) {
  if (!W || !W_prev || !D_M || !D_Q) return NVFP4_ERR_NULL;
  if (C < 0 || D < 0 || ldw < D || t0 < 0) return NVFP4_ERR_SHAPE;
  if (gs_mode < 0 || gs_mode > 2) return NVFP4_ERR_ENUM;
  if (bad_f32(W) || bad_f32(W_prev) || bad_f32(D_M) || bad_f32(D_Q)) return NVFP4_ERR_ALIGN;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 3u) || ws_bytes < nvfp4_osci_workspace_bytes(C, gs_mode))
    return NVFP4_ERR_WORKSPACE;
  if (!device_is_sm100()) return NVFP4_ERR_ARCH;
  if (C == 0 || D == 0) return NVFP4_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (t0 == 0) {
    const int64_t blocks16 = C * ((D + 15) >> 4);
    launch_kernel(osci_init_kernel, dim3((unsigned)((blocks16 + 255) / 256)), dim3(256), 0, st, W, ldw, C, D, W_prev, D_M, D_Q);
    return cudaGetLastError() == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
  }
  uint32_t* cells = static_cast<uint32_t*>(workspace);
  if (gs_mode != kGsBlock128) {
    const int per_row = gs_mode == kGsRow;
    if (cudaMemsetAsync(cells, 0, osci_cells(C, gs_mode) * 4, st) != cudaSuccess) return NVFP4_ERR_CUDA;
    if (run_amax(W, ldw, C, D, cells, per_row, st) != cudaSuccess) return NVFP4_ERR_CUDA;
    if (run_amax(W_prev, D, C, D, cells + (per_row ? C : 1), per_row, st) != cudaSuccess) return NVFP4_ERR_CUDA;
  }
  const int64_t nb = ((D + 127) & ~(int64_t)127) >> 4;
  const dim3 grid((unsigned)((C * nb + 255) / 256));
  if (gs_mode == kGsTensor)
    launch_kernel(osci_update_kernel<kGsTensor>, grid, dim3(256), 0, st, W, ldw, C, D, W_prev, D_M, D_Q, static_cast<const uint32_t*>(cells));
  else if (gs_mode == kGsRow)
    launch_kernel(osci_update_kernel<kGsRow>, grid, dim3(256), 0, st, W, ldw, C, D, W_prev, D_M, D_Q, static_cast<const uint32_t*>(cells));
  else
    launch_kernel(osci_update_kernel<kGsBlock128>, grid, dim3(256), 0, st, W, ldw, C, D, W_prev, D_M, D_Q, static_cast<const uint32_t*>(cells));
  return cudaGetLastError() == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

nvfp4_status nvfp4_osci_suppress(float* W, int64_t ldw, int64_t C, int64_t D, int32_t gs_mode, const float* D_M, const float* D_Q,
                                 float tau, unsigned long long* n_reset, void* workspace, size_t ws_bytes, void* stream) {
  if (!W || !D_M || !D_Q) return NVFP4_ERR_NULL;
  if (C < 0 || D < 0 || ldw < D) return NVFP4_ERR_SHAPE;
  if (gs_mode < 0 || gs_mode > 2) return NVFP4_ERR_ENUM;
  if (bad_f32(W) || bad_f32(D_M) || bad_f32(D_Q) || (n_reset && (reinterpret_cast<uintptr_t>(n_reset) & 7u))) return NVFP4_ERR_ALIGN;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 3u) || ws_bytes < nvfp4_osci_workspace_bytes(C, gs_mode))
    return NVFP4_ERR_WORKSPACE;
  if (!device_is_sm100()) return NVFP4_ERR_ARCH;
  if (C == 0 || D == 0) return NVFP4_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t* cells = static_cast<uint32_t*>(workspace);
  if (gs_mode != kGsBlock128) {
    const int per_row = gs_mode == kGsRow;
    if (cudaMemsetAsync(cells, 0, osci_cells(C, gs_mode) * 4, st) != cudaSuccess) return NVFP4_ERR_CUDA;
    if (run_amax(W, ldw, C, D, cells, per_row, st) != cudaSuccess) return NVFP4_ERR_CUDA;
  }
  const int64_t nb = ((D + 127) & ~(int64_t)127) >> 4;
  const dim3 grid((unsigned)((C * nb + 255) / 256));
  const uint32_t* cc = cells;
  if (gs_mode == kGsTensor)
    launch_kernel(osci_suppress_kernel<kGsTensor>, grid, dim3(256), 0, st, W, ldw, C, D, D_M, D_Q, tau, cc, n_reset);
  else if (gs_mode == kGsRow)
    launch_kernel(osci_suppress_kernel<kGsRow>, grid, dim3(256), 0, st, W, ldw, C, D, D_M, D_Q, tau, cc, n_reset);
  else
    launch_kernel(osci_suppress_kernel<kGsBlock128>, grid, dim3(256), 0, st, W, ldw, C, D, D_M, D_Q, tau, cc, n_reset);
  return cudaGetLastError() == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

}  // extern "C"
