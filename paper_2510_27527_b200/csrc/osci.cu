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

// Q(w) of one 16-block in three steps: BF16 cast + block amax, global scale of its group, scale / round / dequantize.
// w <- BF16(w) in place; returns the block's amax
__device__ __forceinline__ float round_block_bf16(float (&w)[16]) {
  float m = 0.0f;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    w[i] = bf16_bits_to_float(f32_to_bf16_bits(w[i]));
    m = fmaxf(m, fabsf(w[i]));
  }
  return m;
}
// global scale of the block: from the 8 lanes of its 128-group (BLOCK128; every lane of the warp must call this), or from
// the pre-pass cell, which holds max |w| over the master values (BF16 rounding is monotonic, so rounding it gives
// max |bf16(w)|)
template <int GS>
__device__ __forceinline__ float group_scale(float m, uint32_t amax_cell) {
  if (GS == kGsBlock128) {
    uint32_t g = __float_as_uint(m);
    g = max(g, __shfl_xor_sync(0xFFFFFFFFu, g, 1));
    g = max(g, __shfl_xor_sync(0xFFFFFFFFu, g, 2));
    g = max(g, __shfl_xor_sync(0xFFFFFFFFu, g, 4));
    return global_scale_from_amax(__uint_as_float(g));
  }
  return global_scale_from_amax(bf16_bits_to_float(f32_to_bf16_bits(__uint_as_float(amax_cell))));
}
__device__ __forceinline__ void quant_block_with(float (&w)[16], float m, float Sg);

template <int GS>
__device__ __forceinline__ void quant_dequant16(float (&w)[16], uint32_t amax_cell) {
  const float m = round_block_bf16(w);
  quant_block_with(w, m, group_scale<GS>(m, amax_cell));
}

// w (already BF16-rounded, block amax m) -> x_hat for the global scale Sg
__device__ __forceinline__ void quant_block_with(float (&w)[16], float m, float Sg) {
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

// =========================================================================================================
// Memory-efficient statistics (appendix Algorithm 3): only the n_track elements with the largest sensitivity score
// s = |w - Q(w)| / binwidth(Q(w)) at t0 = 0 are tracked. State per tracked element: linear index, master and quantized
// snapshot, the two path lengths.
// =========================================================================================================

// Sensitivity score of every element as a binary32 pattern (non-negative: integer order = value order).
template <int GS>
__global__ void __launch_bounds__(256, 3) osci_score_kernel(const float* __restrict__ W, int64_t ldw, int64_t C, int64_t D,
                                                           const uint32_t* __restrict__ cells, uint32_t* __restrict__ scores) {
  pdl_prologue();
  const int64_t nb = ((D + 127) & ~(int64_t)127) >> 4;
  const int64_t gid = (int64_t)blockIdx.x * 256 + threadIdx.x;
  const bool active = gid < C * nb;
  const int64_t r = active ? gid / nb : 0;
  const int64_t k0 = active ? (gid - r * nb) << 4 : D;
  float w[16], x[16];
  load16f(W + r * ldw, k0, D, (ldw & 3) == 0, w);
  float m = 0.0f;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    x[i] = bf16_bits_to_float(f32_to_bf16_bits(w[i]));
    m = fmaxf(m, fabsf(x[i]));
  }
  float Sg;
  if (GS == kGsBlock128) {
    uint32_t g = __float_as_uint(m);
    g = max(g, __shfl_xor_sync(0xFFFFFFFFu, g, 1));
    g = max(g, __shfl_xor_sync(0xFFFFFFFFu, g, 2));
    g = max(g, __shfl_xor_sync(0xFFFFFFFFu, g, 4));
    Sg = global_scale_from_amax(__uint_as_float(g));
  } else {
    const uint32_t cell = GS == kGsTensor ? cells[0] : cells[r];
    Sg = global_scale_from_amax(bf16_bits_to_float(f32_to_bf16_bits(__uint_as_float(cell))));
  }
  float rcp;
  const uint32_t sb = block_scale(m, Sg, rcp);
  const float Sbf = e4m3_decode(sb);
  const float d = __fmul_rn(Sg, Sbf);
  if (!(active && k0 < D)) return;
  float sc[16];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float ylo = __fmul_rn(x[2 * i], rcp), yhi = __fmul_rn(x[2 * i + 1], rcp);
    uint32_t h2;
    asm("{\n"
        ".reg .b8 t;\n"
        "cvt.rn.satfinite.e2m1x2.f32 t, %2, %1;\n"
        "cvt.rn.f16x2.e2m1x2 %0, t;\n"
        "}"
        : "=r"(h2)
        : "f"(ylo), "f"(yhi));
    const float2 pv = __half22float2(*reinterpret_cast<__half2*>(&h2));
    const float pp[2] = {pv.x, pv.y};
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const float q = __fmul_rn(__fmul_rn(pp[h], Sbf), Sg);
      const float a = fabsf(pp[h]);
      // width of the rounding bin of the E2M1 value: thresholds are the midpoints between neighbouring values
      const float bw = a < 1.75f ? 0.5f : a < 2.5f ? 0.75f : a < 3.5f ? 1.0f : a < 5.0f ? 1.5f : 2.0f;
      const float err = fabsf(__fsub_rn(w[2 * i + h], q));
      sc[2 * i + h] = d == 0.0f ? 0.0f : __fdiv_rn(err, __fmul_rn(bw, d));
    }
  }
  uint32_t* out = scores + r * D + k0;
  if (k0 + 16 <= D && (D & 3) == 0) {
#pragma unroll
    for (int q = 0; q < 4; ++q)
      *reinterpret_cast<uint4*>(out + 4 * q) = make_uint4(__float_as_uint(sc[4 * q]), __float_as_uint(sc[4 * q + 1]),
                                                         __float_as_uint(sc[4 * q + 2]), __float_as_uint(sc[4 * q + 3]));
  } else {
#pragma unroll
    for (int i = 0; i < 16; ++i)
      if (k0 + i < D) out[i] = __float_as_uint(sc[i]);
  }
}

// Radix select of the k-th largest 32-bit pattern, one byte per pass from the top. sel[0] = prefix found so far,
// sel[1] = rank still to resolve inside the candidates, sel[2..257] = histogram of the current byte.
__global__ void __launch_bounds__(256) osci_hist_kernel(const uint32_t* __restrict__ v, int64_t n, uint32_t* sel, int shift) {
  pdl_prologue();
  __shared__ uint32_t h[256];
  h[threadIdx.x] = 0;
  __syncthreads();
  const uint32_t prefix = sel[0];
  const uint32_t mask_hi = shift == 24 ? 0u : (0xFFFFFFFFu << (shift + 8));
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < n; i += (int64_t)gridDim.x * 256) {
    const uint32_t x = v[i];
    if (((x ^ prefix) & mask_hi) == 0) atomicAdd(&h[(x >> shift) & 255u], 1u);
  }
  __syncthreads();
  if (h[threadIdx.x]) atomicAdd(sel + 2 + threadIdx.x, h[threadIdx.x]);
}

__global__ void osci_pick_kernel(uint32_t* sel, int shift) {
  pdl_prologue();
  if (threadIdx.x != 0) return;
  uint32_t k = sel[1], cum = 0;
  int chosen = 0;
  for (int b = 255; b >= 0; --b) {
    const uint32_t c = sel[2 + b];
    if (cum + c >= k) {
      chosen = b;
      break;
    }
    cum += c;
  }
  sel[0] |= (uint32_t)chosen << shift;
  sel[1] = k - cum;
  for (int b = 0; b < 256; ++b) sel[2 + b] = 0;
}

__global__ void osci_sel_init_kernel(uint32_t* sel, uint32_t k) {
  pdl_prologue();
  for (int i = threadIdx.x; i < 258; i += blockDim.x) sel[i] = i == 1 ? k : 0u;
}

// Ordered compaction of the selected elements (value > T, plus the first sel[1] elements equal to T in index order).
// A CTA covers 4096 consecutive elements, a thread 16 consecutive ones.
__global__ void __launch_bounds__(256) osci_count_kernel(const uint32_t* __restrict__ v, int64_t n, const uint32_t* __restrict__ sel,
                                                        uint2* __restrict__ cta_counts) {
  pdl_prologue();
  const uint32_t T = sel[0];
  const int64_t base = ((int64_t)blockIdx.x * 256 + threadIdx.x) * 16;
  uint32_t gt = 0, eq = 0;
  for (int i = 0; i < 16; ++i)
    if (base + i < n) {
      const uint32_t x = v[base + i];
      gt += x > T;
      eq += x == T;
    }
  __shared__ uint32_t sg[8], se[8];
#pragma unroll
  for (int o = 16; o; o >>= 1) {
    gt += __shfl_xor_sync(0xFFFFFFFFu, gt, o);
    eq += __shfl_xor_sync(0xFFFFFFFFu, eq, o);
  }
  if ((threadIdx.x & 31) == 0) {
    sg[threadIdx.x >> 5] = gt;
    se[threadIdx.x >> 5] = eq;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w) {
      gt += sg[w];
      eq += se[w];
    }
    cta_counts[blockIdx.x] = make_uint2(gt, eq);
  }
}

// exclusive scan of the per-CTA counts, in place (one CTA; the running totals are carried over the chunks)
__global__ void __launch_bounds__(1024) osci_scan_kernel(uint2* cta_counts, int64_t n_cta) {
  pdl_prologue();
  __shared__ uint32_t wg[32], we[32];
  __shared__ uint32_t tot_g, tot_e;
  uint32_t run_g = 0, run_e = 0;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  for (int64_t c0 = 0; c0 < n_cta; c0 += 1024) {
    const int64_t i = c0 + threadIdx.x;
    const uint2 v = i < n_cta ? cta_counts[i] : make_uint2(0, 0);
    uint32_t ig = v.x, ie = v.y;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t tg = __shfl_up_sync(0xFFFFFFFFu, ig, o), te = __shfl_up_sync(0xFFFFFFFFu, ie, o);
      if (lane >= o) {
        ig += tg;
        ie += te;
      }
    }
    if (lane == 31) {
      wg[wid] = ig;
      we[wid] = ie;
    }
    __syncthreads();
    if (wid == 0) {
      uint32_t a = wg[lane], b = we[lane], ia = a, ib = b;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t ta = __shfl_up_sync(0xFFFFFFFFu, ia, o), tb = __shfl_up_sync(0xFFFFFFFFu, ib, o);
        if (lane >= o) {
          ia += ta;
          ib += tb;
        }
      }
      wg[lane] = ia - a;
      we[lane] = ib - b;
      if (lane == 31) {
        tot_g = ia;
        tot_e = ib;
      }
    }
    __syncthreads();
    if (i < n_cta) cta_counts[i] = make_uint2(run_g + wg[wid] + ig - v.x, run_e + we[wid] + ie - v.y);
    run_g += tot_g;
    run_e += tot_e;
    __syncthreads();
  }
}

__global__ void __launch_bounds__(256) osci_scatter_kernel(const uint32_t* __restrict__ v, int64_t n, const uint32_t* __restrict__ sel,
                                                          const uint2* __restrict__ cta_base, int32_t* __restrict__ idx) {
  pdl_prologue();
  const uint32_t T = sel[0], need_eq = sel[1];
  const int64_t base = ((int64_t)blockIdx.x * 256 + threadIdx.x) * 16;
  uint32_t x[16];
  uint32_t gt = 0, eq = 0;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    x[i] = base + i < n ? v[base + i] : 0u;
    if (base + i < n) {
      gt += x[i] > T;
      eq += x[i] == T;
    }
  }
  // exclusive scan of (gt, eq) over the CTA's threads
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  uint32_t ig = gt, ie = eq;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t tg = __shfl_up_sync(0xFFFFFFFFu, ig, o), te = __shfl_up_sync(0xFFFFFFFFu, ie, o);
    if (lane >= o) {
      ig += tg;
      ie += te;
    }
  }
  __shared__ uint32_t wg[8], we[8];
  if (lane == 31) {
    wg[wid] = ig;
    we[wid] = ie;
  }
  __syncthreads();
  uint32_t og = 0, oe = 0;
  for (int w = 0; w < wid; ++w) {
    og += wg[w];
    oe += we[w];
  }
  const uint2 cb = cta_base[blockIdx.x];
  uint32_t g_before = cb.x + og + ig - gt, e_before = cb.y + oe + ie - eq;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    if (base + i < n) {
      const bool is_gt = x[i] > T, is_eq = x[i] == T;
      if (is_gt || (is_eq && e_before < need_eq)) idx[g_before + min(e_before, need_eq)] = (int32_t)(base + i);
      g_before += is_gt;
      e_before += is_eq;
    }
  }
}

// amax of every 128-group of a row (BLOCK128 scale mode) as binary32 patterns: cells[r * G + g], G = ceil(D / 128).
__global__ void __launch_bounds__(256) amax_groups_f32_kernel(const float* __restrict__ W, int64_t ldw, int64_t C, int64_t D,
                                                             uint32_t* __restrict__ cells) {
  pdl_prologue();
  const int64_t nb = ((D + 127) & ~(int64_t)127) >> 4;
  const int64_t gid = (int64_t)blockIdx.x * 256 + threadIdx.x;
  const bool active = gid < C * nb;
  const int64_t r = active ? gid / nb : 0;
  const int64_t b = active ? gid - r * nb : 0;
  float w[16];
  load16f(W + r * ldw, active ? b << 4 : D, D, (ldw & 3) == 0, w);
  float m = 0.0f;
#pragma unroll
  for (int i = 0; i < 16; ++i) m = fmaxf(m, fabsf(w[i]));
  uint32_t g = __float_as_uint(m);
  g = max(g, __shfl_xor_sync(0xFFFFFFFFu, g, 1));
  g = max(g, __shfl_xor_sync(0xFFFFFFFFu, g, 2));
  g = max(g, __shfl_xor_sync(0xFFFFFFFFu, g, 4));
  if (active && (b & 7) == 0) cells[r * (nb >> 3) + (b >> 3)] = g;
}

// One tracked element per thread: its 16-block is loaded and quantized with the global scale looked up in the amax
// cells (tensor, row, or the element's 128-group). Returns the master value and Q(w) of the element.
template <int GS>
__device__ __forceinline__ void tracked_values(const float* __restrict__ W, int64_t ldw, int64_t C, int64_t D,
                                               const uint32_t* __restrict__ cells, int32_t e, bool valid, float& wm, float& wq,
                                               bool& mine) {
  const uint32_t ue = valid ? (uint32_t)e : 0u;
  const uint32_t r = ue / (uint32_t)D, c = ue - r * (uint32_t)D;
  const int64_t k0 = valid ? (int64_t)(c & ~15u) : D;
  mine = valid;
  float w[16], q[16];
  load16f(W + (int64_t)r * ldw, k0, D, (ldw & 3) == 0, w);
#pragma unroll
  for (int i = 0; i < 16; ++i) q[i] = w[i];
  const float m = round_block_bf16(q);
  const int64_t G = (D + 127) >> 7;
  const uint32_t cell = GS == kGsTensor ? cells[0] : GS == kGsRow ? cells[r] : cells[(int64_t)r * G + (c >> 7)];
  const float Sg = group_scale<kGsTensor>(m, cell);  // the lookup form (no shuffles) in every mode
  quant_block_with(q, m, Sg);
  wm = 0.0f;
  wq = 0.0f;
  const uint32_t pos = c & 15u;
#pragma unroll
  for (int i = 0; i < 16; ++i)
    if (pos == (uint32_t)i) {
      wm = w[i];
      wq = q[i];
    }
}

template <int GS>
__global__ void __launch_bounds__(256) osci_sparse_update_kernel(const float* __restrict__ W, int64_t ldw, int64_t C, int64_t D,
                                                                const uint32_t* __restrict__ cells, int64_t n_track,
                                                                const int32_t* __restrict__ idx, float* __restrict__ WM,
                                                                float* __restrict__ WQ, float* __restrict__ DM, float* __restrict__ DQ,
                                                                int init) {
  pdl_prologue();
  const int64_t gid = (int64_t)blockIdx.x * 256 + threadIdx.x;
  const int64_t i = gid;
  const bool valid = i < n_track;
  const int32_t e = valid ? idx[i] : 0;
  float wm, wq;
  bool mine;
  tracked_values<GS>(W, ldw, C, D, cells, e, valid, wm, wq, mine);
  if (!mine) return;
  if (init) {
    DM[i] = 0.0f;
    DQ[i] = 0.0f;
  } else {
    DM[i] = __fadd_rn(DM[i], fabsf(__fsub_rn(wm, WM[i])));
    DQ[i] = __fadd_rn(DQ[i], fabsf(__fsub_rn(wq, WQ[i])));
  }
  WM[i] = wm;
  WQ[i] = wq;
}

// Reset in two launches so that no thread reads a weight another thread has already reset: the first computes, per
// tracked element, the value to write (NaN = leave alone) from the untouched matrix, the second applies them.
template <int GS>
__global__ void __launch_bounds__(256) osci_sparse_decide_kernel(const float* __restrict__ W, int64_t ldw, int64_t C, int64_t D,
                                                                const uint32_t* __restrict__ cells, int64_t n_track,
                                                                const int32_t* __restrict__ idx, const float* __restrict__ DM,
                                                                const float* __restrict__ DQ, float tau, float* __restrict__ newval) {
  pdl_prologue();
  const int64_t gid = (int64_t)blockIdx.x * 256 + threadIdx.x;
  const int64_t i = gid;
  const bool valid = i < n_track;
  const int32_t e = valid ? idx[i] : 0;
  float wm, wq;
  bool mine;
  tracked_values<GS>(W, ldw, C, D, cells, e, valid, wm, wq, mine);
  if (!mine) return;
  const float dq = DQ[i], dm = DM[i];
  const bool hit = (dq == 0.0f && tau > 0.0f) ? false : (__fdiv_rn(dq, dm) >= tau);
  newval[i] = hit ? wq : __uint_as_float(0x7FC00000u);
}

__global__ void __launch_bounds__(256) osci_sparse_apply_kernel(float* __restrict__ W, int64_t ldw, int64_t D, int64_t n_track,
                                                               const int32_t* __restrict__ idx, const float* __restrict__ newval,
                                                               unsigned long long* n_reset) {
  pdl_prologue();
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  int n = 0;
  if (i < n_track) {
    const float v = newval[i];
    if (v == v) {
      const uint32_t e = (uint32_t)idx[i];
      const uint32_t r = e / (uint32_t)D, c = e - r * (uint32_t)D;
      W[(int64_t)r * ldw + c] = v;
      n = 1;
    }
  }
  if (n_reset) {
#pragma unroll
    for (int o = 16; o; o >>= 1) n += __shfl_xor_sync(0xFFFFFFFFu, n, o);
    if ((threadIdx.x & 31) == 0 && n) atomicAdd(n_reset, (unsigned long long)n);
  }
}

size_t osci_cells(int64_t C, int32_t gs_mode) { return gs_mode == kGsRow ? (size_t)(2 * std::max<int64_t>(C, 1)) : 2; }

bool bad_f32(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

cudaError_t run_amax(const float* W, int64_t ld, int64_t C, int64_t D, uint32_t* cells, int per_row, cudaStream_t st) {
  const unsigned grid = (unsigned)std::min<int64_t>(C, device_sm_count() * 8);
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
    if (launch_zero_words(cells, (int64_t)osci_cells(C, gs_mode), st) != cudaSuccess) return NVFP4_ERR_CUDA;
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
    if (launch_zero_words(cells, (int64_t)osci_cells(C, gs_mode), st) != cudaSuccess) return NVFP4_ERR_CUDA;
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

// ---- memory-efficient variant --------------------------------------------------------------------------------
namespace {
struct SparseWs {
  uint32_t* cells;      // amax cells of W: 1 word (TENSOR), C words (ROW), C * ceil(D / 128) words (BLOCK128)
  uint32_t* sel;        // selection phase: 258 words of the radix select
  uint2* cta_counts;    // selection phase: one pair per 4096 elements
  uint32_t* scores;     // selection phase: C * D words
  float* newval;        // reset phase: n_track words
};
// phase 0: selection + initial snapshot (t0 = 0); 1: update (t0 > 0); 2: reset
size_t sparse_ws_layout(int64_t C, int64_t D, int32_t gs_mode, int64_t n_track, int phase, void* base, SparseWs* out) {
  size_t off = 0;
  auto take = [&](size_t bytes) {
    const size_t start = (off + 255) & ~(size_t)255;
    off = start + bytes;
    return base ? static_cast<uint8_t*>(base) + start : nullptr;
  };
  uint8_t* p0 = take((gs_mode == kGsBlock128 ? (size_t)C * (size_t)((D + 127) >> 7) : osci_cells(C, gs_mode)) * 4);
  uint8_t* p1 = take(258 * 4);
  const int64_t n = C * D;
  uint8_t* p2 = take(phase == 0 ? (size_t)((n + 4095) / 4096) * 8 : 0);
  uint8_t* p3 = take(phase == 0 ? (size_t)n * 4 : 0);
  uint8_t* p4 = take(phase == 2 ? (size_t)n_track * 4 : 0);
  if (out) {
    out->cells = reinterpret_cast<uint32_t*>(p0);
    out->sel = reinterpret_cast<uint32_t*>(p1);
    out->cta_counts = reinterpret_cast<uint2*>(p2);
    out->scores = reinterpret_cast<uint32_t*>(p3);
    out->newval = reinterpret_cast<float*>(p4);
  }
  return (off + 255) & ~(size_t)255;
}

nvfp4_status sparse_amax(const float* W, int64_t ldw, int64_t C, int64_t D, int32_t gs_mode, uint32_t* cells, cudaStream_t st) {
  if (gs_mode == kGsBlock128) {  // every group is written: no clearing needed
    const int64_t nb = ((D + 127) & ~(int64_t)127) >> 4;
    launch_kernel(amax_groups_f32_kernel, dim3((unsigned)((C * nb + 255) / 256)), dim3(256), 0, st, W, ldw, C, D, cells);
    return cudaGetLastError() == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
  }
  const int per_row = gs_mode == kGsRow;
  if (launch_zero_words(cells, per_row ? C : 1, st) != cudaSuccess) return NVFP4_ERR_CUDA;
  return run_amax(W, ldw, C, D, cells, per_row, st) == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}
}  // namespace

extern "C" {

size_t nvfp4_osci_sparse_workspace_bytes(int64_t C, int64_t D, int32_t gs_mode, int64_t n_track, int32_t phase) {
  if (C <= 0 || D <= 0 || n_track < 0 || phase < 0 || phase > 2) return 256;
  return sparse_ws_layout(C, D, gs_mode, n_track, phase, nullptr, nullptr);
}

nvfp4_status nvfp4_osci_sparse_update(const float* W, int64_t ldw, int64_t C, int64_t D, int32_t gs_mode, int32_t t0,
                                      int64_t n_track, int32_t* idx, float* WM_prev, float* WQ_prev, float* D_M, float* D_Q,
                                      void* workspace, size_t ws_bytes, void* stream) {
  if (!W) return NVFP4_ERR_NULL;
  if (C < 0 || D < 0 || ldw < D || t0 < 0 || n_track < 0 || n_track > C * D) return NVFP4_ERR_SHAPE;
  if (C * D >= ((int64_t)1 << 31)) return NVFP4_ERR_LIMIT;
  if (gs_mode < 0 || gs_mode > 2) return NVFP4_ERR_ENUM;
  if (n_track > 0 && (!idx || !WM_prev || !WQ_prev || !D_M || !D_Q)) return NVFP4_ERR_NULL;
  if (bad_f32(W)) return NVFP4_ERR_ALIGN;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || ws_bytes < nvfp4_osci_sparse_workspace_bytes(C, D, gs_mode, n_track, t0 == 0 ? 0 : 1))
    return NVFP4_ERR_WORKSPACE;
  if (!device_is_sm100()) return NVFP4_ERR_ARCH;
  if (C == 0 || D == 0 || n_track == 0) return NVFP4_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  SparseWs ws{};
  sparse_ws_layout(C, D, gs_mode, n_track, t0 == 0 ? 0 : 1, workspace, &ws);
  nvfp4_status s = sparse_amax(W, ldw, C, D, gs_mode, ws.cells, st);
  if (s != NVFP4_OK) return s;
  const uint32_t* cells = ws.cells;
  const int64_t n = C * D;
  if (t0 == 0) {
    // scores -> k-th largest by radix select -> ordered compaction of the selected indices
    const int64_t nb = ((D + 127) & ~(int64_t)127) >> 4;
    const dim3 sgrid((unsigned)((C * nb + 255) / 256));
    if (gs_mode == kGsTensor) launch_kernel(osci_score_kernel<kGsTensor>, sgrid, dim3(256), 0, st, W, ldw, C, D, cells, ws.scores);
    else if (gs_mode == kGsRow) launch_kernel(osci_score_kernel<kGsRow>, sgrid, dim3(256), 0, st, W, ldw, C, D, cells, ws.scores);
    else launch_kernel(osci_score_kernel<kGsBlock128>, sgrid, dim3(256), 0, st, W, ldw, C, D, cells, ws.scores);
    launch_kernel(osci_sel_init_kernel, dim3(1), dim3(256), 0, st, ws.sel, (uint32_t)n_track);
    const unsigned hgrid = (unsigned)std::min<int64_t>((n + 255) / 256, device_sm_count() * 8);
    for (int shift = 24; shift >= 0; shift -= 8) {
      launch_kernel(osci_hist_kernel, dim3(hgrid), dim3(256), 0, st, static_cast<const uint32_t*>(ws.scores), n, ws.sel, shift);
      launch_kernel(osci_pick_kernel, dim3(1), dim3(32), 0, st, ws.sel, shift);
    }
    const int64_t n_cta = (n + 4095) / 4096;
    launch_kernel(osci_count_kernel, dim3((unsigned)n_cta), dim3(256), 0, st, static_cast<const uint32_t*>(ws.scores), n,
                  static_cast<const uint32_t*>(ws.sel), ws.cta_counts);
    launch_kernel(osci_scan_kernel, dim3(1), dim3(1024), 0, st, ws.cta_counts, n_cta);
    launch_kernel(osci_scatter_kernel, dim3((unsigned)n_cta), dim3(256), 0, st, static_cast<const uint32_t*>(ws.scores), n,
                  static_cast<const uint32_t*>(ws.sel), static_cast<const uint2*>(ws.cta_counts), idx);
    if (cudaGetLastError() != cudaSuccess) return NVFP4_ERR_CUDA;
  }
  const int init = t0 == 0 ? 1 : 0;
  const int64_t threads = n_track;
  const dim3 grid((unsigned)((threads + 255) / 256));
  const int32_t* cidx = idx;
  if (gs_mode == kGsTensor)
    launch_kernel(osci_sparse_update_kernel<kGsTensor>, grid, dim3(256), 0, st, W, ldw, C, D, cells, n_track, cidx, WM_prev, WQ_prev, D_M, D_Q, init);
  else if (gs_mode == kGsRow)
    launch_kernel(osci_sparse_update_kernel<kGsRow>, grid, dim3(256), 0, st, W, ldw, C, D, cells, n_track, cidx, WM_prev, WQ_prev, D_M, D_Q, init);
  else
    launch_kernel(osci_sparse_update_kernel<kGsBlock128>, grid, dim3(256), 0, st, W, ldw, C, D, cells, n_track, cidx, WM_prev, WQ_prev, D_M, D_Q, init);
  return cudaGetLastError() == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

nvfp4_status nvfp4_osci_sparse_suppress(float* W, int64_t ldw, int64_t C, int64_t D, int32_t gs_mode, int64_t n_track,
                                        const int32_t* idx, const float* D_M, const float* D_Q, float tau,
                                        unsigned long long* n_reset, void* workspace, size_t ws_bytes, void* stream) {
  if (!W) return NVFP4_ERR_NULL;
  if (C < 0 || D < 0 || ldw < D || n_track < 0 || n_track > C * D) return NVFP4_ERR_SHAPE;
  if (C * D >= ((int64_t)1 << 31)) return NVFP4_ERR_LIMIT;
  if (gs_mode < 0 || gs_mode > 2) return NVFP4_ERR_ENUM;
  if (n_track > 0 && (!idx || !D_M || !D_Q)) return NVFP4_ERR_NULL;
  if (bad_f32(W) || (n_reset && (reinterpret_cast<uintptr_t>(n_reset) & 7u))) return NVFP4_ERR_ALIGN;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || ws_bytes < nvfp4_osci_sparse_workspace_bytes(C, D, gs_mode, n_track, 2))
    return NVFP4_ERR_WORKSPACE;
  if (!device_is_sm100()) return NVFP4_ERR_ARCH;
  if (C == 0 || D == 0 || n_track == 0) return NVFP4_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  SparseWs ws{};
  sparse_ws_layout(C, D, gs_mode, n_track, 2, workspace, &ws);
  nvfp4_status s = sparse_amax(W, ldw, C, D, gs_mode, ws.cells, st);
  if (s != NVFP4_OK) return s;
  const uint32_t* cells = ws.cells;
  const int64_t threads = n_track;
  const dim3 grid((unsigned)((threads + 255) / 256));
  if (gs_mode == kGsTensor)
    launch_kernel(osci_sparse_decide_kernel<kGsTensor>, grid, dim3(256), 0, st, static_cast<const float*>(W), ldw, C, D, cells, n_track, idx, D_M, D_Q, tau, ws.newval);
  else if (gs_mode == kGsRow)
    launch_kernel(osci_sparse_decide_kernel<kGsRow>, grid, dim3(256), 0, st, static_cast<const float*>(W), ldw, C, D, cells, n_track, idx, D_M, D_Q, tau, ws.newval);
  else
    launch_kernel(osci_sparse_decide_kernel<kGsBlock128>, grid, dim3(256), 0, st, static_cast<const float*>(W), ldw, C, D, cells, n_track, idx, D_M, D_Q, tau, ws.newval);
  if (cudaGetLastError() != cudaSuccess) return NVFP4_ERR_CUDA;
  launch_kernel(osci_sparse_apply_kernel, dim3((unsigned)((n_track + 255) / 256)), dim3(256), 0, st, W, ldw, D, n_track, idx,
                static_cast<const float*>(ws.newval), n_reset);
  return cudaGetLastError() == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

}  // extern "C"
