// Device-side building blocks of the NVFP4 quantizers: format conversions, the element rounding rules and the
// counter-based random generator. Everything that can change a code or a scale is an explicit IEEE binary32
// operation (__fdiv_rn / __fmul_rn, no fast-math, no contraction), in the order the quantizer's contract fixes.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace nvfp4 {

// Programmatic dependent launch: let the next kernel of the stream start its prologue, then wait until the previous
// kernel has completed (its writes are visible, and it no longer reads what this kernel will overwrite). Must run
// before the first global-memory access. A no-op when the kernel was launched without the attribute.
__device__ __forceinline__ void pdl_prologue() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

constexpr int kRoundRTN = 0;
constexpr int kRoundSR = 1;
constexpr int kGsTensor = 0;
constexpr int kGsRow = 1;
constexpr int kGsBlock128 = 2;
constexpr int kSfLinear = 0;
constexpr int kSfTiled = 1;

// ---------------------------------------------------------------------------------------------------------
// BF16 pairs packed in a 32-bit word
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
// |x| of both halves as 16-bit patterns; for finite BF16 the pattern order is the value order.
__device__ __forceinline__ uint32_t bf16x2_abs_bits(uint32_t w) { return w & 0x7FFF7FFFu; }
// max of two packed pairs of non-negative BF16 patterns (as 16-bit unsigned integers == as BF16 values)
__device__ __forceinline__ uint32_t umax16x2(uint32_t a, uint32_t b) {
  const __nv_bfloat162 r = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&a), *reinterpret_cast<const __nv_bfloat162*>(&b));
  return *reinterpret_cast<const uint32_t*>(&r);
}
// max(|a|, |b|) of both halves in one instruction; the sign bits of the result are meaningless (xor of the inputs'),
// callers mask them off once at the end with bf16x2_abs_bits
__device__ __forceinline__ uint32_t amax16x2(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("max.xorsign.abs.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}
__device__ __forceinline__ uint32_t hmax_of_pair(uint32_t m) { return max(m & 0xFFFFu, m >> 16); }
__device__ __forceinline__ float bf16_bits_to_float(uint32_t b16) { return __uint_as_float(b16 << 16); }

// FP32 -> BF16 bit pattern, round to nearest even (finite inputs).
__device__ __forceinline__ uint16_t f32_to_bf16_bits(float v) {
  const uint32_t b = __float_as_uint(v);
  return (uint16_t)((b + 0x7FFFu + ((b >> 16) & 1u)) >> 16);
}

// ---------------------------------------------------------------------------------------------------------
// E4M3 (bias 7, max 448, no infinity): block scales
// ---------------------------------------------------------------------------------------------------------
// Non-negative float -> E4M3 byte: round to nearest, ties to even, saturate to 448.
__device__ __forceinline__ uint32_t e4m3_encode(float s) {
  uint16_t packed;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(packed) : "f"(0.0f), "f"(s));
  return packed & 0xFFu;
}
// E4M3 byte -> float (exact).
__device__ __forceinline__ float e4m3_decode(uint32_t byte) {
  uint32_t h2;
  asm("{.reg .b16 t; cvt.u16.u32 t, %1; cvt.rn.f16x2.e4m3x2 %0, t;}" : "=r"(h2) : "r"(byte & 0xFFu));
  return __half2float(__ushort_as_half((unsigned short)(h2 & 0xFFFFu)));
}

// ---------------------------------------------------------------------------------------------------------
// Scales of the double-block quantizer (paper Sec. 2.2): the pinned operation sequence.
// ---------------------------------------------------------------------------------------------------------
// x / c for a constant c, correctly rounded, in three instructions: q0 = RN(x * rc), rem = x - q0 * c (exact in the FMA),
// q = RN(q0 + rem * rc), rc = RN(1 / c). For c = 6 and c = 2688 this was compared with the IEEE quotient for every one of the
// 2^31 non-negative binary32 inputs: identical whenever the quotient is a normal number (quotients in the subnormal range
// differ in the last bits; there the value only ever feeds an E4M3 conversion that gives 0 either way, or lies below the
// smallest supported amax).
__device__ __forceinline__ float div_const(float x, float c, float rc) {
  const float q0 = __fmul_rn(x, rc);
  const float rem = __fmaf_rn(-q0, c, x);
  return __fmaf_rn(rem, rc, q0);
}
__device__ __forceinline__ float global_scale_from_amax(float amax) {
  return amax == 0.0f ? 1.0f : div_const(amax, 2688.0f, 0x1.861862p-12f);  // amax / (448 * 6)
}
// Returns the E4M3 byte of the block scale and the reciprocal r that maps x to the FP4 grid (0 if the scale is 0).
// round_up: take the smallest E4M3 value >= s instead of the nearest one (448 stays the ceiling), so that no element of
// the block lands beyond +-6 on the FP4 grid and stochastic rounding is unbiased for every element.
__device__ __forceinline__ uint32_t block_scale(float amax_b, float Sg, float& rcp, bool round_up = false) {
  const float t = __fdiv_rn(amax_b, Sg);
  const float s = div_const(t, 6.0f, 0x1.555556p-3f);
  uint32_t sb = e4m3_encode(s);
  float Sbf = e4m3_decode(sb);
  if (round_up && Sbf < s && sb < 0x7Eu) {  // non-negative E4M3 bytes are ordered like their values
    sb += 1u;
    Sbf = e4m3_decode(sb);
  }
  const float d = __fmul_rn(Sg, Sbf);
  rcp = (Sbf == 0.0f) ? 0.0f : __frcp_rn(d);  // the correctly rounded 1 / d
  return sb;
}

// ---------------------------------------------------------------------------------------------------------
// Philox4x32-10
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                               uint32_t k1) {
#pragma unroll
  for (int i = 0; i < 10; ++i) {
    // one widening multiply per product (high and low halves together)
    const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    c0 = n0; c1 = (uint32_t)p1; c2 = n2; c3 = (uint32_t)p0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return make_uint4(c0, c1, c2, c3);
}
// The ten round keys of a 64-bit Philox key, prepared on the host and handed to the kernels as a constant parameter:
// the rounds then read them as constant-bank operands instead of carrying two running additions per round.
struct PhiloxKeys {
  uint32_t k0[10], k1[10];
};
inline PhiloxKeys make_philox_keys(uint64_t seed) {
  PhiloxKeys r;
  uint32_t a = (uint32_t)seed, b = (uint32_t)(seed >> 32);
  for (int i = 0; i < 10; ++i) {
    r.k0[i] = a;
    r.k1[i] = b;
    a += 0x9E3779B9u;
    b += 0xBB67AE85u;
  }
  return r;
}
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, const PhiloxKeys& rk) {
#pragma unroll
  for (int i = 0; i < 10; ++i) {
    const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ rk.k0[i];
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ rk.k1[i];
    c0 = n0; c1 = (uint32_t)p1; c2 = n2; c3 = (uint32_t)p0;
  }
  return make_uint4(c0, c1, c2, c3);
}
// The four 32-bit words holding the 16-bit draws of elements idx8*8 .. idx8*8+7 of the operand.
__device__ __forceinline__ uint4 sr_words(const PhiloxKeys& rk, uint32_t stream_id, uint64_t idx8) {
  return philox4x32_10((uint32_t)idx8, (uint32_t)(idx8 >> 32), stream_id, 0u, rk);
}

// ---------------------------------------------------------------------------------------------------------
// Random Hadamard transformation along k (paper Sec. 4.1): x' = (x S) H with H = diag(H_16, H_16, ...), the orthonormal
// Sylvester matrix (entries +-1/4), and S a random sign diagonal that depends on k only.
//   * sign of k: bit (k % 128) of the Philox block with counter (k / 128, 0, rht_stream, 0x5348), key = seed; set = -1;
//   * arithmetic: v[i] = x[i] * (s_i / 4) (exact), then four butterfly stages h = 1, 2, 4, 8 in binary32.
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 rht_sign_words(uint64_t seed, uint32_t rht_stream, uint64_t group128) {
  return philox4x32_10((uint32_t)group128, (uint32_t)(group128 >> 32), rht_stream, 0x5348u, (uint32_t)seed,
                       (uint32_t)(seed >> 32));
}
__device__ __forceinline__ uint32_t rht_pick_word(const uint4& w, uint32_t q) {
  return q == 0 ? w.x : q == 1 ? w.y : q == 2 ? w.z : w.w;
}
// the 16 sign bits of k0 .. k0 + 15 (k0 a multiple of 16), bit i for k0 + i
__device__ __forceinline__ uint32_t rht_sign16(uint64_t seed, uint32_t rht_stream, int64_t k0) {
  const uint4 w = rht_sign_words(seed, rht_stream, (uint64_t)k0 >> 7);
  return (rht_pick_word(w, ((uint32_t)k0 >> 5) & 3u) >> ((uint32_t)k0 & 16u)) & 0xFFFFu;
}
// +-1/4 for position kk (0..127) of a 128-group
__device__ __forceinline__ float rht_factor(const uint4& w, uint32_t kk) {
  return __uint_as_float(0x3E800000u | ((rht_pick_word(w, kk >> 5) >> (kk & 31u)) << 31));
}
__device__ __forceinline__ void rht_scale16(float (&v)[16], uint32_t sign16) {
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __fmul_rn(v[i], __uint_as_float(0x3E800000u | ((sign16 << (31 - i)) & 0x80000000u)));
}
__device__ __forceinline__ void hadamard16_butterflies(float (&v)[16]) {
#pragma unroll
  for (int h = 1; h < 16; h <<= 1) {
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      if ((i & h) == 0) {
        const float a = v[i], b = v[i + h];
        v[i] = __fadd_rn(a, b);
        v[i + h] = __fsub_rn(a, b);
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------------------
// Element rounding to E2M1 (paper Sec. 2.1). Codes: sign << 3 | magnitude index.
// ---------------------------------------------------------------------------------------------------------
// Stochastic rounding. For an element with 16-bit draw u the rule is
//     round the magnitude up  iff  (u + 0.5) / 65536 < (a - q1) / (q2 - q1),   a = min(|y|, 6) in [q1, q2).
// It is evaluated exactly with one integer multiply-add on the bits of a float z:
//   * for a >= 1, z = a: the E2M1 cell of a is (bits >> 22) - 252 and the low 22 mantissa bits are the position inside
//     the cell in units of 2^-22 of the cell width;
//   * for a < 1 the cells [0, .5) and [.5, 1) are mapped onto [.5, .75) and [.75, 1) by z = 0.5 + a / 2, computed with
//     round-up so that the low bits are ceil(position * 2^22) (an integer n is < x iff n < ceil(x); when the ceiling
//     crosses into the next cell the true position was within 2^-24 of 1, where every draw rounds up);
//     0.5 + a / 2 >= a exactly when a <= 1, so z = max(a, 0.5 + a / 2) picks the right branch;
//   * adding r22 = 2^22 - 1 - ((2u + 1) << 5) = ((~u & 0xFFFF) << 6) | 0x1F to the bits carries into the cell index iff
//     position > (2u + 1) << 5, and adding -(252 << 22) as well leaves the magnitude index 0..7 in bits 22..24 with
//     nothing above. Both additions and a shift by 6 are one multiply-add modulo 2^32:
//         v = bits * 64 + c6,   c6 = ((~u & 0xFFFF) << 12) | 0x7C0 | (4 << 28)      (-252 = 4 modulo 16)
//     has the magnitude index in bits 28..30 and bit 31 clear, i.e. the code's magnitude already sits next to where the
//     sign bit of y lives: one bit-select gives the nibble in the top four bits (e2m1x8_sr below).
// Round-to-nearest (ties to the even code, saturating) of 8 scaled values, packed low nibble first.
__device__ __forceinline__ uint32_t e2m1x8_rtn(const float (&y)[8]) {
  uint32_t out;
  asm("{\n"
      ".reg .b8 b0, b1, b2, b3;\n"
      "cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n"
      "cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n"
      "cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n"
      "cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n"
      "mov.b32 %0, {b0, b1, b2, b3};\n"
      "}"
      : "=r"(out)
      : "f"(y[0]), "f"(y[1]), "f"(y[2]), "f"(y[3]), "f"(y[4]), "f"(y[5]), "f"(y[6]), "f"(y[7]));
  return out;
}

// Stochastic rounding of 8 scaled values with the draws packed in w (two 16-bit draws per word), packed low nibble
// first. The sign bits are those of y. Elements are taken last to first: a funnel shift moves each code's four top bits
// in below the ones already collected, so that element 0 ends in the lowest nibble.
__device__ __forceinline__ uint32_t e2m1x8_sr(const float (&y)[8], const uint4& w) {
  const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
  uint32_t out = 0, u_odd = 0;
#pragma unroll
  for (int e = 7; e >= 0; --e) {
    // The draw u of element e (the even element is the low half of its word), then c6 = ((0xFFFF - u) << 12) | 0x400007C0
    // = 0x4FFFF7C0 - u * 4096. Multiply-adds are written as such on purpose: the logic / shift / min-max pipe is the one
    // this code saturates (half the rate of the multiply-add pipe), so shifts and adds that can be a multiply-add are one.
    uint32_t c6, v;
    if (e & 1) {
      asm("mul.hi.u32 %0, %1, 65536;" : "=r"(u_odd) : "r"(ww[e >> 1]));
      asm("mad.lo.u32 %0, %1, 0xFFFFF000, 0x4FFFF7C0;" : "=r"(c6) : "r"(u_odd));
    } else {
      // the even element's draw is the low half of the same word: w * -4096 = u_even * -4096 - u_odd * 2^28 (mod 2^32),
      // so adding u_odd * 2^28 back gives its c6 without a mask (two multiply-adds instead of a logic op and one)
      uint32_t t;
      asm("mad.lo.u32 %0, %1, 0xFFFFF000, 0x4FFFF7C0;" : "=r"(t) : "r"(ww[e >> 1]));
      asm("mad.lo.u32 %0, %1, 0x10000000, %2;" : "=r"(c6) : "r"(u_odd), "r"(t));
    }
    const float a = fminf(fabsf(y[e]), 6.0f);
    const float z = fmaxf(a, __fmaf_ru(a, 0.5f, 0.5f));
    asm("mad.lo.u32 %0, %1, 64, %2;" : "=r"(v) : "r"(__float_as_uint(z)), "r"(c6));
    // code in bits 28..31 (v has the magnitude index in 28..30 and bit 31 clear); the funnel shift takes those four bits
    out = __funnelshift_l((__float_as_uint(y[e]) & 0x80000000u) | (v & 0x7FFFFFFFu), out, 4);
  }
  return out;
}

// E2M1 code -> value, as float.
__device__ __forceinline__ float e2m1_decode(uint32_t code) {
  const uint32_t m = code & 7u;
  // magnitudes 0, .5, 1, 1.5, 2, 3, 4, 6: exponent field e = m >> 1, mantissa bit m & 1
  const uint32_t e = m >> 1, f = m & 1u;
  const uint32_t bits = (e == 0) ? (f ? 0x3F000000u : 0u) : (((126u + e) << 23) | (f << 22));
  return __uint_as_float(bits | ((code & 8u) << 28));
}

// Decode 8 packed E2M1 codes times one E4M3 scale times the global scale into 8 floats:
// x_hat = (P * S_block) * S_global; the inner product is exact in FP16 (6 significant bits, |value| <= 2688).
__device__ __forceinline__ void decode8(uint32_t word, uint32_t sf_byte, float sg, float* out) {
  uint32_t h[4];
  asm("{\n"
      ".reg .b8 b0, b1, b2, b3;\n"
      "mov.b32 {b0, b1, b2, b3}, %4;\n"
      "cvt.rn.f16x2.e2m1x2 %0, b0;\n"
      "cvt.rn.f16x2.e2m1x2 %1, b1;\n"
      "cvt.rn.f16x2.e2m1x2 %2, b2;\n"
      "cvt.rn.f16x2.e2m1x2 %3, b3;\n"
      "}"
      : "=r"(h[0]), "=r"(h[1]), "=r"(h[2]), "=r"(h[3])
      : "r"(word));
  uint32_t s2;
  asm("{.reg .b16 t; cvt.u16.u32 t, %1; cvt.rn.f16x2.e4m3x2 %0, t;}" : "=r"(s2) : "r"(sf_byte | (sf_byte << 8)));
  const __half2 sb2 = *reinterpret_cast<__half2*>(&s2);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f = __half22float2(__hmul2(*reinterpret_cast<__half2*>(&h[i]), sb2));
    out[2 * i] = __fmul_rn(f.x, sg);
    out[2 * i + 1] = __fmul_rn(f.y, sg);
  }
}

// Decode 8 packed E2M1 codes times one E4M3 scale into four packed FP16 pairs (element 2i in the low half of word i):
// P * S_block, exact in FP16 (at most 7 significant bits, 2^-10 <= |value| <= 2688 or zero).
__device__ __forceinline__ void decode8_h2(uint32_t word, uint32_t sf_byte, uint32_t (&out)[4]) {
  uint32_t h[4];
  asm("{\n"
      ".reg .b8 b0, b1, b2, b3;\n"
      "mov.b32 {b0, b1, b2, b3}, %4;\n"
      "cvt.rn.f16x2.e2m1x2 %0, b0;\n"
      "cvt.rn.f16x2.e2m1x2 %1, b1;\n"
      "cvt.rn.f16x2.e2m1x2 %2, b2;\n"
      "cvt.rn.f16x2.e2m1x2 %3, b3;\n"
      "}"
      : "=r"(h[0]), "=r"(h[1]), "=r"(h[2]), "=r"(h[3])
      : "r"(word));
  uint32_t s2;
  asm("{.reg .b16 t; cvt.u16.u32 t, %1; cvt.rn.f16x2.e4m3x2 %0, t;}" : "=r"(s2) : "r"(sf_byte | (sf_byte << 8)));
  const __half2 sb2 = *reinterpret_cast<__half2*>(&s2);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const __half2 p = __hmul2(*reinterpret_cast<__half2*>(&h[i]), sb2);
    out[i] = *reinterpret_cast<const uint32_t*>(&p);
  }
}

// Scale, round and pack one 16-element inner block (two code words).
template <bool SR>
__device__ __forceinline__ uint2 quantize_block16(const float (&x)[16], float rcp, const PhiloxKeys& pk, uint32_t stream_id,
                                                  uint64_t idx8) {
  float y0[8], y1[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    y0[i] = __fmul_rn(x[i], rcp);
    y1[i] = __fmul_rn(x[8 + i], rcp);
  }
  uint2 out;
  if (SR) {
    out.x = e2m1x8_sr(y0, sr_words(pk, stream_id, idx8));
    out.y = e2m1x8_sr(y1, sr_words(pk, stream_id, idx8 + 1));
  } else {
    out.x = e2m1x8_rtn(y0);
    out.y = e2m1x8_rtn(y1);
  }
  return out;
}

// Byte offset of scale (r, kb) in the TILED128x4 layout with n_ktiles4 = (number of k-blocks, padded to 16) / 4.
__device__ __forceinline__ size_t sf_tiled_offset(int64_t r, int64_t kb, int64_t kb_padded) {
  const int64_t tile = (r >> 7) * (kb_padded >> 2) + (kb >> 2);
  return (size_t)tile * 512 + (size_t)((r & 31) * 16 + ((r >> 5) & 3) * 4 + (kb & 3));
}

}  // namespace nvfp4
