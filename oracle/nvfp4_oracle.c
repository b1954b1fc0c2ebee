/*
 * CPU oracle for the NVFP4 linear-layer path (double-block quantization + dequantize-then-FP64 GEMM).
 *
 * THIS IS TEST INFRASTRUCTURE. It is a slow, plain restatement of the method, written from the paper's
 * formulas, and exists only so that tests, the smoke check and the bench's cpu_baseline leg have something
 * independent to compare the CUDA library with. It shares no code, header, table or constant generator with
 * the CUDA path and must never be linked into, imported by or called from the product.
 *
 * Paper passages followed (TetraJet-v2):
 *   - Sec. 2.1 "NVFP4 Format": the E2M1 value set {0, +-0.5, 1, 1.5, 2, 3, 4, 6}; groups of 16 share one E4M3 scale.
 *   - Sec. 2.1 "Quantization": round_FP4,D (nearest value) and round_FP4,S (stochastic, unbiased on [-6, 6]).
 *   - Sec. 2.2 (double-block quantization equations): S_global = amax / (448*6); S_block = max|X/S_global| / 6;
 *     P = round_FP4(X / (S_global * S_block)); X ~ P * S_global * S_block.
 *   - Sec. 2.3: the six quantizers of the three matrix products; backward re-quantizes the dequantized
 *     forward operands.
 *
 * Readings where the paper is silent (each also listed in the design notes of the repository):
 *   - E4M3 is the OCP "FN" variant: bias 7, subnormals k*2^-9, max 448 (byte 0x7E), 0x7F is NaN, no infinity.
 *   - The block scale is rounded to E4M3 by round-to-nearest, ties to the even code, saturating at 448.
 *   - All scale arithmetic is IEEE binary32, one rounding per operation, in exactly this order:
 *        Sg = amax_g / 2688 ; t = amax_b / Sg ; s = t / 6 ; Sb = e4m3(s) ; d = Sg * Sb ; r = 1 / d ; y = x * r.
 *   - RTN ties go to the even code; |y| > 6 clamps to 6 in both rounding modes.
 *   - SR draws 16 random bits u per element and rounds the magnitude up iff (u + 0.5) / 65536 < f,
 *     f = (a - q1) / (q2 - q1); the sign of the input is re-attached (kept even when the magnitude is 0).
 *   - Random bits: Philox4x32-10, key = seed, counter = (idx / 8, stream_id, 0), idx = row * K16 + k.
 *   - An all-zero outer group takes Sg = 1; a block whose scale rounds to 0 gets all-zero magnitudes.
 *
 *   - Sec. 4.1 (Random Hadamard Transformation): A' = A S H with a block-diagonal Hadamard matrix of block size 16
 *     and a random sign diagonal S, applied along the contraction axis to both operands of the two backward products.
 *
 * Every function is pinned by tests that do not re-use its own formula (exhaustive format tables, hand-derived
 * golden blocks, Philox known-answer vectors, brute-force nearest-value search, unbiasedness statistics,
 * transposition/scaling/sign symmetries, brute-force triple-loop products).
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fopenmp -shared -fPIC nvfp4_oracle.c -o libnvfp4_oracle.so -lm
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_ROUND_RTN 0
#define ORC_ROUND_SR 1
#define ORC_ROUND_SR_SCALE_UP 2 /* SR with S_block rounded up to E4M3: no element beyond +-6, E[Q(x)] = x for all */
#define ORC_GS_TENSOR 0
#define ORC_GS_ROW 1
#define ORC_GS_BLOCK128 2

/* ---------------------------------------------------------------------------------------------------------
 * Formats
 * ------------------------------------------------------------------------------------------------------- */

/* Sec. 2.1: magnitudes of the eight E2M1 codes, in code order (1 exponent-0 subnormal step, then 2^(e-1)*(1+m/2)). */
static const double kE2M1Mag[8] = {0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0};

double orc_e2m1_value(int code) {
    double mag = kE2M1Mag[code & 7];
    return (code & 8) ? -mag : mag;
}

/* E4M3 (OCP FN variant) value of a byte, from the field definition; NaN for 0x7F / 0xFF. */
double orc_e4m3_value(int byte) {
    int sign = (byte >> 7) & 1;
    int e = (byte >> 3) & 15;
    int m = byte & 7;
    double v;
    if (e == 15 && m == 7) return NAN;
    if (e == 0)
        v = ldexp((double)m, -9); /* subnormal: m * 2^-9 */
    else
        v = ldexp(1.0 + (double)m / 8.0, e - 7);
    return sign ? -v : v;
}

/* Non-negative float -> E4M3 byte, round to nearest, ties to the even code, saturating at 448 (0x7E).
 * Written as the definition: scan all 127 finite non-negative values and keep the closest. */
int orc_e4m3_encode(float s) {
    double x = (double)s;
    int best = 0;
    double best_err = fabs(x - 0.0);
    for (int c = 1; c <= 0x7E; ++c) {
        double err = fabs(x - orc_e4m3_value(c));
        if (err < best_err || (err == best_err && (c & 1) == 0)) {
            best = c;
            best_err = err;
        }
    }
    return best;
}

/* Non-negative float -> the smallest E4M3 value that is >= s (byte), 448 (0x7E) if there is none.
 * Variant for strictly unbiased stochastic rounding: with S_block >= amax_b / (6 Sg) every |x| / (Sg S_block) <= 6 up to
 * the float roundings of d, r and y, so the clamp at 6 never removes more than those. Written as the definition. */
int orc_e4m3_encode_up(float s) {
    for (int c = 0; c <= 0x7E; ++c)
        if (orc_e4m3_value(c) >= (double)s) return c;
    return 0x7E;
}

/* ---------------------------------------------------------------------------------------------------------
 * Philox4x32-10 counter-based generator (Salmon et al., "Parallel random numbers: as easy as 1, 2, 3").
 * ------------------------------------------------------------------------------------------------------- */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The 16 random bits that element `idx` (linear index in the operand layout) draws. */
uint32_t orc_sr_bits(uint64_t seed, uint32_t stream_id, uint64_t idx) {
    uint64_t j = idx / 8;
    uint32_t e = (uint32_t)(idx % 8);
    uint32_t ctr[4] = {(uint32_t)j, (uint32_t)(j >> 32), stream_id, 0u};
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t w[4];
    orc_philox4x32_10(ctr, key, w);
    return (w[e >> 1] >> (16u * (e & 1u))) & 0xFFFFu;
}

/* ---------------------------------------------------------------------------------------------------------
 * Element rounding (Sec. 2.1 "Quantization")
 * ------------------------------------------------------------------------------------------------------- */

/* round_FP4,D on a magnitude a in [0, 6]: index of the nearest value; a tie goes to the even index. */
int orc_round_rtn_mag(float a) {
    int best = 0;
    double best_err = fabs((double)a - kE2M1Mag[0]);
    for (int m = 1; m < 8; ++m) {
        double err = fabs((double)a - kE2M1Mag[m]);
        if (err < best_err || (err == best_err && (m & 1) == 0)) {
            best = m;
            best_err = err;
        }
    }
    return best;
}

/* round_FP4,S on a magnitude a in [0, 6] with 16 random bits u.
 * The paper draws xi ~ U(-g/2, g/2), g = q2 - q1, and returns q2 iff a + xi > (q1 + q2) / 2. With xi = g (v - 1/2),
 * v ~ U(0, 1), that is: up iff 1 - v < f, f = (a - q1) / g. 1 - v is again uniform; it is discretised at the
 * mid-points (u + 1/2) / 65536 of 65536 equal bins. */
int orc_round_sr_mag(float a, uint32_t u) {
    if (a >= 6.0f) return 7;
    int lo = 0;
    while (lo < 6 && (double)a >= kE2M1Mag[lo + 1]) ++lo; /* q1 = mag[lo] <= a < q2 = mag[lo + 1] */
    double q1 = kE2M1Mag[lo], q2 = kE2M1Mag[lo + 1];
    double f = ((double)a - q1) / (q2 - q1);
    double v = ((double)u + 0.5) / 65536.0;
    return (v < f) ? lo + 1 : lo;
}

/* ---------------------------------------------------------------------------------------------------------
 * Double-block quantizer (Sec. 2.2) on a matrix x[R, K] (row-major float32, already in operand orientation:
 * quantization groups run along k). K16 = K rounded up to 16.
 *   codes  : uint8[R, K16/2], low nibble = even k, padding nibbles 0
 *   sf     : uint8[R, K16/16] E4M3 block scales (plain row-major)
 *   gscale : float[1] (TENSOR) | float[R] (ROW) | float[R, ceil(K/128)] (BLOCK128)
 * ------------------------------------------------------------------------------------------------------- */
static int64_t round_up(int64_t v, int64_t m) { return (v + m - 1) / m * m; }

static float group_amax(const float *x, int64_t n) {
    float amax = 0.0f;
    for (int64_t i = 0; i < n; ++i) {
        float a = fabsf(x[i]);
        if (a > amax) amax = a;
    }
    return amax;
}

static float global_scale_of(float amax_g) { return (amax_g == 0.0f) ? 1.0f : amax_g / 2688.0f; }

void orc_quantize(const float *x, int64_t R, int64_t K, int rounding, int gs_mode, uint64_t seed,
                  uint32_t stream_id, uint8_t *codes, uint8_t *sf, float *gscale) {
    const int64_t K16 = round_up(K, 16);
    const int64_t nb = K16 / 16;
    const int64_t ng = (K + 127) / 128;
    memset(codes, 0, (size_t)(R * K16 / 2));
    memset(sf, 0, (size_t)(R * nb));

    float Sg_tensor = 1.0f;
    if (gs_mode == ORC_GS_TENSOR) {
        float amax = 0.0f;
        for (int64_t r = 0; r < R; ++r) {
            float a = group_amax(x + r * K, K);
            if (a > amax) amax = a;
        }
        Sg_tensor = global_scale_of(amax);
        gscale[0] = Sg_tensor;
    }

#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < R; ++r) {
        const float *row = x + r * K;
        float Sg_row = 1.0f;
        if (gs_mode == ORC_GS_ROW) {
            Sg_row = global_scale_of(group_amax(row, K));
            gscale[r] = Sg_row;
        }
        for (int64_t b = 0; b < nb; ++b) {
            const int64_t k0 = b * 16;
            const int64_t len = (K - k0 < 16) ? (K - k0) : 16;
            float Sg;
            if (gs_mode == ORC_GS_TENSOR) {
                Sg = Sg_tensor;
            } else if (gs_mode == ORC_GS_ROW) {
                Sg = Sg_row;
            } else {
                const int64_t g = k0 / 128;
                const int64_t g0 = g * 128;
                const int64_t glen = (K - g0 < 128) ? (K - g0) : 128;
                Sg = global_scale_of(group_amax(row + g0, glen));
                gscale[r * ng + g] = Sg;
            }
            /* inner block scale */
            const float amax_b = group_amax(row + k0, len);
            const float t = amax_b / Sg;
            const float s = t / 6.0f;
            const int sb = (rounding == ORC_ROUND_SR_SCALE_UP) ? orc_e4m3_encode_up(s) : orc_e4m3_encode(s);
            const float Sbf = (float)orc_e4m3_value(sb);
            sf[r * nb + b] = (uint8_t)sb;
            const float d = Sg * Sbf;
            const float rcp = (Sbf == 0.0f) ? 0.0f : 1.0f / d;
            for (int64_t i = 0; i < len; ++i) {
                const int64_t k = k0 + i;
                const float xv = row[k];
                const float y = xv * rcp;
                float a = fabsf(y);
                if (a > 6.0f) a = 6.0f;
                int m;
                if (rounding == ORC_ROUND_SR || rounding == ORC_ROUND_SR_SCALE_UP) {
                    const uint64_t idx = (uint64_t)r * (uint64_t)K16 + (uint64_t)k;
                    m = orc_round_sr_mag(a, orc_sr_bits(seed, stream_id, idx));
                } else {
                    m = orc_round_rtn_mag(a);
                }
                const int code = (signbit(xv) ? 8 : 0) | m;
                codes[(r * K16 + k) / 2] |= (uint8_t)(code << (4 * (k & 1)));
            }
        }
    }
}

/* Global scale that applies to element (r, k). */
static float gscale_at(const float *gscale, int gs_mode, int64_t r, int64_t k, int64_t ng) {
    if (gs_mode == ORC_GS_TENSOR) return gscale[0];
    if (gs_mode == ORC_GS_ROW) return gscale[r];
    return gscale[r * ng + k / 128];
}

/* Exact dequantization P * S_block * S_global (Sec. 2.2, last equation) in double, out[R, K16]. */
void orc_dequantize(const uint8_t *codes, const uint8_t *sf, const float *gscale, int64_t R, int64_t K,
                    int gs_mode, double *out) {
    const int64_t K16 = round_up(K, 16);
    const int64_t nb = K16 / 16;
    const int64_t ng = (K + 127) / 128;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < R; ++r)
        for (int64_t k = 0; k < K16; ++k) {
            const int code = (codes[(r * K16 + k) / 2] >> (4 * (k & 1))) & 15;
            const double sb = orc_e4m3_value(sf[r * nb + k / 16]);
            const double sg = (double)gscale_at(gscale, gs_mode, r, k, ng);
            out[r * K16 + k] = orc_e2m1_value(code) * sb * sg;
        }
}

/* The aligned tensor X-hat / W-hat of Sec. 2.3 as the backward quantizers see it: float32, one rounding,
 * x_hat = (P * S_block) * S_global (the inner product is exact in binary32). out[R, K16]. */
void orc_rematerialize_f32(const uint8_t *codes, const uint8_t *sf, const float *gscale, int64_t R, int64_t K,
                           int gs_mode, float *out) {
    const int64_t K16 = round_up(K, 16);
    const int64_t nb = K16 / 16;
    const int64_t ng = (K + 127) / 128;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < R; ++r)
        for (int64_t k = 0; k < K16; ++k) {
            const int code = (codes[(r * K16 + k) / 2] >> (4 * (k & 1))) & 15;
            const float ps = (float)(orc_e2m1_value(code) * orc_e4m3_value(sf[r * nb + k / 16]));
            out[r * K16 + k] = ps * gscale_at(gscale, gs_mode, r, k, ng);
        }
}

/* ---------------------------------------------------------------------------------------------------------
 * Random Hadamard transformation (Sec. 4.1), block size 16, along k:  out[r, 16g .. 16g+15] = (x[r, 16g ..] * s) H_16.
 *   - H_16 is the orthonormal Sylvester matrix H_2 (x) H_2 (x) H_2 (x) H_2, entries +-1/4; it is symmetric.
 *   - s_k = -1 iff bit (k % 128) of the Philox4x32-10 block with counter (k / 128, 0, stream_id, 0x5348) and key = seed
 *     is set (word (k % 128) / 32, bit k % 32). The sign depends on k only: both operands of a product see the same S.
 *   - Readings (the paper fixes only the mathematics): float32 arithmetic; v[i] = x[i] * (s_i / 4) first (exact: a
 *     power of two), then the four butterfly stages in the order h = 1, 2, 4, 8, each replacing (a, b) = (v[i], v[i + h])
 *     for the i with (i & h) == 0 by (a + b, a - b). K is zero-extended to K16; the result has K16 columns.
 * ------------------------------------------------------------------------------------------------------- */
int orc_rht_sign_bit(uint64_t seed, uint32_t stream_id, uint64_t k) {
    uint64_t g = k / 128;
    uint32_t b = (uint32_t)(k % 128);
    uint32_t ctr[4] = {(uint32_t)g, (uint32_t)(g >> 32), stream_id, 0x5348u};
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t w[4];
    orc_philox4x32_10(ctr, key, w);
    return (int)((w[b / 32] >> (b % 32)) & 1u);
}

void orc_rht16(const float *x, int64_t R, int64_t K, uint64_t seed, uint32_t stream_id, float *out) {
    const int64_t K16 = round_up(K, 16);
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < R; ++r)
        for (int64_t k0 = 0; k0 < K16; k0 += 16) {
            float v[16];
            for (int i = 0; i < 16; ++i) {
                const int64_t k = k0 + i;
                const float xv = (k < K) ? x[r * K + k] : 0.0f;
                v[i] = xv * (orc_rht_sign_bit(seed, stream_id, (uint64_t)k) ? -0.25f : 0.25f);
            }
            for (int h = 1; h < 16; h <<= 1)
                for (int i = 0; i < 16; ++i)
                    if ((i & h) == 0) {
                        const float a = v[i], b = v[i + h];
                        v[i] = a + b;
                        v[i + h] = a - b;
                    }
            for (int i = 0; i < 16; ++i) out[r * K16 + k0 + i] = v[i];
        }
}

/* ---------------------------------------------------------------------------------------------------------
 * Matrix products: C[m, n] = sum_k A[m, k] * B[n, k], FP64 accumulation in k order (Sec. 2.3: all three
 * products of the layer have this form once both operands are laid out along the contraction axis).
 * ------------------------------------------------------------------------------------------------------- */
void orc_gemm_tn_f64(const double *A, const double *B, int64_t M, int64_t N, int64_t K, double *C) {
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int64_t k = 0; k < K; ++k) acc += A[m * K + k] * B[n * K + k];
            C[m * N + n] = acc;
        }
}

/* Same product at a list of (m, n) positions only; also returns sum_k |a_k b_k| per position (the scale of the
 * rounding error an FP32 accumulation may legitimately show). */
void orc_gemm_tn_f64_samples(const double *A, const double *B, int64_t K, const int64_t *ms, const int64_t *ns,
                             int64_t count, double *out, double *out_abs) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < count; ++i) {
        const double *a = A + ms[i] * K;
        const double *b = B + ns[i] * K;
        double acc = 0.0, acc_abs = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            acc += a[k] * b[k];
            acc_abs += fabs(a[k] * b[k]);
        }
        out[i] = acc;
        if (out_abs) out_abs[i] = acc_abs;
    }
}
