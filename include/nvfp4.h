/*
 * nvfp4.h — C ABI of the B200 (sm_100a) NVFP4 linear-layer library.
 *
 * The library implements the hot path of the TetraJet-v2 NVFP4 linear layer:
 *   - double-block quantization to NVFP4 (paper Sec. 2.2): FP32 global scale per outer group, one E4M3 scale
 *     per 16 elements, E2M1 codes; round-to-nearest or stochastic rounding (Sec. 2.1), along either axis;
 *   - the three block-scaled FP4 matrix products of the layer (Sec. 2.3):
 *         Y = Q1(X) Q2(W)^T,   dX = Q3(dY) Q4(W-hat),   dW = Q5(dY^T) Q6(X-hat),
 *     where backward re-quantizes the dequantized forward operands X-hat, W-hat;
 *   - OutControl's split (Sec. 4.2, without the Hadamard factors): a static set of outlier channels of X / W
 *     stays in BF16 and goes through high-precision products.
 *
 * Conventions, valid for every entry point unless stated otherwise:
 *   - All data pointers are DEVICE pointers owned by the caller. The library never allocates, frees or
 *     synchronises; every call only enqueues work on `stream` (a cudaStream_t passed as void*).
 *   - Arguments are validated on the host before anything is launched: a non-zero status means nothing ran.
 *   - Matrices are row-major. BF16 matrices have a leading dimension `ld` in elements (multiple of 8) and a
 *     16-byte aligned base.
 *   - Non-finite inputs are outside the contract (results unspecified, no fault).
 *   - Only compute capability 10.x devices are supported (NVFP4_ERR_ARCH otherwise). There is no CPU path.
 */
#ifndef NVFP4_H_
#define NVFP4_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  NVFP4_OK = 0,
  NVFP4_ERR_NULL = 1,      /* a required pointer is NULL */
  NVFP4_ERR_SHAPE = 2,     /* a size is negative, zero where not allowed, or inconsistent */
  NVFP4_ERR_ALIGN = 3,     /* a pointer or leading dimension breaks the alignment rules */
  NVFP4_ERR_ENUM = 4,      /* an enum argument is out of range */
  NVFP4_ERR_WORKSPACE = 5, /* workspace missing or smaller than nvfp4_*_workspace_bytes says */
  NVFP4_ERR_ARCH = 6,      /* current device is not sm_100 */
  NVFP4_ERR_CUDA = 7,      /* a CUDA runtime / driver call failed (launch error, tensor-map encode) */
  NVFP4_ERR_TIMEOUT = 8,   /* reported through dev_status only: a bounded device-side wait ran out */
  NVFP4_ERR_LIMIT = 9      /* a size exceeds a fixed capacity of the entry point (see nvfp4_quantize_static) */
} nvfp4_status;

/* Element rounding (paper Sec. 2.1).
 * RTN: round to nearest, ties to the even code. SR: stochastic rounding with 16 random bits per element.
 * SR_SCALE_UP: SR, and the block scale S_block is the smallest E4M3 value >= amax_b / (6 S_global) instead of the nearest
 *   one (448 stays the ceiling). With the nearest scale about half of the blocks get a scale rounded down, their
 *   largest element lands in (6, 6.43] on the FP4 grid and is clamped, so E[Q(x)] = x (Sec. 2.1, stated for -6 <= x <= 6)
 *   fails for it; with the rounded-up scale every element lies within +-6 and the expectation is exact. A variant the
 *   paper's unbiasedness ablation motivates; not the default of any quantizer. */
typedef enum { NVFP4_ROUND_RTN = 0, NVFP4_ROUND_SR = 1, NVFP4_ROUND_SR_SCALE_UP = 2 } nvfp4_round;

/* Axis along which the 16-element groups run in the SOURCE matrix.
 * ROW: groups along the columns of a row; the operand has the source's shape [rows, cols].
 * COL: groups down the rows of a column; the operand is the transpose, shape [cols, rows]. */
typedef enum { NVFP4_AXIS_ROW = 0, NVFP4_AXIS_COL = 1 } nvfp4_axis;

/* Granularity of the FP32 "global" scale S_global of Sec. 2.2.
 * TENSOR: one per tensor (needs an amax pre-pass). ROW: one per operand row. BLOCK128: one per 128 consecutive
 * k of an operand row — the paper's 1x128 outer block. */
typedef enum { NVFP4_GS_TENSOR = 0, NVFP4_GS_ROW = 1, NVFP4_GS_BLOCK128 = 2 } nvfp4_gs_mode;

/* Memory layout of the E4M3 block scales of an operand [R, Kp].
 * LINEAR:     row-major [R, Kp/16].
 * TILED128x4: what the tensor core reads. 512-byte tiles cover 128 rows x 4 k-blocks; inside a tile the byte
 *             of (r, kb) sits at (r % 32) * 16 + (r / 32) * 4 + (kb % 4); tiles are ordered k-tile fastest
 *             within a 128-row tile; rows are padded to 128 and k-blocks to 16 (zero bytes). */
typedef enum { NVFP4_SF_LINEAR = 0, NVFP4_SF_TILED128x4 = 1 } nvfp4_sf_layout;

typedef enum { NVFP4_DT_BF16 = 0, NVFP4_DT_F32 = 1 } nvfp4_dtype;

/* A quantized GEMM operand [R, K], groups along K. Kp = K rounded up to 128; padding codes and scales are 0.
 *   codes : uint8 [R, Kp/2], two E2M1 codes per byte, low nibble = even k; code = sign<<3 | magnitude index
 *           into {0, .5, 1, 1.5, 2, 3, 4, 6}.
 *   sf    : E4M3 bytes, nvfp4_operand_sf_bytes() of them, layout per sf_layout.
 *   gscale: 1 (TENSOR) | R (ROW) | R * (Kp/128) (BLOCK128) floats, row-major.
 * The struct lives on the host; the three pointers are device memory owned by the caller. R, K, gs_mode and
 * sf_layout are inputs to the quantize calls (they say what the caller allocated) and are validated there. */
typedef struct {
  uint8_t* codes;
  uint8_t* sf;
  float* gscale;
  int64_t R, K;
  int32_t gs_mode;   /* nvfp4_gs_mode */
  int32_t sf_layout; /* nvfp4_sf_layout */
} nvfp4_operand;

/* Host-only size helpers (no CUDA call). K padded to 128; bytes of codes / scales; floats of gscale. */
int64_t nvfp4_padded_k(int64_t K);
size_t nvfp4_operand_codes_bytes(int64_t R, int64_t K);
size_t nvfp4_operand_sf_bytes(int64_t R, int64_t K, int32_t sf_layout);
size_t nvfp4_operand_gscale_count(int64_t R, int64_t K, int32_t gs_mode);

const char* nvfp4_status_string(nvfp4_status s);

/* ---------------------------------------------------------------------------------------------------------
 * nvfp4_quantize — double-block quantization of a BF16 matrix (Sec. 2.2; rounding per Sec. 2.1).
 *
 *   src_bf16 [rows, cols], leading dimension ld.
 *   axis     ROW -> out is [rows, n_keep or cols]; COL -> out is the transpose [n_keep or cols, rows].
 *   rounding RTN: nearest E2M1 value, ties to the even code. SR: 16 random bits u per element from
 *            Philox4x32-10 (key = seed, counter = (idx / 8, stream_id, 0), idx = r * Kp16 + k in the OPERAND,
 *            Kp16 = K rounded up to 16); the magnitude rounds up iff (u + 0.5) / 65536 < (a - q1) / (q2 - q1).
 *            SR_SCALE_UP: the same draws and rule, with S_block rounded up instead of to nearest (see nvfp4_round).
 *   rht_stream_id  0: off. Otherwise the random Hadamard transformation of Sec. 4.1 is applied along the operand's K before
 *            anything else: each aligned block of 16 consecutive k (zero-extended at the end of K) becomes (x S) H_16,
 *            H_16 the orthonormal Sylvester matrix (entries +-1/4), S the sign diagonal with s_k = -1 iff bit (k % 128)
 *            of the Philox block with counter (k / 128, 0, rht_stream_id, 0x5348) and key = seed is set. Binary32:
 *            v_i = x_i * (s_i / 4), then the butterfly stages h = 1, 2, 4, 8, each (a, b) -> (a + b, a - b). Scales and
 *            codes are those of the transformed matrix, whose columns K .. K16-1 are in general non-zero. Two operands
 *            transformed with the same seed and stream multiply to the product of the untransformed ones (up to
 *            rounding). Not combined with keep_cols (NVFP4_ERR_ENUM).
 *   keep_cols optional sorted list (device, int32) of the n_keep source columns that are kept; the others
 *            (OutControl's outlier channels) are skipped and the kept ones are compacted along K. ROW axis only
 *            (NVFP4_ERR_SHAPE otherwise). NULL keeps all columns (n_keep is ignored).
 *   out      operand to fill; out->R / out->K must equal the shape stated above.
 *   workspace at least nvfp4_quantize_workspace_bytes(out->R, gs_mode); holds the amax cells of the TENSOR
 *            and ROW modes.
 *
 * Arithmetic (binary32, one rounding each, in this order): Sg = amax_g / 2688 (1 if the group is all zero);
 * t = amax_b / Sg; s = t / 6; Sb = e4m3_rn_satfinite(s); d = Sg * Sb; r = 1 / d (0 if Sb = 0); y = x * r;
 * magnitude = round(min(|y|, 6)); the input's sign bit is kept.
 * --------------------------------------------------------------------------------------------------------- */
size_t nvfp4_quantize_workspace_bytes(int64_t out_rows, int32_t gs_mode);
nvfp4_status nvfp4_quantize(const void* src_bf16, int64_t rows, int64_t cols, int64_t ld, int32_t axis,
                            int32_t rounding, uint64_t seed, uint32_t stream_id, uint32_t rht_stream_id,
                            const int32_t* keep_cols, int64_t n_keep, const nvfp4_operand* out, void* workspace,
                            size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------------------
 * nvfp4_quantize_static — nvfp4_quantize without a workspace argument. (The paper has no counterpart: this is a
 * packaging variant of the same quantizer, not a step of the method.)
 *
 * For callers that cannot obtain device memory where they call from — code inside an allocator hook or under a
 * framework's no-allocation guard, a plugin that receives tensors but no allocator, a loop whose memory was fixed
 * at start-up. The amax cells live in a fixed array inside the library image (NVFP4_STATIC_MAX_ROWS 32-bit cells,
 * 256 KiB, held by every GPU that loads the library until the process exits). The call allocates and frees
 * nothing. Inputs, outputs, arithmetic and results are those of nvfp4_quantize.
 *   - Capacity: gs_mode ROW needs one cell per operand row; out->R > NVFP4_STATIC_MAX_ROWS returns NVFP4_ERR_LIMIT
 *     and nothing is launched. TENSOR and BLOCK128 have no such limit.
 *   - The first call made with a given device current looks up the array's device address; make that first call
 *     outside any stream capture.
 *   - Every call on a device shares the one array. The cells a call uses are cleared on `stream` before use, so
 *     calls that are ordered (same stream, or ordered by events) are independent; calls whose kernels can overlap
 *     on the GPU (different streams, no ordering) race on the cells and give undefined scales.
 * --------------------------------------------------------------------------------------------------------- */
#define NVFP4_STATIC_MAX_ROWS 65536
int64_t nvfp4_quantize_static_max_rows(void);
nvfp4_status nvfp4_quantize_static(const void* src_bf16, int64_t rows, int64_t cols, int64_t ld, int32_t axis,
                                   int32_t rounding, uint64_t seed, uint32_t stream_id, const int32_t* keep_cols,
                                   int64_t n_keep, const nvfp4_operand* out, void* stream);

/* ---------------------------------------------------------------------------------------------------------
 * nvfp4_quantize_w16x16 / nvfp4_transpose_operand16 -- the two pieces of the 16x16 weight-block recipe (see
 * nvfp4_layer_cfg.weight_block), exposed for tests and for callers that drive the GEMMs themselves.
 *
 *   nvfp4_quantize_w16x16: W_bf16 [C, D] (leading dimension ldw, multiple of 8) -> out [C, D], gs_mode TENSOR, either scale
 *     layout. amax_b is taken over 16x16 squares (ragged squares cover the rows / columns that exist); round to nearest.
 *     workspace: nvfp4_quantize_workspace_bytes(C, NVFP4_GS_TENSOR).
 *   nvfp4_transpose_operand16: in [C, D] made by nvfp4_quantize_w16x16 -> out [D, C] (gs_mode TENSOR): the operand of
 *     W-hat^T with identical values; pure data movement. in and out must not overlap.
 *   Errors: NVFP4_ERR_NULL, _SHAPE (out shape), _ENUM (gs_mode), _ALIGN, _WORKSPACE, _ARCH, _CUDA.
 * ------------------------------------------------------------------------------------------------------- */
nvfp4_status nvfp4_quantize_w16x16(const void* W_bf16, int64_t C, int64_t D, int64_t ldw, const nvfp4_operand* out,
                                   void* workspace, size_t ws_bytes, void* stream);
nvfp4_status nvfp4_transpose_operand16(const nvfp4_operand* in, const nvfp4_operand* out, void* stream);

/* ---------------------------------------------------------------------------------------------------------
 * nvfp4_requantize_t — the backward quantizers Q4 / Q6 of Sec. 2.3: dequantize a forward operand to the
 * aligned tensor (x_hat = (P * S_block) * S_global, one binary32 rounding), and quantize its TRANSPOSE.
 *
 *   in       forward operand [R, K] (any gs_mode, either sf layout).
 *   out      operand [n_rows_out, R]; without a row map n_rows_out = in->K.
 *   row_map  optional (device, int32 [n_rows_out]): output row d takes column row_map[d] of `in` when
 *            row_map[d] >= 0, and column d of the BF16 matrix hp_bf16 [R, >= n_rows_out] (leading dimension
 *            hp_ld) when row_map[d] < 0 — OutControl's W-hat, whose outlier columns come from W itself
 *            (Sec. 4.2). NULL: identity map, hp_bf16 unused.
 *   rounding, seed, stream_id, rht_stream_id, workspace: as in nvfp4_quantize (the transformation runs along the
 *            output operand's K, i.e. along the rows of `in`).
 * --------------------------------------------------------------------------------------------------------- */
nvfp4_status nvfp4_requantize_t(const nvfp4_operand* in, const void* hp_bf16, int64_t hp_ld,
                                const int32_t* row_map, int64_t n_rows_out, int32_t rounding, uint64_t seed,
                                uint32_t stream_id, uint32_t rht_stream_id, const nvfp4_operand* out,
                                void* workspace, size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------------------
 * nvfp4_gemm — block-scaled FP4 product of two operands (the "FP4 MM" of Sec. 2.3):
 *      C[m, n] (+)= sum_k  (Pa * Sba * Sga)[m, k] * (Pb * Sbb * Sgb)[n, k]
 * FP32 accumulation on the tensor cores; TENSOR / ROW global scales are applied in the epilogue, BLOCK128
 * scales per 128-wide k chunk (each chunk's partial product is promoted into FP32 registers; this variant takes
 * K up to 16384 and returns NVFP4_ERR_LIMIT beyond).
 *
 *   A [M, K], B [N, K]: same K and gs_mode, sf_layout = TILED128x4.
 *   C [M, N] row-major, leading dimension ldc (elements), dtype c_dtype; 16-byte aligned rows.
 *   accumulate != 0 adds to the existing C (read in c_dtype, summed in FP32).
 *   dev_status optional device int: set to NVFP4_ERR_TIMEOUT if a bounded wait inside the kernel ran out
 *            (the kernel then drains and exits; C is unspecified). Never written otherwise.
 *   workspace at least nvfp4_gemm_workspace_bytes(M, N, K) bytes; the present kernels need none (the query returns 0 for
 *            every shape and workspace may then be NULL).
 *
 * nvfp4_gemm_ex is the same product with explicit control over what nvfp4_gemm chooses by itself (opts == NULL gives
 * nvfp4_gemm). It exists for tests and for measurements:
 *   variant  AUTO: chosen from the shape. TILE128: one CTA per 128 x 128 output tile, two accumulators. PAIR256: a pair of
 *            CTAs on neighbouring SMs per 256 x 256 tile (cta_group::2), one accumulator. PAIR192: the same pair on
 *            256 x 192 tiles with two accumulators. The pair variants take the TENSOR and ROW scale modes only
 *            (NVFP4_ERR_ENUM with BLOCK128).
 *   wait_limit_cycles  bound of every device-side wait, in SM clock cycles (0: the default, about two seconds).
 *   starve_first_stage  test hook of the bounded waits: when non-zero, the barrier of the first operand stage expects 16
 *            bytes more than will ever arrive, so the first wait of the MMA warp runs out; the kernel then reports
 *            NVFP4_ERR_TIMEOUT through dev_status, every role drains and the call returns. C is unspecified.
 * --------------------------------------------------------------------------------------------------------- */
size_t nvfp4_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K);
nvfp4_status nvfp4_gemm(const nvfp4_operand* A, const nvfp4_operand* B, void* C, int32_t c_dtype, int64_t ldc,
                        int32_t accumulate, int32_t* dev_status, void* workspace, size_t ws_bytes, void* stream);

typedef enum { NVFP4_GEMM_AUTO = 0, NVFP4_GEMM_TILE128 = 1, NVFP4_GEMM_PAIR256 = 2, NVFP4_GEMM_PAIR192 = 3 } nvfp4_gemm_variant;
typedef struct {
  int32_t variant;           /* nvfp4_gemm_variant */
  int32_t starve_first_stage;
  int64_t wait_limit_cycles;
} nvfp4_gemm_opts;
nvfp4_status nvfp4_gemm_ex(const nvfp4_operand* A, const nvfp4_operand* B, void* C, int32_t c_dtype, int64_t ldc,
                           int32_t accumulate, int32_t* dev_status, const nvfp4_gemm_opts* opts, void* workspace,
                           size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------------------
 * The layer (Sec. 2.3; OutControl split of Sec. 4.2). X [N_tok, D], W [C, D], Y / dY [N_tok, C].
 * --------------------------------------------------------------------------------------------------------- */
typedef struct {
  int32_t gs_mode;     /* nvfp4_gs_mode, used by all six quantizers */
  int32_t rounding[6]; /* nvfp4_round of Q1..Q6; the paper's assignment is RTN, RTN, SR, SR, SR, SR */
  uint64_t seed;       /* Philox key; the six quantizers use stream ids 1..6 */
  int32_t y_dtype, dx_dtype, dw_dtype; /* nvfp4_dtype of the three outputs */
  /* OutControl (all NULL / 0 when unused); device int32 arrays prepared by the caller:                       */
  int64_t n_out;               /* number of outlier channels |A|                                             */
  const int32_t* outlier_cols; /* [n_out]      sorted outlier channel indices                                */
  const int32_t* keep_cols;    /* [D - n_out]  sorted complement                                             */
  const int32_t* col_map;      /* [D]          position of channel d in keep_cols, or -1 for an outlier      */
  int32_t* dev_status;         /* optional, see nvfp4_gemm                                                   */
  /* Random Hadamard transformation of both operands of the two backward products (Sec. 4.1): 0 off, 1 on.
   * Q3 and Q4 use sign stream 7 along C, Q5 and Q6 sign stream 8 along the tokens; forward is never transformed. */
  int32_t rht;
  /* Precision of the outlier channels under OutControl (Sec. 4.2 allows "FP8, BF16"; the paper gives no FP8 recipe, this
   * one is the library's): 0 = BF16 as they are. 1 = E4M3 with a per-tensor power-of-two scale: forward replaces
   * X[:, A] and W[:, A] by T8 = E4M3(T / 2^e) 2^e, e the smallest integer with amax|T| / 2^e <= 448 (round to nearest
   * even; exact scalings), and everything that uses the outlier part (forward side product, dW[:, A], W-hat[:, A]) uses
   * T8. T8 is exactly representable in BF16, which is how X_out / W_out hold it; products of T8 accumulated in FP32 equal
   * the FP8 tensor product times the two scales. */
  int32_t outlier_format;
  /* Weight scale group (Sec. 2.3, third difference to NVIDIA's recipe; appendix on the overhead of the 1x16 scheme):
   * 0 = 1x16 blocks, the paper's choice. 1 = 16x16 squares, the recipe it is compared with: Q2 takes amax_b over the
   * square (same pinned scale arithmetic, round to nearest), the 16 rows of a square repeat its scale byte, and dX uses
   * the forward codes transposed as they are -- no Q4, so no rounding, no random bits and no Hadamard factor on the dX
   * product (cfg.rht then applies to dW only). Requires gs_mode TENSOR, n_out = 0 and rounding[1] = RTN (NVFP4_ERR_ENUM). */
  int32_t weight_block;
  /* Optional second stream (all four NULL: everything is enqueued on the call's `stream`). The two backward products
   * share nothing but their inputs, and forward's two quantizers are independent: with a side stream the dX chain (Q3, Q4,
   * product) and the weight quantizer run on it, forked from `stream` by ev_fork at entry and joined into it by ev_join
   * before the call returns (ev_aux orders the shared amax pass of dY before Q5 under OutControl). Work queued on `stream`
   * after the call sees all results; nothing else is observable, and the pattern is legal under stream capture. The
   * stream (a cudaStream_t) and the three events (cudaEvent_t, timing disabled is enough) belong to the caller, must live
   * on the current device and must not be used by another call at the same time; the library creates none. */
  void* side_stream;
  void* ev_fork;
  void* ev_join;
  void* ev_aux;
} nvfp4_layer_cfg;

/* What forward leaves for backward. qx [N_tok, D - n_out] and qw [C, D - n_out] are filled by
 * nvfp4_linear_fwd (buffers are the caller's, sf_layout TILED128x4). With OutControl (n_out > 0) forward also
 * fills X_out [N_tok, Kh] and W_out [C, Kh]: compact BF16 copies of the outlier channels X[:, A], W[:, A], zero-padded
 * to Kh = nvfp4_outlier_pad(n_out) columns (caller-owned device buffers, 16-byte aligned; NULL when n_out = 0).
 * Backward reads only these and the operands; X and W themselves are not touched again. */
typedef struct {
  nvfp4_operand qx, qw;
  const void* X; /* BF16 [N_tok, D] (recorded by forward; informational) */
  const void* W; /* BF16 [C, D]     */
  int64_t ldx, ldw;
  int64_t N_tok, D, C;
  void* X_out; /* BF16 [N_tok, Kh] */
  void* W_out; /* BF16 [C, Kh]     */
} nvfp4_saved;

/* Columns of the compact outlier-channel matrices: n_out rounded up to a multiple of 64 (0 for n_out = 0). */
int64_t nvfp4_outlier_pad(int64_t n_out);

typedef enum { NVFP4_OP_FWD = 0, NVFP4_OP_BWD_DX = 1, NVFP4_OP_BWD_DW = 2, NVFP4_OP_BWD = 3 } nvfp4_op_kind;
size_t nvfp4_linear_workspace_bytes(int32_t op_kind, int64_t N_tok, int64_t D, int64_t C, int64_t n_out,
                                    int32_t gs_mode);

/* Where a backward call keeps its quantized operands inside its workspace (host-only, nothing is launched): fills *out
 * with the descriptor of Q3(dY) [N_tok, C], Q4(W-hat^T) [D, C], Q5(dY^T) [C, N_tok] or Q6(X-hat^T) [D - n_out, N_tok]
 * (which = 3 .. 6; tiled scales) for a workspace that was, or will be, passed to the call of kind op_kind with the same
 * shapes. The contents are valid once that call has run on its stream and until the workspace is used again: a way to
 * inspect what the products of Sec. 2.3 actually consumed. which = 3, 4 go with NVFP4_OP_BWD_DX or NVFP4_OP_BWD, 5, 6 with
 * NVFP4_OP_BWD_DW or NVFP4_OP_BWD (NVFP4_ERR_ENUM otherwise). */
nvfp4_status nvfp4_linear_bwd_operand(int32_t op_kind, int32_t which, int64_t N_tok, int64_t D, int64_t C, int64_t n_out,
                                      int32_t gs_mode, void* workspace, size_t ws_bytes, nvfp4_operand* out);

/* Y = Q1(X[:, keep]) Q2(W[:, keep])^T  +  X[:, outl] W[:, outl]^T (BF16 inputs, FP32 accumulate). */
nvfp4_status nvfp4_linear_fwd(const void* X, int64_t ldx, const void* W, int64_t ldw, int64_t N_tok, int64_t D,
                              int64_t C, const nvfp4_layer_cfg* cfg, void* Y, int64_t ldy, nvfp4_saved* saved,
                              void* workspace, size_t ws_bytes, void* stream);

/* dX = Q3(dY S H) Q4(H^T S^T W-hat): one FP4 product over all D channels; W-hat's outlier columns are W's.
 * (S H is the identity unless cfg->rht is set.) */
nvfp4_status nvfp4_linear_bwd_dx(const void* dY, int64_t lddy, const nvfp4_saved* saved,
                                 const nvfp4_layer_cfg* cfg, void* dX, int64_t lddx, void* workspace,
                                 size_t ws_bytes, void* stream);

/* dW[:, keep] = Q5(dY^T S H) Q6(H^T S^T X-hat[:, keep]);  dW[:, outl] = dY^T X[:, outl] (BF16 inputs, FP32 accumulate,
 * never transformed). */
nvfp4_status nvfp4_linear_bwd_dw(const void* dY, int64_t lddy, const nvfp4_saved* saved,
                                 const nvfp4_layer_cfg* cfg, void* dW, int64_t lddw, void* workspace,
                                 size_t ws_bytes, void* stream);

/* Both backward products of Sec. 2.3 in one call: exactly nvfp4_linear_bwd_dx followed by nvfp4_linear_bwd_dw (bit-identical
 * outputs), except that in the TENSOR scale mode without the Hadamard transformation the per-tensor amax of dY, which Q3
 * and Q5 share, is computed once. workspace: nvfp4_linear_workspace_bytes(NVFP4_OP_BWD, ...).
 *
 * Streams: with cfg->side_stream set, the dX chain runs there beside the dW chain (see nvfp4_layer_cfg). */
nvfp4_status nvfp4_linear_bwd(const void* dY, int64_t lddy, const nvfp4_saved* saved, const nvfp4_layer_cfg* cfg,
                              void* dX, int64_t lddx, void* dW, int64_t lddw, void* workspace, size_t ws_bytes,
                              void* stream);

/* ---------------------------------------------------------------------------------------------------------
 * Simulated FP6 x FP4 products (Sec. 5.4, paragraph "Precision Switching in Final Stage"):
 *     Y = Q6_D(X) Q4_D(W^T),   dX = Q6_S(dY) Q4_S(W-hat),   dW = Q4_S(dY^T) Q6_S(X-hat)
 * (D deterministic, S stochastic rounding; X-hat / W-hat the dequantized forward operands). The paper names FP6 and gives
 * these three products, nothing more; the FP6 quantizer is this library's definition: element format E2M3 (sign, two
 * exponent bits with bias 1, three mantissa bits: 32 magnitudes 0, 1/8, ..., 7/8, 1 ... 1.875, 2 ... 3.75, 4 ... 7.5), the
 * FP4 quantizer's scale sequence (Sec. 2.2) with Q_max = 7.5 in place of 6 (Sg = amax / 3360, t = amax_b / Sg,
 * s = t / 7.5, Sb = e4m3(s), d = Sg Sb, r = 1 / d, y = x r, each one binary32 operation, |y| clamped to 7.5), a per-tensor
 * global scale (TENSOR mode only), NVFP4_ROUND_RTN (ties to the even code) or NVFP4_ROUND_SR with the FP4 quantizer's
 * rule, 16-bit draws and Philox addressing (element idx = row * K16 + k of the operand).
 *
 * No tensor-core instruction multiplies E2M3 by E2M1 values under E4M3 block scales, and the paper simulates as well: the
 * operands of these products are "dense" -- vals = P * S_block as BF16 [R, ld] (exact: at most 4 + 4 significant bits),
 * ld = nvfp4_dense_ld(K) = K rounded up to 64, columns K .. ld - 1 zero, rows 16-byte aligned, plus one FP32 global scale.
 *   nvfp4_fp6_quantize      Q6 along the rows of a BF16 matrix [rows, cols] (leading dimension ld, 16-byte aligned rows as for
 *                           nvfp4_quantize: NVFP4_ERR_ALIGN otherwise; operand K = cols).
 *   nvfp4_fp6_requantize_t  Q6 of the transposed aligned tensor float32(vals * gscale) of a dense operand `in` [R, K]:
 *                           out is [K, R], its blocks run along R (Q6_S(X-hat) of the dW product).
 *   nvfp4_expand_operand    an ordinary FP4 operand (TENSOR mode, either scale layout) as a dense operand: no arithmetic
 *                           beyond P * S_block.
 *   nvfp4_dense_gemm        C [A.R, B.R] = (A.gscale B.gscale) A.vals B.vals^T, A.K == B.K: BF16 tensor-core product with
 *                           FP32 accumulation (the BF16 path of the 128 x 128 GEMM kernel), C BF16 or FP32 with leading
 *                           dimension ldc, 16-byte aligned rows; dev_status as for nvfp4_gemm.
 * workspace (the two quantizers): at least nvfp4_fp6_workspace_bytes() bytes, 16-byte aligned. All pointers device.
 * Errors: NULL / SHAPE / ALIGN / ENUM (rounding, c_dtype, an operand that is not TENSOR mode) / WORKSPACE / ARCH; nothing is
 * launched on an error.
 * --------------------------------------------------------------------------------------------------------- */
typedef struct {
  void* vals;       /* BF16 [R, ld] */
  float* gscale;    /* FP32 [1] */
  int64_t R, K, ld; /* ld == nvfp4_dense_ld(K) */
} nvfp4_dense_operand;
int64_t nvfp4_dense_ld(int64_t K);
size_t nvfp4_fp6_workspace_bytes(void);
nvfp4_status nvfp4_fp6_quantize(const void* src_bf16, int64_t rows, int64_t cols, int64_t ld, int32_t rounding, uint64_t seed,
                                uint32_t stream_id, const nvfp4_dense_operand* out, void* workspace, size_t ws_bytes,
                                void* stream);
nvfp4_status nvfp4_fp6_requantize_t(const nvfp4_dense_operand* in, int32_t rounding, uint64_t seed, uint32_t stream_id,
                                    const nvfp4_dense_operand* out, void* workspace, size_t ws_bytes, void* stream);
nvfp4_status nvfp4_expand_operand(const nvfp4_operand* in, const nvfp4_dense_operand* out, void* stream);
nvfp4_status nvfp4_dense_gemm(const nvfp4_dense_operand* A, const nvfp4_dense_operand* B, void* C, int32_t c_dtype, int64_t ldc,
                              int32_t* dev_status, void* stream);

/* ---------------------------------------------------------------------------------------------------------
 * OutControl calibration (Sec. 4.2, the paragraph defining the outlier index set A): the activation l2-norm of every
 * channel is accumulated over a calibration window; the channels with the largest accumulated value form A.
 *
 * nvfp4_outlier_accumulate — one step of the window:  acc[d] += sqrt(sum_t X[t, d]^2),  X BF16 [N_tok, D] (device,
 *   leading dimension ldx, 16-byte aligned rows), acc FP32 [D] (device, read and written). FP32 arithmetic with a fixed
 *   summation order (bit-reproducible for a given shape). workspace: at least
 *   nvfp4_outlier_accumulate_workspace_bytes(N_tok, D), 16-byte aligned.
 * nvfp4_outlier_select — the n_out channels that come first in the order (acc descending, channel index ascending on
 *   ties; NaN is outside the contract). Writes, all device int32: outlier_cols [n_out] sorted ascending, keep_cols
 *   [D - n_out] sorted ascending, col_map [D] = position of channel d in keep_cols or -1 for an outlier — exactly the
 *   three arrays nvfp4_layer_cfg takes. n_out is the caller's rounding of p % of D.
 * Errors: NULL / SHAPE / ALIGN / WORKSPACE / ARCH as elsewhere; nothing is launched on an error.
 * --------------------------------------------------------------------------------------------------------- */
size_t nvfp4_outlier_accumulate_workspace_bytes(int64_t N_tok, int64_t D);
nvfp4_status nvfp4_outlier_accumulate(const void* X_bf16, int64_t ldx, int64_t N_tok, int64_t D, float* acc,
                                      void* workspace, size_t ws_bytes, void* stream);
nvfp4_status nvfp4_outlier_select(const float* acc, int64_t D, int64_t n_out, int32_t* outlier_cols,
                                  int32_t* keep_cols, int32_t* col_map, void* stream);

/* ---------------------------------------------------------------------------------------------------------
 * OsciReset (Sec. 3.2-3.3): oscillation statistics of the master weights (appendix Algorithm 2,
 * "UpdateOscillationStats") and the reset of high-risk weights to their bin centre (Algorithm 1,
 * "OscillationSuppress"), for one weight matrix.
 *
 *   W      master weights, FP32 [C, D] (device), leading dimension ldw, 16-byte aligned rows for full speed.
 *   W_prev, D_M, D_Q   the state of Algorithm 2: previous step's weights and the two accumulated path lengths, FP32
 *          [C, D] contiguous (device, 16-byte aligned), owned by the caller, 12 B per parameter.
 *   Q(.)   FP4 quant-dequant as the layer's forward weight quantizer defines it: cast to BF16 (nearest even), double-block
 *          quantize along D with round-to-nearest in `gs_mode`, dequantize as float32((P * S_block) * S_global).
 *
 * nvfp4_osci_update, t0 = 0:  D_M = D_Q = 0, W_prev = W.
 *                    t0 > 0:  D_M += |W - W_prev|;  D_Q += |Q(W) - Q(W_prev)|;  W_prev = W   (one binary32 operation each).
 * nvfp4_osci_suppress:        W[i] = Q(W)[i] wherever float32(D_Q[i] / D_M[i]) >= tau (0 / 0 is no reset); Q is taken of
 *                             the weights as they are before any reset. *n_reset (device, optional, 8-byte aligned) is
 *                             incremented by the number of resets. The statistics are not modified.
 * workspace: nvfp4_osci_workspace_bytes(C, gs_mode) bytes (amax cells of the TENSOR / ROW modes), 4-byte aligned.
 * --------------------------------------------------------------------------------------------------------- */
size_t nvfp4_osci_workspace_bytes(int64_t C, int32_t gs_mode);
nvfp4_status nvfp4_osci_update(const float* W, int64_t ldw, int64_t C, int64_t D, int32_t gs_mode, int32_t t0,
                               float* W_prev, float* D_M, float* D_Q, void* workspace, size_t ws_bytes, void* stream);
nvfp4_status nvfp4_osci_suppress(float* W, int64_t ldw, int64_t C, int64_t D, int32_t gs_mode, const float* D_M,
                                 const float* D_Q, float tau, unsigned long long* n_reset, void* workspace,
                                 size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------------------
 * OsciReset, memory-efficient statistics (appendix Algorithm 3, "UpdateOscillationStats_MemoryEfficient"): only the
 * n_track elements with the largest sensitivity score at t0 = 0 are tracked,
 *      s = |w - Q(w)| / binwidth(Q(w)),   binwidth = (upper - lower rounding threshold of the E2M1 value) * S_block * S_global
 * (widths 0.5, 0.5, 0.5, 0.5, 0.75, 1, 1.5, 2 for |P| = 0 .. 6; a block with scale 0 scores 0; binary32, one operation each).
 *
 *   State, all caller-owned device arrays of n_track entries: idx (int32 linear index r * D + c, sorted ascending; ties in
 *   s go to the lower index), WM_prev / WQ_prev (FP32 snapshots of w and Q(w)), D_M / D_Q (FP32 path lengths): 20 B per
 *   tracked element. C * D must be below 2^31 (NVFP4_ERR_LIMIT).
 *
 * nvfp4_osci_sparse_update, t0 = 0: computes the scores, selects idx (radix select + ordered compaction), clears D_M, D_Q
 *                                   and takes the snapshots.
 *                           t0 > 0: D_M += |w - WM_prev|; D_Q += |Q(w) - WQ_prev|; snapshots <- current values.
 * nvfp4_osci_sparse_suppress:       W[idx[i]] = Q(W)[idx[i]] wherever float32(D_Q[i] / D_M[i]) >= tau; Q is taken of the
 *                                   matrix before any reset (two launches); *n_reset as in nvfp4_osci_suppress.
 * workspace: nvfp4_osci_sparse_workspace_bytes(C, D, gs_mode, n_track, phase), 256-byte aligned; phase 0 = update with
 * t0 = 0 (holds one 32-bit score per element of W for the selection), 1 = update with t0 > 0, 2 = suppress.
 * --------------------------------------------------------------------------------------------------------- */
size_t nvfp4_osci_sparse_workspace_bytes(int64_t C, int64_t D, int32_t gs_mode, int64_t n_track, int32_t phase);
nvfp4_status nvfp4_osci_sparse_update(const float* W, int64_t ldw, int64_t C, int64_t D, int32_t gs_mode, int32_t t0,
                                      int64_t n_track, int32_t* idx, float* WM_prev, float* WQ_prev, float* D_M,
                                      float* D_Q, void* workspace, size_t ws_bytes, void* stream);
nvfp4_status nvfp4_osci_sparse_suppress(float* W, int64_t ldw, int64_t C, int64_t D, int32_t gs_mode, int64_t n_track,
                                        const int32_t* idx, const float* D_M, const float* D_Q, float tau,
                                        unsigned long long* n_reset, void* workspace, size_t ws_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* NVFP4_H_ */
