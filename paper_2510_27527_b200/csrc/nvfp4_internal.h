// Internal (non-ABI) declarations shared by the library's translation units.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>
#include <atomic>

namespace nvfp4 {

// Number of kernels this library has enqueued since it was loaded (measurement aid).
extern std::atomic<long long> g_launch_count;

// true if the current device has compute capability 10.x (cached per device)
bool device_is_sm100();
// Number of SMs of the current device (queried once per device).
int device_sm_count();
// Raises a kernel's dynamic shared-memory limit to at least `bytes` on the current device; remembered per device and
// kernel, so the attribute call is made once per pair.
cudaError_t ensure_dynamic_smem(const void* kernel, size_t bytes);

struct QuantRowsArgs {
  const uint16_t* src;  // BF16 [rows, cols_src], leading dimension ld
  int64_t rows, K, cols_src, ld;
  const int32_t* keep;  // optional column list of length K
  const int32_t* excluded;  // optional: the sorted complement of `keep` (cols_src - K entries); enables the masked amax
  // optional (with `excluded`): excl_out[r, j] = src[r, excluded[j]], zero for cols_src - K <= j < ld_excl_out. Written by the
  // masked amax pass where that runs (the matrix is read once for both), else by a separate gather launch.
  uint16_t* excl_out;
  int64_t ld_excl_out;
  uint64_t seed;
  uint32_t stream_id;
  uint32_t rht_stream;  // non-zero: random Hadamard transformation along K with this sign stream (not with `keep`)
  int gs_mode, sr, sf_tiled;  // sr: 0 round to nearest, 1 stochastic, 2 stochastic with the block scale rounded up
  int compute_amax;    // TENSOR mode: run the amax pre-pass (0: gs_cells[0] already holds the amax bits)
  int cells_zeroed;    // the caller has already cleared gs_cells on this stream
  uint32_t* gs_cells;  // workspace: 1 cell (TENSOR) or `rows` cells (ROW)
  uint8_t* codes;
  uint8_t* sf;
  float* gscale;
};

// Source of a transposing quantizer. Operand element (d, k) = source element (row k, column d).
struct TransposeSrc {
  // from BF16: matrix [rowsK, D], leading dimension ld
  const uint16_t* bf16;
  int64_t ld;
  // from a forward operand [rowsK, in_K] (codes + scales + global scales), optionally remapped per d and
  // mixed with the BF16 matrix hp for the rows whose map entry is negative
  const uint8_t* in_codes;
  const uint8_t* in_sf;
  const float* in_gscale;
  int64_t in_K;
  int32_t in_gs_mode, in_sf_tiled;
  const int32_t* row_map;  // [D] or null
  const uint16_t* hp;      // BF16 [rowsK, >= D]
  int64_t hp_ld;
  // output placement and scale coupling (both optional)
  const int32_t* out_rows;       // operand row that source column d produces (null: d itself)
  const float* closed_form_sg;   // TENSOR mode: the tensor maximum is at least float32(2688 * *closed_form_sg)
};

struct QuantTransposeArgs {
  int from_codes;
  int64_t rowsK, D;  // operand [D, rowsK] = transpose of a [rowsK, D] source
  TransposeSrc src;
  uint64_t seed;
  uint32_t stream_id;
  uint32_t rht_stream;  // non-zero: random Hadamard transformation along the operand's K (source rows) with this stream
  int gs_mode, sr, sf_tiled;  // sr: 0 round to nearest, 1 stochastic, 2 stochastic with the block scale rounded up
  int compute_amax;
  int cells_zeroed;        // the caller has already cleared gs_cells on this stream
  int tensor_closed_form;  // set by the launcher
  uint32_t* gs_cells;  // 1 cell (TENSOR) or D cells (ROW)
  uint8_t* codes;
  uint8_t* sf;
  float* gscale;
};

// Every kernel of the library is launched with programmatic stream serialisation: its CTAs may be scheduled while the
// previous kernel of the stream is still draining, run their prologue (barrier setup, tensor-memory allocation) and then
// block in griddepcontrol.wait until that kernel has completed and its writes are visible. Each kernel calls
// pdl_prologue() (see nvfp4_device.cuh) before its first global-memory access.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  g_launch_count.fetch_add(1, std::memory_order_relaxed);
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

cudaError_t launch_quantize_rows(const QuantRowsArgs& a, cudaStream_t st);
cudaError_t launch_quantize_transpose(const QuantTransposeArgs& a, cudaStream_t st);
// amax of a contiguous-row BF16 matrix folded into cells[0] (atomic max; the cell must already hold a valid value)
cudaError_t launch_amax_tensor(const uint16_t* src, int64_t rows, int64_t cols, int64_t ld, uint32_t* cell, cudaStream_t st);
// p[0 .. n) = 0 by a kernel (keeps the programmatic launch chain intact where a memset node would break it)
cudaError_t launch_zero_words(uint32_t* p, int64_t n, cudaStream_t st);
// the same for two matrices in one launch
cudaError_t launch_amax_tensor_pair(const uint16_t* a, int64_t rows_a, int64_t cols_a, int64_t ld_a, uint32_t* cell_a, const uint16_t* b,
                                    int64_t rows_b, int64_t cols_b, int64_t ld_b, uint32_t* cell_b, cudaStream_t st);
// amax of a transposing quantizer's source (from codes or BF16) folded into cells[0]; with a non-zero rht_stream, of the
// source after the random Hadamard transformation along its rows (the operand's K)
cudaError_t launch_amax_transpose_src(const TransposeSrc& s, int from_codes, int64_t rowsK, int64_t D, uint32_t* cell, cudaStream_t st,
                                      uint64_t seed = 0, uint32_t rht_stream = 0);

struct GemmArgs {
  const uint8_t *a_codes, *a_sf, *b_codes, *b_sf;
  const float *a_gscale, *b_gscale;
  int64_t M, N, K;  // logical sizes; operand buffers are padded as the ABI header says
  int gs_mode;
  void* C;
  int c_is_f32;
  int64_t ldc;
  int accumulate;
  // optional high-precision side product (OutControl): C += hp_a [M, hp_Kh] * hp_b [N, hp_Kh]^T, BF16 inputs, FP32
  // accumulation on the tensor cores inside the same kernel (TENSOR / ROW modes)
  const void* hp_a;
  const void* hp_b;
  int64_t hp_Kh;
  int32_t* dev_status;
  void* workspace;
  size_t ws_bytes;
  int variant;               // nvfp4_gemm_variant of the ABI header (0 = chosen from the shape)
  long long wait_limit;      // bound of every device-side wait in clock cycles (<= 0: the default, about two seconds)
  int starve_first_stage;    // test hook of the bounded waits: the first stage's barrier expects bytes that never arrive
};
size_t gemm_workspace_bytes(int64_t M, int64_t N, int64_t K);
int64_t gemm_block128_max_k();  // largest K the BLOCK128 GEMM variant takes
cudaError_t launch_gemm(const GemmArgs& a, cudaStream_t st);
// C = (*a_gscale * *b_gscale) A B^T, A [M, ld] and B [N, ld] BF16 row-major (ld a multiple of 64), FP32 accumulation
cudaError_t launch_dense_gemm(const void* A, const void* B, int64_t M, int64_t N, int64_t ld, const float* a_gscale,
                              const float* b_gscale, void* C, int c_is_f32, int64_t ldc, int32_t* dev_status, cudaStream_t st);

// Simulated FP6 (E2M3) quantizers and the FP4 -> dense expansion (fp6.cu). cell: one workspace word.
cudaError_t launch_fp6_quantize_rows(const uint16_t* src, int64_t rows, int64_t K, int64_t ld, int sr, uint64_t seed, uint32_t stream_id,
                                     uint32_t* cell, uint16_t* out, int64_t ld_out, float* gscale, cudaStream_t st);
cudaError_t launch_fp6_requantize_t(const uint16_t* in, int64_t rowsK, int64_t D, int64_t ld_in, const float* in_gscale, int sr,
                                    uint64_t seed, uint32_t stream_id, uint32_t* cell, uint16_t* out, int64_t ld_out, float* gscale,
                                    cudaStream_t st);
cudaError_t launch_expand_operand(const uint8_t* codes, const uint8_t* sf, int sf_tiled, int64_t R, int64_t K, const float* in_gscale,
                                  uint16_t* out, int64_t ld_out, float* gscale, cudaStream_t st);

// High-precision (BF16 inputs, FP32 accumulate) products over OutControl's outlier channels.
//   fwd: Y[m, n] (+)= sum_j X[m, outl[j]] * W[n, outl[j]]
//   dw : dW[c, outl[j]] = sum_t dY[t, c] * X[t, outl[j]]
// dst[r, j] = src[r, cols[j]] for j < n, zero for n <= j < ld_dst (compact BF16 copy of OutControl's outlier channels)
cudaError_t launch_gather_cols(const uint16_t* src, int64_t ld_src, int64_t rows, const int32_t* cols, int64_t n, uint16_t* dst,
                               int64_t ld_dst, cudaStream_t st);

// 16x16 weight-block recipe: Q2 with one E4M3 scale per 16x16 square (per-tensor global scale from amax_cell, round to
// nearest), and the transposition of such an operand (codes transposed, scales re-indexed) that replaces Q4.
cudaError_t launch_quantize_w16(const uint16_t* src, int64_t C, int64_t D, int64_t ld, const uint32_t* amax_cell, uint8_t* codes,
                                uint8_t* sf, float* gscale, int tiled, cudaStream_t st);
cudaError_t launch_transpose_operand(const uint8_t* in_codes, const uint8_t* in_sf, int in_tiled, const float* in_gscale, int64_t C, int64_t D,
                                     uint8_t* out_codes, uint8_t* out_sf, int out_tiled, float* out_gscale, cudaStream_t st);

// FP8 option of OutControl: both compact side operands ([rows, Kh] BF16, contiguous) snapped in place onto their per-tensor
// power-of-two scaled E4M3 grids; cells2 = two workspace words.
cudaError_t launch_fp8_snap_pair(uint16_t* a, int64_t rows_a, uint16_t* b, int64_t rows_b, int64_t Kh, uint32_t* cells2, cudaStream_t st);

struct HpDwArgs {
  const uint16_t *dY, *X_out;  // dY [T, C]; X_out [T, Kh]: the outlier channels of X, compact, zero-padded to Kh (multiple of 64)
  int64_t lddy, Kh, T, C, n_out;
  const int32_t* outl;
  void* dW;
  int dw_is_f32;
  int64_t lddw;
  float* partial;  // workspace: hp_dw_partial_floats(T, C, Kh) floats
  int32_t* dev_status;
  // optional: the kept channels' product [C, D - n_out] (FP32, compact), placed into dW by the same pass that writes the
  // outlier channels. keep [D - n_out] and col_map [D] describe the placement (D = all channels).
  const float* compact;
  int64_t ld_compact, D;
  const int32_t* keep;
  const int32_t* col_map;
};
size_t hp_dw_partial_floats(int64_t T, int64_t C, int64_t Kh);
bool hp_dw_assemble_fits(int64_t D, int64_t n_out);  // the assembling pass of dW handles this many channels
cudaError_t launch_hp_dw_mma(const uint16_t* dY, int64_t lddy, const uint16_t* X_out, int64_t Kh, int64_t T, int64_t C,
                             float* partial, int n_split, int64_t t_per_split, int32_t* dev_status, cudaStream_t st);
cudaError_t launch_hp_dw(const HpDwArgs& a, cudaStream_t st);  // product, then finish, on one stream
// the two halves, for callers that overlap the side product (which needs only dY and X_out) with other work
cudaError_t launch_hp_dw_product(const HpDwArgs& a, cudaStream_t st);
cudaError_t launch_hp_dw_finish(const HpDwArgs& a, cudaStream_t st);

}  // namespace nvfp4
