// C-ABI entry points: argument validation on the host, workspace carving, and the order in which the layer's
// quantizers and products are enqueued (paper Sec. 2.3; OutControl split of Sec. 4.2). No allocation, no
// synchronisation: everything is enqueued on the caller's stream.
#include "../../include/nvfp4.h"
#include "../../include/nvfp4_measure.h"

#include <map>
#include <mutex>

#include "nvfp4_device.cuh"
#include "nvfp4_internal.h"

using namespace nvfp4;

namespace nvfp4 {
std::atomic<long long> g_launch_count{0};

// Per-device facts and settings (a process may drive several GPUs): compute capability, SM count, and the dynamic
// shared-memory limit already granted to each kernel.
namespace {
constexpr int kMaxDevices = 64;
struct DeviceCache {
  int cc_major = -1;
  int sm_count = 0;
  std::map<const void*, size_t> dyn_smem;
};
std::mutex g_device_mutex;
DeviceCache g_device[kMaxDevices];

DeviceCache* current_device_cache() {  // call with g_device_mutex held
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  DeviceCache& d = g_device[dev];
  if (d.cc_major < 0) {
    int major = 0, sms = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
      return nullptr;
    d.cc_major = major;
    d.sm_count = sms;
  }
  return &d;
}
}  // namespace

int device_sm_count() {
  std::lock_guard<std::mutex> lock(g_device_mutex);
  DeviceCache* d = current_device_cache();
  return d && d->sm_count > 0 ? d->sm_count : 1;
}

cudaError_t ensure_dynamic_smem(const void* kernel, size_t bytes) {
  if (bytes <= 48 * 1024) return cudaSuccess;
  std::lock_guard<std::mutex> lock(g_device_mutex);
  DeviceCache* d = current_device_cache();
  if (!d) return cudaErrorInvalidDevice;
  size_t& have = d->dyn_smem[kernel];
  if (bytes <= have) return cudaSuccess;
  const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess) have = bytes;
  return e;
}
}  // namespace nvfp4

namespace {

// Philox stream ids of the two sign diagonals of the backward products (the six quantizers use 1..6)
constexpr uint32_t kRhtStreamDx = 7, kRhtStreamDw = 8;

inline int64_t round_up(int64_t v, int64_t m) { return (v + m - 1) / m * m; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

nvfp4_status check_arch() {
  std::lock_guard<std::mutex> lock(g_device_mutex);
  DeviceCache* d = current_device_cache();
  if (!d) return NVFP4_ERR_CUDA;
  return d->cc_major == 10 ? NVFP4_OK : NVFP4_ERR_ARCH;
}

bool valid_operand_desc(const nvfp4_operand* o) {
  return o->R >= 0 && o->K >= 0 && o->gs_mode >= 0 && o->gs_mode <= 2 && o->sf_layout >= 0 && o->sf_layout <= 1;
}

nvfp4_status check_operand_ptrs(const nvfp4_operand* o) {
  if (!o) return NVFP4_ERR_NULL;
  if (!valid_operand_desc(o)) return (o->R < 0 || o->K < 0) ? NVFP4_ERR_SHAPE : NVFP4_ERR_ENUM;
  if (o->R == 0 || o->K == 0) return NVFP4_OK;
  if (!o->codes || !o->sf || !o->gscale) return NVFP4_ERR_NULL;
  if (!aligned16(o->codes) || !aligned16(o->sf) || (reinterpret_cast<uintptr_t>(o->gscale) & 3u)) return NVFP4_ERR_ALIGN;
  return NVFP4_OK;
}

// The scale buffer of the tiled layout is padded (rows to 128, k-blocks to 16); kernels write only real entries.
cudaError_t clear_sf_padding(const nvfp4_operand* o, cudaStream_t st) {
  if (o->sf_layout != NVFP4_SF_TILED128x4) return cudaSuccess;
  const int64_t nb = nvfp4_padded_k(o->K) / 16;
  if ((o->R % 128) == 0 && (nb % 16) == 0) return cudaSuccess;
  return cudaMemsetAsync(o->sf, 0, nvfp4_operand_sf_bytes(o->R, o->K, o->sf_layout), st);
}

struct Carver {
  uint8_t* base;
  size_t size, used;
  Carver(void* p, size_t n) : base(static_cast<uint8_t*>(p)), size(n), used(0) {}
  void* take(size_t bytes) {
    const size_t start = (used + 255) & ~(size_t)255;
    used = start + bytes;
    return (base && used <= size) ? base + start : nullptr;
  }
};
inline size_t carve_size(size_t& total, size_t bytes) {
  total = ((total + 255) & ~(size_t)255) + bytes;
  return total;
}

size_t cells_bytes(int64_t rows, int32_t gs_mode) {
  return gs_mode == NVFP4_GS_ROW ? (size_t)std::max<int64_t>(rows, 1) * 4 : 4;
}

// Operand carved from a workspace (tiled scales).
void operand_sizes(size_t& total, int64_t R, int64_t K, int32_t gs_mode) {
  carve_size(total, nvfp4_operand_codes_bytes(R, K));
  carve_size(total, nvfp4_operand_sf_bytes(R, K, NVFP4_SF_TILED128x4));
  carve_size(total, nvfp4_operand_gscale_count(R, K, gs_mode) * 4);
}
bool carve_operand(Carver& c, nvfp4_operand* o, int64_t R, int64_t K, int32_t gs_mode) {
  o->codes = static_cast<uint8_t*>(c.take(nvfp4_operand_codes_bytes(R, K)));
  o->sf = static_cast<uint8_t*>(c.take(nvfp4_operand_sf_bytes(R, K, NVFP4_SF_TILED128x4)));
  o->gscale = static_cast<float*>(c.take(nvfp4_operand_gscale_count(R, K, gs_mode) * 4));
  o->R = R;
  o->K = K;
  o->gs_mode = gs_mode;
  o->sf_layout = NVFP4_SF_TILED128x4;
  return o->codes && o->sf && o->gscale;
}

// Head of the workspace of the two backward calls: amax cells, then the two operands (the rest follows in the callers).
bool carve_bwd_dx(Carver& cv, int64_t N_tok, int64_t D, int64_t C, int32_t gs_mode, uint32_t** cells3, uint32_t** cells4,
                  nvfp4_operand* q3, nvfp4_operand* q4) {
  *cells3 = static_cast<uint32_t*>(cv.take(cells_bytes(N_tok, gs_mode)));
  *cells4 = static_cast<uint32_t*>(cv.take(cells_bytes(D, gs_mode)));
  return carve_operand(cv, q3, N_tok, C, gs_mode) && carve_operand(cv, q4, D, C, gs_mode) && *cells3 && *cells4;
}
bool carve_bwd_dw(Carver& cv, int64_t N_tok, int64_t Dk, int64_t C, int32_t gs_mode, uint32_t** cells5, uint32_t** cells6,
                  nvfp4_operand* q5, nvfp4_operand* q6) {
  *cells5 = static_cast<uint32_t*>(cv.take(cells_bytes(C, gs_mode)));
  *cells6 = static_cast<uint32_t*>(cv.take(cells_bytes(Dk, gs_mode)));
  return carve_operand(cv, q5, C, N_tok, gs_mode) && carve_operand(cv, q6, Dk, N_tok, gs_mode) && *cells5 && *cells6;
}

// The caller's optional second stream with its three events (nvfp4_layer_cfg); null when the call runs on one stream.
struct SideStream {
  cudaStream_t stream = nullptr;
  cudaEvent_t fork = nullptr, join = nullptr, amax = nullptr;
};
static bool side_stream_of(const nvfp4_layer_cfg* cfg, SideStream* out) {
  if (!cfg->side_stream) return false;
  out->stream = static_cast<cudaStream_t>(cfg->side_stream);
  out->fork = static_cast<cudaEvent_t>(cfg->ev_fork);
  out->join = static_cast<cudaEvent_t>(cfg->ev_join);
  out->amax = static_cast<cudaEvent_t>(cfg->ev_aux);
  return true;
}

nvfp4_status do_quantize_rows(const uint16_t* src, int64_t rows, int64_t cols, int64_t ld, int32_t rounding,
                              uint64_t seed, uint32_t stream_id, const int32_t* keep, int64_t n_keep,
                              const nvfp4_operand* out, uint32_t* cells, cudaStream_t st, int cells_zeroed = 0,
                              const int32_t* excluded = nullptr, uint32_t rht_stream = 0, int compute_amax = 1,
                              uint16_t* excl_out = nullptr, int64_t ld_excl_out = 0) {
  if (clear_sf_padding(out, st) != cudaSuccess) return NVFP4_ERR_CUDA;
  QuantRowsArgs a{};
  a.excl_out = keep && excluded ? excl_out : nullptr;
  a.ld_excl_out = ld_excl_out;
  a.src = src;
  a.rows = rows;
  a.K = keep ? n_keep : cols;
  a.cols_src = cols;
  a.ld = ld;
  a.keep = keep;
  a.excluded = keep ? excluded : nullptr;
  a.seed = seed;
  a.stream_id = stream_id;
  a.rht_stream = rht_stream;
  a.gs_mode = out->gs_mode;
  a.sr = rounding == NVFP4_ROUND_SR ? 1 : rounding == NVFP4_ROUND_SR_SCALE_UP ? 2 : 0;
  a.sf_tiled = out->sf_layout == NVFP4_SF_TILED128x4;
  a.compute_amax = compute_amax;
  a.cells_zeroed = cells_zeroed;
  a.gs_cells = cells;
  a.codes = out->codes;
  a.sf = out->sf;
  a.gscale = out->gscale;
  return launch_quantize_rows(a, st) == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

nvfp4_status do_quantize_transpose(const TransposeSrc& src, int from_codes, int64_t rowsK, int64_t D, int32_t rounding,
                                   uint64_t seed, uint32_t stream_id, const nvfp4_operand* out, uint32_t* cells,
                                   cudaStream_t st, int cells_zeroed = 0, uint32_t rht_stream = 0, int compute_amax = 1) {
  if (clear_sf_padding(out, st) != cudaSuccess) return NVFP4_ERR_CUDA;
  QuantTransposeArgs a{};
  a.from_codes = from_codes;
  a.rowsK = rowsK;
  a.D = D;
  a.src = src;
  a.seed = seed;
  a.stream_id = stream_id;
  a.rht_stream = rht_stream;
  a.gs_mode = out->gs_mode;
  a.sr = rounding == NVFP4_ROUND_SR ? 1 : rounding == NVFP4_ROUND_SR_SCALE_UP ? 2 : 0;
  a.sf_tiled = out->sf_layout == NVFP4_SF_TILED128x4;
  a.compute_amax = compute_amax;
  a.cells_zeroed = cells_zeroed;
  a.gs_cells = cells;
  a.codes = out->codes;
  a.sf = out->sf;
  a.gscale = out->gscale;
  return launch_quantize_transpose(a, st) == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

nvfp4_status do_gemm(const nvfp4_operand* A, const nvfp4_operand* B, void* C, int32_t c_dtype, int64_t ldc,
                     int32_t accumulate, int32_t* dev_status, cudaStream_t st, const void* hp_a = nullptr,
                     const void* hp_b = nullptr, int64_t hp_Kh = 0, const nvfp4_gemm_opts* opts = nullptr) {
  if (A->gs_mode == NVFP4_GS_BLOCK128 && nvfp4_padded_k(A->K) > gemm_block128_max_k()) return NVFP4_ERR_LIMIT;
  GemmArgs g{};
  g.a_codes = A->codes;
  g.a_sf = A->sf;
  g.a_gscale = A->gscale;
  g.b_codes = B->codes;
  g.b_sf = B->sf;
  g.b_gscale = B->gscale;
  g.M = A->R;
  g.N = B->R;
  g.K = A->K;
  g.gs_mode = A->gs_mode;
  g.C = C;
  g.c_is_f32 = c_dtype == NVFP4_DT_F32;
  g.ldc = ldc;
  g.accumulate = accumulate;
  g.dev_status = dev_status;
  g.hp_a = hp_a;
  g.hp_b = hp_b;
  g.hp_Kh = hp_Kh;
  if (opts) {
    g.variant = opts->variant;
    g.wait_limit = opts->wait_limit_cycles;
    g.starve_first_stage = opts->starve_first_stage;
  }
  return launch_gemm(g, st) == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

// Clears the amax cells of a layer call (two arrays carved back to back) with one memset, so that the kernels that follow
// are launched kernel-after-kernel and can overlap their prologues with their predecessors' tails.
bool zero_cells(uint32_t* first, uint32_t* second, size_t second_bytes, cudaStream_t st) {
  const size_t span = (reinterpret_cast<uint8_t*>(second) - reinterpret_cast<uint8_t*>(first)) + second_bytes;
  return launch_zero_words(first, (int64_t)((span + 3) / 4), st) == cudaSuccess;
}

nvfp4_status check_cfg(const nvfp4_layer_cfg* cfg, int64_t D) {
  if (!cfg) return NVFP4_ERR_NULL;
  if (cfg->gs_mode < 0 || cfg->gs_mode > 2) return NVFP4_ERR_ENUM;
  for (int i = 0; i < 6; ++i)
    if (cfg->rounding[i] < 0 || cfg->rounding[i] > 2) return NVFP4_ERR_ENUM;
  if (cfg->y_dtype < 0 || cfg->y_dtype > 1 || cfg->dx_dtype < 0 || cfg->dx_dtype > 1 || cfg->dw_dtype < 0 ||
      cfg->dw_dtype > 1 || cfg->rht < 0 || cfg->rht > 1 || cfg->outlier_format < 0 || cfg->outlier_format > 1 ||
      cfg->weight_block < 0 || cfg->weight_block > 1)
    return NVFP4_ERR_ENUM;
  if (cfg->weight_block == 1 && (cfg->gs_mode != NVFP4_GS_TENSOR || cfg->n_out != 0 || cfg->rounding[1] != NVFP4_ROUND_RTN))
    return NVFP4_ERR_ENUM;
  if (cfg->n_out < 0 || cfg->n_out > D) return NVFP4_ERR_SHAPE;
  if (cfg->n_out > 0 && (!cfg->outlier_cols || !cfg->keep_cols || !cfg->col_map)) return NVFP4_ERR_NULL;
  if (cfg->side_stream && (!cfg->ev_fork || !cfg->ev_join || !cfg->ev_aux)) return NVFP4_ERR_NULL;
  return NVFP4_OK;
}

bool bad_matrix(const void* p, int64_t ld, int64_t cols, int elem_bytes) {
  return !aligned16(p) || ld < cols || (ld * elem_bytes) % 16 != 0;
}

}  // namespace

namespace nvfp4 {
bool device_is_sm100() { return check_arch() == NVFP4_OK; }
}  // namespace nvfp4

extern "C" {

int64_t nvfp4_padded_k(int64_t K) { return round_up(K, 128); }

int64_t nvfp4_outlier_pad(int64_t n_out) { return round_up(n_out, 64); }

size_t nvfp4_operand_codes_bytes(int64_t R, int64_t K) { return (size_t)(R * (nvfp4_padded_k(K) / 2)); }

size_t nvfp4_operand_sf_bytes(int64_t R, int64_t K, int32_t sf_layout) {
  const int64_t nb = nvfp4_padded_k(K) / 16;
  if (sf_layout == NVFP4_SF_TILED128x4) return (size_t)(round_up(R, 128) * round_up(nb, 16));
  return (size_t)(R * nb);
}

size_t nvfp4_operand_gscale_count(int64_t R, int64_t K, int32_t gs_mode) {
  if (gs_mode == NVFP4_GS_TENSOR) return 1;
  if (gs_mode == NVFP4_GS_ROW) return (size_t)R;
  return (size_t)(R * (nvfp4_padded_k(K) / 128));
}

long long nvfp4_launch_count(void) { return g_launch_count.load(std::memory_order_relaxed); }

const char* nvfp4_status_string(nvfp4_status s) {
  switch (s) {
    case NVFP4_OK: return "ok";
    case NVFP4_ERR_NULL: return "null pointer";
    case NVFP4_ERR_SHAPE: return "bad shape";
    case NVFP4_ERR_ALIGN: return "bad alignment";
    case NVFP4_ERR_ENUM: return "bad enum value";
    case NVFP4_ERR_WORKSPACE: return "workspace too small";
    case NVFP4_ERR_ARCH: return "device is not sm_100";
    case NVFP4_ERR_CUDA: return "CUDA call failed";
    case NVFP4_ERR_TIMEOUT: return "device-side wait timed out";
    case NVFP4_ERR_LIMIT: return "size exceeds the fixed capacity of this entry point";
  }
  return "unknown status";
}

size_t nvfp4_quantize_workspace_bytes(int64_t out_rows, int32_t gs_mode) {
  return round_up((int64_t)cells_bytes(out_rows, gs_mode), 256);
}

nvfp4_status nvfp4_quantize(const void* src_bf16, int64_t rows, int64_t cols, int64_t ld, int32_t axis,
                            int32_t rounding, uint64_t seed, uint32_t stream_id, uint32_t rht_stream_id,
                            const int32_t* keep_cols, int64_t n_keep, const nvfp4_operand* out, void* workspace,
                            size_t ws_bytes, void* stream) {
  if (!src_bf16 || !out) return NVFP4_ERR_NULL;
  if (axis < 0 || axis > 1 || rounding < 0 || rounding > 2) return NVFP4_ERR_ENUM;
  if (rht_stream_id && keep_cols) return NVFP4_ERR_ENUM;
  if (rows < 0 || cols < 0 || (keep_cols && (n_keep < 0 || n_keep > cols))) return NVFP4_ERR_SHAPE;
  if (keep_cols && axis != NVFP4_AXIS_ROW) return NVFP4_ERR_SHAPE;
  nvfp4_status s = check_operand_ptrs(out);
  if (s != NVFP4_OK) return s;
  const int64_t kept = keep_cols ? n_keep : cols;
  const int64_t R = axis == NVFP4_AXIS_ROW ? rows : kept;
  const int64_t K = axis == NVFP4_AXIS_ROW ? kept : rows;
  if (out->R != R || out->K != K) return NVFP4_ERR_SHAPE;
  if (bad_matrix(src_bf16, ld, cols, 2)) return NVFP4_ERR_ALIGN;
  if (!workspace || ws_bytes < nvfp4_quantize_workspace_bytes(R, out->gs_mode)) return NVFP4_ERR_WORKSPACE;
  if ((s = check_arch()) != NVFP4_OK) return s;
  if (R == 0 || K == 0) return NVFP4_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t* cells = static_cast<uint32_t*>(workspace);
  if (axis == NVFP4_AXIS_ROW)
    return do_quantize_rows(static_cast<const uint16_t*>(src_bf16), rows, cols, ld, rounding, seed, stream_id, keep_cols,
                            n_keep, out, cells, st, 0, nullptr, rht_stream_id);
  TransposeSrc ts{};
  ts.bf16 = static_cast<const uint16_t*>(src_bf16);
  ts.ld = ld;
  return do_quantize_transpose(ts, 0, rows, cols, rounding, seed, stream_id, out, cells, st, 0, rht_stream_id);
}

nvfp4_status nvfp4_quantize_w16x16(const void* W_bf16, int64_t C, int64_t D, int64_t ldw, const nvfp4_operand* out,
                                   void* workspace, size_t ws_bytes, void* stream) {
  if (!W_bf16 || !out) return NVFP4_ERR_NULL;
  if (C < 0 || D < 0) return NVFP4_ERR_SHAPE;
  nvfp4_status s;
  if ((s = check_operand_ptrs(out)) != NVFP4_OK) return s;
  if (out->R != C || out->K != D) return NVFP4_ERR_SHAPE;
  if (out->gs_mode != NVFP4_GS_TENSOR) return NVFP4_ERR_ENUM;
  if (bad_matrix(W_bf16, ldw, D, 2)) return NVFP4_ERR_ALIGN;
  if (!workspace || !aligned16(workspace) || ws_bytes < nvfp4_quantize_workspace_bytes(C, NVFP4_GS_TENSOR)) return NVFP4_ERR_WORKSPACE;
  if ((s = check_arch()) != NVFP4_OK) return s;
  if (C == 0 || D == 0) return NVFP4_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t* cell = static_cast<uint32_t*>(workspace);
  if (clear_sf_padding(out, st) != cudaSuccess) return NVFP4_ERR_CUDA;
  if (launch_zero_words(cell, 1, st) != cudaSuccess) return NVFP4_ERR_CUDA;
  if (launch_amax_tensor(static_cast<const uint16_t*>(W_bf16), C, D, ldw, cell, st) != cudaSuccess) return NVFP4_ERR_CUDA;
  return launch_quantize_w16(static_cast<const uint16_t*>(W_bf16), C, D, ldw, cell, out->codes, out->sf, out->gscale,
                             out->sf_layout == NVFP4_SF_TILED128x4, st) == cudaSuccess
             ? NVFP4_OK
             : NVFP4_ERR_CUDA;
}

static nvfp4_status do_transpose_operand16(const nvfp4_operand* in, const nvfp4_operand* out, cudaStream_t st) {
  if (clear_sf_padding(out, st) != cudaSuccess) return NVFP4_ERR_CUDA;
  return launch_transpose_operand(in->codes, in->sf, in->sf_layout == NVFP4_SF_TILED128x4, in->gscale, in->R, in->K, out->codes, out->sf,
                                  out->sf_layout == NVFP4_SF_TILED128x4, out->gscale, st) == cudaSuccess
             ? NVFP4_OK
             : NVFP4_ERR_CUDA;
}

nvfp4_status nvfp4_transpose_operand16(const nvfp4_operand* in, const nvfp4_operand* out, void* stream) {
  if (!in || !out) return NVFP4_ERR_NULL;
  nvfp4_status s;
  if ((s = check_operand_ptrs(in)) != NVFP4_OK) return s;
  if ((s = check_operand_ptrs(out)) != NVFP4_OK) return s;
  if (out->R != in->K || out->K != in->R) return NVFP4_ERR_SHAPE;
  if (in->gs_mode != NVFP4_GS_TENSOR || out->gs_mode != NVFP4_GS_TENSOR) return NVFP4_ERR_ENUM;
  if ((s = check_arch()) != NVFP4_OK) return s;
  if (in->R == 0 || in->K == 0) return NVFP4_OK;
  return do_transpose_operand16(in, out, static_cast<cudaStream_t>(stream));
}

nvfp4_status nvfp4_requantize_t(const nvfp4_operand* in, const void* hp_bf16, int64_t hp_ld, const int32_t* row_map,
                                int64_t n_rows_out, int32_t rounding, uint64_t seed, uint32_t stream_id,
                                uint32_t rht_stream_id, const nvfp4_operand* out, void* workspace, size_t ws_bytes,
                                void* stream) {
  if (!in || !out) return NVFP4_ERR_NULL;
  if (rounding < 0 || rounding > 2) return NVFP4_ERR_ENUM;
  nvfp4_status s;
  if ((s = check_operand_ptrs(in)) != NVFP4_OK) return s;
  if ((s = check_operand_ptrs(out)) != NVFP4_OK) return s;
  const int64_t D = row_map ? n_rows_out : in->K;
  if (n_rows_out < 0 || out->R != D || out->K != in->R) return NVFP4_ERR_SHAPE;
  if (row_map && !hp_bf16) return NVFP4_ERR_NULL;
  if (row_map && bad_matrix(hp_bf16, hp_ld, D, 2)) return NVFP4_ERR_ALIGN;
  if (!workspace || ws_bytes < nvfp4_quantize_workspace_bytes(D, out->gs_mode)) return NVFP4_ERR_WORKSPACE;
  if ((s = check_arch()) != NVFP4_OK) return s;
  if (D == 0 || in->R == 0) return NVFP4_OK;
  TransposeSrc ts{};
  ts.in_codes = in->codes;
  ts.in_sf = in->sf;
  ts.in_gscale = in->gscale;
  ts.in_K = in->K;
  ts.in_gs_mode = in->gs_mode;
  ts.in_sf_tiled = in->sf_layout == NVFP4_SF_TILED128x4;
  ts.row_map = row_map;
  ts.hp = static_cast<const uint16_t*>(hp_bf16);
  ts.hp_ld = hp_ld;
  return do_quantize_transpose(ts, 1, in->R, D, rounding, seed, stream_id, out, static_cast<uint32_t*>(workspace),
                               static_cast<cudaStream_t>(stream), 0, rht_stream_id);
}

size_t nvfp4_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K) { return gemm_workspace_bytes(M, N, K); }

nvfp4_status nvfp4_gemm(const nvfp4_operand* A, const nvfp4_operand* B, void* C, int32_t c_dtype, int64_t ldc,
                        int32_t accumulate, int32_t* dev_status, void* workspace, size_t ws_bytes, void* stream) {
  return nvfp4_gemm_ex(A, B, C, c_dtype, ldc, accumulate, dev_status, nullptr, workspace, ws_bytes, stream);
}

nvfp4_status nvfp4_gemm_ex(const nvfp4_operand* A, const nvfp4_operand* B, void* C, int32_t c_dtype, int64_t ldc,
                           int32_t accumulate, int32_t* dev_status, const nvfp4_gemm_opts* opts, void* workspace,
                           size_t ws_bytes, void* stream) {
  if (!A || !B || !C) return NVFP4_ERR_NULL;
  if (opts && (opts->variant < 0 || opts->variant > 3 || opts->wait_limit_cycles < 0 ||
               (opts->variant >= NVFP4_GEMM_PAIR256 && A->gs_mode == NVFP4_GS_BLOCK128)))
    return NVFP4_ERR_ENUM;
  nvfp4_status s;
  if ((s = check_operand_ptrs(A)) != NVFP4_OK) return s;
  if ((s = check_operand_ptrs(B)) != NVFP4_OK) return s;
  if (c_dtype < 0 || c_dtype > 1) return NVFP4_ERR_ENUM;
  if (A->K != B->K || A->K <= 0) return NVFP4_ERR_SHAPE;
  if (A->gs_mode != B->gs_mode) return NVFP4_ERR_ENUM;
  if (A->sf_layout != NVFP4_SF_TILED128x4 || B->sf_layout != NVFP4_SF_TILED128x4) return NVFP4_ERR_ENUM;
  if (bad_matrix(C, ldc, B->R, c_dtype == NVFP4_DT_F32 ? 4 : 2)) return NVFP4_ERR_ALIGN;
  const size_t need = nvfp4_gemm_workspace_bytes(A->R, B->R, A->K);
  if (need && (!workspace || ws_bytes < need)) return NVFP4_ERR_WORKSPACE;
  if ((s = check_arch()) != NVFP4_OK) return s;
  return do_gemm(A, B, C, c_dtype, ldc, accumulate, dev_status, static_cast<cudaStream_t>(stream), nullptr, nullptr, 0, opts);
}

int64_t nvfp4_dense_ld(int64_t K) { return (K + 63) & ~(int64_t)63; }
size_t nvfp4_fp6_workspace_bytes(void) { return 16; }

static nvfp4_status check_dense(const nvfp4_dense_operand* o) {
  if (!o || !o->vals || !o->gscale) return NVFP4_ERR_NULL;
  if (o->R <= 0 || o->K <= 0 || o->ld != nvfp4_dense_ld(o->K)) return NVFP4_ERR_SHAPE;
  if (!aligned16(o->vals) || (reinterpret_cast<uintptr_t>(o->gscale) & 3u)) return NVFP4_ERR_ALIGN;
  return NVFP4_OK;
}

nvfp4_status nvfp4_fp6_quantize(const void* src_bf16, int64_t rows, int64_t cols, int64_t ld, int32_t rounding, uint64_t seed,
                                uint32_t stream_id, const nvfp4_dense_operand* out, void* workspace, size_t ws_bytes, void* stream) {
  if (!src_bf16) return NVFP4_ERR_NULL;
  nvfp4_status s;
  if ((s = check_dense(out)) != NVFP4_OK) return s;
  if (rows <= 0 || cols <= 0 || ld < cols || out->R != rows || out->K != cols) return NVFP4_ERR_SHAPE;
  if (rounding != NVFP4_ROUND_RTN && rounding != NVFP4_ROUND_SR) return NVFP4_ERR_ENUM;
  if (bad_matrix(src_bf16, ld, cols, 2)) return NVFP4_ERR_ALIGN;  // 16-byte aligned rows, as for nvfp4_quantize
  if (!workspace || !aligned16(workspace) || ws_bytes < nvfp4_fp6_workspace_bytes()) return NVFP4_ERR_WORKSPACE;
  if ((s = check_arch()) != NVFP4_OK) return s;
  return launch_fp6_quantize_rows(static_cast<const uint16_t*>(src_bf16), rows, cols, ld, rounding == NVFP4_ROUND_SR, seed, stream_id,
                                  static_cast<uint32_t*>(workspace), static_cast<uint16_t*>(out->vals), out->ld, out->gscale,
                                  static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? NVFP4_OK
             : NVFP4_ERR_CUDA;
}

nvfp4_status nvfp4_fp6_requantize_t(const nvfp4_dense_operand* in, int32_t rounding, uint64_t seed, uint32_t stream_id,
                                    const nvfp4_dense_operand* out, void* workspace, size_t ws_bytes, void* stream) {
  nvfp4_status s;
  if ((s = check_dense(in)) != NVFP4_OK) return s;
  if ((s = check_dense(out)) != NVFP4_OK) return s;
  if (out->R != in->K || out->K != in->R) return NVFP4_ERR_SHAPE;
  if (rounding != NVFP4_ROUND_RTN && rounding != NVFP4_ROUND_SR) return NVFP4_ERR_ENUM;
  if (!workspace || !aligned16(workspace) || ws_bytes < nvfp4_fp6_workspace_bytes()) return NVFP4_ERR_WORKSPACE;
  if ((s = check_arch()) != NVFP4_OK) return s;
  return launch_fp6_requantize_t(static_cast<const uint16_t*>(in->vals), in->R, in->K, in->ld, in->gscale, rounding == NVFP4_ROUND_SR, seed,
                                 stream_id, static_cast<uint32_t*>(workspace), static_cast<uint16_t*>(out->vals), out->ld, out->gscale,
                                 static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? NVFP4_OK
             : NVFP4_ERR_CUDA;
}

nvfp4_status nvfp4_expand_operand(const nvfp4_operand* in, const nvfp4_dense_operand* out, void* stream) {
  nvfp4_status s;
  if (!in) return NVFP4_ERR_NULL;
  if ((s = check_operand_ptrs(in)) != NVFP4_OK) return s;
  if ((s = check_dense(out)) != NVFP4_OK) return s;
  if (in->R != out->R || in->K != out->K) return NVFP4_ERR_SHAPE;
  if (in->gs_mode != NVFP4_GS_TENSOR) return NVFP4_ERR_ENUM;
  if ((s = check_arch()) != NVFP4_OK) return s;
  return launch_expand_operand(in->codes, in->sf, in->sf_layout == NVFP4_SF_TILED128x4, in->R, in->K, in->gscale,
                               static_cast<uint16_t*>(out->vals), out->ld, out->gscale, static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? NVFP4_OK
             : NVFP4_ERR_CUDA;
}

nvfp4_status nvfp4_dense_gemm(const nvfp4_dense_operand* A, const nvfp4_dense_operand* B, void* C, int32_t c_dtype, int64_t ldc,
                              int32_t* dev_status, void* stream) {
  nvfp4_status s;
  if (!C) return NVFP4_ERR_NULL;
  if ((s = check_dense(A)) != NVFP4_OK) return s;
  if ((s = check_dense(B)) != NVFP4_OK) return s;
  if (A->K != B->K) return NVFP4_ERR_SHAPE;
  if (c_dtype < 0 || c_dtype > 1) return NVFP4_ERR_ENUM;
  if (bad_matrix(C, ldc, B->R, c_dtype == NVFP4_DT_F32 ? 4 : 2)) return NVFP4_ERR_ALIGN;
  if ((s = check_arch()) != NVFP4_OK) return s;
  return launch_dense_gemm(A->vals, B->vals, A->R, B->R, A->ld, A->gscale, B->gscale, C, c_dtype == NVFP4_DT_F32, ldc, dev_status,
                           static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? NVFP4_OK
             : NVFP4_ERR_CUDA;
}

size_t nvfp4_linear_workspace_bytes(int32_t op_kind, int64_t N_tok, int64_t D, int64_t C, int64_t n_out,
                                    int32_t gs_mode) {
  size_t total = 0;
  const int64_t Dk = D - n_out;
  if (op_kind == NVFP4_OP_FWD) {
    carve_size(total, cells_bytes(N_tok, gs_mode));
    carve_size(total, cells_bytes(C, gs_mode));
    if (n_out > 0) carve_size(total, 16);  // amax cells of the FP8 outlier option
  } else if (op_kind == NVFP4_OP_BWD_DX) {
    carve_size(total, cells_bytes(N_tok, gs_mode));
    carve_size(total, cells_bytes(D, gs_mode));
    operand_sizes(total, N_tok, C, gs_mode);
    operand_sizes(total, D, C, gs_mode);
  } else if (op_kind == NVFP4_OP_BWD) {
    // both halves back to back (each already a multiple of 256 bytes) plus the shared amax cell
    return nvfp4_linear_workspace_bytes(NVFP4_OP_BWD_DX, N_tok, D, C, n_out, gs_mode) +
           nvfp4_linear_workspace_bytes(NVFP4_OP_BWD_DW, N_tok, D, C, n_out, gs_mode) + 256;
  } else {
    carve_size(total, cells_bytes(C, gs_mode));
    carve_size(total, cells_bytes(Dk, gs_mode));
    operand_sizes(total, C, N_tok, gs_mode);
    operand_sizes(total, Dk, N_tok, gs_mode);
    if (n_out > 0) {
      carve_size(total, (size_t)C * (size_t)round_up(Dk, 4) * 4);
      carve_size(total, hp_dw_partial_floats(N_tok, C, nvfp4_outlier_pad(n_out)) * 4);
    }
  }
  return ((total + 255) & ~(size_t)255) + 256;
}

nvfp4_status nvfp4_linear_bwd_operand(int32_t op_kind, int32_t which, int64_t N_tok, int64_t D, int64_t C, int64_t n_out,
                                      int32_t gs_mode, void* workspace, size_t ws_bytes, nvfp4_operand* out) {
  if (!workspace || !out) return NVFP4_ERR_NULL;
  if (gs_mode < 0 || gs_mode > 2 || which < 3 || which > 6) return NVFP4_ERR_ENUM;
  if (N_tok <= 0 || D <= 0 || C <= 0 || n_out < 0 || n_out >= D) return NVFP4_ERR_SHAPE;
  const bool dx = which <= 4;
  if (!(op_kind == NVFP4_OP_BWD || (dx && op_kind == NVFP4_OP_BWD_DX) || (!dx && op_kind == NVFP4_OP_BWD_DW))) return NVFP4_ERR_ENUM;
  if (ws_bytes < nvfp4_linear_workspace_bytes(op_kind, N_tok, D, C, n_out, gs_mode)) return NVFP4_ERR_WORKSPACE;
  uint8_t* base = static_cast<uint8_t*>(workspace);
  size_t size = ws_bytes;
  if (op_kind == NVFP4_OP_BWD && !dx) {  // the dW half follows the dX half
    const size_t need_dx = nvfp4_linear_workspace_bytes(NVFP4_OP_BWD_DX, N_tok, D, C, n_out, gs_mode);
    base += need_dx;
    size -= need_dx;
  }
  Carver cv(base, size);
  uint32_t *ca, *cb;
  nvfp4_operand qa, qb;
  const bool ok = dx ? carve_bwd_dx(cv, N_tok, D, C, gs_mode, &ca, &cb, &qa, &qb)
                     : carve_bwd_dw(cv, N_tok, D - n_out, C, gs_mode, &ca, &cb, &qa, &qb);
  if (!ok) return NVFP4_ERR_WORKSPACE;
  *out = (which == 3 || which == 5) ? qa : qb;
  return NVFP4_OK;
}

nvfp4_status nvfp4_linear_fwd(const void* X, int64_t ldx, const void* W, int64_t ldw, int64_t N_tok, int64_t D,
                              int64_t C, const nvfp4_layer_cfg* cfg, void* Y, int64_t ldy, nvfp4_saved* saved,
                              void* workspace, size_t ws_bytes, void* stream) {
  if (!X || !W || !Y || !saved) return NVFP4_ERR_NULL;
  if (N_tok <= 0 || D <= 0 || C <= 0) return NVFP4_ERR_SHAPE;
  nvfp4_status s;
  if ((s = check_cfg(cfg, D)) != NVFP4_OK) return s;
  const int64_t n_out = cfg->n_out, Dk = D - n_out;
  if (Dk <= 0) return NVFP4_ERR_SHAPE;
  if ((s = check_operand_ptrs(&saved->qx)) != NVFP4_OK) return s;
  if ((s = check_operand_ptrs(&saved->qw)) != NVFP4_OK) return s;
  if (saved->qx.R != N_tok || saved->qx.K != Dk || saved->qw.R != C || saved->qw.K != Dk) return NVFP4_ERR_SHAPE;
  if (saved->qx.gs_mode != cfg->gs_mode || saved->qw.gs_mode != cfg->gs_mode ||
      saved->qx.sf_layout != NVFP4_SF_TILED128x4 || saved->qw.sf_layout != NVFP4_SF_TILED128x4)
    return NVFP4_ERR_ENUM;
  if (bad_matrix(X, ldx, D, 2) || bad_matrix(W, ldw, D, 2) || bad_matrix(Y, ldy, C, cfg->y_dtype == NVFP4_DT_F32 ? 4 : 2))
    return NVFP4_ERR_ALIGN;
  if (!workspace || ws_bytes < nvfp4_linear_workspace_bytes(NVFP4_OP_FWD, N_tok, D, C, n_out, cfg->gs_mode))
    return NVFP4_ERR_WORKSPACE;
  if ((s = check_arch()) != NVFP4_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  Carver cv(workspace, ws_bytes);
  uint32_t* cells_x = static_cast<uint32_t*>(cv.take(cells_bytes(N_tok, cfg->gs_mode)));
  uint32_t* cells_w = static_cast<uint32_t*>(cv.take(cells_bytes(C, cfg->gs_mode)));
  if (!cells_x || !cells_w) return NVFP4_ERR_WORKSPACE;

  const uint16_t* Xp = static_cast<const uint16_t*>(X);
  const uint16_t* Wp = static_cast<const uint16_t*>(W);
  const int32_t* keep = n_out > 0 ? cfg->keep_cols : nullptr;
  // (the 1x128 outer-block mode has no amax cells: its scales come out of the quantizers' own pass)
  if (cfg->gs_mode != NVFP4_GS_BLOCK128 && !zero_cells(cells_x, cells_w, cells_bytes(C, cfg->gs_mode), st)) return NVFP4_ERR_CUDA;
  int amax_pass = 1;
  if (cfg->gs_mode == NVFP4_GS_TENSOR && !keep) {  // the two per-tensor maxima in one launch
    if (launch_amax_tensor_pair(Xp, N_tok, D, ldx, cells_x, Wp, C, D, ldw, cells_w, st) != cudaSuccess) return NVFP4_ERR_CUDA;
    amax_pass = 0;
  }
  // with outlier channels, the quantizers also write the BF16 side operands X[:, outliers] and W[:, outliers]
  const int64_t Kh = n_out > 0 ? nvfp4_outlier_pad(n_out) : 0;
  if (n_out > 0 && (!saved->X_out || !saved->W_out)) return NVFP4_ERR_NULL;
  // Q1 and Q2 (each with its own amax pass where it has one) are independent: the weight side runs on the side stream
  SideStream side_store;
  SideStream* side = side_stream_of(cfg, &side_store) ? &side_store : nullptr;
  if (side && (cudaEventRecord(side->fork, st) != cudaSuccess || cudaStreamWaitEvent(side->stream, side->fork, 0) != cudaSuccess))
    return NVFP4_ERR_CUDA;
  const nvfp4_status s_x = do_quantize_rows(Xp, N_tok, D, ldx, cfg->rounding[0], cfg->seed, 1, keep, Dk, &saved->qx, cells_x, st, 1,
                                            cfg->outlier_cols, 0, amax_pass, static_cast<uint16_t*>(saved->X_out), Kh);
  nvfp4_status s_w;
  if (cfg->weight_block == 1) {  // 16x16 scale squares (TENSOR mode: amax(W) is already in cells_w)
    cudaStream_t sw = side ? side->stream : st;
    s_w = clear_sf_padding(&saved->qw, sw) == cudaSuccess &&
                  launch_quantize_w16(Wp, C, D, ldw, cells_w, saved->qw.codes, saved->qw.sf, saved->qw.gscale, 1, sw) == cudaSuccess
              ? NVFP4_OK
              : NVFP4_ERR_CUDA;
  } else {
    s_w = do_quantize_rows(Wp, C, D, ldw, cfg->rounding[1], cfg->seed, 2, keep, Dk, &saved->qw, cells_w, side ? side->stream : st, 1,
                           cfg->outlier_cols, 0, amax_pass, static_cast<uint16_t*>(saved->W_out), Kh);
  }
  if (side && (cudaEventRecord(side->join, side->stream) != cudaSuccess || cudaStreamWaitEvent(st, side->join, 0) != cudaSuccess))
    return NVFP4_ERR_CUDA;
  if (s_x != NVFP4_OK) return s_x;
  if (s_w != NVFP4_OK) return s_w;
  if (n_out > 0 && cfg->outlier_format == 1) {  // outlier channels on their scaled E4M3 grids from here on
    uint32_t* cells_fp8 = static_cast<uint32_t*>(cv.take(16));
    if (!cells_fp8) return NVFP4_ERR_WORKSPACE;
    if (launch_fp8_snap_pair(static_cast<uint16_t*>(saved->X_out), N_tok, static_cast<uint16_t*>(saved->W_out), C, Kh, cells_fp8, st) !=
        cudaSuccess)
      return NVFP4_ERR_CUDA;
  }
  saved->X = X; saved->W = W; saved->ldx = ldx; saved->ldw = ldw;
  saved->N_tok = N_tok; saved->D = D; saved->C = C;
  if (n_out > 0)  // Y = FP4 product + X_out W_out^T, both inside one kernel
    return do_gemm(&saved->qx, &saved->qw, Y, cfg->y_dtype, ldy, 0, cfg->dev_status, st, saved->X_out, saved->W_out,
                   nvfp4_outlier_pad(n_out));
  return do_gemm(&saved->qx, &saved->qw, Y, cfg->y_dtype, ldy, 0, cfg->dev_status, st);
}

// dy_amax: optional cell already holding the bit pattern of max |dY| (TENSOR mode without the Hadamard transformation):
// the amax pre-pass of the dY quantizer is then skipped.
static nvfp4_status bwd_dx_impl(const void* dY, int64_t lddy, const nvfp4_saved* saved, const nvfp4_layer_cfg* cfg,
                                void* dX, int64_t lddx, void* workspace, size_t ws_bytes, void* stream, uint32_t* dy_amax) {
  if (!dY || !saved || !dX) return NVFP4_ERR_NULL;
  const int64_t N_tok = saved->N_tok, D = saved->D, C = saved->C;
  if (N_tok <= 0 || D <= 0 || C <= 0) return NVFP4_ERR_SHAPE;
  nvfp4_status s;
  if ((s = check_cfg(cfg, D)) != NVFP4_OK) return s;
  const int64_t n_out = cfg->n_out;
  if ((s = check_operand_ptrs(&saved->qw)) != NVFP4_OK) return s;
  if (saved->qw.R != C || saved->qw.K != D - n_out) return NVFP4_ERR_SHAPE;
  if (bad_matrix(dY, lddy, C, 2) || bad_matrix(dX, lddx, D, cfg->dx_dtype == NVFP4_DT_F32 ? 4 : 2)) return NVFP4_ERR_ALIGN;
  if (!workspace || ws_bytes < nvfp4_linear_workspace_bytes(NVFP4_OP_BWD_DX, N_tok, D, C, n_out, cfg->gs_mode))
    return NVFP4_ERR_WORKSPACE;
  if ((s = check_arch()) != NVFP4_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  Carver cv(workspace, ws_bytes);
  uint32_t *cells3, *cells4;
  nvfp4_operand q3, q4;
  if (!carve_bwd_dx(cv, N_tok, D, C, cfg->gs_mode, &cells3, &cells4, &q3, &q4)) return NVFP4_ERR_WORKSPACE;
  // with a shared dY amax and a TENSOR -> TENSOR re-quantization (closed-form maximum) no cell of this call is read
  const bool cells_unused = cfg->gs_mode == NVFP4_GS_BLOCK128 ||
                            (dy_amax && n_out == 0 && cfg->gs_mode == NVFP4_GS_TENSOR && saved->qw.gs_mode == NVFP4_GS_TENSOR && !cfg->rht);
  if (!cells_unused && !zero_cells(cells3, cells4, cells_bytes(D, cfg->gs_mode), st)) return NVFP4_ERR_CUDA;
  // (16x16 weight squares: W-hat^T is the forward operand transposed as it is, so this product takes no Hadamard factor)
  const uint32_t rht = cfg->rht && cfg->weight_block == 0 ? kRhtStreamDx : 0u;
  if ((s = do_quantize_rows(static_cast<const uint16_t*>(dY), N_tok, C, lddy, cfg->rounding[2], cfg->seed, 3, nullptr, 0,
                            &q3, dy_amax ? dy_amax : cells3, st, 1, nullptr, rht, dy_amax ? 0 : 1)) != NVFP4_OK)
    return s;
  if (cfg->weight_block == 1) {
    if ((s = do_transpose_operand16(&saved->qw, &q4, st)) != NVFP4_OK) return s;
    return do_gemm(&q3, &q4, dX, cfg->dx_dtype, lddx, 0, cfg->dev_status, st);
  }
  TransposeSrc ts{};
  ts.in_codes = saved->qw.codes;
  ts.in_sf = saved->qw.sf;
  ts.in_gscale = saved->qw.gscale;
  ts.in_K = saved->qw.K;
  ts.in_gs_mode = saved->qw.gs_mode;
  ts.in_sf_tiled = saved->qw.sf_layout == NVFP4_SF_TILED128x4;
  if (n_out == 0) {
    if ((s = do_quantize_transpose(ts, 1, C, D, cfg->rounding[3], cfg->seed, 4, &q4, cells4, st, 1, rht)) != NVFP4_OK) return s;
  } else {
    // W-hat^T over all D channels in two passes that write disjoint operand rows: the kept channels from the forward
    // operand (compact column j -> row keep[j]) and the outlier channels from the compact BF16 copy (column j -> row
    // outl[j]). Rows are quantized independently; only the TENSOR-mode scale couples them: its maximum is the larger
    // of float32(2688 * Sg) of the forward operand and the BF16 copy's amax, which both passes are told about.
    if (!saved->W_out) return NVFP4_ERR_NULL;
    const int64_t Kh = nvfp4_outlier_pad(n_out);
    if (clear_sf_padding(&q4, st) != cudaSuccess) return NVFP4_ERR_CUDA;
    // (the closed form does not survive the Hadamard transformation: both sources then get a transformed amax pass)
    const bool closed = cfg->gs_mode == NVFP4_GS_TENSOR && saved->qw.gs_mode == NVFP4_GS_TENSOR && !rht;
    TransposeSrc th{};
    th.bf16 = static_cast<const uint16_t*>(saved->W_out);
    th.ld = Kh;
    th.out_rows = cfg->outlier_cols;
    ts.out_rows = cfg->keep_cols;
    QuantTransposeArgs qa{};
    qa.seed = cfg->seed;
    qa.stream_id = 4;
    qa.rht_stream = rht;
    qa.gs_mode = cfg->gs_mode;
    qa.sr = cfg->rounding[3] == NVFP4_ROUND_SR ? 1 : cfg->rounding[3] == NVFP4_ROUND_SR_SCALE_UP ? 2 : 0;
    qa.sf_tiled = 1;
    qa.cells_zeroed = 1;
    qa.gs_cells = cells4;
    qa.codes = q4.codes;
    qa.sf = q4.sf;
    qa.gscale = q4.gscale;
    qa.rowsK = C;
    if (cfg->gs_mode == NVFP4_GS_TENSOR) {
      // one amax pass over the compact BF16 copy (and over the forward operand unless the closed form applies)
      if (rht) {
        if (launch_amax_transpose_src(th, 0, C, n_out, cells4, st, cfg->seed, rht) != cudaSuccess) return NVFP4_ERR_CUDA;
      } else if (launch_amax_tensor(static_cast<const uint16_t*>(saved->W_out), C, Kh, Kh, cells4, st) != cudaSuccess) {
        return NVFP4_ERR_CUDA;
      }
      if (closed) {
        th.closed_form_sg = saved->qw.gscale;
        ts.closed_form_sg = saved->qw.gscale;
      } else if (launch_amax_transpose_src(ts, 1, C, D - n_out, cells4, st, cfg->seed, rht) != cudaSuccess) {
        return NVFP4_ERR_CUDA;
      }
      qa.compute_amax = 0;
    } else {
      qa.compute_amax = 1;  // ROW: per-row cells, each pass fills the rows it owns; BLOCK128: no pre-pass
    }
    qa.from_codes = 1;
    qa.D = D - n_out;
    qa.src = ts;
    if (launch_quantize_transpose(qa, st) != cudaSuccess) return NVFP4_ERR_CUDA;
    qa.from_codes = 0;
    qa.D = n_out;
    qa.src = th;
    if (launch_quantize_transpose(qa, st) != cudaSuccess) return NVFP4_ERR_CUDA;
  }
  return do_gemm(&q3, &q4, dX, cfg->dx_dtype, lddx, 0, cfg->dev_status, st);
}

nvfp4_status nvfp4_linear_bwd_dx(const void* dY, int64_t lddy, const nvfp4_saved* saved, const nvfp4_layer_cfg* cfg,
                                 void* dX, int64_t lddx, void* workspace, size_t ws_bytes, void* stream) {
  return bwd_dx_impl(dY, lddy, saved, cfg, dX, lddx, workspace, ws_bytes, stream, nullptr);
}

static nvfp4_status bwd_dw_impl(const void* dY, int64_t lddy, const nvfp4_saved* saved, const nvfp4_layer_cfg* cfg,
                                void* dW, int64_t lddw, void* workspace, size_t ws_bytes, void* stream, uint32_t* dy_amax,
                                cudaEvent_t dy_amax_ready = nullptr, HpDwArgs* deferred_hp = nullptr) {
  if (!dY || !saved || !dW) return NVFP4_ERR_NULL;
  const int64_t N_tok = saved->N_tok, D = saved->D, C = saved->C;
  if (N_tok <= 0 || D <= 0 || C <= 0) return NVFP4_ERR_SHAPE;
  nvfp4_status s;
  if ((s = check_cfg(cfg, D)) != NVFP4_OK) return s;
  const int64_t n_out = cfg->n_out, Dk = D - n_out;
  if ((s = check_operand_ptrs(&saved->qx)) != NVFP4_OK) return s;
  if (saved->qx.R != N_tok || saved->qx.K != Dk) return NVFP4_ERR_SHAPE;
  if (n_out > 0 && !saved->X_out) return NVFP4_ERR_NULL;
  if (n_out > 0 && !hp_dw_assemble_fits(D, n_out)) return NVFP4_ERR_LIMIT;
  const int dw_f32 = cfg->dw_dtype == NVFP4_DT_F32;
  if (bad_matrix(dY, lddy, C, 2) || bad_matrix(dW, lddw, D, dw_f32 ? 4 : 2)) return NVFP4_ERR_ALIGN;
  if (!workspace || ws_bytes < nvfp4_linear_workspace_bytes(NVFP4_OP_BWD_DW, N_tok, D, C, n_out, cfg->gs_mode))
    return NVFP4_ERR_WORKSPACE;
  if ((s = check_arch()) != NVFP4_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  Carver cv(workspace, ws_bytes);
  uint32_t *cells5, *cells6;
  nvfp4_operand q5, q6;
  if (!carve_bwd_dw(cv, N_tok, Dk, C, cfg->gs_mode, &cells5, &cells6, &q5, &q6)) return NVFP4_ERR_WORKSPACE;
  const int64_t ld_compact = round_up(Dk, 4);
  const int64_t Kh = nvfp4_outlier_pad(n_out);
  float* compact = n_out > 0 ? static_cast<float*>(cv.take((size_t)C * ld_compact * 4)) : nullptr;
  float* hp_partial = n_out > 0 ? static_cast<float*>(cv.take(hp_dw_partial_floats(N_tok, C, Kh) * 4)) : nullptr;
  if (n_out > 0 && (!compact || !hp_partial)) return NVFP4_ERR_WORKSPACE;

  TransposeSrc t5{};
  t5.bf16 = static_cast<const uint16_t*>(dY);
  t5.ld = lddy;
  const bool cells_unused = cfg->gs_mode == NVFP4_GS_BLOCK128 ||
                            (dy_amax && cfg->gs_mode == NVFP4_GS_TENSOR && saved->qx.gs_mode == NVFP4_GS_TENSOR && !cfg->rht);
  if (!cells_unused && !zero_cells(cells5, cells6, cells_bytes(Dk, cfg->gs_mode), st)) return NVFP4_ERR_CUDA;
  const uint32_t rht = cfg->rht ? kRhtStreamDw : 0u;
  // Q6 first: it needs nothing of dY, so it can run while another stream still computes the shared amax of dY
  TransposeSrc t6{};
  t6.in_codes = saved->qx.codes;
  t6.in_sf = saved->qx.sf;
  t6.in_gscale = saved->qx.gscale;
  t6.in_K = saved->qx.K;
  t6.in_gs_mode = saved->qx.gs_mode;
  t6.in_sf_tiled = saved->qx.sf_layout == NVFP4_SF_TILED128x4;
  if ((s = do_quantize_transpose(t6, 1, N_tok, Dk, cfg->rounding[5], cfg->seed, 6, &q6, cells6, st, 1, rht)) != NVFP4_OK) return s;
  if (dy_amax_ready && cudaStreamWaitEvent(st, dy_amax_ready, 0) != cudaSuccess) return NVFP4_ERR_CUDA;
  if ((s = do_quantize_transpose(t5, 0, N_tok, C, cfg->rounding[4], cfg->seed, 5, &q5, dy_amax ? dy_amax : cells5, st, 1, rht,
                                 dy_amax ? 0 : 1)) != NVFP4_OK)
    return s;
  if (n_out == 0) return do_gemm(&q5, &q6, dW, cfg->dw_dtype, lddw, 0, cfg->dev_status, st);

  // kept columns: compact product; one pass then writes dW row by row from it and from the outlier channels' side product
  // (a scattering GEMM epilogue measured slower)
  if ((s = do_gemm(&q5, &q6, compact, NVFP4_DT_F32, ld_compact, 0, cfg->dev_status, st)) != NVFP4_OK) return s;
  HpDwArgs h{};
  h.dY = static_cast<const uint16_t*>(dY); h.X_out = static_cast<const uint16_t*>(saved->X_out);
  h.lddy = lddy; h.Kh = Kh; h.T = N_tok; h.C = C; h.n_out = n_out; h.outl = cfg->outlier_cols;
  h.dW = dW; h.dw_is_f32 = dw_f32; h.lddw = lddw; h.partial = hp_partial; h.dev_status = cfg->dev_status;
  h.compact = compact; h.ld_compact = ld_compact; h.D = D; h.keep = cfg->keep_cols; h.col_map = cfg->col_map;
  if (deferred_hp) {  // the caller runs the side product on another stream and finishes dW after joining it
    *deferred_hp = h;
    return NVFP4_OK;
  }
  return launch_hp_dw(h, st) == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

nvfp4_status nvfp4_linear_bwd_dw(const void* dY, int64_t lddy, const nvfp4_saved* saved, const nvfp4_layer_cfg* cfg,
                                 void* dW, int64_t lddw, void* workspace, size_t ws_bytes, void* stream) {
  return bwd_dw_impl(dY, lddy, saved, cfg, dW, lddw, workspace, ws_bytes, stream, nullptr);
}

nvfp4_status nvfp4_linear_bwd(const void* dY, int64_t lddy, const nvfp4_saved* saved, const nvfp4_layer_cfg* cfg, void* dX,
                              int64_t lddx, void* dW, int64_t lddw, void* workspace, size_t ws_bytes, void* stream) {
  if (!dY || !saved || !cfg || !dX || !dW) return NVFP4_ERR_NULL;
  const int64_t N_tok = saved->N_tok, D = saved->D, C = saved->C;
  if (N_tok <= 0 || D <= 0 || C <= 0) return NVFP4_ERR_SHAPE;
  if (cfg->gs_mode < 0 || cfg->gs_mode > 2 || cfg->n_out < 0 || cfg->n_out > D) return NVFP4_ERR_ENUM;
  const size_t need_dx = nvfp4_linear_workspace_bytes(NVFP4_OP_BWD_DX, N_tok, D, C, cfg->n_out, cfg->gs_mode);
  const size_t need_dw = nvfp4_linear_workspace_bytes(NVFP4_OP_BWD_DW, N_tok, D, C, cfg->n_out, cfg->gs_mode);
  if (!workspace || !aligned16(workspace) || ws_bytes < nvfp4_linear_workspace_bytes(NVFP4_OP_BWD, N_tok, D, C, cfg->n_out, cfg->gs_mode))
    return NVFP4_ERR_WORKSPACE;
  if (bad_matrix(dY, lddy, C, 2)) return NVFP4_ERR_ALIGN;
  uint8_t* base = static_cast<uint8_t*>(workspace);
  uint32_t* shared = nullptr;
  // The two products share nothing but their inputs: the dX chain (Q3, Q4, GEMM) runs on a side stream forked from the
  // caller's stream here and joined before returning, so that its kernels fill the SMs that the other chain's small GEMMs
  // and kernel tails leave idle. (Fork and join are events: the pattern is also legal under stream capture.)
  // (measured: dW chain launched first on the caller's stream, dX chain on the side stream, default priorities, was the
  // best of the launch orders and priorities tried: 0.268 ms per default step against 0.276 ms the other way round and
  // 0.303 ms on one stream)
  nvfp4_status s;
  if ((s = check_arch()) != NVFP4_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cfg->side_stream && (!cfg->ev_fork || !cfg->ev_join || !cfg->ev_aux)) return NVFP4_ERR_NULL;
  SideStream side_store;
  SideStream* side = side_stream_of(cfg, &side_store) ? &side_store : nullptr;
  // Q3 and Q5 quantize the same tensor with the same per-tensor scale: one amax pass serves both. Without OutControl it
  // runs before the fork. With OutControl it runs at the head of the dX chain, and the dW chain, which starts with Q6 (no
  // dY involved), waits for it only before Q5: the bandwidth-bound amax pass and the arithmetic-bound Q6 overlap.
  // (Measured per step, before the fork / overlapped: 0.2675 / 0.2695 ms plain, 0.409 / 0.389 ms with 10 % outlier channels.)
  const bool shared_amax = cfg->gs_mode == NVFP4_GS_TENSOR && !cfg->rht;
  const bool amax_early = shared_amax && cfg->n_out == 0;
  if (amax_early) {
    shared = reinterpret_cast<uint32_t*>(base + need_dx + need_dw);
    if (launch_zero_words(shared, 1, st) != cudaSuccess) return NVFP4_ERR_CUDA;
    if (launch_amax_tensor(static_cast<const uint16_t*>(dY), N_tok, C, lddy, shared, st) != cudaSuccess) return NVFP4_ERR_CUDA;
  }
  if (side && (cudaEventRecord(side->fork, st) != cudaSuccess || cudaStreamWaitEvent(side->stream, side->fork, 0) != cudaSuccess))
    return NVFP4_ERR_CUDA;
  cudaStream_t st_dx = side ? side->stream : st;
  cudaEvent_t amax_ready = nullptr;
  if (shared_amax && !amax_early) {
    shared = reinterpret_cast<uint32_t*>(base + need_dx + need_dw);
    if (launch_zero_words(shared, 1, st_dx) != cudaSuccess) return NVFP4_ERR_CUDA;
    if (launch_amax_tensor(static_cast<const uint16_t*>(dY), N_tok, C, lddy, shared, st_dx) != cudaSuccess) return NVFP4_ERR_CUDA;
    if (side) {
      if (cudaEventRecord(side->amax, st_dx) != cudaSuccess) return NVFP4_ERR_CUDA;
      amax_ready = side->amax;
    }
  }
  // With OutControl the BF16 side product dY^T X_out needs nothing of the FP4 chain: it runs at the end of the (shorter) dX
  // chain on the side stream, and dW is assembled on the caller's stream after the join.
  HpDwArgs hp{};
  const bool defer_hp = side != nullptr && cfg->n_out > 0;
  nvfp4_status s_dw = bwd_dw_impl(dY, lddy, saved, cfg, dW, lddw, base + need_dx, need_dw, stream, shared, amax_ready,
                                  defer_hp ? &hp : nullptr);
  const nvfp4_status s_dx = bwd_dx_impl(dY, lddy, saved, cfg, dX, lddx, base, need_dx, st_dx, shared);
  const bool hp_pending = defer_hp && s_dw == NVFP4_OK && hp.n_out > 0;
  if (hp_pending && launch_hp_dw_product(hp, side->stream) != cudaSuccess) s_dw = NVFP4_ERR_CUDA;
  if (side && (cudaEventRecord(side->join, side->stream) != cudaSuccess || cudaStreamWaitEvent(st, side->join, 0) != cudaSuccess))
    return NVFP4_ERR_CUDA;
  if (hp_pending && s_dw == NVFP4_OK && launch_hp_dw_finish(hp, st) != cudaSuccess) s_dw = NVFP4_ERR_CUDA;
  return s_dx != NVFP4_OK ? s_dx : s_dw;
}

}  // extern "C"
