// nvfp4_quantize_static: the quantizer for callers that cannot provide scratch memory.
//
// nvfp4_quantize needs a few bytes of global scratch (the amax cells of the TENSOR and ROW scale modes) and asks the
// caller for them. Some callers have no way to get device memory at the point of the call: code running inside an
// allocator callback or under a framework's "no allocation" guard, a plugin that is handed tensors but no allocator,
// a real-time loop whose memory was fixed at start-up. For them this entry point keeps the cells in an array that is
// part of the library image: every GPU that loads the library holds those kStaticCells * 4 bytes until the process
// ends, and nothing is allocated or freed here (no cudaMalloc / cudaFree, no allocating library routine).
#include "../../include/nvfp4.h"

#include "nvfp4_internal.h"

namespace {

constexpr int64_t kStaticCells = NVFP4_STATIC_MAX_ROWS;  // one cell per operand row in ROW mode
constexpr int kMaxDevices = 64;

// The scratch itself. In host code this name is only a handle: the device address has to be asked for.
static __device__ __align__(256) uint32_t g_static_cells[kStaticCells];

// Device address of g_static_cells on each device, resolved on the first call made with that device current.
uint32_t* g_cells_addr[kMaxDevices] = {};

nvfp4_status static_cells(uint32_t** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return NVFP4_ERR_CUDA;
  if (!g_cells_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_cells) != cudaSuccess || !p) return NVFP4_ERR_CUDA;
    g_cells_addr[dev] = static_cast<uint32_t*>(p);
  }
  *out = g_cells_addr[dev];
  return NVFP4_OK;
}

}  // namespace

extern "C" {

int64_t nvfp4_quantize_static_max_rows(void) { return kStaticCells; }

nvfp4_status nvfp4_quantize_static(const void* src_bf16, int64_t rows, int64_t cols, int64_t ld, int32_t axis,
                                   int32_t rounding, uint64_t seed, uint32_t stream_id, const int32_t* keep_cols,
                                   int64_t n_keep, const nvfp4_operand* out, void* stream) {
  if (!out) return NVFP4_ERR_NULL;
  // The ROW scale mode needs one cell per operand row; the other modes need one cell.
  if (out->gs_mode == NVFP4_GS_ROW && out->R > kStaticCells) return NVFP4_ERR_LIMIT;
  uint32_t* cells = nullptr;
  const nvfp4_status s = static_cells(&cells);
  if (s != NVFP4_OK) return s;
  // Same validation, same kernels, same order as nvfp4_quantize; only the scratch differs. The launchers zero the
  // cells they use on `stream` before the amax pass, so the previous call's contents never leak into this one.
  return nvfp4_quantize(src_bf16, rows, cols, ld, axis, rounding, seed, stream_id, 0u, keep_cols, n_keep, out, cells,
                        (size_t)kStaticCells * sizeof(uint32_t), stream);
}

}  // extern "C"
