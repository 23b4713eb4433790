// mlpmoe_fade_buffers_static: Fractal Fade's magnitude masking applied to caller-owned buffers,
// with the selection scratch (segment records, radix-select state and histograms) held in a
// fixed array inside the library image instead of memory obtained from cudaMalloc.
//
// It exists for callers that cannot allocate device memory when they need this operation: a
// serving process that handed all device memory to its own arena at start-up (cudaMalloc would
// fail), or a latency-critical path that must not take cudaMalloc's device-wide synchronisation.
// The handle-based mlpmoe_fade needs a layer handle, and creating one allocates.
#include <mutex>
#include <vector>

#include "../../include/mlpmoe.h"
#include "internal.h"

using namespace mlpmoe;

namespace {

constexpr int kMaxSlices = MLPMOE_STATIC_FADE_MAX_SLICES;
// Per slice: one segment record (24 bytes) + selection state (prefix, rank, 256-bin histogram);
// fade_work_bytes() states the exact amount, 1100 bytes bounds it.
constexpr size_t kScratchBytes = static_cast<size_t>(kMaxSlices) * 1100;

// Lives in every device that loads the library, until the process exits (about 275 KB).
static __device__ __align__(256) unsigned char g_fade_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void* g_scratch_addr[kMaxDevices] = {};   // device address of g_fade_scratch, per device ordinal

// The array's name is only a host-side handle for the symbol; the address a kernel can use
// has to be asked for, once per device, with that device current.
mlpmoe_status_t scratch_address(void** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return MLPMOE_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return MLPMOE_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (g_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_fade_scratch) != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return MLPMOE_ERR_CUDA;
    }
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return MLPMOE_OK;
}

}  // namespace

extern "C" mlpmoe_status_t mlpmoe_fade_buffers_static(void* const* slices, const int64_t* m, const double* s,
                                                      int32_t n_slices, mlpmoe_dtype_t dtype, void* stream) {
  if (n_slices < 0 || (n_slices > 0 && (!slices || !m || !s))) return MLPMOE_ERR_INVALID_ARG;
  if (dtype != MLPMOE_BF16 && dtype != MLPMOE_FP32) return MLPMOE_ERR_INVALID_ARG;
  if (n_slices > kMaxSlices) return MLPMOE_ERR_UNSUPPORTED;          // more slices than the fixed scratch holds
  if (fade_work_bytes(n_slices) > kScratchBytes) return MLPMOE_ERR_UNSUPPORTED;
  const int elem_size = dtype == MLPMOE_BF16 ? 2 : 4;
  std::vector<FadeSeg> segs;
  segs.reserve(static_cast<size_t>(n_slices));
  for (int i = 0; i < n_slices; ++i) {
    if (!(s[i] >= 0.0 && s[i] < 1.0)) return MLPMOE_ERR_BAD_SCHEDULE;
    if (m[i] < 0 || (m[i] > 0 && !slices[i])) return MLPMOE_ERR_INVALID_ARG;
    // the kernels read the slice as 2- or 4-byte words: an address off that grid would fault on the device
    if (reinterpret_cast<uintptr_t>(slices[i]) % static_cast<uintptr_t>(elem_size) != 0) return MLPMOE_ERR_INVALID_ARG;
    if (s[i] == 0.0 || m[i] == 0) continue;                            // "leave untouched"
    int64_t lo = 0;
    if (mlpmoe_host_fade_position(s[i], m[i], &lo) != MLPMOE_OK) return MLPMOE_ERR_INVALID_ARG;
    FadeSeg g;
    g.base = slices[i];
    g.m = m[i];
    g.rank = lo;
    segs.push_back(g);
  }
  if (segs.empty()) return MLPMOE_OK;
  void* scratch = nullptr;
  mlpmoe_status_t rc = scratch_address(&scratch);
  if (rc != MLPMOE_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // launch_fade re-initialises every record it uses (rank, prefix, histograms), so what an
  // earlier call left in the array does not matter.
  if (launch_fade(segs.data(), static_cast<int>(segs.size()), scratch, elem_size, st) != cudaSuccess)
    return MLPMOE_ERR_CUDA;
  // the segment records were copied from this function's host memory
  if (cudaStreamSynchronize(st) != cudaSuccess) return MLPMOE_ERR_CUDA;
  return MLPMOE_OK;
}
